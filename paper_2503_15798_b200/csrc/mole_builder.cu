// Re-parameterisation on the GPU (Sec. 3.3, Eq. 6-7 of arXiv 2503.15798): the table of a layer is the
// output of every routed expert on every embedding row, LUT[i][j] = FFN_j(Embedding(i)) -- "a single
// forward pass with the embedding matrix as the input".  This is the one dense contraction of the method,
// so it runs on the 5th-generation tensor cores: two bf16 GEMMs with fp32 accumulation in tensor memory,
//     H = gelu(X . W1^T)      X [V][d] (the embedding rows, optionally RMS-normalised as in the training
//                             listing's expert_layernorm), W1 all experts stacked [N*D][d], H [V][N*D] bf16
//     LUT[:, j, :] = H[:, jD:(j+1)D] . W2_j^T      per expert j, W2_j [d][D], written straight into [V][N][d]
// each a launch of one kernel: C[z][m][n] = epilogue(sum_k A[z][m][k] * B[z][n][k]), both operands K-major.
//
// Kernel: persistent, one block per SM, each walking 128 x 256 output tiles (raster: eight tile rows by all
// tile columns at a time, so that the blocks in flight share operand tiles in L2).  Warp 0 (one thread)
// streams 128 x 64 tiles of A and 256 x 64 tiles of B through a four-stage ring of shared memory with tiled
// bulk tensor copies (128-byte swizzle, each into this block's own shared memory); warp 1 (one thread) issues
// tcgen05.mma 128 x 256 x 16 on the staged tiles and hands stages back with tcgen05.commit; the accumulator
// is double-buffered in tensor memory (2 x 256 of the 512 columns), so that warps 2-9 read tile i back with
// tcgen05.ld, apply the epilogue (GELU for the first GEMM) and store bf16 while the tensor cores already
// work on tile i + 1.  Every wait is bounded; a wait that runs out sets MOLE_STATUS_TIMEOUT and the block
// winds down: copies and MMAs in flight are waited for (again bounded) and tensor memory is freed on every path.
#include <cuda.h>
#include <math.h>
#include <mutex>
#include <string.h>

#include "mole_kernel.cuh"

namespace mole {

constexpr int kBM = 128, kBN = 256, kBK = 64;          // tile; kBK bf16 = one 128-byte swizzle span
constexpr int kGemmStages = 4;                         // 192 KB of operand tiles in flight per SM
constexpr int kTileBytesA = kBM * kBK * 2;             // 16 KB
constexpr int kTileBytesB = kBN * kBK * 2;             // 32 KB
constexpr int kStageBytes = kTileBytesA + kTileBytesB;
constexpr int kAccBuffers = 2;                         // accumulators in tensor memory: 2 x kBN of the 512 columns
constexpr int kTmemCols = kAccBuffers * kBN;
constexpr int kEpiWarps = 8;
constexpr int kGemmThreads = (2 + kEpiWarps) * 32;     // producer warp, MMA warp, eight epilogue warps
constexpr int kRasterRows = 8;                         // tile rows walked together
constexpr int kGemmBarriers = 2 * kGemmStages + 2 * kAccBuffers + 1;
constexpr int kStoreBytes = 32 * 128;                  // an epilogue warp's staging tile: 32 rows x 64 bf16, 128-byte swizzle
constexpr uint32_t kGemmSmem = kGemmStages * kStageBytes + kEpiWarps * kStoreBytes + 1024 /* alignment slack */ + 256 /* barriers */;
static_assert(kGemmSmem <= 232448, "one block's shared memory");
constexpr uint32_t kGemmWaitPolls = 1u << 22;
static_assert(kTmemCols == 512 && kGemmBarriers * 8 <= 128 && kEpiWarps % 4 == 0 && kBN % (8 * kEpiWarps) == 0, "tensor-memory columns are a power of two; barriers fit their block");

struct GemmParams {
    int M, N, K;            // per z slice
    int m_tiles, n_tiles;   // per z slice
    int total_tiles;        // over all z slices
    uint32_t *status;
};

#ifdef __CUDACC__

__device__ __forceinline__ void tma_load_3d(uint32_t smem_dst, const CUtensorMap *map, int c0, int c1, int c2, uint32_t bar)
{
    asm volatile("cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
                 ::"r"(smem_dst), "l"(map), "r"(c0), "r"(c1), "r"(c2), "r"(bar)
                 : "memory");
}
__device__ __forceinline__ void tma_store_3d(const CUtensorMap *map, uint32_t smem_src, int c0, int c1, int c2)
{
    asm volatile("cp.async.bulk.tensor.3d.global.shared::cta.bulk_group [%0, {%1, %2, %3}], [%4];"
                 ::"l"(map), "r"(c0), "r"(c1), "r"(c2), "r"(smem_src)
                 : "memory");
    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
}
__device__ __forceinline__ void st_shared_v4(uint32_t addr, uint32_t a, uint32_t b, uint32_t c, uint32_t d)
{
    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}
__device__ __forceinline__ bool bar_try_wait(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}
__device__ __forceinline__ bool bar_wait_bounded(uint32_t bar, uint32_t parity, volatile int *dead, uint32_t polls = kGemmWaitPolls)
{
    for (uint32_t i = 0; i < polls; ++i) {
        if (bar_try_wait(bar, parity)) return true;
        if (i > 32) {
            __nanosleep(40);
            if ((i & 255u) == 0 && *dead) return false;
        }
    }
    return false;
}
__device__ __forceinline__ void bar_arrive(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
// shared-memory operand descriptor of tcgen05.mma: a K-major tile of rows x 64 bf16, rows 128 bytes apart,
// 128-byte swizzle (as the tensor copy wrote it), 1024 bytes between groups of eight rows
__device__ __forceinline__ uint64_t umma_desc(uint32_t smem_addr)
{
    uint64_t d = 0;
    d |= static_cast<uint64_t>((smem_addr & 0x3FFFFu) >> 4);  // start address, 16-byte units
    d |= static_cast<uint64_t>(1) << 16;                      // leading-dimension offset (unused with a swizzled K-major tile)
    d |= static_cast<uint64_t>(1024 >> 4) << 32;              // stride between 8-row groups
    d |= static_cast<uint64_t>(1) << 46;                      // descriptor version of this architecture
    d |= static_cast<uint64_t>(2) << 61;                      // 128-byte swizzle
    return d;
}
// instruction descriptor: bf16 x bf16 -> fp32, both operands K-major, M = kBM, N = kBN
__device__ __forceinline__ uint32_t umma_idesc()
{
    return (1u << 4) | (1u << 7) | (1u << 10) | (static_cast<uint32_t>(kBN >> 3) << 17) | (static_cast<uint32_t>(kBM >> 4) << 24);
}
__device__ __forceinline__ void umma_bf16(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32])
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]), "=r"(r[9]),
          "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]),
          "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]),
          "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr));
}

// GELU(x) = x Phi(x) = max(x, 0) - |x| erfc(|x| / sqrt 2) / 2, with
// erfc(u) = t (a1 + t (a2 + t (a3 + t (a4 + t a5)))) exp(-u^2), t = 1 / (1 + p u)
// (Abramowitz & Stegun 7.1.26, |error| <= 1.5e-7): within 4e-7 of the exact GELU everywhere, a fraction of the
// bf16 rounding that follows.  Two elements at a time on the packed fp32 pipe; about a third of the
// instructions of erff().
__device__ __forceinline__ float2 splat(float v) { return make_float2(v, v); }
__device__ __forceinline__ float rcp_approx(float v)
{
    float r;
    asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(v));
    return r;
}
__device__ __forceinline__ float ex2_approx(float v)
{
    float r;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(v));
    return r;
}
__device__ __forceinline__ float2 gelu_erf2(float2 x)
{
    constexpr float kP = 0.3275911f * 0.70710678118654752440f;  // p / sqrt 2
    float2 t;
    t.x = rcp_approx(fmaf(fabsf(x.x), kP, 1.0f));
    t.y = rcp_approx(fmaf(fabsf(x.y), kP, 1.0f));
    float2 poly = __ffma2_rn(splat(0.5f * 1.061405429f), t, splat(0.5f * -1.453152027f));  // a_i / 2
    poly = __ffma2_rn(poly, t, splat(0.5f * 1.421413741f));
    poly = __ffma2_rn(poly, t, splat(0.5f * -0.284496736f));
    poly = __ffma2_rn(poly, t, splat(0.5f * 0.254829592f));
    poly = __fmul2_rn(poly, t);
    const float2 arg = __fmul2_rn(__fmul2_rn(x, splat(-0.72134752044448170368f)), x);  // -x^2 / 2 in powers of two
    float2 e;
    e.x = ex2_approx(arg.x);
    e.y = ex2_approx(arg.y);
    const float2 h = __fmul2_rn(poly, e);  // erfc(|x| / sqrt 2) / 2
    float2 g;
    g.x = fmaf(-fabsf(x.x), h.x, fmaxf(x.x, 0.0f));
    g.y = fmaf(-fabsf(x.y), h.y, fmaxf(x.y, 0.0f));
    return g;
}

struct TileCoord {
    int m0, n0, z;
};
// tiles in the order the blocks walk them: z slice by z slice, kRasterRows tile rows at a time, down the rows first
__device__ __forceinline__ TileCoord tile_coord(int tile, const GemmParams &p)
{
    const int per_z = p.m_tiles * p.n_tiles;
    const int z = tile / per_z, r = tile - z * per_z;
    const int band = r / (kRasterRows * p.n_tiles);
    const int first = band * kRasterRows;
    const int rows = min(kRasterRows, p.m_tiles - first);
    const int w = r - band * kRasterRows * p.n_tiles;
    TileCoord t;
    t.m0 = (first + w % rows) * kBM;
    t.n0 = (w / rows) * kBN;
    t.z = z;
    return t;
}

template <int GELU>
__global__ void __launch_bounds__(kGemmThreads, 1) mole_gemm_tn_kernel(const __grid_constant__ CUtensorMap map_a,
                                                                    const __grid_constant__ CUtensorMap map_b,
                                                                    const __grid_constant__ CUtensorMap map_c, const GemmParams p)
{
    extern __shared__ unsigned char smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t tiles = (raw + 1023u) & ~1023u;  // swizzled tiles want 1024-byte alignment
    const uint32_t staging = tiles + kGemmStages * kStageBytes;
    unsigned char *ctl = smem_raw + (tiles - raw) + kGemmStages * kStageBytes + kEpiWarps * kStoreBytes;
    uint64_t *bars = reinterpret_cast<uint64_t *>(ctl);  // full[stages], empty[stages], acc_full[2], acc_empty[2], drain
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(ctl + 128);
    volatile int *dead = reinterpret_cast<volatile int *>(tmem_slot + 1);
    const uint32_t full0 = smem_u32(bars), empty0 = full0 + kGemmStages * 8, acc_full0 = empty0 + kGemmStages * 8,
                   acc_empty0 = acc_full0 + kAccBuffers * 8, drain_bar = acc_empty0 + kAccBuffers * 8;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int ktiles = (p.K + kBK - 1) / kBK;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kGemmBarriers; ++s) {
            const bool acc_empty = s >= 2 * kGemmStages + kAccBuffers && s < 2 * kGemmStages + 2 * kAccBuffers;
            mbar_init(bars + s, acc_empty ? kEpiWarps : 1);  // every epilogue warp hands an accumulator back
        }
        dead[0] = 0;
        dead[1] = 0;  // stays 0: the flag the draining waits look at
        mbar_init_fence();
    }
    if (warp == 1) {  // all of this SM's tensor memory: two 128 x kBN fp32 accumulators (one block per SM)
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(kTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_acc = *tmem_slot;

    if (warp == 0) {
        if (lane == 0) {  // ---- producer: tiles of A and B, kGemmStages ahead, across output tiles ----
            uint32_t it = 0;  // k-tiles issued by this block so far
            bool ok = true;
            for (int tile = blockIdx.x; tile < p.total_tiles && ok; tile += gridDim.x) {
                const TileCoord tc = tile_coord(tile, p);
                for (int kt = 0; kt < ktiles; ++kt, ++it) {
                    const uint32_t s = it % kGemmStages;
                    const uint32_t par = ((it / kGemmStages) & 1u) ^ 1u;  // first pass: the stage has never been used
                    if (!bar_wait_bounded(empty0 + s * 8, par, dead)) {
                        ok = false;
                        break;
                    }
                    const uint32_t a_dst = tiles + s * kStageBytes, b_dst = a_dst + kTileBytesA;
                    mbar_expect_tx(bars + s, kStageBytes);
                    tma_load_3d(a_dst, &map_a, kt * kBK, tc.m0, tc.z, full0 + s * 8);
                    tma_load_3d(b_dst, &map_b, kt * kBK, tc.n0, tc.z, full0 + s * 8);
                }
            }
            if (!ok) {
                if (!*dead && p.status) atomicOr(p.status, MOLE_STATUS_TIMEOUT);
                *dead = 1;
                // the copies already issued land in this block's shared memory: let them, before the block can exit
                const uint32_t first = it > static_cast<uint32_t>(kGemmStages) ? it - kGemmStages : 0u;
                for (uint32_t j = first; j < it; ++j)
                    (void)bar_wait_bounded(full0 + (j % kGemmStages) * 8, (j / kGemmStages) & 1u, dead + 1, kDrainPolls);
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {  // ---- tensor-core issue ----
            const uint32_t idesc = umma_idesc();
            uint32_t it = 0, t = 0;  // k-tiles and output tiles consumed by this block so far
            bool ok = true;
            for (int tile = blockIdx.x; tile < p.total_tiles && ok; tile += gridDim.x, ++t) {
                const uint32_t b = t & 1u;
                // the epilogue warps have read this accumulator's previous tile out
                ok = bar_wait_bounded(acc_empty0 + b * 8, ((t >> 1) & 1u) ^ 1u, dead);
                if (!ok) break;
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const uint32_t acc = tmem_acc + b * kBN;
                for (int kt = 0; kt < ktiles; ++kt, ++it) {
                    const uint32_t s = it % kGemmStages;
                    ok = bar_wait_bounded(full0 + s * 8, (it / kGemmStages) & 1u, dead);
                    if (!ok) break;
                    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                    const uint32_t a_src = tiles + s * kStageBytes, b_src = a_src + kTileBytesA;
                    const uint64_t adesc = umma_desc(a_src), bdesc = umma_desc(b_src);
#pragma unroll
                    for (int k = 0; k < kBK / 16; ++k)  // 16 bf16 = 32 bytes along K inside the swizzle span: +2 in 16-byte units
                        umma_bf16(acc, adesc + 2 * k, bdesc + 2 * k, idesc, (kt > 0 || k > 0) ? 1u : 0u);
                    umma_commit(empty0 + s * 8);  // the stage is free once these have read it
                }
                if (ok) umma_commit(acc_full0 + b * 8);
            }
            if (!ok) {
                if (!*dead && p.status) atomicOr(p.status, MOLE_STATUS_TIMEOUT);
                *dead = 1;
                umma_commit(drain_bar);  // whatever was issued finishes reading shared memory before the block exits
                (void)bar_wait_bounded(drain_bar, 0, dead + 1, kDrainPolls);
            }
        }
    } else {
        // ---- epilogue: warp w reads tensor-memory lanes 32 (w % 4) .., one output row per thread; the warps
        // that share a lane quarter take an equal part of the tile's columns each, 32 at a time.  The rounded
        // values go through a staging tile in shared memory (32 rows x 64 columns, 128-byte swizzle: the eight
        // lanes of a store phase hit eight different 16-byte columns) and leave with one bulk tensor store per
        // 64 columns: whole 128-byte lines, clipped to the matrix by the copy engine ----
        const int quarter = warp & 3;
        const int part = (warp - 2) >> 2;
        constexpr int kColsPerWarp = kBN / (kEpiWarps / 4);
        constexpr int kChunks = kColsPerWarp / 32;
        static_assert(kChunks % 2 == 0, "a staging tile is two chunks wide");
        const uint32_t stage_row = staging + static_cast<uint32_t>((warp - 2) * kStoreBytes + lane * 128);
        uint32_t t = 0;
        bool ok = true;
        for (int tile = blockIdx.x; tile < p.total_tiles && ok; tile += gridDim.x, ++t) {
            const uint32_t b = t & 1u;
            ok = bar_wait_bounded(acc_full0 + b * 8, (t >> 1) & 1u, dead);
            if (!ok) break;
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const TileCoord tc = tile_coord(tile, p);
            const int row0 = tc.m0 + quarter * 32;
            const int ncol0 = tc.n0 + part * kColsPerWarp;
            const uint32_t tsrc = tmem_acc + (static_cast<uint32_t>(quarter * 32) << 16) + b * kBN + static_cast<uint32_t>(part * kColsPerWarp);
            uint32_t r[2][32];
            tmem_ld32(tsrc, r[0]);
#pragma unroll
            for (int c = 0; c < kChunks; ++c) {
                asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
                if (c + 1 < kChunks) {
                    tmem_ld32(tsrc + static_cast<uint32_t>((c + 1) * 32), r[(c + 1) & 1]);
                } else {
                    // this warp's part of the accumulator is in registers: hand the buffer back to the tensor cores
                    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
                    __syncwarp();
                    if (lane == 0) bar_arrive(acc_empty0 + b * 8);
                }
                uint32_t packed[16];  // 32 consecutive columns of this thread's row, rounded in pairs
#pragma unroll
                for (int i = 0; i < 32; i += 2) {
                    float2 x = make_float2(__uint_as_float(r[c & 1][i]), __uint_as_float(r[c & 1][i + 1]));
                    if (GELU) x = gelu_erf2(x);
                    const __nv_bfloat162 v = __floats2bfloat162_rn(x.x, x.y);
                    packed[i / 2] = *reinterpret_cast<const uint32_t *>(&v);
                }
                if ((c & 1) == 0) {  // the staging tile is free once the previous store has read it
                    if (lane == 0) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
                    __syncwarp();
                }
#pragma unroll
                for (int v = 0; v < 4; ++v)
                    st_shared_v4(stage_row + static_cast<uint32_t>((((c & 1) * 4 + v) ^ (lane & 7)) * 16), packed[4 * v], packed[4 * v + 1],
                                 packed[4 * v + 2], packed[4 * v + 3]);
                if (c & 1) {
                    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                    __syncwarp();
                    const int col0 = ncol0 + (c >> 1) * 64;
                    if (lane == 0 && row0 < p.M && col0 < p.N) tma_store_3d(&map_c, stage_row, col0, row0, tc.z);
                }
            }
        }
        if (lane == 0) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");  // this warp's stores have left shared memory and landed
        if (!ok && lane == 0 && !*dead && p.status) atomicOr(p.status, MOLE_STATUS_TIMEOUT);
        if (!ok && lane == 0) *dead = 1;
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 1) {
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_acc), "r"(kTmemCols) : "memory");
    }
}

// y = (x / sqrt(mean(x^2) + eps)) * w, rounded once to bf16: the embedding rows as the routed experts of the
// training listing see them.  One warp per row.
__global__ void mole_rmsnorm_rows_kernel(const __nv_bfloat16 *__restrict__ x, const __nv_bfloat16 *__restrict__ w,
                                         __nv_bfloat16 *__restrict__ y, long long rows, int d, float eps)
{
    const long long row = static_cast<long long>(blockIdx.x) * (blockDim.x / 32) + (threadIdx.x >> 5);
    const int lane = threadIdx.x & 31;
    if (row >= rows) return;
    const __nv_bfloat16 *xr = x + row * d;
    float ss = 0.f;
    for (int c = lane; c < d; c += 32) {
        const float v = __bfloat162float(xr[c]);
        ss = fmaf(v, v, ss);
    }
    ss = warp_sum(ss);
    const float r = 1.0f / sqrtf(ss / static_cast<float>(d) + eps);
    for (int c = lane; c < d; c += 32) y[row * d + c] = __float2bfloat16_rn((__bfloat162float(xr[c]) * r) * __bfloat162float(w[c]));
}

#endif  // __CUDACC__

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *, const cuuint64_t *,
                                  const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_tiled()
{
    static EncodeTiledFn fn = nullptr;
    static std::once_flag once;
    std::call_once(once, [] {
        void *p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess && q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
        else
            (void)cudaGetLastError();
    });
    return fn;
}

// bf16 matrix [z][rows][k], k contiguous: rows row_stride elements apart, z slices z_stride elements apart; tiles of
// box_rows x 64 elements in the 128-byte swizzle (operands and the output alike)
static int make_matrix_map(CUtensorMap *map, const void *base, long long k, long long rows, long long zs, long long row_stride,
                           long long z_stride, int box_rows)
{
    EncodeTiledFn enc = encode_tiled();
    if (!enc) return MOLE_ERR_CUDA;
    const cuuint64_t dims[3] = {static_cast<cuuint64_t>(k), static_cast<cuuint64_t>(rows), static_cast<cuuint64_t>(zs)};
    const cuuint64_t strides[2] = {static_cast<cuuint64_t>(row_stride) * 2, static_cast<cuuint64_t>(z_stride) * 2};
    const cuuint32_t box[3] = {kBK, static_cast<cuuint32_t>(box_rows), 1};
    const cuuint32_t estr[3] = {1, 1, 1};
    const CUresult r = enc(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void *>(base), dims, strides, box, estr,
                           CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                           CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? MOLE_OK : MOLE_ERR_CUDA;
}

// C[z][m][n] = epilogue(sum_k A[z][m][k] B[z][n][k])
static int launch_gemm(const void *a, long long a_row_stride, long long a_z_stride, const void *b, long long b_row_stride,
                       long long b_z_stride, void *c, long long c_row_stride, long long c_z_stride, int M, int N, int K, int Z, int gelu,
                       uint32_t *status, cudaStream_t st)
{
    CUtensorMap map_a, map_b, map_c;
    int rc = make_matrix_map(&map_a, a, K, M, Z, a_row_stride, a_z_stride, kBM);
    if (rc != MOLE_OK) return rc;
    rc = make_matrix_map(&map_b, b, K, N, Z, b_row_stride, b_z_stride, kBN);
    if (rc != MOLE_OK) return rc;
    rc = make_matrix_map(&map_c, c, N, M, Z, c_row_stride, c_z_stride, 32);
    if (rc != MOLE_OK) return rc;
    const void *fn = gelu ? reinterpret_cast<const void *>(mole_gemm_tn_kernel<1>) : reinterpret_cast<const void *>(mole_gemm_tn_kernel<0>);
    rc = ensure_smem_opt_in(fn, static_cast<int>(kGemmSmem));
    if (rc != MOLE_OK) return rc;
    int sms = 0;
    rc = sm_count(&sms);
    if (rc != MOLE_OK) return rc;
    GemmParams p;
    p.M = M;
    p.N = N;
    p.K = K;
    p.m_tiles = (M + kBM - 1) / kBM;
    p.n_tiles = (N + kBN - 1) / kBN;
    const long long total = static_cast<long long>(p.m_tiles) * p.n_tiles * Z;
    if (total > 0x7fffffffLL) return MOLE_ERR_TOO_LARGE;
    p.total_tiles = static_cast<int>(total);
    p.status = status;
    const unsigned grid = static_cast<unsigned>(total < sms ? total : sms);  // persistent: one block per SM
    if (gelu)
        mole_gemm_tn_kernel<1><<<grid, kGemmThreads, kGemmSmem, st>>>(map_a, map_b, map_c, p);
    else
        mole_gemm_tn_kernel<0><<<grid, kGemmThreads, kGemmSmem, st>>>(map_a, map_b, map_c, p);
    MOLE_CUDA_TRY(cudaGetLastError());
    return MOLE_OK;
}

}  // namespace mole

using namespace mole;

extern "C" {

int mole_build_lut_scratch_bytes(int V, int N, int d, int D, int with_norm, int64_t *bytes)
{
    if (!bytes || V < 1 || N < 1 || N > 64 || d < 8 || D < 8 || (d & 7) || (D & 7)) return MOLE_ERR_INVALID_ARG;
    int64_t b = static_cast<int64_t>(V) * N * D * 2;
    if (with_norm) b += (static_cast<int64_t>(V) * d * 2 + 255) / 256 * 256;
    *bytes = b;
    return MOLE_OK;
}

int mole_build_lut(const void *embedding, const void *w1, const void *w2, const void *norm_weight, float norm_eps, void *lut,
                   void *scratch, int V, int N, int d, int D, uint32_t *status, void *stream)
{
    if (V < 1 || N < 1 || N > 64 || d < 8 || D < 8 || (d & 7) || (D & 7)) return MOLE_ERR_UNSUPPORTED_SHAPE;
    if (static_cast<long long>(N) * D > 0x7fffffffLL / 2 || V > 0x7fffffff / 2) return MOLE_ERR_TOO_LARGE;
    if (!embedding || !w1 || !w2 || !lut || !scratch) return MOLE_ERR_INVALID_ARG;
    if (!aligned16(embedding) || !aligned16(w1) || !aligned16(w2) || !aligned16(lut) || !aligned16(scratch)) return MOLE_ERR_INVALID_ARG;
    if (norm_weight && (!aligned16(norm_weight) || !(norm_eps >= 0.f) || norm_eps > 3.0e38f)) return MOLE_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    unsigned char *hbuf = static_cast<unsigned char *>(scratch);
    const void *x = embedding;
    if (norm_weight) {
        __nv_bfloat16 *xn = reinterpret_cast<__nv_bfloat16 *>(hbuf);
        hbuf += (static_cast<int64_t>(V) * d * 2 + 255) / 256 * 256;
        const int warps = 8;
        mole_rmsnorm_rows_kernel<<<static_cast<unsigned>((V + warps - 1) / warps), warps * 32, 0, st>>>(
            static_cast<const __nv_bfloat16 *>(embedding), static_cast<const __nv_bfloat16 *>(norm_weight), xn, V, d, norm_eps);
        MOLE_CUDA_TRY(cudaGetLastError());
        x = xn;
    }
    const long long ND = static_cast<long long>(N) * D;
    // H = gelu(X . W1^T): one GEMM over all experts' first matrices stacked [N*D][d]
    int rc = launch_gemm(x, d, static_cast<long long>(V) * d, w1, d, ND * d, hbuf, ND, static_cast<long long>(V) * ND, V, static_cast<int>(ND), d,
                         1, 1, status, st);
    if (rc != MOLE_OK) return rc;
    // LUT[:, j, :] = H[:, jD:(j+1)D] . W2_j^T: z = expert; A's z slices are D columns apart, C's are d columns apart
    return launch_gemm(hbuf, ND, D, w2, D, static_cast<long long>(d) * D, lut, static_cast<long long>(N) * d, d, V, d, D, N, 0, status, st);
}

}  // extern "C"
