// The one-token-per-cluster form of the fused MoLE layer for sm_100a (Eq. 4 and Eq. 8 of arXiv 2503.15798),
// for the widest layers (d = 2048, N = 16 or 32: 64 or 128 KB of table rows and as much router matrix per
// token and layer).
//
// A thread-block cluster of CS blocks owns one token; block q of the cluster owns the 512 columns
// q * 512 .. q * 512 + 511: that slice of each of the token's N rows (in registers, requested before the
// grid dependency is waited for, as in mole_decode.cuh), that slice of the hidden state, and the matching
// 512 x N slice of the router matrix (one bulk copy into its own shared memory).  Each block reduces its
// slice to N partial logits, PUSHES them into the shared memory of every block of the cluster
// (st.async: the value and its count at the destination's mbarrier travel together), waits -- bounded -- until
// the CS x N values addressed to it have landed, and from there on is the decode kernel again: every warp
// forms the softmax numerators itself and accumulates its rows.  Against a split of the layer over
// independent blocks, where every block computes all logits by itself, the router matrix crosses from L2
// into the SMs once per token instead of once per block (a quarter of the bytes at CS = 4, and a quarter of
// the router arithmetic).
//
// Nobody reads another block's shared memory, so a block may exit as soon as it has received its partials:
// by then every push addressed to it has landed and its own pushes are on their way to blocks that are
// still waiting for them.  The hardware cluster barrier is used once, at the top (arrive) and just before the
// first push (wait): a push must not reach a block that has not initialised its barrier yet.  Every thread of
// every block reaches both unconditionally.
#pragma once

#include "mole_decode.cuh"

namespace mole {

constexpr int kClusterSlice = 512;             // columns per block
constexpr int kClusterThreads = kClusterSlice / 4;
constexpr int kClusterWarps = kClusterThreads / 32;
constexpr int kClusterMaxBlocks = 8;

// shared memory: the router slice [512][N], per-warp partial logits, the partials of the cluster's blocks, the
// per-warp sums of squares, two barriers
__host__ __device__ inline uint32_t cdecode_smem_bytes(int N)
{
    return up128(static_cast<uint32_t>(kClusterSlice) * N * 2) + kClusterWarps * 32 * 4 + kClusterMaxBlocks * 32 * 4 + kClusterWarps * 4 + 32;
}

#ifdef __CUDACC__

__device__ __forceinline__ uint32_t cluster_ctarank()
{
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ void cluster_arrive() { asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory"); }
__device__ __forceinline__ void cluster_wait() { asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory"); }
// the address of this block's shared-memory location `local` in block `rank` of the cluster
__device__ __forceinline__ uint32_t cluster_map(uint32_t local, uint32_t rank)
{
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(local), "r"(rank));
    return r;
}
// one value into another block's shared memory; its four bytes are counted in at that block's barrier when they land
__device__ __forceinline__ void cluster_push_f32(uint32_t remote_addr, float v, uint32_t remote_bar)
{
    asm volatile("st.async.weak.shared::cluster.mbarrier::complete_tx::bytes.f32 [%0], %1, [%2];" ::"r"(remote_addr), "f"(v), "r"(remote_bar)
                 : "memory");
}
__device__ __forceinline__ uint4 ldcg_v4(const void *p)
{
    uint4 v;
    asm volatile("ld.global.cg.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}
__device__ __forceinline__ bool mbar_try_wait_cluster(uint64_t *bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}

// N: experts (16 or 32).  CS: blocks per cluster = d / 512.  NORM: the router reads RMSNorm(hidden) rounded to bf16
// (App. A.2 listing); every block then reads the whole hidden row for the mean of squares.
// Launch: grid = tokens x CS blocks of 128 threads, dynamic shared memory cdecode_smem_bytes(N).
template <int N, int CS, int NORM>
__global__ void __cluster_dims__(CS, 1, 1) __launch_bounds__(kClusterThreads) mole_cdecode_kernel(const DecodeParams p)
{
    using E = Elem<__nv_bfloat16>;
    constexpr int VEC = 8;          // bf16 values per 16-byte vector
    constexpr int NV = VEC;         // accumulators per lane in the sweep
    constexpr int QL = N / VEC;     // vectors per router column
    constexpr int R = N / 2;        // sweep vectors per thread: (512 * N / 8) / 128
    constexpr int T = kClusterThreads;
    static_assert(N == 16 || N == 32, "experts per lane of the exchange");
    static_assert(CS >= 2 && CS <= kClusterMaxBlocks && CS % 2 == 0, "portable cluster sizes; a hidden row is CS / 2 passes of 16 bytes per thread");
    extern __shared__ __align__(128) unsigned char smem[];

    pdl_launch_dependents();

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int d = p.d;  // CS * 512
    const uint32_t q = cluster_ctarank();
    const long long t = blockIdx.x / CS;
    constexpr uint32_t wr_bytes = static_cast<uint32_t>(kClusterSlice) * N * 2;
    float *partial = reinterpret_cast<float *>(smem + up128(wr_bytes));  // [warps][N]
    float *xch = partial + kClusterWarps * 32;                           // [CS][N]: block c's partial logits
    float *scratch = xch + kClusterMaxBlocks * 32;                       // [warps]
    uint64_t *bar = reinterpret_cast<uint64_t *>(scratch + kClusterWarps);
    uint64_t *xbar = bar + 1;

    // ---- requests that do not depend on the previous kernel ----
    if (tid == 0) {
        mbar_init(bar, 1);
        mbar_init(xbar, 1);
        mbar_init_fence();
        mbar_expect_tx(xbar, CS * N * 4);  // armed for the partial logits of all CS blocks (this block's own included)
        mbar_expect_tx(bar, wr_bytes);
        bulk_g2s(smem, static_cast<const unsigned char *>(p.w_router) + static_cast<size_t>(q) * wr_bytes, wr_bytes, bar);
    }
    __syncwarp();
    cluster_arrive();  // (thread 0's initialisation of xbar is ordered before its arrival)
    const long long id = (p.flags & MOLE_FLAG_IDS_INT64) ? __ldg(static_cast<const long long *>(p.row_index) + t)
                                                         : static_cast<long long>(__ldg(static_cast<const int *>(p.row_index) + t));
    const bool valid = id >= 0 && id < p.rows;
    const size_t own = static_cast<size_t>(q) * kClusterSlice * 2 + static_cast<size_t>(tid) * 8;  // this thread's four columns, in bytes
    uint2 rv[N];
    {
        const unsigned char *row = static_cast<const unsigned char *>(p.lut) + static_cast<size_t>(valid ? id : 0) * N * d * 2 + own;
#pragma unroll
        for (int j = 0; j < N; ++j) rv[j] = ldg_stream_v2(row + static_cast<size_t>(j) * d * 2);
    }
    float nw[NORM ? R : 1];
    if constexpr (NORM) {
#pragma unroll
        for (int r = 0; r < R; ++r) {
            const int col = static_cast<int>(q) * kClusterSlice + (tid + r * T) / QL;
            nw[r] = bf16_bits_to_float(__ldg(static_cast<const unsigned short *>(p.norm_weight) + col));
        }
    }
    __syncthreads();  // the barriers are initialised before anybody in this block polls them

    // ---- the previous kernel's output: this block's slice of the token's hidden state (and residual) ----
    pdl_wait();
    const unsigned char *hrow = static_cast<const unsigned char *>(p.hidden) + static_cast<size_t>(t) * d * 2;
    unsigned short hs[R];
#pragma unroll
    for (int r = 0; r < R; ++r) {
        const int col = static_cast<int>(q) * kClusterSlice + (tid + r * T) / QL;  // sweep vector tid + r T covers one column of the slice
        hs[r] = ldcg_u16(hrow + 2 * col);
    }
    uint2 res = ldcg_v2((p.residual ? static_cast<const unsigned char *>(p.residual) + static_cast<size_t>(t) * d * 2 : hrow) + own);

    if constexpr (NORM) {
        // y = (x / sqrt(mean(x^2) + eps)) * w in fp32, rounded once to bf16: what the router reads.  The mean runs over
        // all d columns: every block reads the whole hidden row (4 KB from L2, 32 bytes per thread) and forms the
        // sum of squares itself, in the same order in every block -- cheaper than a second exchange.
        float ss = 0.f;
#pragma unroll
        for (int v = 0; v < CS / 2; ++v) {
            const uint4 hv = ldcg_v4(hrow + (static_cast<size_t>(v) * T + tid) * 16);
            const uint32_t w4[4] = {hv.x, hv.y, hv.z, hv.w};
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const float lo = bf16_bits_to_float(w4[i] & 0xffffu), hi = __uint_as_float(w4[i] & 0xffff0000u);
                ss = fmaf(hi, hi, fmaf(lo, lo, ss));
            }
        }
        ss = warp_sum(ss);
        if (lane == 0) scratch[warp] = ss;
        __syncthreads();
        float total = 0.f;
#pragma unroll
        for (int w = 0; w < kClusterWarps; ++w) total += scratch[w];
        const float rinv = 1.0f / sqrtf(total / static_cast<float>(d) + p.norm_eps);
#pragma unroll
        for (int r = 0; r < R; ++r) hs[r] = float_to_bf16_bits((bf16_bits_to_float(hs[r]) * rinv) * nw[r]);
    }

    // ---- router slice in shared memory? (bounded; after a failure the block goes on with whatever is there) ----
    {
        bool ok = false;
        for (uint32_t i = 0; i < p.wait_polls && !ok; ++i) {
            ok = mbar_try_wait(bar, 0);
            if (!ok && i > 64) __nanosleep(64);
        }
        if (!ok) {
            if (tid == 0 && p.status) atomicOr(p.status, MOLE_STATUS_TIMEOUT);
            for (uint32_t i = 0; i < kDrainPolls && !ok; ++i) {  // let the copy land before the block exits
                ok = mbar_try_wait(bar, 0);
                if (!ok) __nanosleep(64);
            }
        }
    }

    // ---- router sweep over the slice: partial logits per warp ----
    float acc[NV];
#pragma unroll
    for (int i = 0; i < NV; ++i) acc[i] = 0.f;
    const uint32_t wbase = smem_u32(smem);
    {
        uint4 wv[R];
#pragma unroll
        for (int r = 0; r < R; ++r) wv[r] = lds128(wbase + 16u * static_cast<uint32_t>(tid + r * T));
#pragma unroll
        for (int r = 0; r < R; ++r)
#pragma unroll
            for (int e = 0; e < VEC; ++e) E::fma_elem(acc[e], wv[r], e, hs[r]);
    }
    int base = 0;
    lane_reduce_scatter<NV, NV, 16, QL>(acc, lane, base);
    static_assert(ReduceScatterLeft<NV, 16, QL>::value == 1, "one logit share per lane");
    partial[warp * N + (lane % QL) * VEC + base] = acc[0];
    __syncthreads();

    // ---- exchange: warp 0 sums the warps' partials (lane j <-> expert j) and pushes the sum to every block ----
    cluster_wait();  // every block of the cluster has initialised its barriers (since long)
    if (warp == 0 && lane < N) {
        float z = 0.f;
#pragma unroll
        for (int w = 0; w < kClusterWarps; ++w) z += partial[w * N + lane];
        const uint32_t slot = smem_u32(xch + q * N + lane), xb = smem_u32(xbar);
#pragma unroll
        for (int c = 0; c < CS; ++c) cluster_push_f32(cluster_map(slot, c), z, cluster_map(xb, c));
    }
    {
        bool ok = false;
        for (uint32_t i = 0; i < p.wait_polls && !ok; ++i) {
            ok = mbar_try_wait_cluster(xbar, 0);
            if (!ok && i > 64) __nanosleep(64);
        }
        if (!ok) {
            if (tid == 0 && p.status) atomicOr(p.status, MOLE_STATUS_TIMEOUT);
            for (uint32_t i = 0; i < kDrainPolls && !ok; ++i) {  // pushes still on their way land in live shared memory
                ok = mbar_try_wait_cluster(xbar, 0);
                if (!ok) __nanosleep(64);
            }
        }
    }

    // ---- every warp: logits = the blocks' partials in rank order, softmax numerators (Eq. 4) ----
    const float e = softmax_numerator<N>(xch, CS, lane);

    // ---- weighted sum of this block's slice of the rows (Eq. 8), residual, store ----
    float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
    float es[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
    for (int j = 0; j < N; ++j) {
        const float g = __shfl_sync(0xffffffffu, e, j);
        es[j & 3] += g;
        // two values per fma on the packed fp32 pipe (two independent IEEE fmas: the bits of four fmaf)
        const float2 g2 = make_float2(g, g);
        const float2 lo = __ffma2_rn(g2, make_float2(bf16_bits_to_float(rv[j].x & 0xffffu), __uint_as_float(rv[j].x & 0xffff0000u)),
                                     make_float2(a0, a1));
        const float2 hi = __ffma2_rn(g2, make_float2(bf16_bits_to_float(rv[j].y & 0xffffu), __uint_as_float(rv[j].y & 0xffff0000u)),
                                     make_float2(a2, a3));
        a0 = lo.x, a1 = lo.y, a2 = hi.x, a3 = hi.y;
    }
    const float esum = (es[0] + es[1]) + (es[2] + es[3]);
    const float inv = __frcp_rn(esum);
    uint2 o = res;
    if (valid) {
        const __nv_bfloat162 lo = __floats2bfloat162_rn(fmaf(a0, inv, bf16_bits_to_float(res.x & 0xffffu)),
                                                        fmaf(a1, inv, __uint_as_float(res.x & 0xffff0000u)));
        const __nv_bfloat162 hi = __floats2bfloat162_rn(fmaf(a2, inv, bf16_bits_to_float(res.y & 0xffffu)),
                                                        fmaf(a3, inv, __uint_as_float(res.y & 0xffff0000u)));
        o.x = *reinterpret_cast<const uint32_t *>(&lo);
        o.y = *reinterpret_cast<const uint32_t *>(&hi);
    }
    *reinterpret_cast<uint2 *>(static_cast<unsigned char *>(p.out) + static_cast<size_t>(t) * d * 2 + own) = o;
    if (warp == 0 && q == 0) {
        if (p.gates_out && lane < N) p.gates_out[t * N + lane] = e / esum;
        if (!valid && lane == 0 && p.status) atomicOr(p.status, MOLE_STATUS_BAD_ID);
    }
}

#endif  // __CUDACC__

}  // namespace mole
