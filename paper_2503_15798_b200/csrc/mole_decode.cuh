// The decode-batch form of the fused MoLE layer for sm_100a (Eq. 4 and Eq. 8 of arXiv 2503.15798):
// one block per token, one launch per layer, built for the shortest chain from "the previous layer
// has finished" to "this layer's output is stored".
//
// At decode batches a layer moves a few megabytes -- less than a microsecond at HBM speed -- so what
// a chain of layers costs is the latency of one token's path, not bandwidth.  Everything that does
// not depend on the previous layer is therefore requested before the grid dependency is waited for
// and lands while this block waits:
//   - the token's N table rows, straight into registers: thread i owns the four columns 4i .. 4i+3
//     of every expert's row (one 8-byte load per expert, a warp reads 256 consecutive bytes);
//   - the router matrix, one bulk asynchronous copy into shared memory (it is shared by all tokens,
//     so it comes from L2);
//   - with a normalised router, the scale vector's entries this thread will need.
// After the dependency only the hidden state is fetched -- by plain loads into registers, each thread
// exactly the elements it multiplies -- and the arithmetic has one block barrier on its path:
//   sweep over the router matrix (linear, 16 bytes per lane, bank-conflict free; a lane always meets
//   the same experts and keeps min(N, 8) fp32 accumulators) -> shuffle reduce-scatter over the warp ->
//   per-warp partial logits to shared memory -> barrier -> EVERY warp sums the partials and forms the
//   softmax numerators itself (lane j holds expert j; no second barrier, no broadcast through shared
//   memory) -> the numerators are handed round by shuffles while the rows, already in registers, are
//   accumulated -> one reciprocal, residual add, one rounding, one 8-byte store per thread.
// The summation order of the weighted sum (experts in ascending order per column, the numerators' sum
// in four interleaved chains) is the one the ring kernel uses with one lane per column group.
#pragma once

#include <math.h>

#include "mole_kernel.cuh"

namespace mole {

constexpr int kDecodeMaxThreads = 512;  // d <= 2048 (N <= 16); N = 32 keeps twice the registers: 256 threads, d <= 1024
constexpr int kDecodeMaxWarps = kDecodeMaxThreads / 32;
__host__ __device__ constexpr int decode_max_threads(int N) { return N > 16 ? 256 : kDecodeMaxThreads; }

struct DecodeParams {
    const void *hidden, *residual, *row_index, *lut, *w_router, *norm_weight;
    void *out;
    float *gates_out;
    uint32_t *status;
    long long rows;       // table rows that may be addressed
    int d;
    float norm_eps;
    uint32_t flags;
    uint32_t wait_polls;  // polls after which the wait for the router matrix gives up
};

// shared memory: the router matrix [d][N], then one float per (warp, expert), one per warp, the barrier
__host__ __device__ inline uint32_t decode_smem_bytes(int N, int d)
{
    return up128(static_cast<uint32_t>(d) * N * 2) + kDecodeMaxWarps * 64 * 4 + kDecodeMaxWarps * 4 + 16;
}

#ifdef __CUDACC__

__device__ __forceinline__ uint2 ldg_stream_v2(const void *p)
{
    uint2 v;
    asm volatile("ld.global.nc.L1::no_allocate.v2.u32 {%0, %1}, [%2];" : "=r"(v.x), "=r"(v.y) : "l"(p));
    return v;
}
__device__ __forceinline__ uint4 ldg_nc_v4(const void *p)
{
    uint4 v;
    asm volatile("ld.global.nc.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}
__device__ __forceinline__ unsigned short ldcg_u16(const void *p)
{
    unsigned short v;
    asm volatile("ld.global.cg.u16 %0, [%1];" : "=h"(v) : "l"(p));
    return v;
}
__device__ __forceinline__ uint2 ldcg_v2(const void *p)
{
    uint2 v;
    asm volatile("ld.global.cg.v2.u32 {%0, %1}, [%2];" : "=r"(v.x), "=r"(v.y) : "l"(p));
    return v;
}
__device__ __forceinline__ float bf16_bits_to_float(uint32_t b) { return __uint_as_float(b << 16); }
__device__ __forceinline__ unsigned short float_to_bf16_bits(float f)
{
    const __nv_bfloat16 b = __float2bfloat16_rn(f);
    return *reinterpret_cast<const unsigned short *>(&b);
}

// Softmax numerator of expert `lane` (Eq. 4; lanes >= N get 0) from the per-warp partial logits
// partial[w * N + j]: independent loads, one chain of adds in warp order, exp(z - m) with the maximum m
// taken only when some logit is large enough for exp to leave the comfortable range (any shift gives
// the same gates).  Every warp of a block calls it and gets the same values.
template <int N>
__device__ __forceinline__ float softmax_numerator(const float *partial, int nwarps, int lane)
{
    float z = 0.f;
    if (lane < N) {
        float v[kDecodeMaxWarps];
#pragma unroll
        for (int w = 0; w < kDecodeMaxWarps; ++w) v[w] = w < nwarps ? partial[w * N + lane] : 0.f;
#pragma unroll
        for (int w = 0; w < kDecodeMaxWarps; ++w) z += v[w];
    }
    const bool big = lane < N && !(fabsf(z) < 80.f);
    float zmax = 0.f;
    if (__any_sync(0xffffffffu, big)) zmax = warp_max(lane < N ? z : -INFINITY);
    return lane < N ? expf(z - zmax) : 0.f;
}

// N: experts (4, 8, 16 or 32).  NORM: the router reads RMSNorm(hidden) rounded to bf16 (App. A.2 listing).
// Launch: one block per token, blockDim.x == d / 4 (a multiple of 32), dynamic shared memory
// decode_smem_bytes(N, d).
template <int N, int NORM>
__global__ void __launch_bounds__(decode_max_threads(N)) mole_decode_kernel(const DecodeParams p)
{
    using E = Elem<__nv_bfloat16>;
    constexpr int VEC = 8;                     // bf16 values per 16-byte vector
    constexpr int NV = N < VEC ? N : VEC;      // accumulators per lane in the sweep
    constexpr int QL = N >= VEC ? N / VEC : 1; // vectors per router column
    constexpr int CPV = N >= VEC ? 1 : VEC / N;  // router columns per vector
    constexpr int R = N / 2;                   // sweep vectors per thread: (d * N / 8) / (d / 4)
    extern __shared__ __align__(128) unsigned char smem[];

    pdl_launch_dependents();

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int T = blockDim.x, nwarps = T >> 5, d = p.d;
    const long long t = blockIdx.x;
    const uint32_t wr_bytes = static_cast<uint32_t>(d) * N * 2;
    float *partial = reinterpret_cast<float *>(smem + up128(wr_bytes));  // [nwarps][N]
    float *scratch = partial + kDecodeMaxWarps * 64;                         // [nwarps]
    uint64_t *bar = reinterpret_cast<uint64_t *>(scratch + kDecodeMaxWarps);

    // ---- requests that do not depend on the previous kernel ----
    if (tid == 0) {
        mbar_init(bar, 1);
        mbar_init_fence();
        mbar_expect_tx(bar, wr_bytes);
        bulk_g2s(smem, p.w_router, wr_bytes, bar);
    }
    const long long id = (p.flags & MOLE_FLAG_IDS_INT64) ? __ldg(static_cast<const long long *>(p.row_index) + t)
                                                         : static_cast<long long>(__ldg(static_cast<const int *>(p.row_index) + t));
    const bool valid = id >= 0 && id < p.rows;
    uint2 rv[N];
    {
        const unsigned char *row = static_cast<const unsigned char *>(p.lut) + static_cast<size_t>(valid ? id : 0) * N * d * 2 +
                                   static_cast<size_t>(tid) * 8;
#pragma unroll
        for (int j = 0; j < N; ++j) rv[j] = ldg_stream_v2(row + static_cast<size_t>(j) * d * 2);
    }
    // column(s) of sweep vector r of this thread: vector u = tid + r * T covers column u / QL (N >= 8)
    // or columns u * CPV .. (N < 8)
    float nw[NORM ? R * CPV : 1];
    if constexpr (NORM) {
#pragma unroll
        for (int r = 0; r < R; ++r)
#pragma unroll
            for (int cc = 0; cc < CPV; ++cc) {
                const int u = tid + r * T;
                const int col = N >= VEC ? u / QL : u * CPV + cc;
                nw[r * CPV + cc] = bf16_bits_to_float(__ldg(static_cast<const unsigned short *>(p.norm_weight) + col));
            }
    }
    __syncthreads();  // the barrier is initialised before anybody polls it

    // ---- the previous kernel's output: hidden state (and residual) of this token ----
    pdl_wait();
    const unsigned char *hrow = static_cast<const unsigned char *>(p.hidden) + static_cast<size_t>(t) * d * 2;
    unsigned short hs[R * CPV];
#pragma unroll
    for (int r = 0; r < R; ++r)
#pragma unroll
        for (int cc = 0; cc < CPV; ++cc) {
            const int u = tid + r * T;
            const int col = N >= VEC ? u / QL : u * CPV + cc;
            hs[r * CPV + cc] = ldcg_u16(hrow + 2 * col);
        }
    const uint2 hown = ldcg_v2(hrow + static_cast<size_t>(tid) * 8);  // columns 4 tid .. 4 tid + 3
    uint2 res = hown;
    if (p.residual) res = ldcg_v2(static_cast<const unsigned char *>(p.residual) + static_cast<size_t>(t) * d * 2 + static_cast<size_t>(tid) * 8);

    if constexpr (NORM) {
        // y = (x / sqrt(mean(x^2) + eps)) * w in fp32, rounded once to bf16: what the router reads
        const float x0 = bf16_bits_to_float(hown.x & 0xffffu), x1 = __uint_as_float(hown.x & 0xffff0000u);
        const float x2 = bf16_bits_to_float(hown.y & 0xffffu), x3 = __uint_as_float(hown.y & 0xffff0000u);
        float ss = fmaf(x3, x3, fmaf(x2, x2, fmaf(x1, x1, x0 * x0)));
        ss = warp_sum(ss);
        if (lane == 0) scratch[warp] = ss;
        __syncthreads();
        float total = 0.f;
        for (int w = 0; w < nwarps; ++w) total += scratch[w];  // the same order in every thread
        const float rinv = 1.0f / sqrtf(total / static_cast<float>(d) + p.norm_eps);
#pragma unroll
        for (int i = 0; i < R * CPV; ++i) hs[i] = float_to_bf16_bits((bf16_bits_to_float(hs[i]) * rinv) * nw[i]);
    }

    // ---- router matrix in shared memory? (bounded wait; after a failure the block computes on
    // whatever is there -- every address stays in its own shared memory and its own output row --
    // and the status word says that the outputs are meaningless) ----
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

    // ---- router sweep: partial logits of this thread's vectors ----
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
            for (int e = 0; e < VEC; ++e) E::fma_elem(acc[e % NV], wv[r], e, hs[r * CPV + e / NV]);
    }
    int base = 0;
    lane_reduce_scatter<NV, NV, 16, QL>(acc, lane, base);
    static_assert(ReduceScatterLeft<NV, 16, QL>::value == 1, "one logit share per lane");
    partial[warp * N + (N >= VEC ? (lane % QL) * VEC : 0) + base] = acc[0];
    __syncthreads();

    // ---- every warp: logits, softmax numerators (Eq. 4), lane j <-> expert j ----
    const float e = softmax_numerator<N>(partial, nwarps, lane);

    // ---- weighted sum of the rows (Eq. 8), residual, store ----
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
    *reinterpret_cast<uint2 *>(static_cast<unsigned char *>(p.out) + static_cast<size_t>(t) * d * 2 + static_cast<size_t>(tid) * 8) = o;
    if (warp == 0) {
        if (p.gates_out && lane < N) p.gates_out[t * N + lane] = e / esum;
        if (!valid && lane == 0 && p.status) atomicOr(p.status, MOLE_STATUS_BAD_ID);
    }
}

#endif  // __CUDACC__

}  // namespace mole
