// Fused MoLE inference layer for sm_100a: router dot products, softmax over all N experts,
// gather of the token's N table rows, fp32 weighted sum, residual add (Eq. 4 and Eq. 8 of
// arXiv 2503.15798).  One thread block handles one token (or one slice of a token's d
// columns).  The rows are pulled into shared memory by bulk asynchronous copies that are
// issued before anything else, because they depend only on the id; the router runs while
// they are in flight.
#include <atomic>
#include <math.h>
#include <string.h>

#include "mole_common.cuh"

namespace mole {

constexpr int kMaxN = 64;      // experts
constexpr int kMaxWarps = 8;   // 256 threads
constexpr int kMaxSplit = 8;   // blocks per token
constexpr int kMaxThreads = 256;
constexpr int kFixedSmem = (kMaxWarps * kMaxN + kMaxSplit * kMaxN + kMaxWarps * kMaxN) * 4 + 16;
constexpr uint32_t kWaitPolls = 1u << 24;  // >= 1 s of polling before a wait gives up

struct LayerParams {
    const void *hidden, *residual, *row_index, *lut, *w_router;
    void *out;
    float *gates_out;
    uint32_t *status;
    long long M, rows;
    int N, d, S, dc;
    uint32_t flags;
};

// Sum N per-thread values over the 32 lanes of a warp with N-1 (+ a few) shuffles instead of
// 5N: every step halves the number of values a lane still carries.  On return a[0..max(1,N/32))
// holds the warp totals of experts base .. base+cnt-1.
template <int NTOT, int n, int o>
__device__ __forceinline__ void warp_reduce_scatter(float (&a)[NTOT], int lane, int &base)
{
    if constexpr (o >= 1) {
        if constexpr (n > 1) {
            constexpr int half = n / 2;
            const bool up = (lane & o) != 0;
#pragma unroll
            for (int i = 0; i < half; ++i) {
                const float send = up ? a[i] : a[i + half];
                const float keep = up ? a[i + half] : a[i];
                a[i] = keep + __shfl_xor_sync(0xffffffffu, send, o);
            }
            if (up) base += half;
            warp_reduce_scatter<NTOT, half, o / 2>(a, lane, base);
        } else {
            a[0] += __shfl_xor_sync(0xffffffffu, a[0], o);
            warp_reduce_scatter<NTOT, 1, o / 2>(a, lane, base);
        }
    }
}

__device__ __forceinline__ float warp_max(float v)
{
#pragma unroll
    for (int o = 16; o >= 1; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}
__device__ __forceinline__ float warp_sum(float v)
{
#pragma unroll
    for (int o = 16; o >= 1; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// T: storage type.  NFAST: compile-time N of the unrolled router (0 = any N <= 64, slower).
// CLUSTER: the S blocks of a token form a cluster; each computes the logits of its own
// column slice and the partial logits are exchanged through distributed shared memory.
// Otherwise every block recomputes the logits over all d columns.
template <typename T, int NFAST, bool CLUSTER>
__global__ void __launch_bounds__(kMaxThreads) mole_layer_kernel(const LayerParams p)
{
    using E = Elem<T>;
    constexpr int VEC = E::VEC;
    extern __shared__ __align__(128) unsigned char smem[];

    pdl_launch_dependents();

    const int N = NFAST > 0 ? NFAST : p.N;
    const int S = p.S, dc = p.dc, d = p.d;
    const long long t = blockIdx.x / S;
    const int s = static_cast<int>(blockIdx.x % S);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, nwarps = blockDim.x >> 5;

    const uint32_t rows_bytes = static_cast<uint32_t>(N) * dc * sizeof(T);
    float *partial = reinterpret_cast<float *>(smem + ((rows_bytes + 15u) & ~15u));
    float *cl_partial = partial + kMaxWarps * kMaxN;
    float *gates = cl_partial + kMaxSplit * kMaxN;
    uint64_t *bar = reinterpret_cast<uint64_t *>(gates + kMaxWarps * kMaxN);

    // ---- 1. start the gather: needs only the id, so it runs ahead of the previous kernel ----
    long long row;
    if (p.flags & MOLE_FLAG_IDS_INT64) row = __ldg(reinterpret_cast<const long long *>(p.row_index) + t);
    else row = __ldg(reinterpret_cast<const int *>(p.row_index) + t);
    const bool valid = row >= 0 && row < p.rows;
    if (tid == 0) {
        mbar_init(bar, 1);
        mbar_init_fence();
        if (valid) {
            mbar_expect_tx(bar, rows_bytes);
            const unsigned char *src = reinterpret_cast<const unsigned char *>(p.lut) +
                                       (static_cast<size_t>(row) * N * d + static_cast<size_t>(s) * dc) * sizeof(T);
            if (S == 1) {
                bulk_g2s(smem, src, rows_bytes, bar);  // the N rows of an id are contiguous
            } else {
                const uint32_t piece = dc * sizeof(T);
                for (int j = 0; j < N; ++j)
                    bulk_g2s(smem + static_cast<size_t>(j) * piece, src + static_cast<size_t>(j) * d * sizeof(T), piece,
                             bar);
            }
        } else if (p.status) {
            atomicOr(p.status, MOLE_STATUS_BAD_ID);
        }
    }

    // ---- 2. hidden is produced by the previous kernel: wait for it -------------------------
    pdl_wait();

    const uint4 *h_vec = reinterpret_cast<const uint4 *>(p.hidden) + t * (d / VEC);
    const int g_begin = CLUSTER ? s * (dc / VEC) : 0;          // 16-byte column groups this block
    const int g_end = CLUSTER ? (s + 1) * (dc / VEC) : d / VEC;  // covers in the router

    int nparts;
    if constexpr (NFAST > 0) {
        float acc[NFAST];
#pragma unroll
        for (int j = 0; j < NFAST; ++j) acc[j] = 0.f;
        for (int grp = g_begin + tid; grp < g_end; grp += blockDim.x) {
            float hf[VEC];
            E::unpack(__ldcg(h_vec + grp), hf);
            // columns grp*VEC .. grp*VEC+VEC-1 of W_r [d][N] are N consecutive 16-byte vectors
            const uint4 *wp = reinterpret_cast<const uint4 *>(p.w_router) + static_cast<size_t>(grp) * NFAST;
#pragma unroll
            for (int k = 0; k < NFAST; ++k) {
                float wf[VEC];
                E::unpack(__ldg(wp + k), wf);
#pragma unroll
                for (int i = 0; i < VEC; ++i) {
                    const int e = k * VEC + i;  // flat element of the VEC x N block
                    acc[e % NFAST] = fmaf(hf[e / NFAST], wf[i], acc[e % NFAST]);
                }
            }
        }
        int base = 0;
        warp_reduce_scatter<NFAST, NFAST, 16>(acc, lane, base);
        constexpr int cnt = NFAST >= 32 ? NFAST / 32 : 1;
#pragma unroll
        for (int i = 0; i < cnt; ++i) partial[warp * kMaxN + base + i] = acc[i];
        nparts = nwarps;
    } else {
        // any N: one warp per expert, lanes stride over the columns
        const int c_begin = g_begin * VEC, c_end = g_end * VEC;
        for (int j = warp; j < N; j += nwarps) {
            float z = 0.f;
            for (int c = c_begin + lane; c < c_end; c += 32)
                z = fmaf(E::scalar_cg(p.hidden, t * d + c), E::scalar(p.w_router, static_cast<long long>(c) * N + j), z);
            z = warp_sum(z);
            if (lane == 0) partial[j] = z;
        }
        nparts = 1;
    }
    __syncthreads();

    // ---- 3. logits -> softmax over all N experts (every warp keeps its own copy) ------------
    const int j0 = lane, j1 = lane + 32;
    float z0 = -INFINITY, z1 = -INFINITY;
    if constexpr (CLUSTER) {
        if (warp == 0) {
            const uint32_t my_slot = smem_u32(cl_partial + s * kMaxN);
            for (int j = lane; j < N; j += 32) {
                float zc = 0.f;
                for (int w = 0; w < nparts; ++w) zc += partial[w * kMaxN + j];
                for (int peer = 0; peer < S; ++peer) st_cluster_f32(my_slot + j * 4, peer, zc);
            }
        }
        cluster_arrive_release();
        cluster_wait_acquire();
        if (j0 < N) {
            z0 = 0.f;
            for (int q = 0; q < S; ++q) z0 += cl_partial[q * kMaxN + j0];
        }
        if (j1 < N) {
            z1 = 0.f;
            for (int q = 0; q < S; ++q) z1 += cl_partial[q * kMaxN + j1];
        }
    } else {
        if (j0 < N) {
            z0 = 0.f;
            for (int w = 0; w < nparts; ++w) z0 += partial[w * kMaxN + j0];
        }
        if (j1 < N) {
            z1 = 0.f;
            for (int w = 0; w < nparts; ++w) z1 += partial[w * kMaxN + j1];
        }
    }
    const float zmax = warp_max(fmaxf(z0, z1));
    const float e0 = j0 < N ? expf(z0 - zmax) : 0.f;
    const float e1 = j1 < N ? expf(z1 - zmax) : 0.f;
    const float esum = warp_sum(e0 + e1);
    float *my_gates = gates + warp * kMaxN;
    if (j0 < N) my_gates[j0] = e0 / esum;
    if (j1 < N) my_gates[j1] = e1 / esum;
    if (p.gates_out && s == 0 && warp == 0) {
        if (j0 < N) p.gates_out[t * N + j0] = e0 / esum;
        if (j1 < N) p.gates_out[t * N + j1] = e1 / esum;
    }
    __syncwarp();

    // ---- 4. rows must have landed ------------------------------------------------------------
    if (valid && !mbar_wait_bounded(bar, 0, kWaitPolls)) {
        if (tid == 0 && p.status) atomicOr(p.status, MOLE_STATUS_TIMEOUT);
        (void)mbar_wait_bounded(bar, 0, kWaitPolls);  // give copies still in flight a last chance to land
        return;
    }

    // ---- 5. weighted sum over the experts, residual add, one rounding at the store ----------
    const uint4 *res_vec = reinterpret_cast<const uint4 *>(p.residual ? p.residual : p.hidden) + t * (d / VEC) +
                           s * (dc / VEC);
    uint4 *out_vec = reinterpret_cast<uint4 *>(p.out) + t * (d / VEC) + s * (dc / VEC);
    const uint4 *rows_vec = reinterpret_cast<const uint4 *>(smem);
    const int ngrp = dc / VEC;
    for (int grp = tid; grp < ngrp; grp += blockDim.x) {
        float acc[VEC];
#pragma unroll
        for (int i = 0; i < VEC; ++i) acc[i] = 0.f;
        if (valid) {
#pragma unroll 4
            for (int j = 0; j < N; ++j) {
                float vf[VEC];
                E::unpack(rows_vec[j * ngrp + grp], vf);
                const float g = my_gates[j];
#pragma unroll
                for (int i = 0; i < VEC; ++i) acc[i] = fmaf(g, vf[i], acc[i]);
            }
        }
        float rf[VEC];
        E::unpack(__ldcg(res_vec + grp), rf);
#pragma unroll
        for (int i = 0; i < VEC; ++i) acc[i] = rf[i] + acc[i];
        out_vec[grp] = E::pack(acc);
    }
}

// ---- host side ---------------------------------------------------------------------------------

static thread_local char g_cuda_error[256] = "";

void set_cuda_error(cudaError_t e)
{
    const char *s = cudaGetErrorString(e);
    strncpy(g_cuda_error, s ? s : "unknown CUDA error", sizeof(g_cuda_error) - 1);
    g_cuda_error[sizeof(g_cuda_error) - 1] = 0;
    (void)cudaGetLastError();  // clear the sticky-less error so that later calls start clean
}

static int round_up(int a, int b) { return (a + b - 1) / b * b; }

int plan_layer(long long M, int N, int d, int dtype, int variant, int d_split, LayerPlan *plan)
{
    if (dtype != MOLE_DTYPE_BF16 && dtype != MOLE_DTYPE_F32) return MOLE_ERR_INVALID_ARG;
    if (variant < MOLE_VARIANT_AUTO || variant > MOLE_VARIANT_CLUSTER) return MOLE_ERR_INVALID_ARG;
    const int eb = elem_bytes(dtype), vec = 16 / eb;
    if (N < 1 || N > kMaxN || d < vec || d % vec != 0) return MOLE_ERR_UNSUPPORTED_SHAPE;
    const int max_smem = 227 * 1024;
    int S;
    if (d_split != 0) {
        if (d_split != 1 && d_split != 2 && d_split != 4 && d_split != 8) return MOLE_ERR_INVALID_ARG;
        if (d % (d_split * vec) != 0) return MOLE_ERR_UNSUPPORTED_SHAPE;
        S = d_split;
    } else {
        // Split a token over more blocks while (a) one block's rows would not leave room for
        // several blocks per SM, or (b) there are too few tokens to occupy the 148 SMs twice
        // over; stop when a row piece would drop under 512 bytes.
        S = 1;
        while (S < kMaxSplit && d % (2 * S * vec) == 0 && (d / (2 * S)) * eb >= 512 &&
               (static_cast<long long>(N) * (d / S) * eb > 32 * 1024 || M * S < 2 * 148))
            S *= 2;
    }
    while (static_cast<long long>(N) * (d / S) * eb + kFixedSmem > max_smem) {
        if (d_split != 0 || S >= kMaxSplit || d % (2 * S * vec) != 0) return MOLE_ERR_UNSUPPORTED_SHAPE;
        S *= 2;
    }
    plan->d_split = S;
    plan->dc = d / S;
    plan->variant = (S == 1) ? MOLE_VARIANT_REPLICATE : (variant == MOLE_VARIANT_AUTO ? MOLE_VARIANT_CLUSTER : variant);
    const int groups = (plan->variant == MOLE_VARIANT_CLUSTER ? plan->dc : d) / vec;
    plan->threads = round_up(groups < kMaxThreads ? groups : kMaxThreads, 32);
    plan->smem = round_up(N * plan->dc * eb, 16) + kFixedSmem;
    plan->n_fast = (N == 4 || N == 8 || N == 16 || N == 32 || N == 64) ? N : 0;
    return MOLE_OK;
}

typedef void (*LayerKernel)(const LayerParams);

template <typename T, bool CLUSTER>
static LayerKernel pick_n(int n_fast)
{
    switch (n_fast) {
        case 4: return mole_layer_kernel<T, 4, CLUSTER>;
        case 8: return mole_layer_kernel<T, 8, CLUSTER>;
        case 16: return mole_layer_kernel<T, 16, CLUSTER>;
        case 32: return mole_layer_kernel<T, 32, CLUSTER>;
        case 64: return mole_layer_kernel<T, 64, CLUSTER>;
        default: return mole_layer_kernel<T, 0, CLUSTER>;
    }
}

static LayerKernel pick_kernel(int dtype, int n_fast, bool cluster)
{
    if (dtype == MOLE_DTYPE_BF16) return cluster ? pick_n<__nv_bfloat16, true>(n_fast) : pick_n<__nv_bfloat16, false>(n_fast);
    return cluster ? pick_n<float, true>(n_fast) : pick_n<float, false>(n_fast);
}

// Kernels that need more than 48 KB of dynamic shared memory must opt in once per device.
static int ensure_smem(LayerKernel k, int smem)
{
    if (smem <= 48 * 1024) return MOLE_OK;
    struct Slot {
        std::atomic<const void *> fn{nullptr};
        std::atomic<int> dev{-1};
        std::atomic<int> bytes{0};
    };
    static Slot slots[128];
    int dev = 0;
    MOLE_CUDA_TRY(cudaGetDevice(&dev));
    const void *fn = reinterpret_cast<const void *>(k);
    for (auto &sl : slots) {
        if (sl.fn.load() == fn && sl.dev.load() == dev && sl.bytes.load() >= smem) return MOLE_OK;
    }
    MOLE_CUDA_TRY(cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
    for (auto &sl : slots) {
        const void *expect = nullptr;
        if (sl.fn.load() == fn && sl.dev.load() == dev) {
            sl.bytes.store(smem);
            break;
        }
        if (sl.fn.compare_exchange_strong(expect, fn)) {
            sl.dev.store(dev);
            sl.bytes.store(smem);
            break;
        }
    }
    return MOLE_OK;
}

int launch_layer(const LayerLaunch &a)
{
    if (a.M == 0) return MOLE_OK;
    LayerPlan plan;
    int rc = plan_layer(a.M, a.N, a.d, a.dtype, a.variant, a.d_split, &plan);
    if (rc != MOLE_OK) return rc;
    if (a.M * plan.d_split > 0x7fffffffLL) return MOLE_ERR_TOO_LARGE;
    const bool cluster = plan.variant == MOLE_VARIANT_CLUSTER;
    // In place (out == hidden) with replicated routers would let one block overwrite columns
    // another block of the same token still has to read for its router.
    if (!cluster && plan.d_split > 1 && a.out == a.hidden) return MOLE_ERR_INVALID_ARG;

    LayerParams p;
    p.hidden = a.hidden;
    p.residual = a.residual;
    p.row_index = a.row_index;
    p.lut = a.lut;
    p.w_router = a.w_router;
    p.out = a.out;
    p.gates_out = a.gates_out;
    p.status = a.status;
    p.M = a.M;
    p.rows = a.rows;
    p.N = a.N;
    p.d = a.d;
    p.S = plan.d_split;
    p.dc = plan.dc;
    p.flags = a.flags;

    LayerKernel k = pick_kernel(a.dtype, plan.n_fast, cluster);
    rc = ensure_smem(k, plan.smem);
    if (rc != MOLE_OK) return rc;

    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof cfg);
    cfg.gridDim = dim3(static_cast<unsigned>(a.M * plan.d_split), 1, 1);
    cfg.blockDim = dim3(plan.threads, 1, 1);
    cfg.dynamicSmemBytes = plan.smem;
    cfg.stream = a.stream;
    cudaLaunchAttribute attrs[2];
    unsigned na = 0;
    if (a.flags & MOLE_FLAG_CHAIN) {
        attrs[na].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attrs[na].val.programmaticStreamSerializationAllowed = 1;
        ++na;
    }
    if (cluster) {
        attrs[na].id = cudaLaunchAttributeClusterDimension;
        attrs[na].val.clusterDim.x = plan.d_split;
        attrs[na].val.clusterDim.y = 1;
        attrs[na].val.clusterDim.z = 1;
        ++na;
    }
    cfg.attrs = attrs;
    cfg.numAttrs = na;
    MOLE_CUDA_TRY(cudaLaunchKernelEx(&cfg, k, p));
    return MOLE_OK;
}

static int check_common(const void *hidden, const void *ids, const void *lut, const void *w_router, const void *out,
                        const void *residual, int B, int T, int N, int d, int V, int dtype)
{
    if (dtype != MOLE_DTYPE_BF16 && dtype != MOLE_DTYPE_F32) return MOLE_ERR_INVALID_ARG;
    if (B < 0 || T < 0) return MOLE_ERR_INVALID_ARG;
    const int vec = 16 / elem_bytes(dtype);
    if (N < 1 || N > kMaxN || V < 1 || d < vec || d % vec != 0) return MOLE_ERR_UNSUPPORTED_SHAPE;
    if (static_cast<long long>(B) * T == 0) return MOLE_OK;
    if (!hidden || !ids || !lut || !w_router || !out) return MOLE_ERR_INVALID_ARG;
    if (!aligned16(hidden) || !aligned16(lut) || !aligned16(w_router) || !aligned16(out)) return MOLE_ERR_INVALID_ARG;
    if (residual && !aligned16(residual)) return MOLE_ERR_INVALID_ARG;
    return MOLE_OK;
}

}  // namespace mole

using namespace mole;

extern "C" {

int mole_layer_forward_ex(const mole_args *a)
{
    if (!a || a->struct_size != sizeof(mole_args)) return MOLE_ERR_INVALID_ARG;
    if (a->flags & ~(MOLE_FLAG_IDS_INT64 | MOLE_FLAG_CHAIN)) return MOLE_ERR_INVALID_ARG;
    int rc = check_common(a->hidden, a->ids, a->lut, a->w_router, a->out, a->residual, a->B, a->T, a->N, a->d, a->V,
                          a->dtype);
    if (rc != MOLE_OK) return rc;
    const uintptr_t id_align = (a->flags & MOLE_FLAG_IDS_INT64) ? 7u : 3u;
    if (reinterpret_cast<uintptr_t>(a->ids) & id_align) return MOLE_ERR_INVALID_ARG;
    if (a->residual && a->residual != a->hidden && a->residual == a->out) return MOLE_ERR_INVALID_ARG;
    LayerLaunch L;
    L.hidden = a->hidden;
    L.residual = a->residual;
    L.row_index = a->ids;
    L.lut = a->lut;
    L.w_router = a->w_router;
    L.out = a->out;
    L.gates_out = a->gates_out;
    L.status = a->status;
    L.M = static_cast<long long>(a->B) * a->T;
    L.N = a->N;
    L.d = a->d;
    L.rows = a->V;
    L.dtype = a->dtype;
    L.flags = a->flags;
    L.variant = a->variant;
    L.d_split = a->d_split;
    L.stream = static_cast<cudaStream_t>(a->stream);
    return launch_layer(L);
}

int mole_layer_forward(const void *hidden, const int32_t *ids, const void *lut, const void *w_router, void *out, int B,
                       int T, int N, int d, int V, void *stream)
{
    mole_args a;
    memset(&a, 0, sizeof a);
    a.struct_size = sizeof a;
    a.hidden = hidden;
    a.ids = ids;
    a.lut = lut;
    a.w_router = w_router;
    a.out = out;
    a.B = B;
    a.T = T;
    a.N = N;
    a.d = d;
    a.V = V;
    a.dtype = MOLE_DTYPE_BF16;
    a.stream = stream;
    return mole_layer_forward_ex(&a);
}

int mole_decode_step(const void *hidden_in, const int32_t *ids, const void *lut_base, int64_t lut_layer_stride_bytes,
                     const void *w_router_base, int64_t wr_layer_stride_bytes, void *out, void *tmp, uint32_t *status,
                     int L, int B, int T, int N, int d, int V, int dtype, void *stream)
{
    if (L < 1) return MOLE_ERR_INVALID_ARG;
    int rc = check_common(hidden_in, ids, lut_base, w_router_base, out, nullptr, B, T, N, d, V, dtype);
    if (rc != MOLE_OK) return rc;
    if (static_cast<long long>(B) * T == 0) return MOLE_OK;
    if ((lut_layer_stride_bytes & 15) || (wr_layer_stride_bytes & 15)) return MOLE_ERR_INVALID_ARG;
    if (L > 1 && (!tmp || !aligned16(tmp) || out == hidden_in || tmp == hidden_in || tmp == out))
        return MOLE_ERR_INVALID_ARG;
    // ping-pong so that the last layer writes `out` and hidden_in is never written
    const void *src = hidden_in;
    for (int l = 0; l < L; ++l) {
        void *dst = ((L - 1 - l) % 2 == 0) ? out : tmp;
        LayerLaunch a;
        a.hidden = src;
        a.residual = nullptr;
        a.row_index = ids;
        a.lut = static_cast<const unsigned char *>(lut_base) + static_cast<int64_t>(l) * lut_layer_stride_bytes;
        a.w_router = static_cast<const unsigned char *>(w_router_base) + static_cast<int64_t>(l) * wr_layer_stride_bytes;
        a.out = dst;
        a.gates_out = nullptr;
        a.status = status;
        a.M = static_cast<long long>(B) * T;
        a.N = N;
        a.d = d;
        a.rows = V;
        a.dtype = dtype;
        a.flags = MOLE_FLAG_CHAIN;
        a.variant = MOLE_VARIANT_AUTO;
        a.d_split = 0;
        a.stream = static_cast<cudaStream_t>(stream);
        rc = launch_layer(a);
        if (rc != MOLE_OK) return rc;
        src = dst;
    }
    return MOLE_OK;
}

int mole_decode_step_host(const void *hidden_host, const int32_t *ids_host, void *out_host, void *dev_hidden,
                          int32_t *dev_ids, void *dev_out, void *dev_tmp, const void *lut_base,
                          int64_t lut_layer_stride_bytes, const void *w_router_base, int64_t wr_layer_stride_bytes,
                          uint32_t *status, int L, int B, int T, int N, int d, int V, int dtype, void *stream)
{
    if (B < 0 || T < 0 || (dtype != MOLE_DTYPE_BF16 && dtype != MOLE_DTYPE_F32)) return MOLE_ERR_INVALID_ARG;
    const long long M = static_cast<long long>(B) * T;
    if (M == 0) return MOLE_OK;
    if (!hidden_host || !ids_host || !out_host || !dev_hidden || !dev_ids || !dev_out) return MOLE_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const size_t act_bytes = static_cast<size_t>(M) * d * elem_bytes(dtype);
    MOLE_CUDA_TRY(cudaMemcpyAsync(dev_ids, ids_host, static_cast<size_t>(M) * sizeof(int32_t), cudaMemcpyHostToDevice, st));
    MOLE_CUDA_TRY(cudaMemcpyAsync(dev_hidden, hidden_host, act_bytes, cudaMemcpyHostToDevice, st));
    int rc = mole_decode_step(dev_hidden, dev_ids, lut_base, lut_layer_stride_bytes, w_router_base, wr_layer_stride_bytes,
                              dev_out, dev_tmp, status, L, B, T, N, d, V, dtype, stream);
    if (rc != MOLE_OK) return rc;
    MOLE_CUDA_TRY(cudaMemcpyAsync(out_host, dev_out, act_bytes, cudaMemcpyDeviceToHost, st));
    return MOLE_OK;
}

int mole_plan(int M, int N, int d, int dtype, int variant, int d_split, int *out_d_split, int *out_threads,
              int *out_smem_bytes, int *out_variant)
{
    LayerPlan plan;
    int rc = plan_layer(M, N, d, dtype, variant, d_split, &plan);
    if (rc != MOLE_OK) return rc;
    if (out_d_split) *out_d_split = plan.d_split;
    if (out_threads) *out_threads = plan.threads;
    if (out_smem_bytes) *out_smem_bytes = plan.smem;
    if (out_variant) *out_variant = plan.variant;
    return MOLE_OK;
}

const char *mole_status_string(int code)
{
    switch (code) {
        case MOLE_OK: return "ok";
        case MOLE_ERR_INVALID_ARG: return "invalid argument";
        case MOLE_ERR_UNSUPPORTED_SHAPE: return "unsupported shape";
        case MOLE_ERR_CUDA: return "CUDA runtime error";
        case MOLE_ERR_NOMEM: return "out of memory";
        case MOLE_ERR_TOO_LARGE: return "size beyond the stated maximum";
        default: return "unknown status";
    }
}

const char *mole_last_cuda_error(void) { return g_cuda_error; }

int mole_version(void) { return MOLE_VERSION; }

}  // extern "C"
