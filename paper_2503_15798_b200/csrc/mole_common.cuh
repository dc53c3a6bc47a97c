// Shared device helpers and host-side error plumbing of the MoLE sm_100a library.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "mole.h"

namespace mole {

// ---- host side -----------------------------------------------------------------------------
void set_cuda_error(cudaError_t e);  // remembers the text for mole_last_cuda_error()

#define MOLE_CUDA_TRY(expr)                       \
    do {                                          \
        cudaError_t e__ = (expr);                 \
        if (e__ != cudaSuccess) {                 \
            ::mole::set_cuda_error(e__);          \
            return MOLE_ERR_CUDA;                 \
        }                                         \
    } while (0)

inline bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
inline int elem_bytes(int dtype) { return dtype == MOLE_DTYPE_BF16 ? 2 : 4; }

// Launch description of the fused kernel (filled by plan_step, pure host arithmetic).
// A block owns whole tokens; it walks over its tokens and, for every token, over the L layers,
// pulling the router matrix (when it streams) and the table rows of each (token, layer) item, cut
// into d_split chunks, through a ring of `stages` shared-memory slots.
struct StepPlan {
    int d_split;        // chunks per item (of the router matrix, and of the rows)
    int dc;             // columns per router chunk (and per rows chunk when the rows are cut by columns)
    int consumers;      // threads that compute (a multiple of 32); one more warp issues the copies
    int threads;        // consumers + 32
    int stages;         // ring depth, in chunks
    int hring;          // hidden states of tokens in flight
    int slot_bytes;     // one ring slot
    int wr_in_ring;     // 1: the router chunks travel through the ring; 0: router matrix loaded once per block
    int smem;           // dynamic shared memory, bytes
    int blocks_per_sm;  // resident blocks per SM the shared memory allows
    int n_fast;         // N if the unrolled router path exists for it, else 0
    int rows_by_expert; // several chunks per item: 1 = the rows are cut by experts, 0 = by columns
    int lanes;          // combine: lanes per 16-byte column group (by columns) or column groups per lane (by experts)
};
// `by_columns`: never cut the rows by experts (kernel variants that exist for the column cut only)
// `sms`: SM count the plan is laid out for (< 1: the nominal 148 of a B200); `norm`: room for RMSNorm(hidden)
int plan_step(long long M, int L, int N, int d, int dtype, int d_split, StepPlan *plan, bool by_columns = false, int sms = 0,
              bool norm = false);

// One launch of the fused kernel over L chained layers (L == 1: a single layer).
// `row_index` is ids (resident mode) or slot (offload mode); `rows` the number of table rows
// that may be addressed.
struct StepLaunch {
    const void *hidden, *residual, *row_index, *lut, *w_router;
    void *out;
    float *gates_out;
    uint32_t *status;
    long long lut_stride, wr_stride;  // bytes between consecutive layers
    long long M;
    int L, N, d;
    long long rows;
    int dtype;
    uint32_t flags;
    int d_split;
    cudaStream_t stream;
    const void *norm_weight = nullptr;  // [d], dtype: the router reads RMSNorm(hidden); NULL: hidden itself
    long long norm_stride = 0;          // bytes between the scale vectors of consecutive layers
    float norm_eps = 0.f;
    int kernel = 0;  // MOLE_KERNEL_*: which kernel family runs the launch (0: the library's choice)
};
int launch_step(const StepLaunch &a);

// kernels that need more than 48 KB of dynamic shared memory opt in once per device
int ensure_smem_opt_in(const void *fn, int smem);
int sm_count(int *out, int *dev_out = nullptr);  // SM count of the current device, asked once per device
// poll limit of the bounded device-side waits (the default unless a debugging variable shortens it)
uint32_t current_wait_polls();

// the fused layer over a quantised table (mole_quant.cu): single layer, bf16 activations
bool quant_layer_shape_ok(int N, int d, int format, int block);
const char *quant_variant_name(int N, int format, bool norm);
int launch_quant_layer(const StepLaunch &a, int format, int block, uint32_t wait_polls);

#ifdef __CUDACC__
// ---- device side ---------------------------------------------------------------------------

__device__ __forceinline__ uint32_t smem_u32(const void *p)
{
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

// mbarrier + bulk-copy (TMA, untiled, each copy into this block's own shared memory only) primitives
__device__ __forceinline__ void mbar_init(uint64_t *bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_init_fence()
{
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t *bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes)
                 : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t *bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}
// Global -> this block's shared memory; both addresses 16-byte aligned, bytes a multiple of 16.
__device__ __forceinline__ void bulk_g2s(void *dst_smem, const void *src_gmem, uint32_t bytes, uint64_t *bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                     smem_u32(dst_smem)),
                 "l"(src_gmem), "r"(bytes), "r"(smem_u32(bar))
                 : "memory");
}

// Ask L2 for a span of global memory (no destination, no completion to wait for); address 16-byte aligned,
// bytes a multiple of 16.
__device__ __forceinline__ void bulk_prefetch_l2(const void *src_gmem, uint32_t bytes)
{
    asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(src_gmem), "r"(bytes) : "memory");
}

// Bounded wait on a bulk-copy barrier.  Returns false if the data never arrived.
__device__ __forceinline__ bool mbar_wait_bounded(uint64_t *bar, uint32_t parity, uint32_t max_polls)
{
    for (uint32_t i = 0; i < max_polls; ++i) {
        if (mbar_try_wait(bar, parity)) return true;
        if (i > 64) __nanosleep(64);
    }
    return false;
}

__device__ __forceinline__ void mbar_arrive(uint64_t *bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
// Barrier over a subset of the block's warps (id 1..15, count a multiple of 32).
__device__ __forceinline__ void named_bar_sync(int id, int count)
{
    asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(count) : "memory");
}
// Count this warp in at a named barrier without waiting for it.
__device__ __forceinline__ void named_bar_arrive(int id, int count)
{
    asm volatile("bar.arrive %0, %1;" ::"r"(id), "r"(count) : "memory");
}
__device__ __forceinline__ void fence_proxy_async_global() { asm volatile("fence.proxy.async.global;" ::: "memory"); }

// programmatic dependent launch
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

// Explicit shared-space accesses (32-bit shared addresses): the hot loops index slots of the
// ring through run-time offsets, and these keep every access on the shared-memory path.
__device__ __forceinline__ uint4 lds128(uint32_t a)
{
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(a));
    return v;
}
__device__ __forceinline__ uint2 lds64(uint32_t a)
{
    uint2 v;
    asm volatile("ld.shared.v2.u32 {%0, %1}, [%2];" : "=r"(v.x), "=r"(v.y) : "r"(a));
    return v;
}
__device__ __forceinline__ uint32_t lds32(uint32_t a)
{
    uint32_t v;
    asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(a));
    return v;
}
__device__ __forceinline__ uint32_t lds16(uint32_t a)
{
    unsigned short v;
    asm volatile("ld.shared.u16 %0, [%1];" : "=h"(v) : "r"(a));
    return v;
}
__device__ __forceinline__ void sts128(uint32_t a, const uint4 &v)
{
    asm volatile("st.shared.v4.u32 [%0], {%1, %2, %3, %4};" ::"r"(a), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}
__device__ __forceinline__ void sts64(uint32_t a, const uint2 &v)
{
    asm volatile("st.shared.v2.u32 [%0], {%1, %2};" ::"r"(a), "r"(v.x), "r"(v.y) : "memory");
}
__device__ __forceinline__ void sts32(uint32_t a, uint32_t v)
{
    asm volatile("st.shared.u32 [%0], %1;" ::"r"(a), "r"(v) : "memory");
}

// 16-byte vectors of the two storage types
template <typename T>
struct Elem;
template <>
struct Elem<__nv_bfloat16> {
    static constexpr int VEC = 8;
    static __device__ __forceinline__ void unpack(const uint4 &v, float (&f)[8])
    {
        f[0] = __uint_as_float(v.x << 16);
        f[1] = __uint_as_float(v.x & 0xffff0000u);
        f[2] = __uint_as_float(v.y << 16);
        f[3] = __uint_as_float(v.y & 0xffff0000u);
        f[4] = __uint_as_float(v.z << 16);
        f[5] = __uint_as_float(v.z & 0xffff0000u);
        f[6] = __uint_as_float(v.w << 16);
        f[7] = __uint_as_float(v.w & 0xffff0000u);
    }
    // acc[0..7] += g * (the 8 values of v): the weighted sum's inner step.  Two values per instruction on the
    // packed fp32 pipe (fma.rn.f32x2: two independent IEEE fmas, the same bits as eight fmaf).
    static __device__ __forceinline__ void fma_row(float (&acc)[8], const uint4 &v, float g)
    {
        const float2 g2 = make_float2(g, g);
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const float2 r = __ffma2_rn(g2, make_float2(__uint_as_float(w[k] << 16), __uint_as_float(w[k] & 0xffff0000u)),
                                        make_float2(acc[2 * k], acc[2 * k + 1]));
            acc[2 * k] = r.x;
            acc[2 * k + 1] = r.y;
        }
    }
    // element i of an array in shared memory (32-bit shared address)
    static __device__ __forceinline__ float lds_scalar(uint32_t base, int i) { return __uint_as_float(lds16(base + 2 * i) << 16); }
    // the same element as a raw 16-bit operand of the mixed-precision fma below
    typedef unsigned short H;
    static __device__ __forceinline__ H lds_h(uint32_t base, int i)
    {
        unsigned short v;
        asm volatile("ld.shared.u16 %0, [%1];" : "=h"(v) : "r"(base + 2u * i));
        return v;
    }
    // acc[e] += v[e] * h for the 8 values of a vector, through sm_100's mixed-precision fma
    // (fma.rn.f32.bf16: bf16 x bf16 products are exact in fp32, one rounding at the add -- the
    // same result as widening both operands and calling fmaf, without the widening instructions)
    static __device__ __forceinline__ void fma_elem(float &acc, const uint4 &v, int e, H h)
    {
        const uint32_t w = e < 2 ? v.x : (e < 4 ? v.y : (e < 6 ? v.z : v.w));
        unsigned short lo, hi;
        asm("mov.b32 {%0, %1}, %2;" : "=h"(lo), "=h"(hi) : "r"(w));
        asm("fma.rn.f32.bf16 %0, %1, %2, %0;" : "+f"(acc) : "h"((e & 1) ? hi : lo), "h"(h));
    }
};
template <>
struct Elem<float> {
    static constexpr int VEC = 4;
    static __device__ __forceinline__ void unpack(const uint4 &v, float (&f)[4])
    {
        f[0] = __uint_as_float(v.x);
        f[1] = __uint_as_float(v.y);
        f[2] = __uint_as_float(v.z);
        f[3] = __uint_as_float(v.w);
    }
    static __device__ __forceinline__ void fma_row(float (&acc)[4], const uint4 &v, float g)
    {
        acc[0] = fmaf(g, __uint_as_float(v.x), acc[0]);
        acc[1] = fmaf(g, __uint_as_float(v.y), acc[1]);
        acc[2] = fmaf(g, __uint_as_float(v.z), acc[2]);
        acc[3] = fmaf(g, __uint_as_float(v.w), acc[3]);
    }
    static __device__ __forceinline__ float lds_scalar(uint32_t base, int i) { return __uint_as_float(lds32(base + 4 * i)); }
    typedef float H;
    static __device__ __forceinline__ H lds_h(uint32_t base, int i) { return __uint_as_float(lds32(base + 4 * i)); }
    static __device__ __forceinline__ void fma_elem(float &acc, const uint4 &v, int e, H h)
    {
        const uint32_t w = e == 0 ? v.x : (e == 1 ? v.y : (e == 2 ? v.z : v.w));
        acc = fmaf(h, __uint_as_float(w), acc);
    }
};
#endif  // __CUDACC__

}  // namespace mole
