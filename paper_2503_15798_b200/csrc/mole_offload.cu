// Offload mode of the MoLE layer: the table stays in pinned host memory (the paper keeps the
// re-parameterised table on a storage device and moves only the looked-up rows, Sec. 3.3);
// per step the distinct ids are found on the device, their rows are read across the host
// link by the GPU itself into a dense staging buffer, and the fused layer gathers from there.
#include <mutex>
#include <new>
#include <string.h>

#include "mole_common.cuh"

namespace mole {

constexpr int kDedupThreads = 1024;
constexpr int kFetchThreads = 256;
constexpr int kFetchVecPerThread = 4;  // 16-byte loads in flight per thread
constexpr int kFetchChunk = kFetchThreads * kFetchVecPerThread * 16;

// Distinct ids of a step, one thread block.  table[V] is all zero on entry and on exit.
//  1. table[id] = max over the id's tokens of (M - t): the first occurrence wins.
//  2. tokens that won are the representatives; an ordered block scan numbers them, so uniq
//     comes out in order of first occurrence and the result does not depend on timing.
//  3. every token copies its representative's number; representatives clear their table entry.
__global__ void __launch_bounds__(kDedupThreads) mole_dedup_kernel(const int32_t *__restrict__ ids, int M, int V,
                                                                   int32_t *table, int32_t *uniq, int32_t *slot,
                                                                   int32_t *count, uint32_t *status)
{
    __shared__ int warp_tot[kDedupThreads / 32];
    __shared__ int total;
    const int tid = threadIdx.x, nt = blockDim.x;
    const int per = (M + nt - 1) / nt;  // contiguous run of tokens per thread
    const int t0 = min(tid * per, M), t1 = min(t0 + per, M);
    bool bad = false;

    for (int t = t0; t < t1; ++t) {
        const int id = ids[t];
        if (id >= 0 && id < V) atomicMax(&table[id], M - t);
        else bad = true;
    }
    __syncthreads();

    int mine = 0;
    for (int t = t0; t < t1; ++t) {
        const int id = ids[t];
        if (id >= 0 && id < V && table[id] == M - t) ++mine;
    }
    // exclusive scan of `mine` over the block
    const int lane = tid & 31, warp = tid >> 5;
    int incl = mine;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int v = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += v;
    }
    if (lane == 31) warp_tot[warp] = incl;
    __syncthreads();
    if (warp == 0) {
        int w = (lane < nt / 32) ? warp_tot[lane] : 0;
        int wi = w;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int v = __shfl_up_sync(0xffffffffu, wi, o);
            if (lane >= o) wi += v;
        }
        if (lane < nt / 32) warp_tot[lane] = wi - w;
        if (lane == 31) total = wi;
    }
    __syncthreads();
    int pos = warp_tot[warp] + incl - mine;
    for (int t = t0; t < t1; ++t) {
        const int id = ids[t];
        if (id >= 0 && id < V && table[id] == M - t) {
            uniq[pos] = id;
            slot[t] = pos;
            ++pos;
        }
    }
    __syncthreads();
    for (int t = t0; t < t1; ++t) {
        const int id = ids[t];
        if (id >= 0 && id < V) {
            const int rep = M - table[id];
            if (rep != t) slot[t] = slot[rep];
        } else {
            slot[t] = -1;
        }
    }
    __syncthreads();
    for (int t = t0; t < t1; ++t) {
        const int id = ids[t];
        if (id >= 0 && id < V && table[id] == M - t) table[id] = 0;
    }
    if (tid == 0) *count = total;
    if (bad && status) atomicOr(status, MOLE_STATUS_BAD_ID);
}

// staging[z][u] = table_host[z][uniq[u]] for u < *count.  blockIdx.y = u, blockIdx.x = 16 KB chunk
// of the row, blockIdx.z = z, one of several layers' tables (table_stride bytes apart on the host,
// staging_stride bytes apart in the staging area) fetched for the same ids in one launch.  All of
// a thread's loads are issued before its first store so that many reads are in flight on the host link.
// Hot rows: ids with hot_slot[id] >= 0 have their rows of every layer cached in device memory
// (hot_base[(hot_layer0 + z) * hot_rows + hot_slot[id]]); those are copied from there and never touch
// the host link.
struct HotRows {
    const int32_t *slot;        // [V] position in the cache or -1; NULL: no cache
    const unsigned char *base;  // [layers][rows][row_bytes]
    long long rows;
    int layer0;                 // cache layer of this launch's z = 0
    unsigned long long *hits;   // rows served from the cache (one count per row and layer), or NULL
};
__global__ void __launch_bounds__(kFetchThreads) mole_fetch_kernel(const unsigned char *__restrict__ table_host,
                                                                   const int32_t *__restrict__ uniq,
                                                                   const int32_t *__restrict__ count, long long row_bytes,
                                                                   unsigned char *__restrict__ staging, long long table_stride,
                                                                   long long staging_stride, const HotRows hot)
{
    const int u = blockIdx.y;
    if (u >= *count) return;
    const long long row = uniq[u];
    const long long chunk0 = static_cast<long long>(blockIdx.x) * kFetchChunk;
    const long long z = blockIdx.z;
    const unsigned char *from = table_host + z * table_stride + row * row_bytes;
    if (hot.slot) {
        const int hs = hot.slot[row];
        if (hs >= 0) {
            from = hot.base + ((hot.layer0 + z) * hot.rows + hs) * row_bytes;
            if (hot.hits && blockIdx.x == 0 && threadIdx.x == 0) atomicAdd(hot.hits, 1ull);
        }
    }
    const uint4 *src = reinterpret_cast<const uint4 *>(from + chunk0);
    uint4 *dst = reinterpret_cast<uint4 *>(staging + z * staging_stride + static_cast<long long>(u) * row_bytes + chunk0);
    const long long nvec = min(static_cast<long long>(kFetchChunk), row_bytes - chunk0) / 16;
    uint4 v[kFetchVecPerThread];
#pragma unroll
    for (int k = 0; k < kFetchVecPerThread; ++k) {
        const long long i = static_cast<long long>(k) * kFetchThreads + threadIdx.x;
        if (i < nvec) v[k] = __ldcs(src + i);
    }
#pragma unroll
    for (int k = 0; k < kFetchVecPerThread; ++k) {
        const long long i = static_cast<long long>(k) * kFetchThreads + threadIdx.x;
        if (i < nvec) dst[i] = v[k];
    }
}

static int launch_dedup(const int32_t *ids, int M, int V, int32_t *scratch, int32_t *uniq, int32_t *slot, int32_t *count,
                        uint32_t *status, cudaStream_t st)
{
    mole_dedup_kernel<<<1, kDedupThreads, 0, st>>>(ids, M, V, scratch, uniq, slot, count, status);
    MOLE_CUDA_TRY(cudaGetLastError());
    return MOLE_OK;
}

// Device alias of a pinned host allocation; the last answer is remembered per thread (a decoding loop asks
// for the same table again and again).
static int device_alias(const void *host, const unsigned char **out)
{
    thread_local const void *last_host = nullptr;
    thread_local const unsigned char *last_dev = nullptr;
    thread_local int last_device = -1;
    int dev = 0;
    MOLE_CUDA_TRY(cudaGetDevice(&dev));
    if (host == last_host && dev == last_device && last_dev) {
        *out = last_dev;
        return MOLE_OK;
    }
    void *alias = nullptr;
    MOLE_CUDA_TRY(cudaHostGetDevicePointer(&alias, const_cast<void *>(host), 0));
    last_host = host;
    last_dev = static_cast<const unsigned char *>(alias);
    last_device = dev;
    *out = last_dev;
    return MOLE_OK;
}

// `layers` tables, table_stride bytes apart from lut_host on (one pinned allocation), into staging areas
// staging_stride bytes apart
static int launch_fetch(const void *lut_host, const int32_t *uniq, const int32_t *count, int max_rows, long long row_bytes,
                        void *staging, cudaStream_t st, int layers = 1, long long table_stride = 0, long long staging_stride = 0,
                        const HotRows *hot = nullptr)
{
    const unsigned char *dev_alias = nullptr;
    int rc = device_alias(lut_host, &dev_alias);
    if (rc != MOLE_OK) return rc;
    dim3 grid(static_cast<unsigned>((row_bytes + kFetchChunk - 1) / kFetchChunk), static_cast<unsigned>(max_rows),
              static_cast<unsigned>(layers));
    HotRows none;
    memset(&none, 0, sizeof none);
    mole_fetch_kernel<<<grid, kFetchThreads, 0, st>>>(dev_alias, uniq, count, row_bytes, static_cast<unsigned char *>(staging),
                                                      table_stride, staging_stride, hot ? *hot : none);
    MOLE_CUDA_TRY(cudaGetLastError());
    return MOLE_OK;
}

}  // namespace mole

using namespace mole;

struct mole_offload_ctx {
    int max_tokens, N, d, V, dtype, n_buffers;
    int lut_format, lut_block;  // MOLE_LUT_*: rows are plain elements, or the packed records of a quantised table
    long long row_bytes;
    int32_t *table;  // [V] dedup scratch, kept all zero between kernels
    // hot rows: the rows of hot_rows ids of hot_layers layers kept in device memory
    int32_t *hot_slot;        // [V]: position in the cache or -1
    unsigned char *hot_base;  // [hot_layers][hot_rows][row_bytes]
    long long hot_rows;
    int hot_layers;
    const unsigned char *hot_host_base;  // the host tables the cache mirrors: layer l at + l * hot_host_stride
    long long hot_host_stride;
    unsigned long long *hot_hits;  // device counter
    cudaEvent_t step_begin;  // orders the side stream after the main stream at the start of a whole step
    struct Buffer {
        unsigned char *staging;  // [max_tokens][N][d]
        int32_t *uniq, *slot, *count;
        cudaEvent_t ready, consumed;
        int M;  // tokens of the prefetch in flight
    } *buf;
};

extern "C" {

int mole_dedup_ids(const int32_t *ids, int M, int V, int32_t *scratch, int32_t *uniq, int32_t *slot, int32_t *count,
                   uint32_t *status, void *stream)
{
    if (M < 0 || V < 1) return MOLE_ERR_INVALID_ARG;
    if (M > MOLE_DEDUP_MAX_TOKENS) return MOLE_ERR_TOO_LARGE;
    if (!count || !scratch || (M > 0 && (!ids || !uniq || !slot))) return MOLE_ERR_INVALID_ARG;
    return launch_dedup(ids, M, V, scratch, uniq, slot, count, status, static_cast<cudaStream_t>(stream));
}

int mole_fetch_rows(const void *lut_host, const int32_t *uniq, const int32_t *count, int max_rows, int64_t row_bytes,
                    void *staging, void *stream)
{
    if (max_rows < 0 || row_bytes < 16 || (row_bytes & 15)) return MOLE_ERR_INVALID_ARG;
    if (max_rows == 0) return MOLE_OK;
    if (max_rows > 65535) return MOLE_ERR_TOO_LARGE;
    if (!lut_host || !uniq || !count || !staging || !aligned16(lut_host) || !aligned16(staging)) return MOLE_ERR_INVALID_ARG;
    return launch_fetch(lut_host, uniq, count, max_rows, row_bytes, staging, static_cast<cudaStream_t>(stream));
}

int mole_host_alloc(void **ptr, size_t bytes)
{
    if (!ptr || bytes == 0) return MOLE_ERR_INVALID_ARG;
    *ptr = nullptr;
    cudaError_t e = cudaHostAlloc(ptr, bytes, cudaHostAllocMapped | cudaHostAllocPortable);
    if (e == cudaErrorMemoryAllocation) {
        set_cuda_error(e);
        return MOLE_ERR_NOMEM;
    }
    MOLE_CUDA_TRY(e);
    return MOLE_OK;
}

int mole_host_free(void *ptr)
{
    if (!ptr) return MOLE_OK;
    MOLE_CUDA_TRY(cudaFreeHost(ptr));
    return MOLE_OK;
}

int mole_offload_destroy(mole_offload_ctx *c)
{
    if (!c) return MOLE_OK;
    if (c->buf) {
        for (int b = 0; b < c->n_buffers; ++b) {
            mole_offload_ctx::Buffer &B = c->buf[b];
            if (B.staging) cudaFree(B.staging);
            if (B.uniq) cudaFree(B.uniq);
            if (B.slot) cudaFree(B.slot);
            if (B.count) cudaFree(B.count);
            if (B.ready) cudaEventDestroy(B.ready);
            if (B.consumed) cudaEventDestroy(B.consumed);
        }
        delete[] c->buf;
    }
    if (c->table) cudaFree(c->table);
    if (c->hot_slot) cudaFree(c->hot_slot);
    if (c->hot_base) cudaFree(c->hot_base);
    if (c->hot_hits) cudaFree(c->hot_hits);
    if (c->step_begin) cudaEventDestroy(c->step_begin);
    delete c;
    (void)cudaGetLastError();
    return MOLE_OK;
}

int mole_offload_create(mole_offload_ctx **out, int max_tokens, int N, int d, int V, int dtype, int n_buffers)
{
    return mole_offload_create_ex(out, max_tokens, N, d, V, dtype, n_buffers, MOLE_LUT_PLAIN, 0);
}

int mole_offload_create_ex(mole_offload_ctx **out, int max_tokens, int N, int d, int V, int dtype, int n_buffers, int lut_format,
                           int lut_block)
{
    if (!out) return MOLE_ERR_INVALID_ARG;
    *out = nullptr;
    if (dtype != MOLE_DTYPE_BF16 && dtype != MOLE_DTYPE_F32) return MOLE_ERR_INVALID_ARG;
    if (lut_format != MOLE_LUT_PLAIN && lut_format != MOLE_LUT_NF4 && lut_format != MOLE_LUT_NF3) return MOLE_ERR_INVALID_ARG;
    if (max_tokens < 1 || n_buffers < 1 || n_buffers > 16) return MOLE_ERR_INVALID_ARG;
    if (max_tokens > 65535) return MOLE_ERR_TOO_LARGE;
    StepPlan plan;
    int rc = plan_step(max_tokens, 1, N, d, dtype, 0, &plan);
    if (rc != MOLE_OK) return rc;
    if (V < 1) return MOLE_ERR_UNSUPPORTED_SHAPE;
    int64_t rec_bytes = 0;
    if (lut_format != MOLE_LUT_PLAIN) {
        if (dtype != MOLE_DTYPE_BF16 || !quant_layer_shape_ok(N, d, lut_format, lut_block)) return MOLE_ERR_UNSUPPORTED_SHAPE;
        rc = mole_quant_record_bytes(N, d, lut_format, lut_block, &rec_bytes);
        if (rc != MOLE_OK) return rc;
    }
    mole_offload_ctx *c = new (std::nothrow) mole_offload_ctx;
    if (!c) return MOLE_ERR_NOMEM;
    memset(c, 0, sizeof *c);
    c->max_tokens = max_tokens;
    c->N = N;
    c->d = d;
    c->V = V;
    c->dtype = dtype;
    c->n_buffers = n_buffers;
    c->lut_format = lut_format;
    c->lut_block = lut_block;
    c->row_bytes = lut_format != MOLE_LUT_PLAIN ? rec_bytes : static_cast<long long>(N) * d * elem_bytes(dtype);
    c->buf = new (std::nothrow) mole_offload_ctx::Buffer[n_buffers];
    if (!c->buf) {
        delete c;
        return MOLE_ERR_NOMEM;
    }
    memset(c->buf, 0, sizeof(mole_offload_ctx::Buffer) * n_buffers);
    cudaError_t e = cudaMalloc(&c->table, sizeof(int32_t) * static_cast<size_t>(V));
    if (e == cudaSuccess) e = cudaMemset(c->table, 0, sizeof(int32_t) * static_cast<size_t>(V));
    if (e == cudaSuccess) e = cudaEventCreateWithFlags(&c->step_begin, cudaEventDisableTiming);
    for (int b = 0; b < n_buffers && e == cudaSuccess; ++b) {
        mole_offload_ctx::Buffer &B = c->buf[b];
        e = cudaMalloc(&B.staging, static_cast<size_t>(c->row_bytes) * max_tokens);
        if (e == cudaSuccess) e = cudaMalloc(&B.uniq, sizeof(int32_t) * max_tokens);
        if (e == cudaSuccess) e = cudaMalloc(&B.slot, sizeof(int32_t) * max_tokens);
        if (e == cudaSuccess) e = cudaMalloc(&B.count, sizeof(int32_t));
        if (e == cudaSuccess) e = cudaMemset(B.count, 0, sizeof(int32_t));
        if (e == cudaSuccess) e = cudaEventCreateWithFlags(&B.ready, cudaEventDisableTiming);
        if (e == cudaSuccess) e = cudaEventCreateWithFlags(&B.consumed, cudaEventDisableTiming);
    }
    if (e != cudaSuccess) {
        set_cuda_error(e);
        mole_offload_destroy(c);
        return e == cudaErrorMemoryAllocation ? MOLE_ERR_NOMEM : MOLE_ERR_CUDA;
    }
    *out = c;
    return MOLE_OK;
}

// The cache as the fetch kernel sees it for tables starting at `lut_host` (layer 0 of the launch): only if
// that address is one of the mirrored host tables.
static bool hot_for(const mole_offload_ctx *c, const void *lut_host, long long table_stride, int layers, HotRows *h)
{
    if (!c->hot_slot || !c->hot_base || c->hot_rows == 0) return false;
    const long long off = static_cast<const unsigned char *>(lut_host) - c->hot_host_base;
    if (off < 0) return false;
    long long layer0 = 0;
    if (c->hot_layers > 1) {
        if (c->hot_host_stride <= 0 || off % c->hot_host_stride != 0) return false;
        layer0 = off / c->hot_host_stride;
        if (layers > 1 && table_stride != c->hot_host_stride) return false;
    } else if (off != 0) {
        return false;
    }
    if (layer0 + layers > c->hot_layers) return false;
    h->slot = c->hot_slot;
    h->base = c->hot_base;
    h->rows = c->hot_rows;
    h->layer0 = static_cast<int>(layer0);
    h->hits = c->hot_hits;
    return true;
}

int mole_offload_set_hot_rows(mole_offload_ctx *c, const int32_t *hot_ids_host, int n_hot, const void *lut_host_base,
                              int64_t lut_layer_stride_bytes, int L)
{
    if (!c || n_hot < 0 || L < 1) return MOLE_ERR_INVALID_ARG;
    MOLE_CUDA_TRY(cudaDeviceSynchronize());  // nothing of this context may be in flight while the cache changes
    if (c->hot_slot) cudaFree(c->hot_slot);
    if (c->hot_base) cudaFree(c->hot_base);
    if (c->hot_hits) cudaFree(c->hot_hits);
    c->hot_slot = nullptr;
    c->hot_base = nullptr;
    c->hot_hits = nullptr;
    c->hot_rows = 0;
    c->hot_layers = 0;
    if (n_hot == 0) return MOLE_OK;
    if (!hot_ids_host || !lut_host_base || !aligned16(lut_host_base) || (lut_layer_stride_bytes & 15)) return MOLE_ERR_INVALID_ARG;
    if (n_hot > c->V) return MOLE_ERR_TOO_LARGE;
    int32_t *slot_host = new (std::nothrow) int32_t[c->V];
    if (!slot_host) return MOLE_ERR_NOMEM;
    for (int i = 0; i < c->V; ++i) slot_host[i] = -1;
    for (int i = 0; i < n_hot; ++i) {
        const int id = hot_ids_host[i];
        if (id < 0 || id >= c->V || slot_host[id] != -1) {  // outside the table, or listed twice
            delete[] slot_host;
            return MOLE_ERR_INVALID_ARG;
        }
        slot_host[id] = i;
    }
    cudaError_t e = cudaMalloc(&c->hot_slot, sizeof(int32_t) * static_cast<size_t>(c->V));
    if (e == cudaSuccess) e = cudaMalloc(&c->hot_base, static_cast<size_t>(L) * n_hot * c->row_bytes);
    if (e == cudaSuccess) e = cudaMalloc(&c->hot_hits, sizeof(unsigned long long));
    if (e == cudaSuccess) e = cudaMemset(c->hot_hits, 0, sizeof(unsigned long long));
    if (e == cudaSuccess) e = cudaMemcpy(c->hot_slot, slot_host, sizeof(int32_t) * static_cast<size_t>(c->V), cudaMemcpyHostToDevice);
    for (int l = 0; l < L && e == cudaSuccess; ++l)
        for (int i = 0; i < n_hot && e == cudaSuccess; ++i)
            e = cudaMemcpyAsync(c->hot_base + (static_cast<size_t>(l) * n_hot + i) * c->row_bytes,
                                static_cast<const unsigned char *>(lut_host_base) + static_cast<int64_t>(l) * lut_layer_stride_bytes +
                                    static_cast<int64_t>(hot_ids_host[i]) * c->row_bytes,
                                static_cast<size_t>(c->row_bytes), cudaMemcpyHostToDevice, nullptr);
    if (e == cudaSuccess) e = cudaDeviceSynchronize();
    delete[] slot_host;
    if (e != cudaSuccess) {
        set_cuda_error(e);
        if (c->hot_slot) cudaFree(c->hot_slot);
        if (c->hot_base) cudaFree(c->hot_base);
        if (c->hot_hits) cudaFree(c->hot_hits);
        c->hot_slot = nullptr;
        c->hot_base = nullptr;
        c->hot_hits = nullptr;
        return e == cudaErrorMemoryAllocation ? MOLE_ERR_NOMEM : MOLE_ERR_CUDA;
    }
    c->hot_rows = n_hot;
    c->hot_layers = L;
    c->hot_host_base = static_cast<const unsigned char *>(lut_host_base);
    c->hot_host_stride = lut_layer_stride_bytes;
    return MOLE_OK;
}

int mole_offload_hot_hits(mole_offload_ctx *c, uint64_t *hits, int reset)
{
    if (!c || !hits) return MOLE_ERR_INVALID_ARG;
    *hits = 0;
    if (!c->hot_hits) return MOLE_OK;
    unsigned long long v = 0;
    MOLE_CUDA_TRY(cudaMemcpy(&v, c->hot_hits, sizeof v, cudaMemcpyDeviceToHost));  // waits for the device's work queued so far
    *hits = v;
    if (reset) MOLE_CUDA_TRY(cudaMemset(c->hot_hits, 0, sizeof v));
    return MOLE_OK;
}

int mole_offload_prefetch(mole_offload_ctx *c, int b, const int32_t *ids, int M, const void *lut_host_layer,
                          void *side_stream)
{
    if (!c || b < 0 || b >= c->n_buffers || M < 0) return MOLE_ERR_INVALID_ARG;
    if (M > c->max_tokens) return MOLE_ERR_TOO_LARGE;
    mole_offload_ctx::Buffer &B = c->buf[b];
    B.M = M;
    if (M == 0) return MOLE_OK;
    if (!ids || !lut_host_layer || !aligned16(lut_host_layer)) return MOLE_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(side_stream);
    // the staging area may still be read by the layer that consumed this buffer last
    MOLE_CUDA_TRY(cudaStreamWaitEvent(st, B.consumed, 0));
    int rc = launch_dedup(ids, M, c->V, c->table, B.uniq, B.slot, B.count, nullptr, st);
    if (rc != MOLE_OK) return rc;
    HotRows hot;
    const bool use_hot = hot_for(c, lut_host_layer, 0, 1, &hot);
    rc = launch_fetch(lut_host_layer, B.uniq, B.count, M, c->row_bytes, B.staging, st, 1, 0, 0, use_hot ? &hot : nullptr);
    if (rc != MOLE_OK) return rc;
    MOLE_CUDA_TRY(cudaEventRecord(B.ready, st));
    return MOLE_OK;
}

int mole_layer_forward_offload(mole_offload_ctx *c, int b, const void *hidden, const void *w_router, void *out,
                               uint32_t *status, int B_, int T, void *stream)
{
    if (!c || b < 0 || b >= c->n_buffers || B_ < 0 || T < 0) return MOLE_ERR_INVALID_ARG;
    mole_offload_ctx::Buffer &B = c->buf[b];
    const long long M = static_cast<long long>(B_) * T;
    if (M != B.M) return MOLE_ERR_INVALID_ARG;
    if (M == 0) return MOLE_OK;
    if (!hidden || !w_router || !out || !aligned16(hidden) || !aligned16(w_router) || !aligned16(out))
        return MOLE_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    MOLE_CUDA_TRY(cudaStreamWaitEvent(st, B.ready, 0));
    StepLaunch a;
    a.hidden = hidden;
    a.residual = nullptr;
    a.row_index = B.slot;  // gather from staging[slot[t]]; slot is -1 for an id outside [0, V)
    a.lut = B.staging;
    a.w_router = w_router;
    a.out = out;
    a.gates_out = nullptr;
    a.status = status;
    a.lut_stride = 0;
    a.wr_stride = 0;
    a.M = M;
    a.L = 1;
    a.N = c->N;
    a.d = c->d;
    a.rows = c->max_tokens;
    a.dtype = c->dtype;
    a.flags = 0;
    a.d_split = 0;
    a.stream = st;
    int rc = c->lut_format != MOLE_LUT_PLAIN ? launch_quant_layer(a, c->lut_format, c->lut_block, current_wait_polls()) : launch_step(a);
    if (rc != MOLE_OK) return rc;
    MOLE_CUDA_TRY(cudaEventRecord(B.consumed, st));
    return MOLE_OK;
}

int mole_offload_decode_step(mole_offload_ctx *c, const void *hidden_in, const int32_t *ids, const void *lut_host_base,
                             int64_t lut_layer_stride_bytes, const void *w_router_base, int64_t wr_layer_stride_bytes,
                             void *out, void *tmp, uint32_t *status, int L, int B_, int T, void *stream, void *side_stream)
{
    if (!c || c->n_buffers < 2 || L < 1 || B_ < 0 || T < 0 || stream == side_stream) return MOLE_ERR_INVALID_ARG;
    const long long M = static_cast<long long>(B_) * T;
    if (M > c->max_tokens) return MOLE_ERR_TOO_LARGE;
    if (M == 0) return MOLE_OK;
    if (!hidden_in || !ids || !lut_host_base || !w_router_base || !out) return MOLE_ERR_INVALID_ARG;
    if (!aligned16(hidden_in) || !aligned16(lut_host_base) || !aligned16(w_router_base) || !aligned16(out) ||
        (lut_layer_stride_bytes & 15) || (wr_layer_stride_bytes & 15))
        return MOLE_ERR_INVALID_ARG;
    if (L > 1 && (!tmp || !aligned16(tmp) || out == hidden_in || tmp == hidden_in || tmp == out)) return MOLE_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream), side = static_cast<cudaStream_t>(side_stream);
    mole_offload_ctx::Buffer &B0 = c->buf[0], &B1 = c->buf[1];

    // the side stream starts after whatever the caller has queued on the main stream (ids, tables) and
    // after the previous step's layers have stopped reading the slot map and both staging areas
    MOLE_CUDA_TRY(cudaEventRecord(c->step_begin, st));
    MOLE_CUDA_TRY(cudaStreamWaitEvent(side, c->step_begin, 0));
    // While `stream` is being captured into a CUDA graph the waits on the previous call's events are
    // left out (a captured stream may not depend on work outside the capture): the step then relies
    // on the stream order of whole graph launches, which step_begin already carries to the side stream.
    cudaStreamCaptureStatus capturing = cudaStreamCaptureStatusNone;
    MOLE_CUDA_TRY(cudaStreamIsCapturing(st, &capturing));
    if (capturing == cudaStreamCaptureStatusNone) {
        MOLE_CUDA_TRY(cudaStreamWaitEvent(side, B0.consumed, 0));
        MOLE_CUDA_TRY(cudaStreamWaitEvent(side, B1.consumed, 0));
    }
    // one dedup for the whole step: every layer looks up the same ids (slot map and distinct ids in buffer 0)
    int rc = launch_dedup(ids, static_cast<int>(M), c->V, c->table, B0.uniq, B0.slot, B0.count, status, side);
    if (rc != MOLE_OK) return rc;
    B0.M = B1.M = static_cast<int>(M);

    // A staging area holds max_tokens rows; a step of M tokens needs at most M per layer, so one area
    // takes the rows of g = max_tokens / M consecutive layers (the ids are the same for all of them):
    // one fetch launch per group of g layers into staging area (group & 1), issued before the previous
    // group's layers so that it runs under them.  Fewer, larger fetches: at small batches the step is
    // bound by the launch + PCIe round trip of every fetch, not by the link.
    int g = static_cast<int>(c->max_tokens / M);
    g = g < 1 ? 1 : (g > L ? L : g);
    // ... but unless the whole step's rows are a small transfer, keep at least three groups so that all fetches
    // but the first run under the previous group's layers.  Small: 256 KB (measured, one token of the 410M shape,
    // 786 KB per step: 54.9 -> 49.8 us with three groups); 1 MB when a hot-row cache is set, since most of a
    // small step's rows then do not cross the link at all (42 us in one group against 45 us in three).
    const long long small_step = c->hot_rows > 0 ? (1LL << 20) : (1LL << 18);
    if (M * c->row_bytes * L > small_step && g > (L + 2) / 3) g = (L + 2) / 3;
    const int groups = (L + g - 1) / g;
    const long long area = M * c->row_bytes;  // one layer's rows inside a staging area
    auto fetch = [&](int k) -> int {
        mole_offload_ctx::Buffer &Bk = c->buf[k & 1];
        const int l0 = k * g, n = (l0 + g <= L) ? g : L - l0;
        if (k >= 2) MOLE_CUDA_TRY(cudaStreamWaitEvent(side, Bk.consumed, 0));
        const unsigned char *tables = static_cast<const unsigned char *>(lut_host_base) + static_cast<int64_t>(l0) * lut_layer_stride_bytes;
        HotRows hot;
        const bool use_hot = hot_for(c, tables, lut_layer_stride_bytes, n, &hot);
        int r = launch_fetch(tables, B0.uniq, B0.count, static_cast<int>(M), c->row_bytes, Bk.staging, side, n, lut_layer_stride_bytes,
                             area, use_hot ? &hot : nullptr);
        if (r != MOLE_OK) return r;
        MOLE_CUDA_TRY(cudaEventRecord(Bk.ready, side));
        return MOLE_OK;
    };
    const void *src = hidden_in;
    if ((rc = fetch(0)) != MOLE_OK) return rc;
    for (int k = 0; k < groups; ++k) {
        if (k + 1 < groups && (rc = fetch(k + 1)) != MOLE_OK) return rc;  // queued before group k's layers: they overlap
        mole_offload_ctx::Buffer &Bk = c->buf[k & 1];
        MOLE_CUDA_TRY(cudaStreamWaitEvent(st, Bk.ready, 0));
        const int l0 = k * g, n = (l0 + g <= L) ? g : L - l0;
        StepLaunch a;
        a.residual = nullptr;
        a.row_index = B0.slot;  // gather from staging[slot[t]]; slot is -1 for an id outside [0, V)
        a.gates_out = nullptr;
        a.status = status;
        a.lut_stride = area;
        a.wr_stride = wr_layer_stride_bytes;
        a.M = M;
        a.N = c->N;
        a.d = c->d;
        a.rows = M;  // a slot never exceeds the number of distinct ids
        a.dtype = c->dtype;
        a.d_split = 0;
        a.stream = st;
        if (c->lut_format != MOLE_LUT_PLAIN) {
            // quantised records: layer by layer from the staging area (the layers of a group chained to one
            // another with programmatic dependent launch), ping-pong so that the last layer writes `out`
            for (int i = 0; i < n; ++i) {
                const int l = l0 + i;
                void *dst = ((L - 1 - l) % 2 == 0) ? out : tmp;
                a.hidden = src;
                a.lut = Bk.staging + static_cast<long long>(i) * area;
                a.w_router = static_cast<const unsigned char *>(w_router_base) + static_cast<int64_t>(l) * wr_layer_stride_bytes;
                a.out = dst;
                a.L = 1;
                a.flags = i > 0 ? MOLE_FLAG_CHAIN : 0;
                rc = launch_quant_layer(a, c->lut_format, c->lut_block, current_wait_polls());
                if (rc != MOLE_OK) return rc;
                src = dst;
            }
        } else {
            // the group's layers in ONE launch: their rows lie `area` bytes apart in the staging area, which is
            // all the fused step kernel needs (a token's chain through the n layers stays on chip).  The last
            // group writes `out`, the groups before it alternate between tmp and out.
            void *dst = (groups - 1 - k) % 2 == 0 ? out : tmp;
            a.hidden = src;
            a.lut = Bk.staging;
            a.w_router = static_cast<const unsigned char *>(w_router_base) + static_cast<int64_t>(l0) * wr_layer_stride_bytes;
            a.out = dst;
            a.L = n;
            a.flags = 0;
            a.kernel = MOLE_KERNEL_RING;  // every group on one kernel family: the step's bits do not depend on how it is grouped
            rc = launch_step(a);
            if (rc != MOLE_OK) return rc;
            src = dst;
        }
        MOLE_CUDA_TRY(cudaEventRecord(Bk.consumed, st));
    }
    return MOLE_OK;
}

int mole_offload_buffers(mole_offload_ctx *c, int b, const int32_t **uniq, const int32_t **slot, const int32_t **count,
                         const void **staging)
{
    if (!c || b < 0 || b >= c->n_buffers) return MOLE_ERR_INVALID_ARG;
    if (uniq) *uniq = c->buf[b].uniq;
    if (slot) *slot = c->buf[b].slot;
    if (count) *count = c->buf[b].count;
    if (staging) *staging = c->buf[b].staging;
    return MOLE_OK;
}

}  // extern "C"

// ---------------------------------------------------------------------------------------------
// Dedup for callers that cannot allocate device memory.
//
// Some hosts of this library have no way to get a V-entry scratch table for mole_dedup_ids:
// a plug-in inside an inference server whose allocator already owns all of HBM (a raw
// cudaMalloc there fails or fragments the pool), or a decode loop that must never run into
// cudaMalloc's device-wide synchronisation.  For them the scratch table lives in the library
// image itself: a fixed array in device global memory that every GPU loading the library
// carries (MOLE_STATIC_DEDUP_MAX_V * 4 bytes = 256 KB) until the process exits.
//
// In host code the array's name is only a stand-in symbol, not an address a kernel can use, so
// its device address is looked up with cudaGetSymbolAddress once per device (with that device
// current) and cached; the kernel gets that address.
// ---------------------------------------------------------------------------------------------
namespace mole {

static __device__ __align__(256) int32_t g_static_dedup_table[MOLE_STATIC_DEDUP_MAX_V];

constexpr int kMaxDevices = 64;
static std::mutex g_static_mutex;
static int32_t *g_static_table_addr[kMaxDevices] = {nullptr};

// Device address of g_static_dedup_table on the current device (looked up on first use).
static int static_table_for_current_device(int32_t **out)
{
    int dev = -1;
    MOLE_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDevices) return MOLE_ERR_INVALID_ARG;
    std::lock_guard<std::mutex> lock(g_static_mutex);
    if (!g_static_table_addr[dev]) {
        void *p = nullptr;
        MOLE_CUDA_TRY(cudaGetSymbolAddress(&p, g_static_dedup_table));
        if (!p) return MOLE_ERR_CUDA;
        g_static_table_addr[dev] = static_cast<int32_t *>(p);
    }
    *out = g_static_table_addr[dev];
    return MOLE_OK;
}

}  // namespace mole

extern "C" int mole_dedup_ids_static(const int32_t *ids, int M, int V, int32_t *uniq, int32_t *slot, int32_t *count,
                                     uint32_t *status, void *stream)
{
    if (M < 0 || V < 1) return MOLE_ERR_INVALID_ARG;
    if (V > MOLE_STATIC_DEDUP_MAX_V) return MOLE_ERR_TOO_LARGE;  // the built-in table has no room for this vocabulary
    if (M > MOLE_DEDUP_MAX_TOKENS) return MOLE_ERR_TOO_LARGE;
    if (!count || (M > 0 && (!ids || !uniq || !slot))) return MOLE_ERR_INVALID_ARG;
    int32_t *table = nullptr;
    int rc = static_table_for_current_device(&table);
    if (rc != MOLE_OK) return rc;
    // The table is zero when the library is loaded and every run of the kernel zeroes the
    // entries it touched before it ends, so nothing has to be cleared here.
    return launch_dedup(ids, M, V, table, uniq, slot, count, status, static_cast<cudaStream_t>(stream));
}
