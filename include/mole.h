/*
 * mole.h -- C ABI of the B200 (sm_100a) inference-time Mixture-of-Lookup-Experts layer
 * (arXiv 2503.15798, "Mixture of Lookup Experts").
 *
 * What the layer computes (Eq. 4 and Eq. 8 of the paper, shared expert left to the caller):
 * for every token t with hidden state h_t (d values) and input id i_t,
 *
 *     z_j   = sum_c h_t[c] * W_r[c][j]                     j = 0..N-1      (router logits)
 *     g     = softmax(z)   over ALL N experts, no top-k                     (Eq. 4)
 *     out_t = res_t + sum_j g_j * LUT[i_t][j][:]                            (Eq. 8)
 *
 * LUT is the per-layer table of pre-computed expert outputs of Eq. 6-7,
 * LUT[i][j] = FFN_j(Embedding(i)), row-major [V][N][d]; res_t = h_t unless a separate
 * residual is given.  Arithmetic: logits, softmax and the weighted sum are fp32; gates are
 * never rounded below fp32; the only rounding to the storage type is at the store of out.
 *
 * Conventions shared by every entry point
 *  - All functions return an int: MOLE_OK (0) or a positive MOLE_ERR_* code.  Nothing is
 *    thrown, printed or aborted.  mole_status_string() names a code; mole_last_cuda_error()
 *    gives the CUDA runtime's text for the calling thread's last MOLE_ERR_CUDA.
 *  - "device" pointers are device memory of the CURRENT CUDA device; "host" pointers are
 *    host memory.  The caller owns every buffer; the library allocates nothing except inside
 *    mole_offload_create()/mole_host_alloc() (freed by their destroy/free calls).
 *  - Calls are asynchronous: work is enqueued on `stream` (a cudaStream_t passed as void*,
 *    NULL = the legacy default stream) and MOLE_OK means "enqueued".  No call synchronises
 *    the device or the stream.
 *  - Shapes: M = B*T tokens, flattened; position (b, t) uses ids[b*T + t], its own input id.
 *    B*T == 0 is a successful no-op.  1 <= N <= 64, V >= 1, d a multiple of 8 (bf16) or
 *    4 (fp32) so that every row piece is a whole number of 16-byte vectors.
 *  - Alignment: hidden, residual, lut, w_router, out must be 16-byte aligned; ids 4-byte
 *    (8-byte for 64-bit ids).
 *  - Aliasing: out may be exactly hidden (in place).  Any other overlap of out with an input
 *    is the caller's error and is not detected.
 *  - An id outside [0, V) never reads out of bounds: that token gets out_t = res_t and, if a
 *    status word was supplied, MOLE_STATUS_BAD_ID is OR-ed into it.
 *  - Results are deterministic: no atomics in the arithmetic, fixed summation order, and a
 *    token's result does not depend on the batch it is in.
 */
#ifndef MOLE_H
#define MOLE_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define MOLE_VERSION 300

/* every entry point is exported from the shared library with default visibility */
#if defined(__GNUC__)
#define MOLE_API __attribute__((visibility("default")))
#else
#define MOLE_API
#endif

/* return codes */
#define MOLE_OK 0
#define MOLE_ERR_INVALID_ARG 1       /* null / misaligned pointer, negative size, bad enum */
#define MOLE_ERR_UNSUPPORTED_SHAPE 2 /* N outside 1..64, d not a multiple of the vector width, ... */
#define MOLE_ERR_CUDA 3              /* a CUDA runtime call failed; see mole_last_cuda_error() */
#define MOLE_ERR_NOMEM 4             /* an allocation inside create()/host_alloc() failed */
#define MOLE_ERR_TOO_LARGE 5         /* size beyond a stated maximum */
#define MOLE_ERR_IO 6                /* a table file could not be opened, read or written, or is not a table file */

/* bits OR-ed by kernels into an optional device status word (uint32_t, caller zeroes it) */
#define MOLE_STATUS_BAD_ID 1u  /* some id was outside [0, V) */
#define MOLE_STATUS_TIMEOUT 2u /* a bounded wait inside a kernel gave up; the launch's outputs are undefined */

/* element type of hidden / residual / lut / w_router / out */
#define MOLE_DTYPE_BF16 0
#define MOLE_DTYPE_F32 1

/* mole_args.flags */
#define MOLE_FLAG_IDS_INT64 1u /* ids are int64_t instead of int32_t */
#define MOLE_FLAG_CHAIN 2u     /* launch with programmatic dependent launch: the kernel may start, \
                                  and may read ids / lut / w_router, before the previous kernel    \
                                  on the stream has finished; it reads hidden / residual only      \
                                  after it has.  Only valid if ids, lut and w_router are not       \
                                  written by that previous kernel. */

/* which kernel family runs a single-layer launch (mole_args.kernel, mole_step_args.kernel) */
#define MOLE_KERNEL_AUTO 0   /* the library's choice: the ring kernel, except d = 2048 with N = 32 at up to 128 tokens (on \
                                148 SMs), where the one-token-per-cluster kernel of MOLE_KERNEL_DECODE runs */
#define MOLE_KERNEL_RING 1   /* persistent blocks, rows and router chunks streamed through a shared-memory ring: any shape */
#define MOLE_KERNEL_DECODE 2 /* one block per token (single layer: rows held in registers; fused step: rows through a ring, \
                                router matrix through registers): bf16, N of 4, 8, 16 or 32, d a multiple of 128 up to   \
                                2048 (single layer with N = 32: up to 1024), d_split 0.  A single layer with d = 2048 and \
                                N of 16 or 32 runs one token per thread-block cluster of four blocks (512 columns each,    \
                                partial router logits exchanged through distributed shared memory) */

/* storage of a table (mole_args.lut_format): plain elements of `dtype`, or the quantised records of Sec. 4.5 / Table 8 */
#define MOLE_LUT_PLAIN 0
#define MOLE_LUT_NF4 1 /* 4-bit NormalFloat codes, one float32 absmax scale per block (paper: block 768 -> 25.3 % of FP16) */
#define MOLE_LUT_NF3 2 /* 3-bit NormalFloat codes, one float16 absmax scale per block (paper: block 128 -> 19.5 % of FP16) */

/* mole_decode_step_ex mode: how the L layers of a step are launched */
#define MOLE_STEP_AUTO 0    /* fused unless the batch is large (then chained); also chained at up to 16 tokens where \
                               MOLE_KERNEL_AUTO runs the cluster kernel and a tmp buffer was given */
#define MOLE_STEP_FUSED 1   /* ONE launch: every block walks its tokens through all L layers */
#define MOLE_STEP_CHAINED 2 /* L launches chained with programmatic dependent launch */

/*
 * mole_layer_forward -- the fused layer, bf16, Eq. 4 + Eq. 8 (router, softmax over all N
 * experts, gather of the N rows selected by the id, fp32 weighted sum, residual add).
 *   hidden   device, bf16 [B*T][d]          router input and residual
 *   ids      device, int32 [B*T]            0 <= id < V
 *   lut      device, bf16 [V][N][d]         one layer's table (Eq. 7)
 *   w_router device, bf16 [d][N]            logits = hidden @ w_router  (a torch
 *                                           nn.Linear(d, N).weight must be transposed)
 *   out      device, bf16 [B*T][d]          may be == hidden
 * Errors: MOLE_ERR_INVALID_ARG, MOLE_ERR_UNSUPPORTED_SHAPE, MOLE_ERR_CUDA; nothing is
 * launched when an error is returned.
 */
MOLE_API int mole_layer_forward(const void *hidden, const int32_t *ids, const void *lut, const void *w_router,
                       void *out, int B, int T, int N, int d, int V, void *stream);

/*
 * mole_layer_forward_ex -- the same operation with every option.  The appendix listing of
 * the paper (App. A.2) routes on the normalised hidden state but adds the un-normalised residual
 * plus the shared expert's output: `norm_weight` fuses that normalisation in front of the router,
 * `residual` takes (residual + shared expert output).
 */
typedef struct mole_args {
    uint32_t struct_size;  /* sizeof(mole_args), checked */
    uint32_t flags;        /* MOLE_FLAG_* */
    const void *hidden;    /* device [M][d], dtype */
    const void *ids;       /* device [M], int32 (int64 with MOLE_FLAG_IDS_INT64) */
    const void *lut;       /* device [V][N][d], dtype */
    const void *w_router;  /* device [d][N], dtype */
    void *out;             /* device [M][d], dtype */
    const void *residual;  /* device [M][d], dtype, or NULL => hidden.  Must not alias out unless it is hidden */
    float *gates_out;      /* device [M][N] fp32 softmax weights, or NULL */
    uint32_t *status;      /* device status word (MOLE_STATUS_* bits OR-ed in), or NULL */
    int32_t B, T, N, d, V;
    int32_t dtype;         /* MOLE_DTYPE_* */
    int32_t kernel;        /* MOLE_KERNEL_*; AUTO is the ring kernel (measured at least as fast at every batch size on
                              B200).  The two families add the same fp32 terms in a different order, so their outputs may
                              differ in a rounding decision; within one family and launch shape a token's result is the
                              same bits whatever batch it is in.  MOLE_ERR_UNSUPPORTED_SHAPE if DECODE is asked for a
                              shape it does not cover. */
    int32_t d_split;       /* chunks a token's router matrix and rows are streamed in (1, 2, 4, 8 or 16; d/d_split must
                              stay a multiple of the vector width); 0 = auto: the fewest chunks of at most 32 KB.
                              The router matrix is cut by columns.  The rows are cut by experts (whole rows of
                              N/d_split experts, one contiguous copy) when d_split > 1 divides N, N is 4, 8, 16, 32
                              or 64, dtype is bf16, d <= 4096 and the router matrix streams with them (several
                              layers in one launch, or a matrix above 96 KB); otherwise by columns.  Chunking and
                              cut fix the order of the fp32 sums: the same launch shape gives the same bits. */
    void *stream;          /* cudaStream_t */
    const void *norm_weight; /* device [d], dtype, or NULL.  Not NULL: the router reads RMSNorm(hidden) =
                              (hidden / sqrt(mean(hidden^2) + norm_eps)) * norm_weight, rounded once to dtype, while
                              the residual stays `residual` (or hidden itself) -- the decoder layer of the paper's
                              App. A.2 listing, whose router input is the normalised state and whose residual is
                              not.  The normalisation happens in shared memory inside the same kernel. */
    float norm_eps;        /* >= 0; read only with norm_weight */
    int32_t lut_format;    /* MOLE_LUT_*.  NF4 / NF3: `lut` points to V packed records of mole_quant_record_bytes() bytes
                              each (written by mole_quantize_lut) instead of [V][N][d] elements; the layer gathers a
                              token's record and de-quantises inside the weighted sum: out = res + sum_j g_j *
                              (codebook[code] * scale).  bf16 activations, N of 4, 8, 16 or 32, d a multiple of 128 up
                              to 2048, d_split 0; MOLE_ERR_UNSUPPORTED_SHAPE otherwise. */
    int32_t lut_block;     /* elements per quantisation block (a multiple of 32 that divides d); read only with NF4 / NF3 */
    int32_t reserved2;     /* must be 0 */
} mole_args;

MOLE_API int mole_layer_forward_ex(const mole_args *args);

/*
 * mole_decode_step -- L layers back to back (Eq. 8 applied layer after layer; the attention
 * and shared-expert blocks that a full model runs in between are not part of this library).
 * Layer l reads table lut_base + l*lut_layer_stride_bytes and router w_router_base +
 * l*wr_layer_stride_bytes; its output, rounded to the storage type, is the next layer's hidden.
 *   hidden_in device [M][d], read only (FUSED mode also accepts out == hidden_in)
 *   out       device [M][d] final result
 *   tmp       device [M][d] scratch for the ping-pong of CHAINED mode (may be NULL when L == 1
 *             or when the mode is MOLE_STEP_FUSED)
 * dtype as MOLE_DTYPE_*.  status (device, may be NULL) as in mole_args.
 *
 * Two ways to run it (bit-identical when the rows travel in one chunk; with several chunks the two
 * may cut the rows differently -- see d_split -- and differ in the order of the fp32 sums, i.e. now
 * and then in a rounding decision):
 *  - FUSED: tokens are independent and a token's chain h_0 -> h_1 -> ... -> h_L needs nothing
 *    but its own rows, so one launch lets each block keep a token's running hidden slice in
 *    shared memory across all L layers while the rows of later layers (which depend only on
 *    the id) are already streaming in.  No hidden state travels through global memory between
 *    layers and there are no L-1 launch boundaries.
 *  - CHAINED: L launches of the single-layer kernel with programmatic dependent launch; layer
 *    l+1's first row gathers are in flight while layer l finishes.  This is what a model that
 *    runs other work between the layers gets by calling mole_layer_forward_ex per layer.
 * mole_decode_step picks FUSED up to 4096 tokens and CHAINED above; _ex lets the caller choose
 * and force d_split (0 = auto).  The first launch of a step waits for everything before it on the
 * stream (see mole_decode_step_args for the flag that lets it start early).
 */
MOLE_API int mole_decode_step(const void *hidden_in, const int32_t *ids, const void *lut_base,
                     int64_t lut_layer_stride_bytes, const void *w_router_base,
                     int64_t wr_layer_stride_bytes, void *out, void *tmp, uint32_t *status, int L, int B,
                     int T, int N, int d, int V, int dtype, void *stream);
MOLE_API int mole_decode_step_ex(const void *hidden_in, const int32_t *ids, const void *lut_base,
                     int64_t lut_layer_stride_bytes, const void *w_router_base,
                     int64_t wr_layer_stride_bytes, void *out, void *tmp, uint32_t *status, int L, int B,
                     int T, int N, int d, int V, int dtype, int mode, int d_split, void *stream);

/*
 * mole_decode_step_args -- the L-layer step with every option, among them the decoder layer of the
 * paper's App. A.2 listing in every layer: with norm_weight_base set, layer l's router reads
 * RMSNorm(hidden) with the scale vector at norm_weight_base + l*norm_layer_stride_bytes (see
 * mole_args.norm_weight) while the residual stays the un-normalised hidden state.  Both modes take it.
 * The first launch of a step is an ordinary launch: it starts after everything that precedes it on the
 * stream.  MOLE_FLAG_CHAIN in `flags` lets it start early as well (programmatic dependent launch); only
 * valid if the kernel before it on the stream writes none of ids, the tables, the router weights and the
 * norm weights.  Later layers of a CHAINED step are always chained to their predecessor.
 */
typedef struct mole_step_args {
    uint32_t struct_size;  /* sizeof(mole_step_args), checked */
    uint32_t flags;        /* 0 or MOLE_FLAG_CHAIN */
    const void *hidden_in; /* device [M][d], dtype, read only */
    const void *ids;       /* device int32 [M] */
    const void *lut_base;  /* device; layer l's table [V][N][d] at + l*lut_layer_stride_bytes */
    int64_t lut_layer_stride_bytes;
    const void *w_router_base; /* device; layer l's router [d][N] at + l*wr_layer_stride_bytes */
    int64_t wr_layer_stride_bytes;
    const void *norm_weight_base; /* device [d] per layer, dtype, or NULL: routers read hidden itself */
    int64_t norm_layer_stride_bytes;
    void *out;             /* device [M][d] */
    void *tmp;             /* device [M][d] scratch of CHAINED mode (NULL when L == 1 or FUSED) */
    uint32_t *status;      /* device status word or NULL */
    int32_t L, B, T, N, d, V;
    int32_t dtype;         /* MOLE_DTYPE_* */
    int32_t mode;          /* MOLE_STEP_* */
    int32_t d_split;       /* as mole_args.d_split */
    int32_t kernel;        /* as mole_args.kernel: the family of the single-layer launches of CHAINED mode and of the
                              one launch of FUSED mode */
    float norm_eps;        /* >= 0; read only with norm_weight_base */
    int32_t lut_format;    /* as mole_args.lut_format; quantised tables run as CHAINED steps (AUTO picks that) */
    int32_t lut_block;     /* as mole_args.lut_block */
    int32_t reserved;      /* must be 0 */
    void *stream;          /* cudaStream_t */
} mole_step_args;

MOLE_API int mole_decode_step_args(const mole_step_args *args);

/*
 * mole_decode_step_host -- mole_decode_step for a caller whose activations live in HOST
 * memory, all on `stream`.  When the three host buffers are pinned and mapped (cudaHostAlloc,
 * cudaHostRegister) and the step runs as one launch (L == 1 or up to 4096 tokens), the launch reads
 * hidden_host and ids_host across the host link itself and stores the last layer's output into
 * out_host: the device buffers are not touched.  Otherwise hidden_host and ids_host are copied to
 * the device buffers, the L layers run there, and the result is copied to out_host (asynchronous
 * when the host buffers are pinned).  The result is the same bits either way.
 *   hidden_host, out_host  host [M][d] (distinct)      ids_host host int32 [M]
 *   dev_hidden, dev_out, dev_tmp device [M][d] scratch owned by the caller; dev_ids device int32 [M]
 * The result is in out_host once the stream has been synchronised.
 */
MOLE_API int mole_decode_step_host(const void *hidden_host, const int32_t *ids_host, void *out_host, void *dev_hidden,
                          int32_t *dev_ids, void *dev_out, void *dev_tmp, const void *lut_base,
                          int64_t lut_layer_stride_bytes, const void *w_router_base,
                          int64_t wr_layer_stride_bytes, uint32_t *status, int L, int B, int T, int N, int d,
                          int V, int dtype, void *stream);

/*
 * mole_prefetch_rows -- ask L2 for the table rows a step will gather, ahead of the layers that gather
 * them.  The rows of every layer depend only on the input ids (Sec. 3.3: the experts' inputs are
 * embedding tokens), so a caller whose model runs other work between the lookup layers can issue this
 * at the start of a step, or a few layers ahead: one L2 prefetch per (token, layer) row of N*d elements,
 * for `layers` consecutive tables from lut_base on (layer l at + l*lut_layer_stride_bytes).  A hint
 * only: nothing is written, no result changes, ids outside [0, V) are skipped.  What stays in L2 until
 * the layer runs is the hardware's business; keep layers * M * row bytes well under the L2 size.
 *   ids device int32 [M] (int64 with MOLE_FLAG_IDS_INT64); lut_base device, 16-byte aligned.
 */
MOLE_API int mole_prefetch_rows(const void *ids, int M, const void *lut_base, int64_t lut_layer_stride_bytes, int layers,
                                int N, int d, int V, int dtype, uint32_t flags, void *stream);

/* ---------------------------------------------------------------------------------------
 * Quantised tables (Sec. 4.5, Table 8): post-training quantisation of a 16-bit table to the NF4 / NF3
 * NormalFloat types of the QLoRA paper, block-wise absmax scaling.  Per block: scale = max |x| (stored as
 * float32 for NF4, as the float16 rounding of min(max, 65504) for NF3); every element takes the code of the
 * codebook value nearest to x / scale (decided in float32, a value on a midpoint takes the lower code);
 * de-quantised value = codebook[code] * scale.  A block never straddles two (id, expert) rows.
 * Record of one id, the unit that is gathered (zero padded to a multiple of 16 bytes):
 *   NF4: N rows of d/2 bytes (byte i: code 2i in the low, code 2i+1 in the high nibble), then N*d/block float32 scales;
 *   NF3: N rows of d/4 bytes with the codes' two low bits (byte i: codes 4i..4i+3, code 4i+k at bits 2k, 2k+1), N rows
 *        of d/8 bytes with their high bits (byte i: codes 8i..8i+7, code 8i+k at bit k), then N*d/block float16 scales.
 * ------------------------------------------------------------------------------------- */

/* the 16 (NF4) or 8 (NF3) codebook values in ascending order: quantiles of N(0,1) at evenly spaced
 * probabilities, one more on the positive side so that zero is exact, scaled to [-1, 1].  Host arithmetic. */
MOLE_API int mole_nf_codebook(int lut_format, float *values);

/* bytes of one id's record; N 1..64, d a multiple of 32, block a multiple of 32 that divides d */
MOLE_API int mole_quant_record_bytes(int N, int d, int lut_format, int block, int64_t *bytes);

/* mole_quantize_lut -- quantise a bf16 table on the device.
 *   lut    device bf16 [V][N][d]           packed device, V * record_bytes bytes (16-byte aligned; padding bytes of a
 *                                           record are not written: zero the buffer once if records are compared)
 * Asynchronous on `stream`. */
MOLE_API int mole_quantize_lut(const void *lut, void *packed, int64_t V, int N, int d, int lut_format, int block,
                      void *stream);

/* ---------------------------------------------------------------------------------------
 * Offload mode: the table lives off the accelerator, in pinned host memory, and only the
 * looked-up rows move (Sec. 3.3 and the inference listing of App. A.2).
 * Per step the distinct ids are found on the device and only their rows cross the host link.
 * ------------------------------------------------------------------------------------- */

/*
 * mole_dedup_ids -- distinct ids of one step.
 *   ids     device int32 [M]
 *   scratch device int32 [V]; must be all zero on entry (zero it once after allocation);
 *           the kernel leaves it all zero again.  Calls sharing one scratch array must not
 *           overlap on the GPU.
 *   uniq    device int32 [>= min(M, V)]: the distinct in-range ids, in order of first occurrence
 *   slot    device int32 [M]: uniq[slot[t]] == ids[t]; -1 for an id outside [0, V)
 *   count   device int32 [1]: number of distinct in-range ids
 * M <= MOLE_DEDUP_MAX_TOKENS.  M == 0 writes count = 0.
 */
#define MOLE_DEDUP_MAX_TOKENS (1 << 20)
MOLE_API int mole_dedup_ids(const int32_t *ids, int M, int V, int32_t *scratch, int32_t *uniq, int32_t *slot,
                   int32_t *count, uint32_t *status, void *stream);

/*
 * mole_dedup_ids_static -- mole_dedup_ids for callers that cannot allocate device memory.
 * (The paper has no counterpart; this is a deployment convenience of this library.)
 *
 * Who needs it: code that runs where cudaMalloc is not an option -- a plug-in inside a server
 * whose own allocator already holds all of the GPU's memory, or a decode loop that must never
 * hit the device-wide synchronisation an allocation implies.  Such a caller still passes its
 * inputs and outputs, but the V-entry scratch table is a fixed array inside the library's
 * device image instead of a caller buffer: MOLE_STATIC_DEDUP_MAX_V int32 entries (256 KB) that
 * every GPU which loads the library holds until the process exits.
 *
 *   ids, uniq, slot, count, status, stream: exactly as in mole_dedup_ids; results are identical.
 *   V > MOLE_STATIC_DEDUP_MAX_V returns MOLE_ERR_TOO_LARGE and launches nothing.
 *
 * The call allocates nothing: no cudaMalloc, cudaFree or allocating library routine.  The
 * first call on each device looks up the array's device address (cudaGetSymbolAddress, with
 * that device current) and caches it; make that first call outside any stream capture.
 * All calls on a device share the one array.  The kernel expects it all zero and leaves it all
 * zero (it clears exactly the entries it set), so consecutive calls on one stream need no
 * clearing in between -- but two calls that overlap on the GPU (different streams without an
 * ordering between them) race on the array and give wrong results.
 */
#define MOLE_STATIC_DEDUP_MAX_V 65536
MOLE_API int mole_dedup_ids_static(const int32_t *ids, int M, int V, int32_t *uniq, int32_t *slot, int32_t *count,
                          uint32_t *status, void *stream);

/*
 * mole_fetch_rows -- copy rows uniq[0..count) of a table in pinned, device-mapped host
 * memory into a dense device staging buffer: staging[u] = lut_host[uniq[u]] (row_bytes each,
 * a multiple of 16).  The reads are issued by the GPU across the host link; `count` is read on
 * the device, so there is no host round trip.  lut_host is the HOST pointer of memory from
 * mole_host_alloc() / cudaHostAlloc / cudaHostRegister; max_rows bounds the launch
 * (count <= max_rows, staging holds max_rows rows).
 */
MOLE_API int mole_fetch_rows(const void *lut_host, const int32_t *uniq, const int32_t *count, int max_rows,
                    int64_t row_bytes, void *staging, void *stream);

/* pinned, device-mapped host memory for a table (cudaHostAlloc); free with mole_host_free */
MOLE_API int mole_host_alloc(void **ptr, size_t bytes);
MOLE_API int mole_host_free(void *ptr);

/*
 * Offload context: owns n_buffers staging buffers [max_tokens][N][d], their uniq / slot /
 * count arrays, one V-entry dedup scratch table and the events that order the side stream
 * against the main stream.  Not thread-safe; use one context per decoding stream.
 */
typedef struct mole_offload_ctx mole_offload_ctx;

MOLE_API int mole_offload_create(mole_offload_ctx **ctx, int max_tokens, int N, int d, int V, int dtype, int n_buffers);
/* ... for a quantised host table (lut_format MOLE_LUT_NF4 / NF3, lut_block as in mole_args): the host
 * table holds V packed records per layer, only the distinct ids' records cross the host link (25.3 % /
 * 19.5 % of the 16-bit bytes with the paper's blocks), and the layers de-quantise from the staging area.
 * MOLE_LUT_PLAIN gives mole_offload_create. */
MOLE_API int mole_offload_create_ex(mole_offload_ctx **ctx, int max_tokens, int N, int d, int V, int dtype, int n_buffers,
                           int lut_format, int lut_block);
MOLE_API int mole_offload_destroy(mole_offload_ctx *ctx);

/*
 * mole_offload_set_hot_rows -- a cache of hot rows in device memory in front of the host link.  Token ids
 * follow a heavy-tailed distribution, so a few ids account for most look-ups: the rows of the n_hot ids
 * listed (distinct, in [0, V), HOST array) are copied once, for all L layers of the host tables at
 * lut_host_base + l*lut_layer_stride_bytes, into n_hot*L*row_bytes bytes of device memory (plus a V-entry
 * index); every later fetch from one of those tables takes a listed id's row from there instead of across
 * the link.  Results do not change by a bit.  Synchronous (it waits for the device); replaces an earlier
 * set; n_hot == 0 frees it.  The host tables must not change while they are mirrored.
 * mole_offload_hot_hits reads (and optionally resets) the number of (row, layer) fetches the cache served;
 * it waits for the device's queued work.
 */
MOLE_API int mole_offload_set_hot_rows(mole_offload_ctx *ctx, const int32_t *hot_ids_host, int n_hot,
                              const void *lut_host_base, int64_t lut_layer_stride_bytes, int L);
MOLE_API int mole_offload_hot_hits(mole_offload_ctx *ctx, uint64_t *hits, int reset);

/*
 * mole_offload_prefetch -- on side_stream: wait until buffer `buf`'s previous consumer has
 * finished, deduplicate ids (device), fetch the distinct rows of lut_host_layer (HOST pointer,
 * pinned + mapped, [V][N][d]) into the buffer's staging area, record the buffer's ready event.
 * ids must stay unchanged until the work has run.
 */
MOLE_API int mole_offload_prefetch(mole_offload_ctx *ctx, int buf, const int32_t *ids, int M, const void *lut_host_layer,
                          void *side_stream);

/*
 * mole_layer_forward_offload -- on stream: wait for buffer `buf`'s ready event, run the fused
 * layer with the gather reading staging[slot[t]], record the buffer's consumed event.
 * B*T must equal the M given to the matching prefetch.  Output is bit-identical to
 * mole_layer_forward on the same inputs (the same kernel choice, the same order of sums).
 */
MOLE_API int mole_layer_forward_offload(mole_offload_ctx *ctx, int buf, const void *hidden, const void *w_router, void *out,
                               uint32_t *status, int B, int T, void *stream);

/*
 * mole_offload_decode_step -- a whole L-layer decode step in offload mode, one call: the ids
 * are deduplicated ONCE (they are the same for every layer), then the distinct rows of the next
 * layers are fetched from their host tables on side_stream while the current layers combine on
 * stream (the paper issues the row transfer first so that it overlaps the rest of the layer, App. A.2
 * listing).  A staging area holds max_tokens rows, so with B*T tokens one fetch launch brings the rows
 * of up to max_tokens / (B*T) consecutive layers (at least one; at least three groups per step once the
 * step's rows exceed 256 KB (1 MB with a hot-row cache), so that fetches overlap layers), and one fused launch then runs those layers:
 * a context created for the largest batch serves small batches with few, large fetches and few launches.
 * Needs a context with n_buffers >= 2.
 *   hidden_in device [M][d], read only;  out device [M][d] final result;  tmp device [M][d]
 *   scratch (may be NULL when L == 1);  lut_host_base HOST pointer (pinned + mapped) of layer 0's
 *   table, layer l at + l*lut_layer_stride_bytes;  w_router_base device, layer l at
 *   + l*wr_layer_stride_bytes.
 * Every group runs on the ring kernel: the output is bit-identical to L single-layer calls with
 * kernel = MOLE_KERNEL_RING when the rows travel in one chunk (see d_split; otherwise equal up to the order
 * of the fp32 sums).  stream and side_stream must differ.
 * The call may be captured into a CUDA graph (stream capturing, side_stream an ordinary stream: it
 * joins the capture and is joined back before the call returns).  While capturing, the call does not
 * wait for the events of the previous call on the same context -- a captured stream may not depend on
 * work outside the capture -- so the graphs of one context must be launched into one stream (or
 * otherwise ordered), and the context should not go back to uncaptured calls afterwards.
 */
MOLE_API int mole_offload_decode_step(mole_offload_ctx *ctx, const void *hidden_in, const int32_t *ids,
                             const void *lut_host_base, int64_t lut_layer_stride_bytes, const void *w_router_base,
                             int64_t wr_layer_stride_bytes, void *out, void *tmp, uint32_t *status, int L, int B, int T,
                             void *stream, void *side_stream);

/* device pointers of a buffer's arrays, for inspection: uniq [max_tokens], slot [max_tokens], count [1], staging */
MOLE_API int mole_offload_buffers(mole_offload_ctx *ctx, int buf, const int32_t **uniq, const int32_t **slot,
                         const int32_t **count, const void **staging);

/* ---------------------------------------------------------------------------------------
 * Re-parameterisation (Sec. 3.3, Eq. 6-7): build a layer's table from its routed experts,
 *     LUT[i][j][:] = FFN_j(x_i),   FFN_j(x) = W2_j . gelu(W1_j . x)   (two matrices, no bias, the erf GELU
 *     x Phi(x), evaluated to within 4e-7 of its exact value before the rounding to bf16),
 *     x_i = Embedding(i), or RMSNorm(Embedding(i)) * norm_weight when norm_weight is given (the
 *     expert_layernorm of the training listing in App. A.1, folded into the table),
 * as one forward pass over the whole embedding matrix: two bf16 tensor-core GEMMs with fp32 accumulation;
 * the hidden activations gelu(W1 x) and the normalised rows are materialised in bf16.
 *   embedding  device bf16 [V][d]          w1 device bf16 [N][D][d]          w2 device bf16 [N][d][D]
 *   norm_weight device bf16 [d] or NULL    lut device bf16 [V][N][d] (written)
 *   scratch    device, mole_build_lut_scratch_bytes() bytes (V*N*D bf16, plus V*d with a norm), 16-byte aligned
 * d and D multiples of 8.  Asynchronous on `stream`; status as elsewhere (MOLE_STATUS_TIMEOUT if a bounded
 * wait inside the kernel ran out: the table is then undefined).
 * ------------------------------------------------------------------------------------- */
MOLE_API int mole_build_lut_scratch_bytes(int V, int N, int d, int D, int with_norm, int64_t *bytes);
MOLE_API int mole_build_lut(const void *embedding, const void *w1, const void *w2, const void *norm_weight, float norm_eps,
                   void *lut, void *scratch, int V, int N, int d, int D, uint32_t *status, void *stream);

/* ---------------------------------------------------------------------------------------
 * Table files: the tables of all L layers on a storage device below host memory (Sec. 3.3: the tables stay
 * offloaded; Sec. 4.2: lower-tier storage).  Layout: a 4096-byte header (magic "MOLELUT1", version, shapes,
 * element type, table format, bytes per row), then layer after layer, V rows of row_bytes each -- plain
 * [N][d] elements or the packed records of a quantised table.  Host calls, no CUDA; MOLE_ERR_IO on any
 * file error (missing, short, not a table file).
 * ------------------------------------------------------------------------------------- */
typedef struct mole_table_info {
    int64_t L, V;
    int32_t N, d;
    int32_t dtype;      /* MOLE_DTYPE_* of plain elements (and of the activations a quantised table serves) */
    int32_t lut_format; /* MOLE_LUT_* */
    int32_t lut_block;  /* quantisation block, 0 for plain tables */
    int32_t reserved;
    int64_t row_bytes;  /* bytes of one id's row: N*d elements, or one packed record */
} mole_table_info;

/* write L tables from host memory (layer l at tables_host + l*layer_stride_bytes, V rows each) */
MOLE_API int mole_table_file_write(const char *path, const void *tables_host, int64_t layer_stride_bytes, int L, int V,
                          int N, int d, int dtype, int lut_format, int lut_block);
MOLE_API int mole_table_file_info(const char *path, mole_table_info *info);
/* read layers layer0 .. layer0 + n_layers - 1 into host memory (e.g. from mole_host_alloc), dst_layer_stride_bytes apart */
MOLE_API int mole_table_file_read(const char *path, void *dst_host, int64_t dst_layer_stride_bytes, int layer0, int n_layers);
/* read the rows of n ids of one layer, densely, into dst_host (n * row_bytes): a tier that leaves the file on disk */
MOLE_API int mole_table_file_read_rows(const char *path, int layer, const int32_t *ids_host, int n, void *dst_host);

/* --------------------------------------------------------------------------------------- */

MOLE_API const char *mole_status_string(int code);
MOLE_API const char *mole_last_cuda_error(void);
MOLE_API int mole_version(void);

/*
 * Debugging aids.  The library reads these environment variables ONCE, at the first launch or plan
 * (unset or 0: no effect); mole_reload_debug_env() reads them again (tests flip them between launches).
 * They override parts of the launch plan and never change what is computed beyond the order of fp32 sums:
 *   MOLE_FORCE_STAGES (2..8: ring depth), MOLE_FORCE_TARGET_BLOCKS (resident blocks per SM aimed at),
 *   MOLE_FORCE_BLOCKS_PER_SM (upper bound on the grid), MOLE_FORCE_LANES (1, 2, 4: lanes per column
 *   group in the combine), MOLE_FORCE_COLUMN_CHUNKS (1: cut the rows by columns even where the expert
 *   cut exists), MOLE_FORCE_KERNEL (1, 2: MOLE_KERNEL_* for launches that leave the choice open).
 * One of them shortens the bounded waits inside the kernels, to let a test see a wait run out:
 *   MOLE_DEBUG_WAIT_LIMIT (n >= 1: a wait gives up after n polls; negative: after none -- any wait that
 *   is not satisfied at once gives up).  The launch then returns normally with MOLE_STATUS_TIMEOUT in
 *   the status word and undefined outputs; nothing faults and the stream stays usable.
 */
MOLE_API int mole_reload_debug_env(void);

/* launch shape the ring kernel would get for M tokens and L layers in one launch (L = 1: a single
 * layer): column chunks per token, threads per block, dynamic shared memory, depth of the ring,
 * resident blocks per SM.  Host arithmetic only; the SM count is the current device's if there is
 * one, else the 148 of a B200. */
MOLE_API int mole_plan(int M, int L, int N, int d, int dtype, int d_split, int *out_d_split, int *out_threads,
              int *out_smem_bytes, int *out_stages, int *out_blocks_per_sm);

/* Name of the kernel instantiation a launch of this shape runs ("decode<N,NORM>", "fstep<N,DB,NORM>",
 * "qdecode<N,nfB,NORM>" or "step<storage,N,P,MODE,SHAPE,DIRECT,NORM>"), with its block size and dynamic
 * shared memory: lets a test list which instantiations a workload reaches.  norm != 0: with a normalised
 * router; kernel as mole_args.kernel; lut_format / lut_block as mole_args (a quantised table: L must be 1).
 * name receives at most name_bytes - 1 characters and a terminator.  Launches nothing. */
MOLE_API int mole_variant(int M, int L, int N, int d, int dtype, int d_split, int norm, int kernel, int lut_format,
                 int lut_block, char *name, int name_bytes, int *out_threads, int *out_smem_bytes);

#ifdef __cplusplus
}
#endif
#endif /* MOLE_H */
