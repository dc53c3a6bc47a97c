// Quantised lookup tables (Sec. 4.5 and Table 8 of arXiv 2503.15798): the tables are compressed after
// training to the 4-bit and 3-bit NormalFloat types of the QLoRA paper with block-wise absmax scaling,
// which cuts the bytes gathered per token to 25.3 % / 19.5 % of the 16-bit table.  This file holds the
// codebooks, the GPU quantiser that packs a bf16 table into per-id records, and the fused layer that
// gathers a token's packed record and de-quantises inside the weighted sum.
//
// Record of one id (the unit that is gathered; a multiple of 16 bytes, zero padded):
//   NF4: N rows of d/2 bytes -- byte i of a row holds code 2i in its low and code 2i+1 in its high
//        nibble -- then N * d/block float32 scales (the blocks' absolute maxima), row after row.
//   NF3: N rows of d/4 bytes with the two low bits of every code (byte i: codes 4i .. 4i+3, code 4i+k at
//        bits 2k, 2k+1), then N rows of d/8 bytes with the high bits (byte i: codes 8i .. 8i+7, code
//        8i+k at bit k), then N * d/block float16 scales.
// With the paper's blocks (768 for NF4, 128 for NF3) that is 388 bytes per 768 elements and 50 bytes per
// 128 elements: the 25.3 % and 19.5 % of Table 8.  A block never straddles two rows.
#include <cuda_fp16.h>
#include <math.h>
#include <mutex>
#include <string.h>

#include "mole_decode.cuh"

namespace mole {

// ---- codebooks -----------------------------------------------------------------------------------
// k-bit NormalFloat (QLoRA, Sec. 3): quantiles of N(0,1) at evenly spaced probabilities, 2^(k-1) of them
// for the negative half and 2^(k-1) + 1 for the positive half (both counts include the median, so that
// zero is a value of its own), divided by the largest magnitude.  The outermost probability is
// 1 - delta, delta the mean of 1/(2 (2^k - 1)) and 1/(2 2^k).
static double normal_quantile(double prob)
{
    // bisection on the normal CDF written with erfc; the CDF is monotone and 1e-17 wide brackets
    // are far below float32 resolution
    double lo = -12.0, hi = 12.0;
    for (int it = 0; it < 200; ++it) {
        const double mid = 0.5 * (lo + hi);
        const double cdf = 0.5 * erfc(-mid * 0.70710678118654752440);
        if (cdf < prob) lo = mid;
        else hi = mid;
    }
    return 0.5 * (lo + hi);
}

static void build_codebook(int bits, float *out)
{
    const int n = 1 << bits, half = n / 2;
    const double delta = 0.5 * (1.0 / (2.0 * (n - 1)) + 1.0 / (2.0 * n));
    double v[16];
    // positive half: half + 1 probabilities from 1/2 to 1 - delta; index half - 1 is the median (zero)
    for (int i = 0; i <= half; ++i) {
        const double prob = 0.5 + (0.5 - delta) * i / half;
        v[half - 1 + i] = i == 0 ? 0.0 : normal_quantile(prob);
    }
    // negative half: half probabilities from 1/2 down to delta; the median is shared
    for (int i = 1; i < half; ++i) {
        const double prob = 0.5 + (0.5 - delta) * i / (half - 1);
        v[half - 1 - i] = -normal_quantile(prob);
    }
    const double top = v[n - 1] > -v[0] ? v[n - 1] : -v[0];
    for (int i = 0; i < n; ++i) out[i] = static_cast<float>(v[i] / top);
}

struct Codebooks {
    float nf4[16], nf3[8];
};
static const Codebooks &codebooks()
{
    static Codebooks cb;
    static std::once_flag once;
    std::call_once(once, [] {
        build_codebook(4, cb.nf4);
        build_codebook(3, cb.nf3);
    });
    return cb;
}

static int format_bits(int format) { return format == MOLE_LUT_NF4 ? 4 : (format == MOLE_LUT_NF3 ? 3 : 0); }
static int scale_bytes(int format) { return format == MOLE_LUT_NF4 ? 4 : 2; }

static long long record_bytes(int N, int d, int format, int block)
{
    const long long codes = format == MOLE_LUT_NF4 ? static_cast<long long>(N) * d / 2 : static_cast<long long>(N) * (d / 4 + d / 8);
    const long long scales = static_cast<long long>(N) * (d / block) * scale_bytes(format);
    return (codes + scales + 15) / 16 * 16;
}

static int check_format(int N, int d, int format, int block)
{
    if (format != MOLE_LUT_NF4 && format != MOLE_LUT_NF3) return MOLE_ERR_INVALID_ARG;
    if (N < 1 || N > 64 || d < 32 || d % 32 != 0) return MOLE_ERR_UNSUPPORTED_SHAPE;
    if (block < 32 || block % 32 != 0 || d % block != 0) return MOLE_ERR_UNSUPPORTED_SHAPE;
    return MOLE_OK;
}

struct CodebookParam {
    float value[16];
    float mid[15];  // midpoints of adjacent values: a normalised element takes the code = number of midpoints below it
};
static CodebookParam codebook_param(int format)
{
    CodebookParam c;
    memset(&c, 0, sizeof c);
    const int n = 1 << format_bits(format);
    const float *src = format == MOLE_LUT_NF4 ? codebooks().nf4 : codebooks().nf3;
    for (int i = 0; i < n; ++i) c.value[i] = src[i];
    for (int i = 0; i + 1 < n; ++i) c.mid[i] = 0.5f * (src[i] + src[i + 1]);
    for (int i = n - 1; i < 15; ++i) c.mid[i] = INFINITY;
    return c;
}

// ---- quantiser: one block of threads per id ---------------------------------------------------------
// Pass 1: a warp per quantisation block finds the absolute maximum and stores the scale (float32, or the
// float16 rounding of min(max, 65504)).  Pass 2: a thread per 8 consecutive elements divides by the stored
// scale in float32 (IEEE division), counts the midpoints below the quotient and packs the 8 codes.
constexpr int kQuantThreads = 256;

template <int BITS>
__global__ void __launch_bounds__(kQuantThreads) mole_quantize_kernel(const uint4 *__restrict__ src, unsigned char *__restrict__ dst,
                                                                      long long V, int N, int d, int block, long long rec_bytes,
                                                                      const CodebookParam cb)
{
    extern __shared__ float s_scale[];  // [N * d / block] effective scales of this id
    const long long id = blockIdx.x;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, nwarps = kQuantThreads / 32;
    const int nblk = d / block, total_blocks = N * nblk;
    const uint4 *row0 = src + id * (static_cast<long long>(N) * d / 8);
    unsigned char *rec = dst + id * rec_bytes;
    const long long code_bytes = BITS == 4 ? static_cast<long long>(N) * d / 2 : static_cast<long long>(N) * (d / 4 + d / 8);
    for (int b = warp; b < total_blocks; b += nwarps) {
        const int j = b / nblk, kb = b % nblk;
        const uint4 *p = row0 + (static_cast<long long>(j) * d + static_cast<long long>(kb) * block) / 8;
        float m = 0.f;
        for (int g = lane; g < block / 8; g += 32) {
            float f[8];
            Elem<__nv_bfloat16>::unpack(__ldg(p + g), f);
#pragma unroll
            for (int i = 0; i < 8; ++i) m = fmaxf(m, fabsf(f[i]));
        }
        m = warp_max(m);
        if (lane == 0) {
            if constexpr (BITS == 4) {
                reinterpret_cast<float *>(rec + code_bytes)[b] = m;
                s_scale[b] = m;
            } else {
                const __half h = __float2half_rn(fminf(m, 65504.f));
                reinterpret_cast<__half *>(rec + code_bytes)[b] = h;
                s_scale[b] = __half2float(h);
            }
        }
    }
    __syncthreads();
    const int groups = N * d / 8;  // groups of 8 consecutive elements
    for (int g = tid; g < groups; g += kQuantThreads) {
        const int j = g / (d / 8), c8 = g % (d / 8);
        const float s = s_scale[j * nblk + (c8 * 8) / block];
        float f[8];
        Elem<__nv_bfloat16>::unpack(__ldg(row0 + g), f);
        uint32_t code[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const float y = s > 0.f ? __fdiv_rn(f[i], s) : 0.f;
            uint32_t k = 0;
#pragma unroll
            for (int t = 0; t < (1 << BITS) - 1; ++t) k += y > cb.mid[t] ? 1u : 0u;
            code[i] = k;
        }
        if constexpr (BITS == 4) {
            uint32_t w = 0;
#pragma unroll
            for (int i = 0; i < 8; ++i) w |= code[i] << (4 * i);
            reinterpret_cast<uint32_t *>(rec)[g] = w;  // 4 bytes: codes 8 c8 .. 8 c8 + 7 of row j
        } else {
            uint32_t a = 0, b = 0;
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                a |= (code[i] & 3u) << (2 * i);
                b |= ((code[i] >> 2) & 1u) << i;
            }
            reinterpret_cast<unsigned short *>(rec)[g] = static_cast<unsigned short>(a);                   // low bits, 2 bytes
            rec[static_cast<long long>(N) * (d / 4) + g] = static_cast<unsigned char>(b);                // high bits, 1 byte
        }
    }
    // padding bytes after the scales stay as the caller left them (zero them once after allocation if
    // records are to compare equal byte for byte)
}

// ---- the fused layer over packed records: one block per token (see mole_decode.cuh for the structure) ----
struct QDecodeParams {
    const void *hidden, *residual, *row_index, *lut, *w_router, *norm_weight;
    void *out;
    float *gates_out;
    uint32_t *status;
    long long rows, rec_bytes;
    int d, block;
    float norm_eps;
    uint32_t flags, wait_polls;
    float cb[16];
};

__host__ __device__ inline uint32_t qdecode_smem_bytes(int N, int d, long long rec_bytes)
{
    return up128(static_cast<uint32_t>(d) * N * 2) + up128(static_cast<uint32_t>(rec_bytes)) + kDecodeMaxWarps * 64 * 4 +
           kDecodeMaxWarps * 4 + 16 * 4 + 32;
}

template <int N, int BITS, int NORM>
__global__ void __launch_bounds__(kDecodeMaxThreads) mole_qdecode_kernel(const QDecodeParams p)
{
    using E = Elem<__nv_bfloat16>;
    constexpr int VEC = 8;
    constexpr int NV = N < VEC ? N : VEC;
    constexpr int QL = N >= VEC ? N / VEC : 1;
    constexpr int CPV = N >= VEC ? 1 : VEC / N;
    constexpr int R = N / 2;
    extern __shared__ __align__(128) unsigned char smem[];

    pdl_launch_dependents();

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int T = blockDim.x, nwarps = T >> 5, d = p.d;
    const long long t = blockIdx.x;
    const uint32_t wr_bytes = static_cast<uint32_t>(d) * N * 2, rec_bytes = static_cast<uint32_t>(p.rec_bytes);
    unsigned char *rec = smem + up128(wr_bytes);
    float *partial = reinterpret_cast<float *>(rec + up128(rec_bytes));
    float *scratch = partial + kDecodeMaxWarps * 64;
    float *cbs = scratch + kDecodeMaxWarps;
    uint64_t *bar = reinterpret_cast<uint64_t *>(cbs + 16);  // [0]: router matrix, [1]: the token's record

    const long long id = (p.flags & MOLE_FLAG_IDS_INT64) ? __ldg(static_cast<const long long *>(p.row_index) + t)
                                                         : static_cast<long long>(__ldg(static_cast<const int *>(p.row_index) + t));
    const bool valid = id >= 0 && id < p.rows;
    if (tid == 0) {
        mbar_init(bar, 1);
        mbar_init(bar + 1, 1);
        mbar_init_fence();
        mbar_expect_tx(bar, wr_bytes);
        bulk_g2s(smem, p.w_router, wr_bytes, bar);
        mbar_expect_tx(bar + 1, rec_bytes);
        bulk_g2s(rec, static_cast<const unsigned char *>(p.lut) + static_cast<size_t>(valid ? id : 0) * rec_bytes, rec_bytes, bar + 1);
    }
    if (tid < 16) cbs[tid] = p.cb[tid];
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
    __syncthreads();

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
    const uint2 hown = ldcg_v2(hrow + static_cast<size_t>(tid) * 8);
    uint2 res = hown;
    if (p.residual) res = ldcg_v2(static_cast<const unsigned char *>(p.residual) + static_cast<size_t>(t) * d * 2 + static_cast<size_t>(tid) * 8);

    if constexpr (NORM) {
        const float x0 = bf16_bits_to_float(hown.x & 0xffffu), x1 = __uint_as_float(hown.x & 0xffff0000u);
        const float x2 = bf16_bits_to_float(hown.y & 0xffffu), x3 = __uint_as_float(hown.y & 0xffff0000u);
        float ss = fmaf(x3, x3, fmaf(x2, x2, fmaf(x1, x1, x0 * x0)));
        ss = warp_sum(ss);
        if (lane == 0) scratch[warp] = ss;
        __syncthreads();
        float total = 0.f;
        for (int w = 0; w < nwarps; ++w) total += scratch[w];
        const float rinv = 1.0f / sqrtf(total / static_cast<float>(d) + p.norm_eps);
#pragma unroll
        for (int i = 0; i < R * CPV; ++i) hs[i] = float_to_bf16_bits((bf16_bits_to_float(hs[i]) * rinv) * nw[i]);
    }

    // bounded waits for the two bulk copies; after a failure the block computes on whatever its shared
    // memory holds (every address stays inside it and inside its own output row) and says so
    bool timed_out = false;
#pragma unroll
    for (int which = 0; which < 2; ++which) {
        bool ok = false;
        for (uint32_t i = 0; i < p.wait_polls && !ok; ++i) {
            ok = mbar_try_wait(bar + which, 0);
            if (!ok && i > 64) __nanosleep(64);
        }
        if (!ok) {
            timed_out = true;
            for (uint32_t i = 0; i < kDrainPolls && !ok; ++i) {
                ok = mbar_try_wait(bar + which, 0);
                if (!ok) __nanosleep(64);
            }
        }
    }
    if (timed_out && tid == 0 && p.status) atomicOr(p.status, MOLE_STATUS_TIMEOUT);

    float acc[NV];
#pragma unroll
    for (int i = 0; i < NV; ++i) acc[i] = 0.f;
    const uint32_t wbase = smem_u32(smem);
#pragma unroll
    for (int r = 0; r < R; ++r) {
        const uint4 wv = lds128(wbase + 16u * static_cast<uint32_t>(tid + r * T));
#pragma unroll
        for (int e = 0; e < VEC; ++e) E::fma_elem(acc[e % NV], wv, e, hs[r * CPV + e / NV]);
    }
    int base = 0;
    lane_reduce_scatter<NV, NV, 16, QL>(acc, lane, base);
    partial[warp * N + (N >= VEC ? (lane % QL) * VEC : 0) + base] = acc[0];
    __syncthreads();

    const float e = softmax_numerator<N>(partial, nwarps, lane);

    // ---- weighted sum over the de-quantised rows: value = codebook[code] * scale of its block ----
    const uint32_t rec_s = smem_u32(rec), cb_s = smem_u32(cbs);
    const int nblk = d / p.block, blk = (4 * tid) / p.block;
    const uint32_t code_bytes = BITS == 4 ? static_cast<uint32_t>(N) * d / 2 : static_cast<uint32_t>(N) * (d / 4 + d / 8);
    float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
    float es[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
    for (int j = 0; j < N; ++j) {
        const float g = __shfl_sync(0xffffffffu, e, j);
        es[j & 3] += g;
        float s;
        uint32_t c0, c1, c2, c3;
        if constexpr (BITS == 4) {
            s = __uint_as_float(lds32(rec_s + code_bytes + 4u * (j * nblk + blk)));
            const uint32_t c = lds16(rec_s + static_cast<uint32_t>(j) * (d / 2) + 2u * tid);
            c0 = c & 15u, c1 = (c >> 4) & 15u, c2 = (c >> 8) & 15u, c3 = (c >> 12) & 15u;
        } else {
            const unsigned short hb = static_cast<unsigned short>(lds16(rec_s + code_bytes + 2u * (j * nblk + blk)));
            s = __half2float(*reinterpret_cast<const __half *>(&hb));
            uint32_t a, b;
            asm volatile("ld.shared.u8 %0, [%1];" : "=r"(a) : "r"(rec_s + static_cast<uint32_t>(j) * (d / 4) + tid));
            asm volatile("ld.shared.u8 %0, [%1];" : "=r"(b) : "r"(rec_s + static_cast<uint32_t>(N) * (d / 4) + static_cast<uint32_t>(j) * (d / 8) + (tid >> 1)));
            b >>= 4 * (tid & 1);
            c0 = (a & 3u) | ((b & 1u) << 2);
            c1 = ((a >> 2) & 3u) | (((b >> 1) & 1u) << 2);
            c2 = ((a >> 4) & 3u) | (((b >> 2) & 1u) << 2);
            c3 = ((a >> 6) & 3u) | (((b >> 3) & 1u) << 2);
        }
        const float gs = g * s;
        a0 = fmaf(gs, __uint_as_float(lds32(cb_s + 4u * c0)), a0);
        a1 = fmaf(gs, __uint_as_float(lds32(cb_s + 4u * c1)), a1);
        a2 = fmaf(gs, __uint_as_float(lds32(cb_s + 4u * c2)), a2);
        a3 = fmaf(gs, __uint_as_float(lds32(cb_s + 4u * c3)), a3);
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

typedef void (*QDecodeKernel)(const QDecodeParams);
struct QVariant {
    QDecodeKernel fn;
    const char *name;
};
#define MOLE_QV(N, BITS, NORM) QVariant { mole_qdecode_kernel<N, BITS, NORM>, "qdecode<" #N ",nf" #BITS "," #NORM ">" }
static QVariant pick_qdecode(int N, int bits, bool norm)
{
    if (bits == 4) {
        switch (N) {
            case 4: return norm ? MOLE_QV(4, 4, 1) : MOLE_QV(4, 4, 0);
            case 8: return norm ? MOLE_QV(8, 4, 1) : MOLE_QV(8, 4, 0);
            case 16: return norm ? MOLE_QV(16, 4, 1) : MOLE_QV(16, 4, 0);
            case 32: return norm ? MOLE_QV(32, 4, 1) : MOLE_QV(32, 4, 0);
        }
    } else {
        switch (N) {
            case 4: return norm ? MOLE_QV(4, 3, 1) : MOLE_QV(4, 3, 0);
            case 8: return norm ? MOLE_QV(8, 3, 1) : MOLE_QV(8, 3, 0);
            case 16: return norm ? MOLE_QV(16, 3, 1) : MOLE_QV(16, 3, 0);
            case 32: return norm ? MOLE_QV(32, 3, 1) : MOLE_QV(32, 3, 0);
        }
    }
    return QVariant{nullptr, "none"};
}

bool quant_layer_shape_ok(int N, int d, int format, int block)
{
    if (check_format(N, d, format, block) != MOLE_OK) return false;
    if (N != 4 && N != 8 && N != 16 && N != 32) return false;
    if (d % 128 != 0 || d / 4 > kDecodeMaxThreads) return false;
    return qdecode_smem_bytes(N, d, record_bytes(N, d, format, block)) <= 227u * 1024u;
}

const char *quant_variant_name(int N, int format, bool norm) { return pick_qdecode(N, format_bits(format), norm).name; }

int launch_quant_layer(const StepLaunch &a, int format, int block, uint32_t wait_polls)
{
    if (a.M == 0) return MOLE_OK;
    if (a.dtype != MOLE_DTYPE_BF16 || a.L != 1 || !quant_layer_shape_ok(a.N, a.d, format, block)) return MOLE_ERR_UNSUPPORTED_SHAPE;
    if (a.M > 0x7fffffffLL) return MOLE_ERR_TOO_LARGE;
    const QVariant v = pick_qdecode(a.N, format_bits(format), a.norm_weight != nullptr);
    if (!v.fn) return MOLE_ERR_UNSUPPORTED_SHAPE;
    QDecodeParams p;
    p.hidden = a.hidden;
    p.residual = a.residual;
    p.row_index = a.row_index;
    p.lut = a.lut;
    p.w_router = a.w_router;
    p.norm_weight = a.norm_weight;
    p.out = a.out;
    p.gates_out = a.gates_out;
    p.status = a.status;
    p.rows = a.rows;
    p.rec_bytes = record_bytes(a.N, a.d, format, block);
    p.d = a.d;
    p.block = block;
    p.norm_eps = a.norm_eps;
    p.flags = a.flags;
    p.wait_polls = wait_polls;
    const CodebookParam cb = codebook_param(format);
    for (int i = 0; i < 16; ++i) p.cb[i] = cb.value[i];
    const int smem = static_cast<int>(qdecode_smem_bytes(a.N, a.d, p.rec_bytes));
    int rc = ensure_smem_opt_in(reinterpret_cast<const void *>(v.fn), smem);
    if (rc != MOLE_OK) return rc;
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof cfg);
    cfg.gridDim = dim3(static_cast<unsigned>(a.M), 1, 1);
    cfg.blockDim = dim3(a.d / 4, 1, 1);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = a.stream;
    cudaLaunchAttribute attrs[1];
    unsigned na = 0;
    if (a.flags & MOLE_FLAG_CHAIN) {
        attrs[na].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attrs[na].val.programmaticStreamSerializationAllowed = 1;
        ++na;
    }
    cfg.attrs = attrs;
    cfg.numAttrs = na;
    MOLE_CUDA_TRY(cudaLaunchKernelEx(&cfg, v.fn, p));
    return MOLE_OK;
}

}  // namespace mole

using namespace mole;

extern "C" {

int mole_nf_codebook(int format, float *values)
{
    if (!values || (format != MOLE_LUT_NF4 && format != MOLE_LUT_NF3)) return MOLE_ERR_INVALID_ARG;
    const int n = 1 << format_bits(format);
    const float *src = format == MOLE_LUT_NF4 ? codebooks().nf4 : codebooks().nf3;
    for (int i = 0; i < n; ++i) values[i] = src[i];
    return MOLE_OK;
}

int mole_quant_record_bytes(int N, int d, int format, int block, int64_t *bytes)
{
    if (!bytes) return MOLE_ERR_INVALID_ARG;
    int rc = check_format(N, d, format, block);
    if (rc != MOLE_OK) return rc;
    *bytes = record_bytes(N, d, format, block);
    return MOLE_OK;
}

int mole_quantize_lut(const void *lut, void *packed, int64_t V, int N, int d, int format, int block, void *stream)
{
    int rc = check_format(N, d, format, block);
    if (rc != MOLE_OK) return rc;
    if (V < 0) return MOLE_ERR_INVALID_ARG;
    if (V == 0) return MOLE_OK;
    if (V > 0x7fffffffLL) return MOLE_ERR_TOO_LARGE;
    if (!lut || !packed || !aligned16(lut) || !aligned16(packed)) return MOLE_ERR_INVALID_ARG;
    const long long rb = record_bytes(N, d, format, block);
    const int smem = N * (d / block) * 4;
    if (smem > 48 * 1024) return MOLE_ERR_UNSUPPORTED_SHAPE;
    const CodebookParam cb = codebook_param(format);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (format == MOLE_LUT_NF4)
        mole_quantize_kernel<4><<<static_cast<unsigned>(V), kQuantThreads, smem, st>>>(static_cast<const uint4 *>(lut), static_cast<unsigned char *>(packed), V, N, d, block, rb, cb);
    else
        mole_quantize_kernel<3><<<static_cast<unsigned>(V), kQuantThreads, smem, st>>>(static_cast<const uint4 *>(lut), static_cast<unsigned char *>(packed), V, N, d, block, rb, cb);
    MOLE_CUDA_TRY(cudaGetLastError());
    return MOLE_OK;
}

}  // extern "C"
