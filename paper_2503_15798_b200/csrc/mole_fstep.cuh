// The fused L-layer decode step for sm_100a (Eq. 8 of arXiv 2503.15798 applied layer after layer): one
// launch, a block walks whole tokens through all L layers with the running hidden state on chip, the
// arithmetic of the one-block-per-token kernel (mole_decode.cuh) and the data movement of the ring
// kernel (mole_kernel.cuh).
//
// A token's chain h_0 -> h_1 -> ... -> h_L is serial, so a step of few tokens costs L times the latency of
// one (token, layer) item; this kernel keeps that item short:
//   - d / 4 compute threads: thread i owns columns 4i .. 4i+3 of the hidden state (in registers, fp32
//     arithmetic, rounded to bf16 after every layer as a layer-by-layer execution would) and of every
//     expert's row;
//   - one producer warp streams, `stages` chunks ahead through a ring of 32 KB shared-memory slots, the
//     chunks of the token's rows (whole rows of N / kr experts, one contiguous bulk copy each); rows depend
//     only on the id, so they run ahead of the arithmetic by several layers.  The layer's router matrix
//     comes from L2 straight into the compute threads' registers one item ahead (up to 16 experts), or
//     through the same ring in column chunks in front of the rows (32 experts);
//   - two block barriers per item: partial logits written / new hidden state written.  Every warp forms
//     the softmax numerators itself from the per-warp partial logits (lane j <-> expert j) and hands them
//     round by shuffles inside the weighted sum.
// The fp32 sums run in the order of mole_decode_kernel, so a fused step gives the bits of L chained
// launches of that kernel.
#pragma once

#include "mole_decode.cuh"

namespace mole {

constexpr uint32_t kFStepSlotBytes = 32 * 1024;
constexpr int kFBarLogits = 4, kFBarHidden = 5, kFBarNorm = 6;  // named barriers of the compute threads

struct FStepParams {
    const void *hidden, *row_index, *lut, *w_router, *norm_weight;
    void *out;
    uint32_t *status;
    long long lut_stride, wr_stride, norm_stride;  // bytes between layers
    long long M, rows;
    int d, L, stages;
    int kr, rexp;  // rows chunks per item, experts per chunk (kr * rexp == N)
    float norm_eps;
    uint32_t flags, wait_polls;
};

struct FStepSmem {
    uint32_t off_hid, off_norm, off_partial, off_scratch, off_meta, off_bars, total;
};
__host__ __device__ inline FStepSmem fstep_smem(int N, int d, int stages, int norm)
{
    FStepSmem m;
    m.off_hid = static_cast<uint32_t>(stages) * kFStepSlotBytes;
    m.off_norm = m.off_hid + up128(static_cast<uint32_t>(d) * 2);
    m.off_partial = m.off_norm + (norm ? up128(static_cast<uint32_t>(d) * 2) : 0u);
    m.off_scratch = m.off_partial + kDecodeMaxWarps * 64 * 4;
    m.off_meta = m.off_scratch + kDecodeMaxWarps * 4;
    m.off_bars = m.off_meta + up128((kMaxStages + 3) * 4);
    m.total = m.off_bars + 2 * kMaxStages * 8;
    (void)N;
    return m;
}

#ifdef __CUDACC__

// How an item is cut into 32 KB ring slots, fixed by N and the width class DB (0: d <= 512, 1: d <= 1024,
// 2: d <= 2048) so that the loops over chunks and experts unroll completely (a rolled weighted sum took
// five times as long): the router matrix in KW column chunks, the rows in chunks of REXP whole experts.
template <int N, int DB>
struct FStepCut {
    static constexpr int dmax = DB == 0 ? 512 : (DB == 1 ? 1024 : 2048);
    static constexpr int kw_raw = N * dmax * 2 / static_cast<int>(kFStepSlotBytes);
    static constexpr int KW = kw_raw < 1 ? 1 : kw_raw;
    static constexpr int rexp_raw = static_cast<int>(kFStepSlotBytes) / (2 * dmax) > 16 ? 16 : static_cast<int>(kFStepSlotBytes) / (2 * dmax);
    static constexpr int REXP = N < rexp_raw ? N : rexp_raw;  // at most 16: a chunk is held in registers while it is summed
    static constexpr int KR = N / REXP;
};

// N: experts (4, 8, 16, 32).  DB: width class (see FStepCut).  NORM: routers read RMSNorm(hidden) rounded
// to bf16.  Launch: blockDim.x == d / 4 + 32, p.kr == KR, p.rexp == REXP.
template <int N, int DB, int NORM>
__global__ void __launch_bounds__(FStepCut<N, DB>::dmax / 4 + 32) mole_fstep_kernel(const FStepParams p)
{
    constexpr int KW = FStepCut<N, DB>::KW, REXP = FStepCut<N, DB>::REXP, KR = FStepCut<N, DB>::KR;
    using E = Elem<__nv_bfloat16>;
    constexpr int VEC = 8;
    constexpr int NV = N < VEC ? N : VEC;
    constexpr int QL = N >= VEC ? N / VEC : 1;
    constexpr int CPV = N >= VEC ? 1 : VEC / N;
    constexpr int RQ = N / 2 / KW;  // sweep vectors per thread and router chunk
    static_assert(RQ >= 1 && RQ * KW * 2 == N, "chunk count must divide N / 2");
    // Up to 16 experts the router matrix does not travel through the ring at all: every compute thread loads
    // its N / 2 vectors of the NEXT item's matrix straight from global memory (L2: all blocks share it) into
    // registers as soon as the current sweep has used them up.  The ring then carries rows only -- half the
    // bytes per item, twice the items in flight -- which is what a block's copy pipeline can keep up with.
    constexpr bool WREG = N <= 16;
    constexpr int KWR = WREG ? 0 : KW;  // router chunks per item in the ring
    constexpr int RW = N / 2;           // vectors of a whole matrix per thread
    extern __shared__ __align__(128) unsigned char smem[];

    pdl_launch_dependents();

    const int d = p.d, L = p.L, stages = p.stages, T = d / 4;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, nwarps = T >> 5;
    const long long G = gridDim.x, b0 = blockIdx.x;
    const int ntok = b0 < p.M ? static_cast<int>((p.M - b0 + G - 1) / G) : 0;
    constexpr int kr = KR, rexp = REXP, cpi = KWR + KR;  // chunks per item
    const FStepSmem m = fstep_smem(N, d, stages, NORM);
    const uint32_t wchunk_bytes = static_cast<uint32_t>(d) * N * 2 / KW, rchunk_bytes = static_cast<uint32_t>(rexp) * d * 2;

    volatile int *meta = reinterpret_cast<volatile int *>(smem + m.off_meta);
    volatile int *dead = meta + kMaxStages;
    volatile int *issued = meta + kMaxStages + 1;
    uint64_t *full = reinterpret_cast<uint64_t *>(smem + m.off_bars), *empty = full + kMaxStages;

    if (tid == 0) {
        for (int st = 0; st < stages; ++st) {
            mbar_init(full + st, 1);
            mbar_init(empty + st, nwarps);
        }
        *dead = 0;
        *issued = 0;
        meta[kMaxStages + 2] = 0;  // a flag nobody raises: lets the drain waits run their full (short) course
        mbar_init_fence();
    }
    __syncthreads();

    if (tid >= T) {
        // ================= producer warp =================
        // ids, tables and router weights are not written by the previous kernel of a chained launch, so
        // nothing here waits for it
        const bool ids64 = (p.flags & MOLE_FLAG_IDS_INT64) != 0;
        long long batch = -1, row = -1;
        int k = 0, l = 0, q = 0, pst = 0;
        uint32_t pph = 1;
        const long long total = static_cast<long long>(ntok) * L * cpi;
        for (long long ci = 0; ci < total; ++ci) {
            if (ci >= stages) {
                int ok = 1;
                if (lane == 0) {
                    ok = wait_or_give_up(empty + pst, pph, dead, p.wait_polls, true);
                    if (!ok) report_timeout(dead, p.status);
                }
                ok = __shfl_sync(0xffffffffu, ok, 0);
                if (!ok) break;
            }
            if (l == 0 && q == 0) {
                if ((k & 31) == 0) {  // ids of the next 32 tokens of this block, one per lane
                    const int kk = k + lane;
                    batch = -1;
                    if (kk < ntok) {
                        const long long t = b0 + static_cast<long long>(kk) * G;
                        batch = ids64 ? __ldg(static_cast<const long long *>(p.row_index) + t)
                                      : static_cast<long long>(__ldg(static_cast<const int *>(p.row_index) + t));
                    }
                }
                row = __shfl_sync(0xffffffffu, batch, k & 31);
            }
            const bool valid = row >= 0 && row < p.rows;
            unsigned char *slot = smem + static_cast<size_t>(pst) * kFStepSlotBytes;
            if (lane == 0) {
                if (q < KWR) {
                    mbar_expect_tx(full + pst, wchunk_bytes);
                    bulk_g2s(slot,
                             static_cast<const unsigned char *>(p.w_router) + static_cast<size_t>(l) * p.wr_stride +
                                 static_cast<size_t>(q) * wchunk_bytes,
                             wchunk_bytes, full + pst);
                } else {
                    // whole rows of experts (q - KW) * rexp ..: contiguous.  An id outside the table gathers
                    // row 0 (always present); its routed term is dropped by the consumers.
                    meta[pst] = valid ? 1 : 0;
                    if (!valid && l == 0 && q == KWR && p.status) atomicOr(p.status, MOLE_STATUS_BAD_ID);
                    mbar_expect_tx(full + pst, rchunk_bytes);
                    bulk_g2s(slot,
                             static_cast<const unsigned char *>(p.lut) + static_cast<size_t>(l) * p.lut_stride +
                                 (static_cast<size_t>(valid ? row : 0) * N + static_cast<size_t>(q - KWR) * rexp) * d * 2,
                             rchunk_bytes, full + pst);
                }
                *issued = static_cast<int>(ci + 1 < 0x7fffffff ? ci + 1 : 0x7fffffff);
            }
            __syncwarp();
            if (++q == cpi) {
                q = 0;
                if (++l == L) {
                    l = 0;
                    ++k;
                }
            }
            if (++pst == stages) {
                pst = 0;
                pph ^= 1u;
            }
        }
        return;
    }

    // ================= compute threads =================
    pdl_wait();  // hidden may still be written, and out still read, by the previous kernel
    const uint32_t smem_base = smem_u32(smem);
    const uint32_t hid_s = smem_base + m.off_hid, norm_s = smem_base + m.off_norm;
    float *partial = reinterpret_cast<float *>(smem + m.off_partial);
    float *scratch = reinterpret_cast<float *>(smem + m.off_scratch);
    bool alive = true;
    long long ci = 0;
    int st = 0;
    uint32_t ph = 0;
    auto acquire = [&]() {
        if (alive && mbar_try_wait(full + st, ph)) return;
        alive = acquire_slow(full + st, ph, dead, alive, ci < *issued, p.status, lane, p.wait_polls);
    };
    auto release = [&]() {
        __syncwarp();
        if (lane == 0) mbar_arrive(empty + st);
        ++ci;
        if (++st == stages) {
            st = 0;
            ph ^= 1u;
        }
    };

    uint4 wreg[WREG ? RW : 1];
    auto load_router = [&](int l) {  // this thread's vectors of layer l's matrix: u = tid + r * T, 16 bytes per lane, coalesced
        const uint4 *w = reinterpret_cast<const uint4 *>(static_cast<const unsigned char *>(p.w_router) + static_cast<size_t>(l) * p.wr_stride);
#pragma unroll
        for (int r = 0; r < RW; ++r) wreg[r] = ldg_nc_v4(w + tid + r * T);
    };
    if constexpr (WREG) {
        if (ntok > 0) load_router(0);
    }

#pragma unroll 1
    for (int k = 0; k < ntok; ++k) {
        const long long t = b0 + static_cast<long long>(k) * G;
        const size_t tbyte = static_cast<size_t>(t) * d * 2 + static_cast<size_t>(tid) * 8;
        uint2 own = ldcg_v2(static_cast<const unsigned char *>(p.hidden) + tbyte);  // columns 4 tid .. 4 tid + 3
        sts64(hid_s + 8u * tid, own);
        named_bar_sync(kFBarHidden, T);
#pragma unroll 1
        for (int l = 0; l < L; ++l) {
            uint32_t rd_s = hid_s;  // what the router reads
            if constexpr (NORM) {
                const float x0 = bf16_bits_to_float(own.x & 0xffffu), x1 = __uint_as_float(own.x & 0xffff0000u);
                const float x2 = bf16_bits_to_float(own.y & 0xffffu), x3 = __uint_as_float(own.y & 0xffff0000u);
                float ss = fmaf(x3, x3, fmaf(x2, x2, fmaf(x1, x1, x0 * x0)));
                ss = warp_sum(ss);
                if (lane == 0) scratch[warp] = ss;
                named_bar_sync(kFBarNorm, T);
                float total = 0.f;
                for (int w = 0; w < nwarps; ++w) total += scratch[w];
                const float rinv = 1.0f / sqrtf(total / static_cast<float>(d) + p.norm_eps);
                const uint2 wq = __ldg(reinterpret_cast<const uint2 *>(static_cast<const unsigned char *>(p.norm_weight) +
                                                                       static_cast<size_t>(l) * p.norm_stride) + tid);
                const __nv_bfloat162 y01 = __floats2bfloat162_rn((x0 * rinv) * bf16_bits_to_float(wq.x & 0xffffu),
                                                                 (x1 * rinv) * __uint_as_float(wq.x & 0xffff0000u));
                const __nv_bfloat162 y23 = __floats2bfloat162_rn((x2 * rinv) * bf16_bits_to_float(wq.y & 0xffffu),
                                                                 (x3 * rinv) * __uint_as_float(wq.y & 0xffff0000u));
                sts64(norm_s + 8u * tid, make_uint2(*reinterpret_cast<const uint32_t *>(&y01), *reinterpret_cast<const uint32_t *>(&y23)));
                named_bar_sync(kFBarNorm, T);
                rd_s = norm_s;
            }

            // ---- router sweep over the KW column chunks ----
            float acc[NV];
#pragma unroll
            for (int i = 0; i < NV; ++i) acc[i] = 0.f;
            if constexpr (WREG) {
                unsigned short hs[RW * CPV];
#pragma unroll
                for (int r = 0; r < RW; ++r) {
                    const int u = tid + r * T;
#pragma unroll
                    for (int cc = 0; cc < CPV; ++cc) hs[r * CPV + cc] = static_cast<unsigned short>(lds16(rd_s + 2u * (N >= VEC ? u / QL : u * CPV + cc)));
                }
#pragma unroll
                for (int r = 0; r < RW; ++r)
#pragma unroll
                    for (int e = 0; e < VEC; ++e) E::fma_elem(acc[e % NV], wreg[r], e, hs[r * CPV + e / NV]);
                // the registers are free again: request the next item's matrix (the next layer's, or layer 0's for
                // the block's next token); it lands while this item's softmax and weighted sum run
                if (l + 1 < L) load_router(l + 1);
                else if (k + 1 < ntok) load_router(0);
            } else {
#pragma unroll
                for (int q = 0; q < KW; ++q) {
                    acquire();
                    const uint32_t wbase = smem_base + static_cast<uint32_t>(st) * kFStepSlotBytes;
                    uint4 wv[RQ];
                    unsigned short hs[RQ * CPV];
#pragma unroll
                    for (int r = 0; r < RQ; ++r) {
                        wv[r] = lds128(wbase + 16u * static_cast<uint32_t>(tid + r * T));
                        const int u = tid + (q * RQ + r) * T;  // vector index in the whole matrix
#pragma unroll
                        for (int cc = 0; cc < CPV; ++cc) hs[r * CPV + cc] = static_cast<unsigned short>(lds16(rd_s + 2u * (N >= VEC ? u / QL : u * CPV + cc)));
                    }
                    release();  // the chunk is in registers
#pragma unroll
                    for (int r = 0; r < RQ; ++r)
#pragma unroll
                        for (int e = 0; e < VEC; ++e) E::fma_elem(acc[e % NV], wv[r], e, hs[r * CPV + e / NV]);
                }
            }
            int base = 0;
            lane_reduce_scatter<NV, NV, 16, QL>(acc, lane, base);
            partial[warp * N + (N >= VEC ? (lane % QL) * VEC : 0) + base] = acc[0];
            named_bar_sync(kFBarLogits, T);

            // ---- softmax numerators, every warp for itself (Eq. 4) ----
            const float e = softmax_numerator<N>(partial, nwarps, lane);

            // ---- weighted sum over the rows chunks (Eq. 8) ----
            float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
            float es[4] = {0.f, 0.f, 0.f, 0.f};
            bool valid = true;
#pragma unroll
            for (int c = 0; c < KR; ++c) {
                acquire();
                valid = meta[st] != 0;
                const uint32_t rbase = smem_base + static_cast<uint32_t>(st) * kFStepSlotBytes + 8u * tid;
                uint2 rv[REXP];
                float g[REXP];
#pragma unroll
                for (int i = 0; i < REXP; ++i) rv[i] = lds64(rbase + static_cast<uint32_t>(i) * d * 2);
#pragma unroll
                for (int i = 0; i < REXP; ++i) g[i] = __shfl_sync(0xffffffffu, e, c * REXP + i);
                release();  // the chunk is in registers
#pragma unroll
                for (int i = 0; i < REXP; ++i) {
                    es[i & 3] += g[i];
                    a0 = fmaf(g[i], bf16_bits_to_float(rv[i].x & 0xffffu), a0);
                    a1 = fmaf(g[i], __uint_as_float(rv[i].x & 0xffff0000u), a1);
                    a2 = fmaf(g[i], bf16_bits_to_float(rv[i].y & 0xffffu), a2);
                    a3 = fmaf(g[i], __uint_as_float(rv[i].y & 0xffff0000u), a3);
                }
            }
            const float esum = (es[0] + es[1]) + (es[2] + es[3]);
            const float inv = __frcp_rn(esum);
            if (valid) {
                const __nv_bfloat162 lo = __floats2bfloat162_rn(fmaf(a0, inv, bf16_bits_to_float(own.x & 0xffffu)),
                                                                fmaf(a1, inv, __uint_as_float(own.x & 0xffff0000u)));
                const __nv_bfloat162 hi = __floats2bfloat162_rn(fmaf(a2, inv, bf16_bits_to_float(own.y & 0xffffu)),
                                                                fmaf(a3, inv, __uint_as_float(own.y & 0xffff0000u)));
                own.x = *reinterpret_cast<const uint32_t *>(&lo);
                own.y = *reinterpret_cast<const uint32_t *>(&hi);
            }
            if (l + 1 < L) {
                sts64(hid_s + 8u * tid, own);
                named_bar_sync(kFBarHidden, T);
            } else {
                *reinterpret_cast<uint2 *>(static_cast<unsigned char *>(p.out) + tbyte) = own;
            }
        }
    }
}

#endif  // __CUDACC__

}  // namespace mole
