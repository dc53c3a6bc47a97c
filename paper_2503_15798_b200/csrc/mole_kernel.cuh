// The fused MoLE kernel for sm_100a (Eq. 4 and Eq. 8 of arXiv 2503.15798): router dot products,
// softmax over all N experts, gather of the token's N table rows, fp32 weighted sum, residual
// add -- for one layer or for L chained layers in one launch.
//
// Work decomposition.  A block owns whole tokens: it walks over its tokens t = b, b + G, b + 2G,
// ... (G blocks in the grid) and, per token, over the layers l = 0 .. L-1; one (token, layer)
// pair is an "item".  The chain h_{l+1} = h_l + sum_j g_j(h_l) LUT_l[id][j] of a token never
// leaves the block: the running hidden state stays in shared memory, rounded to the storage
// type after every layer exactly as a layer-by-layer execution would round it.  There is no
// communication between blocks.
//
// Data movement.  An item is cut into K chunks.  Everything it needs is pulled through a ring of
// shared-memory slots, one chunk per slot, by bulk asynchronous copies (TMA engine, untiled, every
// copy into the block's own shared memory) that one extra "producer" warp issues `stages` chunks
// ahead: first (when the router
// matrix streams: L > 1, or a matrix too large to stay resident) the K chunks [dcc][N] of the
// layer's router matrix, dcc = d / K columns each, then the K chunks of the token's table rows --
// [N][dcc], N short pieces per chunk, or, where K divides N (MODE 3), the whole rows [N/K][d] of
// N/K experts in one contiguous copy, which the copy engine moves three times as fast.  The rows
// depend only on the id, so they run ahead of the arithmetic and, in a chained launch, ahead of
// the previous kernel.  A token's hidden state arrives with its first chunk in a small ring of
// its own (in DIRECT kernels the block's first token excepted: the compute warps load it
// themselves).  Completion is counted on one mbarrier per slot ("full"); the consumer warps hand
// a slot back through a second one ("empty").  Otherwise (L == 1, small matrix) the router matrix
// is loaded once per block and stays.
//
// Arithmetic per item (consumer warps): a conflict-free linear sweep over the router chunks in
// shared memory gives per-lane partial logits, a shuffle reduce-scatter sums them over the warp
// and shared memory over the warps; warp 0 evaluates the softmax numerators (fp32, expf) for
// the block, and every warp combines the row chunks of the column groups it owns, dividing by
// the sum of the numerators.
#pragma once

#include <math.h>

#include "mole_common.cuh"

namespace mole {

constexpr int kMaxN = 64;           // experts
constexpr int kMaxChunks = 16;      // column chunks per token
constexpr int kMaxConsumers = 256;  // compute threads per block
constexpr int kMaxStages = 8;       // ring depth
constexpr int kBarLogits = 1;       // named barriers of the consumer warps: partial logits written,
constexpr int kBarGates = 2;        // softmax numerators written,
constexpr int kBarHidden = 3;       // running hidden state written
constexpr uint32_t kWaitPolls = 1u << 24;   // default poll limit: >= 1 s of polling before a wait gives up
constexpr uint32_t kDrainPolls = 1u << 14;  // after a failure: short waits for copies still in flight

struct StepParams {
    const void *hidden, *residual, *row_index, *lut, *w_router;
    const void *norm_weight;  // [d] scale of the RMSNorm in front of the router (NORM kernels), else unused
    long long norm_stride;    // bytes between the scale vectors of consecutive layers
    float norm_eps;
    void *out;
    float *gates_out;
    uint32_t *status;
    long long lut_stride, wr_stride;  // bytes between layers
    long long M, rows;
    int N, d, K, dcc, L;
    int stages, hring, wr_in_ring, consumers;
    uint32_t flags;
    uint32_t wait_polls;  // polls after which a wait on the ring gives up (kWaitPolls unless a test shortens it)
};

// Shared-memory map, computed the same way on the host (for the size) and in the kernel.
struct SmemMap {
    uint32_t chunk_bytes;  // one ring slot: a [dcc][N] router chunk or an [N][dcc] rows chunk
    uint32_t hid_bytes;    // one hidden state: d elements
    uint32_t off_wr, off_hring, off_hid, off_norm, off_partial, off_gates, off_meta, off_bars, total;
};
__host__ __device__ inline uint32_t up128(uint32_t x) { return (x + 127u) & ~127u; }
__host__ __device__ inline SmemMap smem_map(int N, int d, int dcc, int eb, int stages, int hring, int wr_in_ring,
                                            int consumers, int norm)
{
    SmemMap m;
    m.chunk_bytes = static_cast<uint32_t>(N) * dcc * eb;
    m.hid_bytes = static_cast<uint32_t>(d) * eb;
    const uint32_t warps = consumers / 32;
    m.off_wr = stages * up128(m.chunk_bytes);                                             // resident router matrix (L == 1)
    m.off_hring = m.off_wr + (wr_in_ring ? 0u : up128(static_cast<uint32_t>(d) * N * eb));  // hidden states of the tokens in flight
    m.off_hid = m.off_hring + hring * up128(m.hid_bytes);                                 // running hidden state between layers
    m.off_norm = m.off_hid + up128(m.hid_bytes);                                          // RMSNorm(hidden), what a normalised router reads
    m.off_partial = m.off_norm + (norm ? up128(m.hid_bytes) : 0u);
    m.off_gates = m.off_partial + up128(warps * N * 4);
    m.off_meta = m.off_gates + up128(N * 4);
    m.off_bars = m.off_meta + up128((kMaxStages + 3) * 4);
    m.total = m.off_bars + (2 * kMaxStages + 1) * 8;
    return m;
}

#ifdef __CUDACC__

// Sum n per-lane values over the lanes that differ in bits o, o/2, .., omin: every step halves
// the number of values a lane still carries (n - 1 + a few shuffles instead of log2 * n).  On
// return a[0 .. left) hold the totals of values base .. base + left - 1; lanes that end up with
// the same values hold identical copies.
template <int NTOT, int n, int o, int omin>
__device__ __forceinline__ void lane_reduce_scatter(float (&a)[NTOT], int lane, int &base)
{
    if constexpr (o >= omin) {
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
            lane_reduce_scatter<NTOT, half, o / 2, omin>(a, lane, base);
        } else {
            a[0] += __shfl_xor_sync(0xffffffffu, a[0], o);
            lane_reduce_scatter<NTOT, 1, o / 2, omin>(a, lane, base);
        }
    }
}
// number of values a lane is left with after lane_reduce_scatter<.., n, o, omin>
template <int n, int o, int omin>
struct ReduceScatterLeft {
    static constexpr int value = (o >= omin && n > 1) ? ReduceScatterLeft<n / 2, o / 2, omin>::value : n;
};
template <int n, int omin>
struct ReduceScatterLeft<n, 0, omin> {
    static constexpr int value = n;
};

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

// Bounded wait shared by producer and consumers.  `dead` (shared memory) is raised by whoever
// gives up first; everyone else then stops waiting at once.
// `patient`: sleep after every failed poll (the producer, which runs several items ahead and
// must not take issue slots from the warps that compute).
static __device__ __noinline__ bool wait_or_give_up(uint64_t *bar, uint32_t parity, volatile int *dead, uint32_t polls,
                                             bool patient = false)
{
#pragma unroll 1
    for (uint32_t i = 0; i < polls; ++i) {
        if (mbar_try_wait(bar, parity)) return true;
        if (patient || i > 64) {
            __nanosleep(64);
            if ((i & 127u) == 0 && *dead) return false;
        }
    }
    return false;
}

// Partial router logits over one chunk of columns, fast path (N a power of two the kernel is
// compiled for).  The router chunk [ncols][N] is swept linearly, 16 bytes per lane, so a warp
// reads 512 consecutive bytes per step (no bank conflicts for any N).  A 16-byte vector holds
// either VEC consecutive experts of one column (N >= VEC) or VEC / N whole columns (N < VEC);
// since the sweep stride is a multiple of 32 vectors, a lane always meets the same experts and
// keeps only min(VEC, N) fp32 accumulators across all chunks of an item.
template <typename T, int NFAST>
struct Sweep {
    using E = Elem<T>;
    using H = typename E::H;
    static constexpr int VEC = E::VEC;
    static constexpr int NV = NFAST < VEC ? NFAST : VEC;        // accumulators per lane
    static constexpr int QL = NFAST >= VEC ? NFAST / VEC : 1;   // vectors per column
    static constexpr int CPV = NFAST >= VEC ? 1 : VEC / NFAST;  // columns per vector
    static constexpr int UNR = 16;  // vectors in flight per lane: a whole chunk for the widths of Table 2 (measured best)
    float acc[NV];

    __device__ __forceinline__ void clear()
    {
#pragma unroll
        for (int i = 0; i < NV; ++i) acc[i] = 0.f;
    }
    // one vector: its VEC values times the hidden value(s) of its column(s)
    __device__ __forceinline__ void mac(const uint4 &w, const H (&h)[CPV])
    {
#pragma unroll
        for (int e = 0; e < VEC; ++e) E::fma_elem(acc[e % NV], w, e, h[e / NV]);
    }
    static __device__ __forceinline__ void hidden_of(uint32_t haddr, int u, H (&h)[CPV])
    {
#pragma unroll
        for (int cc = 0; cc < CPV; ++cc) h[cc] = E::lds_h(haddr, NFAST >= VEC ? u / QL : u * CPV + cc);
    }
    // waddr: the chunk in shared memory; haddr: the hidden values of the chunk's first column on
    __device__ __forceinline__ void chunk(uint32_t waddr, uint32_t haddr, int ncols, int tid, int nc)
    {
        const int nvec = ncols * NFAST / VEC;
        int u0 = tid;
#pragma unroll 1
        for (; u0 + (UNR - 1) * nc < nvec; u0 += UNR * nc) {  // full batches: all loads first
            uint4 wv[UNR];
            H hv[UNR][CPV];
#pragma unroll
            for (int r = 0; r < UNR; ++r) {
                wv[r] = lds128(waddr + 16u * (u0 + r * nc));
                hidden_of(haddr, u0 + r * nc, hv[r]);
            }
#pragma unroll
            for (int r = 0; r < UNR; ++r) mac(wv[r], hv[r]);
        }
#pragma unroll 1
        for (; u0 < nvec; u0 += nc) {  // tail
            H h[CPV];
            const uint4 w = lds128(waddr + 16u * u0);
            hidden_of(haddr, u0, h);
            mac(w, h);
        }
    }
    // sum over the lanes of the warp; partial_warp[j] = this warp's share of logit j
    __device__ __forceinline__ void finish(int lane, float *partial_warp)
    {
        int base = 0;
        lane_reduce_scatter<NV, NV, 16, QL>(acc, lane, base);
        constexpr int left = ReduceScatterLeft<NV, 16, QL>::value;
        const int first = (NFAST >= VEC ? (lane % QL) * VEC : 0) + base;
#pragma unroll
        for (int i = 0; i < left; ++i) partial_warp[first + i] = acc[i];
    }
};
// any N <= 64: one warp per expert, lanes stride over the columns; partial[j] accumulates over chunks
template <typename T>
struct Sweep<T, 0> {
    using E = Elem<T>;
    __device__ __forceinline__ void clear() {}
    __device__ __forceinline__ void chunk_any(uint32_t waddr, uint32_t haddr, int ncols, int N, int warp, int lane,
                                              int nwarps, bool first, float *partial)
    {
        for (int j = warp; j < N; j += nwarps) {
            float z = 0.f;
            for (int cc = lane; cc < ncols; cc += 32) z = fmaf(E::lds_scalar(haddr, cc), E::lds_scalar(waddr, cc * N + j), z);
            z = warp_sum(z);
            if (lane == 0) partial[j] = first ? z : partial[j] + z;
        }
    }
};

// Weighted sum of one item (Eq. 8): out = res + sum_j g_j * row_j over one chunk of columns,
// with g_j = e_j / sum_k e_k given as the un-normalised e_j: the lanes add up the e_j of their
// experts next to the rows, so the normalisation costs no reduction of its own -- one reciprocal
// and one multiply per column at the end.
// A warp covers 32 / P column groups of 16 bytes; the P lanes that share a group (lane bits
// above log2(32 / P), so that the 8 lanes of a quarter warp read 8 different groups and never
// collide on a bank) each sum a contiguous chunk of the experts, a shuffle reduce-scatter adds
// the P partial sums and leaves every lane with VEC / P finished columns, to which it adds the
// residual, rounds once and stores 16 / P bytes (to global memory, or to the running hidden
// slice in shared memory when dst_g is null).
template <typename T, int P>
__device__ __forceinline__ void combine_item(uint32_t rows, uint32_t haddr, uint32_t gates, const unsigned char *residual_g,
                                             unsigned char *dst_g, uint32_t dst_s, int N, int ngrp, bool valid, int warp,
                                             int lane, int nwarps)
{
    using E = Elem<T>;
    constexpr int VEC = E::VEC;
    constexpr int GPW = 32 / P;   // column groups per warp
    constexpr int W = 4 / P;      // 32-bit words a lane finishes
    constexpr int VPW = VEC / 4;  // values per word: 2 (bf16) or 1 (fp32)
    constexpr int UNR = 16;       // rows in flight per lane: all N = 16 experts of a column group (measured best)
    const int part = lane / GPW, gl = lane % GPW;
    const int chunk = (N + P - 1) / P;
    const int jb = part * chunk, je = (jb + chunk < N) ? jb + chunk : N;
#pragma unroll 1
    for (int g0 = warp * GPW; g0 < ngrp; g0 += nwarps * GPW) {
        const int grp = g0 + gl;
        const bool in = grp < ngrp;
        const int gg = in ? grp : ngrp - 1;
        float acc[VEC];
        float esum = 0.f;
#pragma unroll
        for (int i = 0; i < VEC; ++i) acc[i] = 0.f;
        if (valid) {
            int j0 = jb;
#pragma unroll 1
            for (; j0 + UNR <= je; j0 += UNR) {  // full batches: all loads first
                uint4 rv[UNR];
                float gv[UNR];
#pragma unroll
                for (int r = 0; r < UNR; ++r) rv[r] = lds128(rows + 16u * ((j0 + r) * ngrp + gg));
                if ((j0 & 3) == 0) {  // the batch's softmax numerators: four per (broadcast) load when aligned
#pragma unroll
                    for (int r = 0; r < UNR; r += 4) {
                        const uint4 g4 = lds128(gates + 4u * (j0 + r));
                        gv[r] = __uint_as_float(g4.x), gv[r + 1] = __uint_as_float(g4.y);
                        gv[r + 2] = __uint_as_float(g4.z), gv[r + 3] = __uint_as_float(g4.w);
                    }
                } else {
#pragma unroll
                    for (int r = 0; r < UNR; ++r) gv[r] = __uint_as_float(lds32(gates + 4u * (j0 + r)));
                }
                float es[4] = {0.f, 0.f, 0.f, 0.f};  // their sum, four short chains instead of one long one
#pragma unroll
                for (int r = 0; r < UNR; ++r) {
                    es[r & 3] += gv[r];
                    E::fma_row(acc, rv[r], gv[r]);
                }
                esum += (es[0] + es[1]) + (es[2] + es[3]);
            }
#pragma unroll 1
            for (; j0 < je; ++j0) {  // tail
                const uint4 rv = lds128(rows + 16u * (j0 * ngrp + gg));
                const float g = __uint_as_float(lds32(gates + 4u * j0));
                esum += g;
                E::fma_row(acc, rv, g);
            }
        }
        int base = 0;
        if constexpr (P > 1) {
            lane_reduce_scatter<VEC, VEC, 16, GPW>(acc, lane, base);
#pragma unroll
            for (int o = 16; o >= GPW; o >>= 1) esum += __shfl_xor_sync(0xffffffffu, esum, o);
        }
        const float inv = __frcp_rn(esum);
        const int word = gg * 4 + base / VPW;  // first 32-bit word of this lane's columns
        uint32_t rw[W];
        if (residual_g) {
            const uint32_t *rsrc = reinterpret_cast<const uint32_t *>(residual_g) + word;
            if constexpr (W == 4) {
                const uint4 v = __ldcg(reinterpret_cast<const uint4 *>(rsrc));
                rw[0] = v.x, rw[1] = v.y, rw[2] = v.z, rw[3] = v.w;
            } else if constexpr (W == 2) {
                const uint2 v = __ldcg(reinterpret_cast<const uint2 *>(rsrc));
                rw[0] = v.x, rw[1] = v.y;
            } else {
                rw[0] = __ldcg(rsrc);
            }
        } else {
            const uint32_t rsrc = haddr + 4u * word;
            if constexpr (W == 4) {
                const uint4 v = lds128(rsrc);
                rw[0] = v.x, rw[1] = v.y, rw[2] = v.z, rw[3] = v.w;
            } else if constexpr (W == 2) {
                const uint2 v = lds64(rsrc);
                rw[0] = v.x, rw[1] = v.y;
            } else {
                rw[0] = lds32(rsrc);
            }
        }
        if (valid) {
#pragma unroll
            for (int w = 0; w < W; ++w) {
                if constexpr (VPW == 2) {
                    const float lo = fmaf(acc[2 * w], inv, __uint_as_float(rw[w] << 16));
                    const float hi = fmaf(acc[2 * w + 1], inv, __uint_as_float(rw[w] & 0xffff0000u));
                    const __nv_bfloat162 b = __floats2bfloat162_rn(lo, hi);
                    rw[w] = *reinterpret_cast<const uint32_t *>(&b);
                } else {
                    rw[w] = __float_as_uint(fmaf(acc[w], inv, __uint_as_float(rw[w])));
                }
            }
        }
        if (in) {
            if (dst_g) {
                uint32_t *o = reinterpret_cast<uint32_t *>(dst_g) + word;
                if constexpr (W == 4) *reinterpret_cast<uint4 *>(o) = make_uint4(rw[0], rw[1], rw[2], rw[3]);
                else if constexpr (W == 2) *reinterpret_cast<uint2 *>(o) = make_uint2(rw[0], rw[1]);
                else *o = rw[0];
            } else {
                const uint32_t o = dst_s + 4u * word;
                if constexpr (W == 4) sts128(o, make_uint4(rw[0], rw[1], rw[2], rw[3]));
                else if constexpr (W == 2) sts64(o, make_uint2(rw[0], rw[1]));
                else sts32(o, rw[0]);
            }
        }
    }
}

// The same weighted sum when an item's rows arrive cut by EXPERTS instead of by columns: chunk kk
// holds the whole rows of experts kk*ne .. kk*ne + ne - 1, contiguous in the table, so that one bulk
// copy brings it (a column chunk of several rows is N short pieces, which the copy engine moves at a
// third of the rate).  A lane owns up to GPL column groups of 16 bytes (group = tid + i * nc) over
// ALL d columns and carries their fp32 sums from chunk to chunk; after the last chunk it divides by
// the sum of the numerators, adds the residual, rounds once and stores.
template <typename T, int GPL>
struct RowSums {
    using E = Elem<T>;
    static constexpr int VEC = E::VEC;
    static constexpr int UNR = 8;  // experts in flight per column group
    float acc[GPL][VEC];
    float esum;

    __device__ __forceinline__ void clear()
    {
#pragma unroll
        for (int i = 0; i < GPL; ++i)
#pragma unroll
            for (int e = 0; e < VEC; ++e) acc[i][e] = 0.f;
        esum = 0.f;
    }
    // rows: the chunk [ne][d] in shared memory; gates: numerators of its first expert on
    __device__ __forceinline__ void chunk(uint32_t rows, uint32_t gates, int ne, int ngrp, int tid, int nc)
    {
        int j0 = 0;
#pragma unroll 1
        for (; j0 + UNR <= ne; j0 += UNR) {  // full batches: all loads first
            uint4 rv[GPL][UNR];
            float gv[UNR];
#pragma unroll
            for (int i = 0; i < GPL; ++i) {
                const int g = tid + i * nc;
                const int gg = g < ngrp ? g : ngrp - 1;
#pragma unroll
                for (int r = 0; r < UNR; ++r) rv[i][r] = lds128(rows + 16u * ((j0 + r) * ngrp + gg));
            }
#pragma unroll
            for (int r = 0; r < UNR; r += 4) {  // UNR and every chunk's first expert are multiples of four here
                const uint4 g4 = lds128(gates + 4u * (j0 + r));
                gv[r] = __uint_as_float(g4.x), gv[r + 1] = __uint_as_float(g4.y);
                gv[r + 2] = __uint_as_float(g4.z), gv[r + 3] = __uint_as_float(g4.w);
            }
            float es[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
            for (int r = 0; r < UNR; ++r) es[r & 3] += gv[r];
            esum += (es[0] + es[1]) + (es[2] + es[3]);
#pragma unroll
            for (int i = 0; i < GPL; ++i)
#pragma unroll
                for (int r = 0; r < UNR; ++r) E::fma_row(acc[i], rv[i][r], gv[r]);
        }
#pragma unroll 1
        for (; j0 < ne; ++j0) {  // tail (and every chunk of fewer than UNR experts)
            const float g = __uint_as_float(lds32(gates + 4u * j0));
            esum += g;
#pragma unroll
            for (int i = 0; i < GPL; ++i) {
                const int grp = tid + i * nc;
                const int gg = grp < ngrp ? grp : ngrp - 1;
                const uint4 rv = lds128(rows + 16u * (j0 * ngrp + gg));
                E::fma_row(acc[i], rv, g);
            }
        }
    }
    // residual from global memory (residual_g) or from the hidden state in shared memory (haddr);
    // result to global memory (dst_g) or to the running hidden state in shared memory (dst_s)
    __device__ __forceinline__ void finish(uint32_t haddr, const unsigned char *residual_g, unsigned char *dst_g, uint32_t dst_s,
                                           int ngrp, bool valid, int tid, int nc)
    {
        constexpr int VPW = VEC / 4;
        const float inv = __frcp_rn(esum);
#pragma unroll
        for (int i = 0; i < GPL; ++i) {
            const int grp = tid + i * nc;
            if (grp < ngrp) {
                uint4 v = residual_g ? __ldcg(reinterpret_cast<const uint4 *>(residual_g) + grp) : lds128(haddr + 16u * grp);
                if (valid) {
                    uint32_t rw[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
                    for (int w = 0; w < 4; ++w) {
                        if constexpr (VPW == 2) {
                            const float lo = fmaf(acc[i][2 * w], inv, __uint_as_float(rw[w] << 16));
                            const float hi = fmaf(acc[i][2 * w + 1], inv, __uint_as_float(rw[w] & 0xffff0000u));
                            const __nv_bfloat162 b = __floats2bfloat162_rn(lo, hi);
                            rw[w] = *reinterpret_cast<const uint32_t *>(&b);
                        } else {
                            rw[w] = __float_as_uint(fmaf(acc[i][w], inv, __uint_as_float(rw[w])));
                        }
                    }
                    v = make_uint4(rw[0], rw[1], rw[2], rw[3]);
                }
                if (dst_g) *(reinterpret_cast<uint4 *>(dst_g) + grp) = v;
                else sts128(dst_s + 16u * grp, v);
            }
        }
    }
};

// The normalisation in front of the router of the paper's decoder layer (App. A.2 listing: the router
// reads the normalised hidden state, the residual stays as it was): y = (x / sqrt(mean(x^2) + eps)) * w,
// rounded once to the storage type, as a model that materialises the normalised activations would
// hold it.  src: the token's hidden state in shared memory; dst: where the router sweep will read.
// `scratch` holds one float per warp; two block barriers (`bar`) separate the three phases.
template <typename T>
__device__ __forceinline__ void rmsnorm_to_shared(uint32_t src, uint32_t dst, const void *weight_g, float eps, int d,
                                                  float *scratch, int bar, int tid, int nc, int lane, int warp, int nwarps)
{
    using E = Elem<T>;
    constexpr int VEC = E::VEC;
    const int ngrp = d / VEC;
    const uint4 *wg = static_cast<const uint4 *>(weight_g);
    // this thread's first vector of the scale comes from L2: asked for before the sum of squares, not after it
    uint4 w_first = make_uint4(0u, 0u, 0u, 0u);
    if (tid < ngrp) w_first = __ldg(wg + tid);
    float ss = 0.f;
    for (int g = tid; g < ngrp; g += nc) {
        float x[VEC];
        E::unpack(lds128(src + 16u * g), x);
#pragma unroll
        for (int i = 0; i < VEC; ++i) ss = fmaf(x[i], x[i], ss);
    }
    ss = warp_sum(ss);
    if (lane == 0) scratch[warp] = ss;
    named_bar_sync(bar, nc);
    float total = 0.f;
    for (int w = 0; w < nwarps; ++w) total += scratch[w];  // the same order in every thread
    const float r = 1.0f / sqrtf(total / static_cast<float>(d) + eps);
    for (int g = tid; g < ngrp; g += nc) {
        float x[VEC], w[VEC];
        E::unpack(lds128(src + 16u * g), x);
        E::unpack(g == tid ? w_first : __ldg(wg + g), w);
        uint32_t o[4];
        if constexpr (VEC == 8) {
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const __nv_bfloat162 b = __floats2bfloat162_rn((x[2 * i] * r) * w[2 * i], (x[2 * i + 1] * r) * w[2 * i + 1]);
                o[i] = *reinterpret_cast<const uint32_t *>(&b);
            }
        } else {
#pragma unroll
            for (int i = 0; i < 4; ++i) o[i] = __float_as_uint((x[i] * r) * w[i]);
        }
        sts128(dst + 16u * g, make_uint4(o[0], o[1], o[2], o[3]));
    }
    named_bar_sync(bar, nc);  // the normalised state is complete (and `scratch` free again)
}

// Cold paths, kept out of the consumers' loop body (its size shows in instruction-fetch stalls).
static __device__ __noinline__ void report_timeout(volatile int *dead, uint32_t *status)
{
    if (!*dead && status) atomicOr(status, MOLE_STATUS_TIMEOUT);
    *dead = 1;
}
static __device__ __noinline__ void write_gates(float *gates_out, long long t, int N, int lane, float e0, float e1)
{
    const float esum = warp_sum(e0 + e1);
    if (lane < N) gates_out[t * N + lane] = e0 / esum;
    if (lane + 32 < N) gates_out[t * N + lane + 32] = e1 / esum;
}
static __device__ __noinline__ float logit_max(float z0, float z1, int N, int lane)
{
    return warp_max(fmaxf(lane < N ? z0 : -INFINITY, lane + 32 < N ? z1 : -INFINITY));
}

// Everything about a ring slot that is not the first, successful poll: the bounded wait of a warp
// that is still computing (returns whether the data arrived; reports the timeout otherwise), or --
// for a warp that has given up -- a short wait that lets copies already issued land, so that none
// is in flight when the block exits.
static __device__ __noinline__ bool acquire_slow(uint64_t *bar, uint32_t parity, volatile int *dead, bool alive, bool issued,
                                          uint32_t *status, int lane, uint32_t polls)
{
    if (alive) {
        if (wait_or_give_up(bar, parity, dead, polls)) return true;
        if (lane == 0) report_timeout(dead, status);
        if (issued) (void)wait_or_give_up(bar, parity, dead + 2, kDrainPolls);  // this chunk's copies may still be on their way
        return false;
    }
    if (issued) (void)wait_or_give_up(bar, parity, dead + 2, kDrainPolls);
    return false;
}

// T: storage type.  NFAST: compile-time N of the unrolled router (0 = any N <= 64, slower).
// P: lanes that share one 16-byte column group in the combine (MODE 3: column groups per lane).
// MODE: the common launch shapes with their flags fixed at compile time (a smaller loop body:
// measured 10 % faster), 0 = any: 1 = router chunks in the ring, one chunk per item; 2 = router
// resident, one chunk per item; 3 = router chunks in the ring, several chunks per item, the rows
// cut by experts (K divides N) instead of by columns.
// SHAPE: the layer widths of the paper's Table 2 with d, the chunk width and the number of compute
// threads as constants (0 = any): 1: d = 768; 2: d = 1024; 3: d = 2048 in chunks of 512; 4: d = 2048 in
// chunks of 1024 (fused steps of at most one token per SM).
// DIRECT: the compute warps load the hidden state of the block's first token themselves, with plain
// 16-byte loads, instead of waiting for the producer's bulk copy (a variant of its own because any
// growth of the loop body costs the other launches 2 - 6 %).
// NORM: the router reads RMSNorm(hidden) -- normalised into a buffer of its own in shared memory
// after the hidden state has landed (layer l of a fused step with the l-th scale vector) -- while
// the residual stays the hidden state itself (App. A.2 listing).
template <int SHAPE>
struct ShapeOf {
    static constexpr int d = SHAPE == 1 ? 768 : (SHAPE == 2 ? 1024 : 2048);
    static constexpr int dcc = SHAPE == 1 ? 768 : (SHAPE == 2 ? 1024 : (SHAPE == 3 ? 512 : 1024));
    static constexpr int consumers = SHAPE == 1 ? 96 : 128;
};
template <typename T, int NFAST, int P, int MODE, int SHAPE, int DIRECT = 0, int NORM = 0>
__global__ void __launch_bounds__(kMaxConsumers + 32) mole_step_kernel(const StepParams p)
{
    using E = Elem<T>;
    constexpr int VEC = E::VEC;
    constexpr int EB = static_cast<int>(sizeof(T));
    extern __shared__ __align__(128) unsigned char smem[];

    pdl_launch_dependents();

    const int N = NFAST > 0 ? NFAST : p.N;
    const int K = (MODE == 1 || MODE == 2) ? 1 : p.K, L = p.L, stages = p.stages, HR = p.hring;
    const int dcc = SHAPE ? ShapeOf<SHAPE>::dcc : p.dcc, d = SHAPE ? ShapeOf<SHAPE>::d : p.d;
    const int nc = SHAPE ? ShapeOf<SHAPE>::consumers : p.consumers;
    const bool ring = MODE == 0 ? (p.wr_in_ring != 0) : (MODE != 2);  // router chunks travel through the ring
    constexpr bool kRowsByExpert = MODE == 3;  // rows chunk kk = the whole rows of experts kk*N/K ..
    const SmemMap m = smem_map(N, d, dcc, EB, stages, HR, ring, nc, NORM);
    const uint32_t slot_bytes = up128(m.chunk_bytes), hid_stride = up128(m.hid_bytes);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const long long G = gridDim.x, b0 = blockIdx.x;
    const int ntok = b0 < p.M ? static_cast<int>((p.M - b0 + G - 1) / G) : 0;  // tokens of this block
    const int cpi = (ring ? 2 : 1) * K;                                // chunks per item

    volatile int *meta = reinterpret_cast<volatile int *>(smem + m.off_meta);  // [stages] row valid
    volatile int *dead = meta + kMaxStages;        // somebody gave up waiting
    volatile int *issued = meta + kMaxStages + 1;  // chunks whose copies have been issued
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem + m.off_bars);
    uint64_t *full = bars, *empty = bars + kMaxStages, *wrbar = bars + 2 * kMaxStages;

    if (tid == 0) {
        for (int st = 0; st < stages; ++st) {
            mbar_init(full + st, 1);
            mbar_init(empty + st, nc / 32);
        }
        mbar_init(wrbar, 1);
        *dead = 0;
        *issued = 0;
        meta[kMaxStages + 2] = 0;  // a flag nobody raises: lets the drain waits run their full (short) course
        mbar_init_fence();
    }
    __syncthreads();

    if (tid >= nc) {
        // ================= producer warp: issues every copy, `stages` chunks ahead ================
        const bool ids64 = (p.flags & MOLE_FLAG_IDS_INT64) != 0;
        long long batch = -1, row = -1;
        int k = 0, l = 0, q = 0;  // token of this block, layer, chunk of the item: the next chunk to issue
        int pst = 0, he = 0;      // its ring slot; hidden-ring entry of token k
        uint32_t pph = 1;         // parity of the `empty` phase that frees that slot (first reuse: phase 0 done)
        const long long total = static_cast<long long>(ntok) * L * cpi;
        if (!ring && ntok > 0 && lane == 0) {
            const uint32_t wr_bytes = static_cast<uint32_t>(d) * N * EB;
            mbar_expect_tx(wrbar, wr_bytes);
            bulk_g2s(smem + m.off_wr, p.w_router, wr_bytes, wrbar);
        }
        auto hidden_copy = [&](int tok, int entry, int st) {
            const long long t = b0 + static_cast<long long>(tok) * G;
            bulk_g2s(smem + m.off_hring + static_cast<size_t>(entry) * hid_stride,
                     static_cast<const unsigned char *>(p.hidden) + static_cast<size_t>(t) * d * EB, m.hid_bytes, full + st);
        };
        // Issue the next chunk; the hidden state (first chunk of a token) only if with_hidden.  With
        // DIRECT the block's first token is the exception: the compute warps fetch its hidden state
        // themselves.
        constexpr int k_first_copied = DIRECT ? 1 : 0;
        auto issue = [&](long long ci, bool with_hidden) {
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
            const bool first = l == 0 && q == 0;
            const int st = pst;
            unsigned char *slot = smem + static_cast<size_t>(st) * slot_bytes;
            if (lane == 0) {
                meta[st] = valid ? 1 : 0;
                if (!valid && first && p.status) atomicOr(p.status, MOLE_STATUS_BAD_ID);
                mbar_expect_tx(full + st, m.chunk_bytes + (first && k >= k_first_copied ? m.hid_bytes : 0u));
                *issued = static_cast<int>(ci + 1 < 0x7fffffff ? ci + 1 : 0x7fffffff);
            }
            __syncwarp();
            if (ring && q < K) {
                // router chunk: columns q*dcc .. of W_r[l], contiguous
                if (lane == 0)
                    bulk_g2s(slot,
                             static_cast<const unsigned char *>(p.w_router) + static_cast<size_t>(l) * p.wr_stride +
                                 static_cast<size_t>(q) * m.chunk_bytes,
                             m.chunk_bytes, full + st);
            } else {
                // rows chunk: columns kk*dcc .. of the N rows of the id.  An id outside the table
                // gathers row 0 (always present); its routed term is dropped later.
                const int kk = ring ? q - K : q;
                const unsigned char *src = static_cast<const unsigned char *>(p.lut) + static_cast<size_t>(l) * p.lut_stride +
                                           (static_cast<size_t>(valid ? row : 0) * N * d + static_cast<size_t>(kk) * dcc) * EB;
                if (kRowsByExpert) {
                    // N / K whole rows, contiguous: the same number of bytes as a column chunk
                    if (lane == 0)
                        bulk_g2s(slot, src + (static_cast<size_t>(kk) * (N / K) * d - static_cast<size_t>(kk) * dcc) * EB,
                                 m.chunk_bytes, full + st);
                } else if (K == 1) {
                    if (lane == 0) bulk_g2s(slot, src, m.chunk_bytes, full + st);  // the N rows of an id are contiguous
                } else {
                    const uint32_t piece = static_cast<uint32_t>(dcc) * EB;
                    for (int j = lane; j < N; j += 32)
                        bulk_g2s(slot + static_cast<size_t>(j) * piece, src + static_cast<size_t>(j) * d * EB, piece, full + st);
                }
            }
            if (with_hidden && first && k >= k_first_copied && lane == 31) hidden_copy(k, he, st);
            if (++q == cpi) {
                q = 0;
                if (++l == L) {
                    l = 0;
                    ++k;
                    if (++he == HR) he = 0;
                }
            }
            if (++pst == stages) {
                pst = 0;
                pph ^= 1u;
            }
        };
        // The first `stages` chunks need no free slot and -- except for hidden, which the previous
        // kernel of a chained launch writes -- nothing upstream: issue them before the grid
        // dependency is waited for.
        const long long pre = total < stages ? total : stages;
        for (long long ci = 0; ci < pre; ++ci) issue(ci, false);
        pdl_wait();
        fence_proxy_async_global();
        if (lane == 31) {
            const int per_tok = L * cpi;  // chunk tok*per_tok is the first chunk of token tok
            for (int tok = k_first_copied; static_cast<long long>(tok) * per_tok < pre; ++tok)
                hidden_copy(tok, tok % HR, static_cast<int>((static_cast<long long>(tok) * per_tok) % stages));
        }
        for (long long ci = pre; ci < total; ++ci) {
            int ok = 1;
            if (lane == 0) {
                ok = wait_or_give_up(empty + pst, pph, dead, p.wait_polls, true);
                if (!ok) report_timeout(dead, p.status);
            }
            ok = __shfl_sync(0xffffffffu, ok, 0);
            if (!ok) break;
            issue(ci, true);
        }
    } else {
        // ================= consumer warps: router, softmax, combine ================================
        pdl_wait();  // out may still be read, and hidden / residual written, by the previous kernel
        const int nwarps = nc / 32;
        const int ngrp = dcc / VEC;  // 16-byte column groups of one chunk
        float *partial = reinterpret_cast<float *>(smem + m.off_partial);  // [nwarps][N]
        float *gates = reinterpret_cast<float *>(smem + m.off_gates);      // [N] softmax numerators of the current item
        const uint32_t smem_base = smem_u32(smem);
        const uint32_t hid_s = smem_base + m.off_hid, norm_s = smem_base + m.off_norm, gates_s = smem_u32(gates);
        const uint32_t chunk_cols_bytes = static_cast<uint32_t>(dcc) * EB;
        // After a wait has timed out (`alive` false) the warp stops waiting but keeps going through the
        // arithmetic and the barriers on whatever the slots hold -- every address stays inside shared
        // memory and the block's own rows of `out` -- so that no other warp is left at a barrier; the
        // status word says that the outputs are meaningless.
        bool alive = true;
        constexpr bool direct = DIRECT != 0;

        auto give_up = [&]() {
            if (lane == 0) report_timeout(dead, p.status);
            alive = false;
        };
        // Make the ring slot `st` usable (its copies have landed) -- or, after a failure, give
        // copies that were issued a short time to land so that none is in flight at exit.
        long long ci = 0;  // chunks consumed so far
        auto acquire = [&](int st, uint32_t ph) {
            if (alive && mbar_try_wait(full + st, ph)) return;  // the usual case: the copies have landed
            alive = acquire_slow(full + st, ph, dead, alive, ci < *issued, p.status, lane, p.wait_polls);
        };
        if (!ring && ntok > 0) {
            if (!wait_or_give_up(wrbar, 0, dead, p.wait_polls)) {
                give_up();
                (void)wait_or_give_up(wrbar, 0, dead + 2, kDrainPolls);  // let the router matrix land before the block can exit
            }
        }

        int st = 0, he = 0;  // ring slot of the next chunk, hidden-ring entry of the current token
        uint32_t ph = 0;     // parity of the slot's current use
        auto release = [&]() {  // hand the current slot back and move on to the next
            __syncwarp();
            if (lane == 0) mbar_arrive(empty + st);
            ++ci;
            if (++st == stages) {
                st = 0;
                ph ^= 1u;
            }
        };
        Sweep<T, NFAST> sweep;
#pragma unroll 1
        for (int k = 0; k < ntok; ++k) {
            const long long t = b0 + static_cast<long long>(k) * G;
            const size_t tbyte = static_cast<size_t>(t) * d * EB;
#pragma unroll 1
            for (int l = 0; l < L; ++l) {
                // the item's hidden state: as loaded (first layer) or as left by the previous layer
                const uint32_t haddr = (l == 0) ? smem_base + m.off_hring + static_cast<uint32_t>(he) * hid_stride : hid_s;

                if (k == 0 && l == 0 && direct) {
                    // first token of the block: plain 16-byte loads straight after the grid dependency
                    // (measured faster than the bulk copy for chained one-token blocks once a launch has
                    // more than about a hundred of them, slower below)
                    const uint4 *src = reinterpret_cast<const uint4 *>(static_cast<const unsigned char *>(p.hidden) + tbyte);
                    for (int g = tid; g < d / VEC; g += nc) sts128(haddr + 16u * g, __ldcg(src + g));
                    named_bar_sync(kBarHidden, nc);
                }

                // ---- router: partial logits over all d columns ----
                const uint32_t raddr = NORM ? norm_s : haddr;  // what the router reads: RMSNorm(hidden) or hidden itself
                const void *norm_w = static_cast<const unsigned char *>(p.norm_weight) + static_cast<size_t>(l) * p.norm_stride;
                sweep.clear();
                if (ring) {
#pragma unroll 1
                    for (int q = 0; q < K; ++q) {
                        acquire(st, ph);
                        if constexpr (NORM) {  // the hidden state came with the item's first chunk
                            if (q == 0)
                                rmsnorm_to_shared<T>(haddr, norm_s, norm_w, p.norm_eps, d, partial, kBarHidden, tid, nc, lane,
                                                     warp, nwarps);
                        }
                        {
                            const uint32_t waddr = smem_base + static_cast<uint32_t>(st) * slot_bytes;
                            if constexpr (NFAST > 0) sweep.chunk(waddr, raddr + q * chunk_cols_bytes, dcc, tid, nc);
                            else sweep.chunk_any(waddr, raddr + q * chunk_cols_bytes, dcc, N, warp, lane, nwarps, q == 0, partial);
                        }
                        release();
                    }
                } else {
                    if (k > 0 || !direct) acquire(st, ph);  // the first rows chunk brings the hidden state with it
                    if constexpr (NORM)
                        rmsnorm_to_shared<T>(haddr, norm_s, norm_w, p.norm_eps, d, partial, kBarHidden, tid, nc, lane, warp,
                                             nwarps);
                    {
                        if constexpr (NFAST > 0) sweep.chunk(smem_base + m.off_wr, raddr, d, tid, nc);
                        else sweep.chunk_any(smem_base + m.off_wr, raddr, d, N, warp, lane, nwarps, true, partial);
                    }
                }
                if constexpr (NFAST > 0) {
                    sweep.finish(lane, partial + warp * N);
                }

                // ---- warp 0 turns the partial logits into softmax numerators for everybody ----
                if (warp != 0) {
                    named_bar_arrive(kBarLogits, nc);
                } else {
                    named_bar_sync(kBarLogits, nc);
                    {
                        const int j0 = lane, j1 = lane + 32;
                        float z0 = 0.f, z1 = 0.f;
                        if constexpr (NFAST > 0) {
                            // fixed trip count, loads independent of one another (rows past nwarps repeat row 0, weight 0)
#pragma unroll
                            for (int w = 0; w < kMaxConsumers / 32; ++w) {
                                const int ww = w < nwarps ? w : 0;
                                const float a0 = j0 < N ? partial[ww * N + j0] : 0.f;
                                z0 += w < nwarps ? a0 : 0.f;
                                if constexpr (NFAST > 32) {
                                    const float a1 = partial[ww * N + j1];
                                    z1 += w < nwarps ? a1 : 0.f;
                                }
                            }
                        } else {
                            if (j0 < N) z0 = partial[j0];
                            if (j1 < N) z1 = partial[j1];
                        }
                        // softmax over all N experts (Eq. 4).  Only the numerators e_j = exp(z_j - m)
                        // are formed here; the combine divides by their sum.  Any shift m gives the same
                        // gates, so the (shuffle-heavy) maximum is taken only when some logit is large
                        // enough for exp to leave the comfortable range.
                        const bool big = (j0 < N && !(fabsf(z0) < 80.f)) || (j1 < N && !(fabsf(z1) < 80.f));
                        float zmax = 0.f;
                        if (__any_sync(0xffffffffu, big)) zmax = logit_max(z0, z1, N, lane);
                        const float e0 = j0 < N ? expf(z0 - zmax) : 0.f;
                        const float e1 = j1 < N ? expf(z1 - zmax) : 0.f;
                        if (j0 < N) gates[j0] = e0;
                        if (j1 < N) gates[j1] = e1;
                        if (p.gates_out) write_gates(p.gates_out, t, N, lane, e0, e1);
                    }
                }
                named_bar_sync(kBarGates, nc);

                // ---- weighted sum of the rows, chunk by chunk (Eq. 8) ----
                if constexpr (kRowsByExpert) {
                    RowSums<T, P> sums;
                    sums.clear();
                    const int ne = N / K, ngrp_all = d / VEC;
                    bool valid = true;
#pragma unroll 1
                    for (int kk = 0; kk < K; ++kk) {
                        acquire(st, ph);
                        valid = meta[st] != 0;
                        sums.chunk(smem_base + static_cast<uint32_t>(st) * slot_bytes, gates_s + 4u * (kk * ne), ne, ngrp_all, tid, nc);
                        release();
                    }
                    const unsigned char *res_g = p.residual ? static_cast<const unsigned char *>(p.residual) + tbyte : nullptr;
                    unsigned char *dst = (l == L - 1) ? static_cast<unsigned char *>(p.out) + tbyte : nullptr;
                    sums.finish(haddr, res_g, dst, hid_s, ngrp_all, valid, tid, nc);
                } else {
#pragma unroll 1
                    for (int kk = 0; kk < K; ++kk) {
                        if (ring || kk > 0 || direct) acquire(st, ph);
                        {
                            const bool valid = meta[st] != 0;
                            const uint32_t off = kk * chunk_cols_bytes;
                            const unsigned char *res_g =
                                p.residual ? static_cast<const unsigned char *>(p.residual) + tbyte + off : nullptr;
                            unsigned char *dst = (l == L - 1) ? static_cast<unsigned char *>(p.out) + tbyte + off : nullptr;
                            combine_item<T, P>(smem_base + static_cast<uint32_t>(st) * slot_bytes, haddr + off, gates_s, res_g,
                                               dst, hid_s + off, N, ngrp, valid, warp, lane, nwarps);
                        }
                        release();
                    }
                }
                // the next layer's router reads the hidden state that all warps have just written
                if (l + 1 < L) named_bar_sync(kBarHidden, nc);
            }
            if (++he == HR) he = 0;
        }
    }
}

#endif  // __CUDACC__

}  // namespace mole
