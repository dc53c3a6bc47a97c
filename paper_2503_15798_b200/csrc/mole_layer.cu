// Host side of the fused MoLE kernel: launch planning, argument checks and the C entry points
// for a single layer and for a chained L-layer decode step (Eq. 4 and Eq. 8 of arXiv
// 2503.15798).  The kernel itself is in mole_kernel.cuh.
#include <atomic>
#include <mutex>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include "mole_cdecode.cuh"
#include "mole_decode.cuh"
#include "mole_fstep.cuh"
#include "mole_kernel.cuh"

namespace mole {

static thread_local char g_cuda_error[256] = "";

void set_cuda_error(cudaError_t e)
{
    const char *s = cudaGetErrorString(e);
    strncpy(g_cuda_error, s ? s : "unknown CUDA error", sizeof(g_cuda_error) - 1);
    g_cuda_error[sizeof(g_cuda_error) - 1] = 0;
    (void)cudaGetLastError();  // clear the error so that later calls start clean
}

static int round_up(int a, int b) { return (a + b - 1) / b * b; }

constexpr int kNumSMs = 148;                  // B200; used when no device can be asked (mole_plan on a machine without one)
constexpr int kSmemPerBlockMax = 227 * 1024;  // opt-in limit per block
constexpr int kSmemPerSM = 228 * 1024;        // per SM, of which every resident block reserves 1 KB
constexpr long long kFusedMaxTokens = 4096;   // above this a step runs as L chained launches

// ---- debugging aids: the MOLE_FORCE_* / MOLE_DEBUG_* variables, read once ---------------------------
struct DebugEnv {
    int lanes, column_chunks, target_blocks, stages, blocks_per_sm, kernel;
    long long wait_limit;
};
static std::mutex g_env_mutex;
static DebugEnv g_env;
static std::atomic<int> g_env_generation{0};  // 0: not read yet; bumped by every (re)load

static int env_int(const char *name)
{
    const char *f = getenv(name);
    return f ? atoi(f) : 0;
}
static void load_env_locked()
{
    g_env.lanes = env_int("MOLE_FORCE_LANES");
    g_env.column_chunks = env_int("MOLE_FORCE_COLUMN_CHUNKS");
    g_env.target_blocks = env_int("MOLE_FORCE_TARGET_BLOCKS");
    g_env.stages = env_int("MOLE_FORCE_STAGES");
    g_env.blocks_per_sm = env_int("MOLE_FORCE_BLOCKS_PER_SM");
    g_env.kernel = env_int("MOLE_FORCE_KERNEL");
    const char *w = getenv("MOLE_DEBUG_WAIT_LIMIT");
    g_env.wait_limit = w ? atoll(w) : 0;
    g_env_generation.fetch_add(1);
}
static DebugEnv debug_env(int *generation = nullptr)
{
    std::lock_guard<std::mutex> lock(g_env_mutex);
    if (g_env_generation.load() == 0) load_env_locked();
    if (generation) *generation = g_env_generation.load();
    return g_env;
}
// polls after which a device-side wait gives up: the default, or what MOLE_DEBUG_WAIT_LIMIT says
// (n >= 1: n polls; negative: none at all, every wait that is not satisfied at once gives up)
static uint32_t wait_polls_from(const DebugEnv &e)
{
    if (e.wait_limit < 0) return 0u;
    if (e.wait_limit > 0) return e.wait_limit > 0x7fffffffLL ? 0x7fffffffu : static_cast<uint32_t>(e.wait_limit);
    return kWaitPolls;
}

uint32_t current_wait_polls() { return wait_polls_from(debug_env()); }

// Lanes per 16-byte column group in the combine (1, 2 or 4).
static int lanes_per_group(int dcc, int vec, const DebugEnv &env)
{
    const int groups = dcc / vec;
    const int forced = env.lanes;
    if ((forced == 1 || forced == 2 || forced == 4) && groups * forced <= kMaxConsumers) return forced;
    // about four compute warps -- one per SM sub-partition -- measured best: more warps repeat the
    // per-item bookkeeping, fewer lengthen the chain of an item
    return groups * 4 <= 128 ? 4 : (groups * 2 <= 128 ? 2 : 1);
}
static int consumers_for(int dcc, int vec, const DebugEnv &env)
{
    const int lanes = (dcc / vec) * lanes_per_group(dcc, vec, env);
    return round_up(lanes < kMaxConsumers ? lanes : kMaxConsumers, 32);
}
// Several chunks per item: the rows are cut by experts -- whole rows, one bulk copy per chunk --
// where the kernel exists for it (bf16, a compiled-in N that the chunk count divides, router
// chunks in the ring) and a lane can carry the sums of its column groups (at most four, over
// about four warps) from chunk to chunk; otherwise by columns.
static int groups_per_lane(int d, int vec)
{
    const int groups = d / vec;
    return groups <= 128 ? 1 : (groups <= 256 ? 2 : 4);
}
static bool rows_by_expert(int dtype, int N, int d, int K, int in_ring, bool by_columns, const DebugEnv &env)
{
    if (by_columns) return false;
    const bool n_fast = N == 4 || N == 8 || N == 16 || N == 32 || N == 64;
    if (env.column_chunks > 0) return false;  // debugging aid
    return dtype == MOLE_DTYPE_BF16 && n_fast && K > 1 && N % K == 0 && in_ring && d / 8 <= 4 * 128;
}
static int consumers_by_expert(int d, int vec)
{
    const int gpl = groups_per_lane(d, vec);
    return round_up((d / vec + gpl - 1) / gpl, 32);
}

int plan_step(long long M, int L, int N, int d, int dtype, int d_split, StepPlan *plan, bool by_columns, int sms, bool norm)
{
    if (dtype != MOLE_DTYPE_BF16 && dtype != MOLE_DTYPE_F32) return MOLE_ERR_INVALID_ARG;
    if (L < 1 || M < 0) return MOLE_ERR_INVALID_ARG;
    if (sms < 1) sms = kNumSMs;
    const DebugEnv env = debug_env();
    const int eb = elem_bytes(dtype), vec = 16 / eb;
    if (N < 1 || N > kMaxN || d < vec || d % vec != 0) return MOLE_ERR_UNSUPPORTED_SHAPE;
    // the router matrix stays resident only for a single layer, and only if it leaves room for the ring
    const int in_ring = (L > 1 || static_cast<long long>(d) * N * eb > 96 * 1024) ? 1 : 0;
    const int per_tok = L * (in_ring ? 2 : 1);  // chunks per token, per column chunk
    auto total_smem = [&](int K, int stages) {
        const int dcc = d / K;
        const int hring = (stages + per_tok * K - 1) / (per_tok * K) + 1;
        const int consumers = rows_by_expert(dtype, N, d, K, in_ring, by_columns, env) ? consumers_by_expert(d, vec)
                                                                                         : consumers_for(dcc, vec, env);
        return smem_map(N, d, dcc, eb, stages, hring, in_ring, consumers, norm ? 1 : 0).total;
    };
    int K;
    if (d_split != 0) {
        if (d_split != 1 && d_split != 2 && d_split != 4 && d_split != 8 && d_split != 16) return MOLE_ERR_INVALID_ARG;
        if (d % (d_split * vec) != 0) return MOLE_ERR_UNSUPPORTED_SHAPE;
        K = d_split;
        if (total_smem(K, 2) > static_cast<uint32_t>(kSmemPerBlockMax)) return MOLE_ERR_UNSUPPORTED_SHAPE;
    } else {
        // the fewest chunks that keep one chunk at or under 32 KB (and a ring of two in shared memory).  A
        // launch of at most one token per SM has the SM's whole shared memory for one block: chunks of up
        // to 64 KB in a ring of three then halve the per-chunk bookkeeping (measured on d = 2048, N = 32,
        // 16 layers, 1 to 148 tokens: 84 -> 56-62 us per step; chained single-layer launches 3 - 12 % less)
        const bool roomy = M <= sms && (L > 1 || in_ring);
        const long long chunk_cap = roomy ? 64 * 1024 : 32 * 1024;
        const int ring_min = roomy ? 3 : 2;
        K = 1;
        while (static_cast<long long>(N) * (d / K) * eb > chunk_cap ||
               total_smem(K, ring_min) > static_cast<uint32_t>(kSmemPerBlockMax)) {
            if (K >= kMaxChunks || d % (2 * K * vec) != 0) {
                if (total_smem(K, 2) <= static_cast<uint32_t>(kSmemPerBlockMax)) break;  // larger chunks, but they fit
                return MOLE_ERR_UNSUPPORTED_SHAPE;
            }
            K *= 2;
        }
    }
    const int dcc = d / K;
    const bool by_expert = rows_by_expert(dtype, N, d, K, in_ring, by_columns, env);
    const int consumers = by_expert ? consumers_by_expert(d, vec) : consumers_for(dcc, vec, env);
    // Resident blocks per SM aimed at: one per token while tokens are few (each with the deepest ring
    // that fits), up to four token chains per SM when there are many (shallower rings, more overlap).
    int want = static_cast<int>((M + sms - 1) / sms);
    want = want < 1 ? 1 : (want > 4 ? 4 : want);
    if (env.target_blocks > 0) want = env.target_blocks;
    int stages = 0;
    for (; want >= 1 && stages == 0; --want) {
        const uint32_t budget = static_cast<uint32_t>(kSmemPerSM / want - 1024);
        for (int s = kMaxStages; s >= 2; --s) {
            const uint32_t need = total_smem(K, s);
            if (need <= budget && need <= static_cast<uint32_t>(kSmemPerBlockMax)) {
                stages = s;
                break;
            }
        }
    }
    if (stages == 0) stages = 2;  // total_smem(K, 2) fits a block (checked above)
    // no deeper than the chunks a block will see
    const long long cap = static_cast<long long>(sms) * 4;
    const long long blocks = M < cap ? (M > 0 ? M : 1) : cap;
    const long long chunks = ((M + blocks - 1) / blocks) * per_tok * K;
    if (stages > chunks) stages = chunks < 2 ? 2 : static_cast<int>(chunks);
    // A single layer with its router matrix resident and more tokens than two-slot blocks fit at once, but no more
    // than one-slot blocks do: one token per block, all of them resident, instead of two tokens in a row per block
    // (measured, 160M shape, 512 tokens: 4.66 -> 3.80 us per layer).
    if (L == 1 && !in_ring && K == 1) {
        auto fit = [&](int s) {
            int n = kSmemPerSM / (static_cast<int>(total_smem(K, s)) + 1024);
            const int by_threads = 2048 / (consumers + 32);
            return n < by_threads ? n : by_threads;
        };
        if (M > static_cast<long long>(fit(2)) * sms && M <= static_cast<long long>(fit(1)) * sms) stages = 1;
    }
    const int forced = env.stages;
    if (forced >= 2 && forced <= kMaxStages && total_smem(K, forced) <= static_cast<uint32_t>(kSmemPerBlockMax)) stages = forced;
    const int hring = (stages + per_tok * K - 1) / (per_tok * K) + 1;
    const SmemMap m = smem_map(N, d, dcc, eb, stages, hring, in_ring, consumers, norm ? 1 : 0);
    plan->d_split = K;
    plan->dc = dcc;
    plan->consumers = consumers;
    plan->threads = consumers + 32;
    plan->stages = stages;
    plan->hring = hring;
    plan->slot_bytes = static_cast<int>(up128(m.chunk_bytes));
    plan->wr_in_ring = in_ring;
    plan->smem = static_cast<int>(m.total);
    int per_sm = kSmemPerSM / (plan->smem + 1024);
    if (per_sm > 2048 / plan->threads) per_sm = 2048 / plan->threads;
    if (per_sm > 32) per_sm = 32;
    if (per_sm < 1) per_sm = 1;
    plan->blocks_per_sm = per_sm;
    plan->rows_by_expert = by_expert ? 1 : 0;
    plan->lanes = by_expert ? groups_per_lane(d, vec) : lanes_per_group(dcc, vec, env);
    plan->n_fast = (N == 4 || N == 8 || N == 16 || N == 32 || N == 64) ? N : 0;
    return MOLE_OK;
}

// A kernel instantiation and its name ("step<storage,NFAST,P,MODE,SHAPE,DIRECT,NORM>" for the ring
// kernel, "decode<N,NORM>" for the one-block-per-token kernel): what mole_variant() reports, so that a
// test can tell which instantiations a workload reaches.
typedef void (*StepKernel)(const StepParams);
typedef void (*DecodeKernel)(const DecodeParams);
struct Variant {
    StepKernel fn;
    const char *name;
};
#define MOLE_V(T, TN, NF, P, MODE, SHAPE, DIRECT, NORM) \
    Variant { mole_step_kernel<T, NF, P, MODE, SHAPE, DIRECT, NORM>, "step<" TN "," #NF "," #P "," #MODE "," #SHAPE "," #DIRECT "," #NORM ">" }
#define MOLE_VB(NF, P, MODE, SHAPE, DIRECT, NORM) MOLE_V(__nv_bfloat16, "bf16", NF, P, MODE, SHAPE, DIRECT, NORM)
#define MOLE_VF(NF, P, MODE, SHAPE, DIRECT, NORM) MOLE_V(float, "f32", NF, P, MODE, SHAPE, DIRECT, NORM)
static const Variant kNoVariant = {nullptr, "none"};

// bf16, compile-time launch flags (MODE 1, 2, 3), any of the unrolled N
#define MOLE_PICK_N_BF16(P, MODE, NORM)                      \
    switch (n_fast) {                                        \
        case 4: return MOLE_VB(4, P, MODE, 0, 0, NORM);      \
        case 8: return MOLE_VB(8, P, MODE, 0, 0, NORM);      \
        case 16: return MOLE_VB(16, P, MODE, 0, 0, NORM);    \
        case 32: return MOLE_VB(32, P, MODE, 0, 0, NORM);    \
        case 64: return MOLE_VB(64, P, MODE, 0, 0, NORM);    \
        default: return kNoVariant;                          \
    }
#define MOLE_PICK_N_F32(P, MODE, NORM)                       \
    switch (n_fast) {                                        \
        case 4: return MOLE_VF(4, P, MODE, 0, 0, NORM);      \
        case 8: return MOLE_VF(8, P, MODE, 0, 0, NORM);      \
        case 16: return MOLE_VF(16, P, MODE, 0, 0, NORM);    \
        case 32: return MOLE_VF(32, P, MODE, 0, 0, NORM);    \
        case 64: return MOLE_VF(64, P, MODE, 0, 0, NORM);    \
        default: return kNoVariant;                          \
    }
template <int MODE>
static Variant pick_bf16(int n_fast, int lanes)
{
    if (lanes == 4) { MOLE_PICK_N_BF16(4, MODE, 0) }
    if (lanes == 2) { MOLE_PICK_N_BF16(2, MODE, 0) }
    MOLE_PICK_N_BF16(1, MODE, 0)
}
static Variant pick_f32(int n_fast, int lanes)
{
    if (lanes == 4) { MOLE_PICK_N_F32(4, 0, 0) }
    if (lanes == 2) { MOLE_PICK_N_F32(2, 0, 0) }
    MOLE_PICK_N_F32(1, 0, 0)
}

// The generic-N router and the fp32 storage type exist only with run-time flags (MODE 0); bf16 with
// a compiled-in N also in the specialised shapes.
static Variant pick_kernel(int dtype, int n_fast, int lanes, int chunks, int in_ring, int d, int dcc, int consumers,
                           int by_expert, bool direct)
{
    // the layer widths of the paper's Table 2 (160M, 410M and 1B models) with their sizes compiled in;
    // `direct`: single-layer launches of 128 tokens up to one token per resident block, where the compute
    // warps loading the hidden state themselves measured 6 % faster per chained layer (slower below)
    if (dtype == MOLE_DTYPE_BF16) {
        if (n_fast == 16 && lanes == 1 && chunks == 1 && d == 768 && consumers == 96)
            return in_ring ? MOLE_VB(16, 1, 1, 1, 0, 0) : (direct ? MOLE_VB(16, 1, 2, 1, 1, 0) : MOLE_VB(16, 1, 2, 1, 0, 0));
        if (n_fast == 16 && lanes == 1 && chunks == 1 && d == 1024 && consumers == 128)
            return in_ring ? MOLE_VB(16, 1, 1, 2, 0, 0) : (direct ? MOLE_VB(16, 1, 2, 2, 1, 0) : MOLE_VB(16, 1, 2, 2, 0, 0));
        if (n_fast == 32 && lanes == 2 && chunks == 4 && d == 2048 && dcc == 512 && consumers == 128 && by_expert)
            return MOLE_VB(32, 2, 3, 3, 0, 0);
        if (n_fast == 32 && lanes == 2 && chunks == 2 && d == 2048 && dcc == 1024 && consumers == 128 && by_expert)
            return MOLE_VB(32, 2, 3, 4, 0, 0);
        if (by_expert) return pick_bf16<3>(n_fast, lanes);
    }
    if (n_fast == 0) {
        if (dtype == MOLE_DTYPE_BF16)
            return lanes == 4 ? MOLE_VB(0, 4, 0, 0, 0, 0) : (lanes == 2 ? MOLE_VB(0, 2, 0, 0, 0, 0) : MOLE_VB(0, 1, 0, 0, 0, 0));
        return lanes == 4 ? MOLE_VF(0, 4, 0, 0, 0, 0) : (lanes == 2 ? MOLE_VF(0, 2, 0, 0, 0, 0) : MOLE_VF(0, 1, 0, 0, 0, 0));
    }
    if (dtype != MOLE_DTYPE_BF16) return pick_f32(n_fast, lanes);
    if (chunks == 1) return in_ring ? pick_bf16<1>(n_fast, lanes) : pick_bf16<2>(n_fast, lanes);
    return pick_bf16<0>(n_fast, lanes);
}

// The kernels whose router reads RMSNorm(hidden): run-time launch flags, rows cut by columns ...
static Variant pick_norm_kernel(int dtype, int n_fast, int lanes)
{
    if (dtype == MOLE_DTYPE_BF16) {
        if (n_fast == 0) return lanes == 4 ? MOLE_VB(0, 4, 0, 0, 0, 1) : (lanes == 2 ? MOLE_VB(0, 2, 0, 0, 0, 1) : MOLE_VB(0, 1, 0, 0, 0, 1));
        if (lanes == 4) { MOLE_PICK_N_BF16(4, 0, 1) }
        if (lanes == 2) { MOLE_PICK_N_BF16(2, 0, 1) }
        MOLE_PICK_N_BF16(1, 0, 1)
    }
    if (n_fast == 0) return lanes == 4 ? MOLE_VF(0, 4, 0, 0, 0, 1) : (lanes == 2 ? MOLE_VF(0, 2, 0, 0, 0, 1) : MOLE_VF(0, 1, 0, 0, 0, 1));
    if (lanes == 4) { MOLE_PICK_N_F32(4, 0, 1) }
    if (lanes == 2) { MOLE_PICK_N_F32(2, 0, 1) }
    MOLE_PICK_N_F32(1, 0, 1)
}
// ... and, for the paper's three layer widths, with the sizes compiled in (single layers and fused steps)
static Variant pick_norm_shape_kernel(const StepPlan &plan, int dtype, int d, bool direct)
{
    if (dtype != MOLE_DTYPE_BF16) return kNoVariant;
    if (plan.n_fast == 16 && plan.lanes == 1 && plan.d_split == 1) {
        if (!plan.wr_in_ring) {
            if (d == 768 && plan.consumers == 96) return direct ? MOLE_VB(16, 1, 2, 1, 1, 1) : MOLE_VB(16, 1, 2, 1, 0, 1);
            if (d == 1024 && plan.consumers == 128) return direct ? MOLE_VB(16, 1, 2, 2, 1, 1) : MOLE_VB(16, 1, 2, 2, 0, 1);
        } else {
            if (d == 768 && plan.consumers == 96) return MOLE_VB(16, 1, 1, 1, 0, 1);
            if (d == 1024 && plan.consumers == 128) return MOLE_VB(16, 1, 1, 2, 0, 1);
        }
    }
    if (plan.n_fast == 32 && plan.lanes == 2 && d == 2048 && plan.consumers == 128 && plan.rows_by_expert) {
        if (plan.d_split == 4 && plan.dc == 512) return MOLE_VB(32, 2, 3, 3, 0, 1);
        if (plan.d_split == 2 && plan.dc == 1024) return MOLE_VB(32, 2, 3, 4, 0, 1);
    }
    return kNoVariant;
}

// The one-block-per-token kernel (mole_decode.cuh): bf16, N of 4, 8, 16 or 32, d a multiple of 128
// with d / 4 threads, a single layer, the launch's own chunking (d_split 0), up to 2048 tokens.
struct DecodeVariant {
    DecodeKernel fn;
    const char *name;
};
static bool decode_shape_ok(int dtype, int N, int d)
{
    if (dtype != MOLE_DTYPE_BF16 || d % 128 != 0) return false;
    if (N != 4 && N != 8 && N != 16 && N != 32) return false;
    return d / 4 <= decode_max_threads(N) && decode_smem_bytes(N, d) <= static_cast<uint32_t>(kSmemPerBlockMax);
}
static DecodeVariant pick_decode(int N, bool norm)
{
    switch (N) {
        case 4: return norm ? DecodeVariant{mole_decode_kernel<4, 1>, "decode<4,1>"} : DecodeVariant{mole_decode_kernel<4, 0>, "decode<4,0>"};
        case 8: return norm ? DecodeVariant{mole_decode_kernel<8, 1>, "decode<8,1>"} : DecodeVariant{mole_decode_kernel<8, 0>, "decode<8,0>"};
        case 16: return norm ? DecodeVariant{mole_decode_kernel<16, 1>, "decode<16,1>"} : DecodeVariant{mole_decode_kernel<16, 0>, "decode<16,0>"};
        case 32: return norm ? DecodeVariant{mole_decode_kernel<32, 1>, "decode<32,1>"} : DecodeVariant{mole_decode_kernel<32, 0>, "decode<32,0>"};
        default: return DecodeVariant{nullptr, "none"};
    }
}

// The one-token-per-cluster kernel (mole_cdecode.cuh): bf16, d = 2048 (four blocks of 512 columns), N of 16 or 32,
// a single layer, the launch's own chunking.
constexpr int kClusterBlocks = 4;
static bool cdecode_shape_ok(int dtype, int N, int d)
{
    return dtype == MOLE_DTYPE_BF16 && (N == 16 || N == 32) && d == kClusterBlocks * kClusterSlice;
}
// Measured on B200 (1B-shaped layers, chained steps): the cluster kernel is ahead of the ring kernel while all of a
// launch's blocks (four per SM) are resident at once with room left for the next layer's blocks to prefetch under
// them -- up to 128 tokens on 148 SMs -- and behind it from there on (a second wave of blocks cannot prefetch).
static bool cdecode_preferred(long long M, int N, int sms)
{
    return N == 32 && M * kClusterBlocks * 8 <= 4LL * sms * 7;
}
static DecodeVariant pick_cdecode(int N, bool norm)
{
    if (N == 32)
        return norm ? DecodeVariant{mole_cdecode_kernel<32, kClusterBlocks, 1>, "cdecode<32,4,1>"}
                    : DecodeVariant{mole_cdecode_kernel<32, kClusterBlocks, 0>, "cdecode<32,4,0>"};
    if (N == 16)
        return norm ? DecodeVariant{mole_cdecode_kernel<16, kClusterBlocks, 1>, "cdecode<16,4,1>"}
                    : DecodeVariant{mole_cdecode_kernel<16, kClusterBlocks, 0>, "cdecode<16,4,0>"};
    return DecodeVariant{nullptr, "none"};
}

// The fused step with the decode arithmetic (mole_fstep.cuh): bf16, N of 4, 8, 16 or 32, d a multiple of
// 128 with d / 4 <= 512 compute threads, router matrix in 1, 2 or 4 column chunks of at most 32 KB, rows in
// chunks of whole experts of at most 32 KB.
typedef void (*FStepKernel)(const FStepParams);
struct FStepVariant {
    FStepKernel fn;
    const char *name;
};
struct FStepPlan {
    int db, kw, kr, rexp, stages, blocks_per_sm, threads, smem;
};
static bool plan_fstep(long long M, int L, int N, int d, int dtype, bool norm, int sms, FStepPlan *f)
{
    if (dtype != MOLE_DTYPE_BF16 || d % 128 != 0 || d / 4 > kDecodeMaxThreads) return false;
    if (N != 4 && N != 8 && N != 16 && N != 32) return false;
    // the cut of an item into ring slots follows the width class (FStepCut): column chunks of the router
    // matrix, chunks of whole experts' rows, neither above 32 KB
    const int db = d <= 512 ? 0 : (d <= 1024 ? 1 : 2);
    const int dmax = db == 0 ? 512 : (db == 1 ? 1024 : 2048);
    int kw = N * dmax * 2 / static_cast<int>(kFStepSlotBytes);
    if (kw < 1) kw = 1;
    int rexp = static_cast<int>(kFStepSlotBytes) / (2 * dmax);
    if (rexp > 16) rexp = 16;
    if (rexp > N) rexp = N;
    if (N / 2 / kw < 1 || rexp < 4) return false;
    // blocks per SM aimed at: one per token while tokens are few (the deepest ring that fits), two or three
    // token chains per SM when there are more tokens than SMs
    int want = static_cast<int>((M + sms - 1) / sms);
    want = want < 1 ? 1 : (want > 3 ? 3 : want);
    const DebugEnv env = debug_env();
    if (env.target_blocks > 0) want = env.target_blocks;
    int stages = 0;
    for (; want >= 1 && stages < 2; --want) {
        const long long budget = kSmemPerSM / want - 1024;
        stages = 0;
        for (int s = kMaxStages; s >= 2; --s)
            if (fstep_smem(N, d, s, norm ? 1 : 0).total <= budget && fstep_smem(N, d, s, norm ? 1 : 0).total <= static_cast<uint32_t>(kSmemPerBlockMax)) {
                stages = s;
                break;
            }
        if (stages >= 2) break;
    }
    if (stages < 2) return false;
    if (env.stages >= 2 && env.stages <= kMaxStages && fstep_smem(N, d, env.stages, norm ? 1 : 0).total <= static_cast<uint32_t>(kSmemPerBlockMax))
        stages = env.stages;
    const long long chunks = ((M + static_cast<long long>(sms) * 3 - 1) / (static_cast<long long>(sms) * 3)) * L * (kw + N / rexp);
    (void)chunks;
    f->db = db;
    f->kw = kw;
    f->rexp = rexp;
    f->kr = N / rexp;
    f->stages = stages;
    f->threads = d / 4 + 32;
    f->smem = static_cast<int>(fstep_smem(N, d, stages, norm ? 1 : 0).total);
    int per_sm = kSmemPerSM / (f->smem + 1024);
    if (per_sm > 2048 / f->threads) per_sm = 2048 / f->threads;
    f->blocks_per_sm = per_sm < 1 ? 1 : per_sm;
    return true;
}
#define MOLE_FV(N, DB, NORM) FStepVariant { mole_fstep_kernel<N, DB, NORM>, "fstep<" #N "," #DB "," #NORM ">" }
#define MOLE_FV_N(N)                                                          \
    switch (db * 2 + (norm ? 1 : 0)) {                                        \
        case 0: return MOLE_FV(N, 0, 0);                                      \
        case 1: return MOLE_FV(N, 0, 1);                                      \
        case 2: return MOLE_FV(N, 1, 0);                                      \
        case 3: return MOLE_FV(N, 1, 1);                                      \
        case 4: return MOLE_FV(N, 2, 0);                                      \
        default: return MOLE_FV(N, 2, 1);                                     \
    }
static FStepVariant pick_fstep(int N, int db, bool norm)
{
    switch (N) {
        case 4: MOLE_FV_N(4)
        case 8: MOLE_FV_N(8)
        case 16: MOLE_FV_N(16)
        case 32: MOLE_FV_N(32)
        default: return FStepVariant{nullptr, "none"};
    }
}

// Kernels that need more than 48 KB of dynamic shared memory must opt in once per device.
int ensure_smem_opt_in(const void *fn, int smem)
{
    if (smem <= 48 * 1024) return MOLE_OK;
    struct Slot {
        std::atomic<const void *> fn{nullptr};
        std::atomic<int> dev{-1};
        std::atomic<int> bytes{0};
    };
    static Slot slots[256];
    int dev = 0;
    MOLE_CUDA_TRY(cudaGetDevice(&dev));
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

// SM count of the current device, asked once per device.
int sm_count(int *out, int *dev_out)
{
    static std::atomic<int> cache[64];
    int dev = 0;
    MOLE_CUDA_TRY(cudaGetDevice(&dev));
    if (dev_out) *dev_out = dev;
    if (dev >= 0 && dev < 64 && cache[dev].load() > 0) {
        *out = cache[dev].load();
        return MOLE_OK;
    }
    int n = 0;
    MOLE_CUDA_TRY(cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev));
    if (n < 1) n = kNumSMs;
    if (dev >= 0 && dev < 64) cache[dev].store(n);
    *out = n;
    return MOLE_OK;
}

// Everything about a launch that depends only on its shape: found once, then looked up.
struct ShapeKey {
    long long M;
    int L, N, d, dtype, d_split, norm, kernel, dev, env_generation;
    bool operator==(const ShapeKey &o) const
    {
        return M == o.M && L == o.L && N == o.N && d == o.d && dtype == o.dtype && d_split == o.d_split && norm == o.norm &&
               kernel == o.kernel && dev == o.dev && env_generation == o.env_generation;
    }
};
struct LaunchChoice {
    bool decode;        // the one-block-per-token kernel; otherwise the ring kernel with `plan`
    bool fstep;         // the fused step with the decode arithmetic, with `fplan`
    FStepPlan fplan;
    FStepKernel fstep_fn;
    StepPlan plan;
    StepKernel step_fn;
    DecodeKernel decode_fn;
    const char *name;
    int threads, smem;
    long long grid;
    uint32_t wait_polls;
};

// `sms` / `dev` < 0: no device is asked (nominal B200 figures, nothing is prepared for a launch).
static int choose_launch(long long M, int L, int N, int d, int dtype, int d_split, bool norm, int kernel, int sms, bool prepare,
                         LaunchChoice *c)
{
    int generation = 0;
    const DebugEnv env = debug_env(&generation);
    if (kernel == MOLE_KERNEL_AUTO && env.kernel > 0) kernel = env.kernel;
    if (kernel != MOLE_KERNEL_AUTO && kernel != MOLE_KERNEL_RING && kernel != MOLE_KERNEL_DECODE) return MOLE_ERR_INVALID_ARG;
    c->wait_polls = wait_polls_from(env);
    StepPlan plan;
    int rc = plan_step(M, L, N, d, dtype, d_split, &plan, false, sms, norm);  // also validates the shape
    if (rc != MOLE_OK) return rc;
    const bool decode_ok = L == 1 && d_split == 0 && decode_shape_ok(dtype, N, d);
    c->decode = c->fstep = false;
    FStepPlan fplan;
    const bool fstep_ok = L > 1 && d_split == 0 && plan_fstep(M, L, N, d, dtype, norm, sms, &fplan);
    const bool cdecode_ok = L == 1 && d_split == 0 && cdecode_shape_ok(dtype, N, d);
    if (kernel == MOLE_KERNEL_DECODE && !(decode_ok || fstep_ok || cdecode_ok)) return MOLE_ERR_UNSUPPORTED_SHAPE;
    // MOLE_KERNEL_AUTO takes the ring kernel for plain tables, except for the widest layers at up to 128 tokens (the
    // cluster kernel, see cdecode_preferred): measured on B200, neither the one-block-per-token kernel (chained steps)
    // nor the fused step built on it beats it -- a decode batch is bound by the latency of one token's dependent
    // instruction stream, which the two families execute at about the same length.  They run on request
    // (MOLE_KERNEL_DECODE), and their structure carries the quantised tables.
    if (fstep_ok && kernel == MOLE_KERNEL_DECODE) {
        const FStepVariant v = pick_fstep(N, fplan.db, norm);
        if (!v.fn) return MOLE_ERR_UNSUPPORTED_SHAPE;
        c->fstep = true;
        c->fplan = fplan;
        c->fstep_fn = v.fn;
        c->plan = plan;
        c->step_fn = nullptr;
        c->decode_fn = nullptr;
        c->name = v.name;
        c->threads = fplan.threads;
        c->smem = fplan.smem;
        int per_sm = fplan.blocks_per_sm;
        if (prepare) {
            rc = ensure_smem_opt_in(reinterpret_cast<const void *>(v.fn), fplan.smem);
            if (rc != MOLE_OK) return rc;
            MOLE_CUDA_TRY(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, v.fn, fplan.threads, fplan.smem));
        }
        if (per_sm < 1) per_sm = 1;
        if (env.blocks_per_sm >= 1 && env.blocks_per_sm < per_sm) per_sm = env.blocks_per_sm;
        c->grid = static_cast<long long>(per_sm) * sms;
        if (c->grid > M) c->grid = M;
        return MOLE_OK;
    }
    if (cdecode_ok && (kernel == MOLE_KERNEL_DECODE || (kernel == MOLE_KERNEL_AUTO && cdecode_preferred(M, N, sms)))) {
        const DecodeVariant v = pick_cdecode(N, norm);
        if (!v.fn) return MOLE_ERR_UNSUPPORTED_SHAPE;
        c->decode = true;
        c->plan = plan;
        c->step_fn = nullptr;
        c->decode_fn = v.fn;
        c->name = v.name;
        c->threads = kClusterThreads;
        c->smem = static_cast<int>(cdecode_smem_bytes(N));
        c->grid = M * kClusterBlocks;  // one cluster per token
        if (prepare) return ensure_smem_opt_in(reinterpret_cast<const void *>(v.fn), c->smem);
        return MOLE_OK;
    }
    if (decode_ok && kernel == MOLE_KERNEL_DECODE) {
        const DecodeVariant v = pick_decode(N, norm);
        if (!v.fn) return MOLE_ERR_UNSUPPORTED_SHAPE;
        c->decode = true;
        c->plan = plan;
        c->step_fn = nullptr;
        c->decode_fn = v.fn;
        c->name = v.name;
        c->threads = d / 4;
        c->smem = static_cast<int>(decode_smem_bytes(N, d));
        c->grid = M;
        if (prepare) return ensure_smem_opt_in(reinterpret_cast<const void *>(v.fn), c->smem);
        return MOLE_OK;
    }
    const bool direct = M >= 128 && M <= 4LL * sms;  // see pick_kernel
    Variant v = kNoVariant;
    if (norm) {
        v = pick_norm_shape_kernel(plan, dtype, d, direct && L == 1);
        if (!v.fn) {
            rc = plan_step(M, L, N, d, dtype, d_split, &plan, true, sms, true);  // the general kernels cut the rows by columns
            if (rc != MOLE_OK) return rc;
            v = pick_norm_kernel(dtype, plan.n_fast, plan.lanes);
        }
    } else {
        v = pick_kernel(dtype, plan.n_fast, plan.lanes, plan.d_split, plan.wr_in_ring, d, plan.dc, plan.consumers, plan.rows_by_expert,
                        direct);
    }
    if (!v.fn) return MOLE_ERR_UNSUPPORTED_SHAPE;
    c->decode = false;
    c->plan = plan;
    c->step_fn = v.fn;
    c->decode_fn = nullptr;
    c->name = v.name;
    c->threads = plan.threads;
    c->smem = plan.smem;
    int per_sm = plan.blocks_per_sm;
    if (prepare) {
        rc = ensure_smem_opt_in(reinterpret_cast<const void *>(v.fn), plan.smem);
        if (rc != MOLE_OK) return rc;
        // a persistent grid: as many blocks as fit at once, never more than the tokens
        MOLE_CUDA_TRY(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, v.fn, plan.threads, plan.smem));
    }
    if (per_sm < 1) per_sm = 1;
    if (env.blocks_per_sm >= 1 && env.blocks_per_sm < per_sm) per_sm = env.blocks_per_sm;
    c->grid = static_cast<long long>(per_sm) * sms;
    if (c->grid > M) c->grid = M;
    return MOLE_OK;
}

// The calling thread's last few shapes (a decoding loop repeats a handful of them).
static int cached_launch(const StepLaunch &a, const LaunchChoice **out)
{
    constexpr int kEntries = 32;
    struct Entry {
        bool used = false;
        ShapeKey key;
        LaunchChoice choice;
    };
    thread_local Entry cache[kEntries];
    thread_local int next = 0;
    int sms = kNumSMs, dev = 0;
    int rc = sm_count(&sms, &dev);
    if (rc != MOLE_OK) return rc;
    int generation = 0;
    (void)debug_env(&generation);
    const ShapeKey key = {a.M, a.L, a.N, a.d, a.dtype, a.d_split, a.norm_weight ? 1 : 0, a.kernel, dev, generation};
    for (int i = 0; i < kEntries; ++i)
        if (cache[i].used && cache[i].key == key) {
            *out = &cache[i].choice;
            return MOLE_OK;
        }
    LaunchChoice c;
    rc = choose_launch(a.M, a.L, a.N, a.d, a.dtype, a.d_split, a.norm_weight != nullptr, a.kernel, sms, true, &c);
    if (rc != MOLE_OK) return rc;
    Entry &e = cache[next];
    next = (next + 1) % kEntries;
    e.used = true;
    e.key = key;
    e.choice = c;
    *out = &e.choice;
    return MOLE_OK;
}

int launch_step(const StepLaunch &a)
{
    if (a.M == 0) return MOLE_OK;
    if (a.M * a.L > 0x3fffffffLL) return MOLE_ERR_TOO_LARGE;
    const LaunchChoice *c = nullptr;
    int rc = cached_launch(a, &c);
    if (rc != MOLE_OK) return rc;

    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof cfg);
    cfg.gridDim = dim3(static_cast<unsigned>(c->grid), 1, 1);
    cfg.blockDim = dim3(c->threads, 1, 1);
    cfg.dynamicSmemBytes = c->smem;
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

    if (c->fstep) {
        FStepParams p;
        p.hidden = a.hidden;
        p.row_index = a.row_index;
        p.lut = a.lut;
        p.w_router = a.w_router;
        p.norm_weight = a.norm_weight;
        p.out = a.out;
        p.status = a.status;
        p.lut_stride = a.lut_stride;
        p.wr_stride = a.wr_stride;
        p.norm_stride = a.norm_stride;
        p.M = a.M;
        p.rows = a.rows;
        p.d = a.d;
        p.L = a.L;
        p.stages = c->fplan.stages;
        p.kr = c->fplan.kr;
        p.rexp = c->fplan.rexp;
        p.norm_eps = a.norm_eps;
        p.flags = a.flags;
        p.wait_polls = c->wait_polls;
        MOLE_CUDA_TRY(cudaLaunchKernelEx(&cfg, c->fstep_fn, p));
        return MOLE_OK;
    }
    if (c->decode) {
        DecodeParams p;
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
        p.d = a.d;
        p.norm_eps = a.norm_eps;
        p.flags = a.flags;
        p.wait_polls = c->wait_polls;
        MOLE_CUDA_TRY(cudaLaunchKernelEx(&cfg, c->decode_fn, p));
        return MOLE_OK;
    }
    const StepPlan &plan = c->plan;
    StepParams p;
    p.hidden = a.hidden;
    p.residual = a.residual;
    p.row_index = a.row_index;
    p.lut = a.lut;
    p.w_router = a.w_router;
    p.norm_weight = a.norm_weight;
    p.norm_stride = a.norm_stride;
    p.norm_eps = a.norm_eps;
    p.out = a.out;
    p.gates_out = a.gates_out;
    p.status = a.status;
    p.lut_stride = a.lut_stride;
    p.wr_stride = a.wr_stride;
    p.M = a.M;
    p.rows = a.rows;
    p.N = a.N;
    p.d = a.d;
    p.K = plan.d_split;
    p.dcc = plan.dc;
    p.L = a.L;
    p.stages = plan.stages;
    p.hring = plan.hring;
    p.wr_in_ring = plan.wr_in_ring;
    p.consumers = plan.consumers;
    p.flags = a.flags;
    p.wait_polls = c->wait_polls;
    MOLE_CUDA_TRY(cudaLaunchKernelEx(&cfg, c->step_fn, p));
    return MOLE_OK;
}

// One thread per (token, layer): an L2 prefetch of the token's N rows of that layer's table, in pieces of at most
// 32 KB.  A hint: nothing is written, nothing waits for it.
constexpr uint32_t kPrefetchPiece = 32 * 1024;
__global__ void mole_prefetch_rows_kernel(const void *ids, long long M, const unsigned char *lut_base, long long lut_stride,
                                          long long row_bytes, long long rows, int ids64)
{
    const long long t = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x;
    if (t >= M) return;
    const long long id = ids64 ? static_cast<const long long *>(ids)[t] : static_cast<long long>(static_cast<const int *>(ids)[t]);
    if (id < 0 || id >= rows) return;
    const unsigned char *row = lut_base + static_cast<size_t>(blockIdx.y) * lut_stride + static_cast<size_t>(id) * row_bytes;
    for (long long off = 0; off < row_bytes; off += kPrefetchPiece) {
        const long long left = row_bytes - off;
        bulk_prefetch_l2(row + off, static_cast<uint32_t>(left < kPrefetchPiece ? left : kPrefetchPiece));
    }
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
    if (a->reserved2 != 0) return MOLE_ERR_INVALID_ARG;
    if (a->lut_format != MOLE_LUT_PLAIN && a->lut_format != MOLE_LUT_NF4 && a->lut_format != MOLE_LUT_NF3) return MOLE_ERR_INVALID_ARG;
    if (a->kernel != MOLE_KERNEL_AUTO && a->kernel != MOLE_KERNEL_RING && a->kernel != MOLE_KERNEL_DECODE) return MOLE_ERR_INVALID_ARG;
    if (a->norm_weight && (!aligned16(a->norm_weight) || !(a->norm_eps >= 0.f) || a->norm_eps > 3.0e38f)) return MOLE_ERR_INVALID_ARG;
    int rc = check_common(a->hidden, a->ids, a->lut, a->w_router, a->out, a->residual, a->B, a->T, a->N, a->d, a->V,
                          a->dtype);
    if (rc != MOLE_OK) return rc;
    const uintptr_t id_align = (a->flags & MOLE_FLAG_IDS_INT64) ? 7u : 3u;
    if (reinterpret_cast<uintptr_t>(a->ids) & id_align) return MOLE_ERR_INVALID_ARG;
    if (a->residual && a->residual != a->hidden && a->residual == a->out) return MOLE_ERR_INVALID_ARG;
    StepLaunch s;
    s.hidden = a->hidden;
    s.residual = a->residual;
    s.row_index = a->ids;
    s.lut = a->lut;
    s.w_router = a->w_router;
    s.out = a->out;
    s.gates_out = a->gates_out;
    s.status = a->status;
    s.lut_stride = 0;
    s.wr_stride = 0;
    s.M = static_cast<long long>(a->B) * a->T;
    s.L = 1;
    s.N = a->N;
    s.d = a->d;
    s.rows = a->V;
    s.dtype = a->dtype;
    s.flags = a->flags;
    s.d_split = a->d_split;
    s.stream = static_cast<cudaStream_t>(a->stream);
    s.norm_weight = a->norm_weight;
    s.norm_eps = a->norm_eps;
    s.kernel = a->kernel;
    if (a->lut_format != MOLE_LUT_PLAIN) {
        // a quantised table: the one-block-per-token kernel that de-quantises inside the weighted sum
        if (a->dtype != MOLE_DTYPE_BF16 || a->d_split != 0 || a->kernel == MOLE_KERNEL_RING) return MOLE_ERR_UNSUPPORTED_SHAPE;
        if (!quant_layer_shape_ok(a->N, a->d, a->lut_format, a->lut_block)) return MOLE_ERR_UNSUPPORTED_SHAPE;
        return launch_quant_layer(s, a->lut_format, a->lut_block, current_wait_polls());
    }
    return launch_step(s);
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

int mole_decode_step_args(const mole_step_args *a)
{
    if (!a || a->struct_size != sizeof(mole_step_args)) return MOLE_ERR_INVALID_ARG;
    if ((a->flags & ~MOLE_FLAG_CHAIN) || a->reserved != 0) return MOLE_ERR_INVALID_ARG;
    if (a->lut_format != MOLE_LUT_PLAIN && a->lut_format != MOLE_LUT_NF4 && a->lut_format != MOLE_LUT_NF3) return MOLE_ERR_INVALID_ARG;
    const bool quant = a->lut_format != MOLE_LUT_PLAIN;
    const int L = a->L;
    int mode = a->mode;
    if (L < 1 || mode < MOLE_STEP_AUTO || mode > MOLE_STEP_CHAINED) return MOLE_ERR_INVALID_ARG;
    if (a->kernel != MOLE_KERNEL_AUTO && a->kernel != MOLE_KERNEL_RING && a->kernel != MOLE_KERNEL_DECODE) return MOLE_ERR_INVALID_ARG;
    int rc = check_common(a->hidden_in, a->ids, a->lut_base, a->w_router_base, a->out, nullptr, a->B, a->T, a->N, a->d, a->V,
                          a->dtype);
    if (rc != MOLE_OK) return rc;
    const long long M = static_cast<long long>(a->B) * a->T;
    if (M == 0) return MOLE_OK;
    if ((a->lut_layer_stride_bytes & 15) || (a->wr_layer_stride_bytes & 15)) return MOLE_ERR_INVALID_ARG;
    if (a->norm_weight_base &&
        (!aligned16(a->norm_weight_base) || (a->norm_layer_stride_bytes & 15) || !(a->norm_eps >= 0.f) || a->norm_eps > 3.0e38f))
        return MOLE_ERR_INVALID_ARG;
    if (mode == MOLE_STEP_AUTO) {
        mode = (quant || (L > 1 && M > kFusedMaxTokens)) ? MOLE_STEP_CHAINED : MOLE_STEP_FUSED;
        // the widest layers at up to 16 tokens: L chained launches of the cluster kernel are ahead of the fused launch
        // (measured: 2.7 - 3.3 us against 3.5 - 3.65 us per layer); they need the caller's second buffer
        int sms = kNumSMs;
        if (mode == MOLE_STEP_FUSED && L > 1 && M <= 16 && a->d_split == 0 && a->kernel == MOLE_KERNEL_AUTO && debug_env(nullptr).kernel <= 0 &&
            cdecode_shape_ok(a->dtype, a->N, a->d) && sm_count(&sms) == MOLE_OK &&
            cdecode_preferred(M, a->N, sms) && a->tmp && aligned16(a->tmp) && a->out != a->hidden_in && a->tmp != a->hidden_in && a->tmp != a->out)
            mode = MOLE_STEP_CHAINED;
    }
    if (quant) {
        // quantised tables run layer by layer (one block per token de-quantising inside the weighted sum)
        if (mode == MOLE_STEP_FUSED && L > 1) return MOLE_ERR_UNSUPPORTED_SHAPE;
        mode = MOLE_STEP_CHAINED;
        if (a->dtype != MOLE_DTYPE_BF16 || a->d_split != 0 || a->kernel == MOLE_KERNEL_RING) return MOLE_ERR_UNSUPPORTED_SHAPE;
        if (!quant_layer_shape_ok(a->N, a->d, a->lut_format, a->lut_block)) return MOLE_ERR_UNSUPPORTED_SHAPE;
    }

    StepLaunch s;
    s.residual = nullptr;
    s.row_index = a->ids;
    s.gates_out = nullptr;
    s.status = a->status;
    s.lut_stride = a->lut_layer_stride_bytes;
    s.wr_stride = a->wr_layer_stride_bytes;
    s.norm_stride = a->norm_layer_stride_bytes;
    s.norm_eps = a->norm_eps;
    s.M = M;
    s.N = a->N;
    s.d = a->d;
    s.rows = a->V;
    s.dtype = a->dtype;
    s.d_split = a->d_split;
    s.kernel = a->kernel;
    s.stream = static_cast<cudaStream_t>(a->stream);
    if (mode == MOLE_STEP_FUSED) {
        // one launch: every block walks its tokens through all L layers
        s.hidden = a->hidden_in;
        s.lut = a->lut_base;
        s.w_router = a->w_router_base;
        s.norm_weight = a->norm_weight_base;
        s.out = a->out;
        s.L = L;
        s.flags = a->flags & MOLE_FLAG_CHAIN;
        return launch_step(s);
    }
    if (L > 1 && (!a->tmp || !aligned16(a->tmp) || a->out == a->hidden_in || a->tmp == a->hidden_in || a->tmp == a->out))
        return MOLE_ERR_INVALID_ARG;
    // L launches; ping-pong so that the last layer writes `out` and hidden_in is never written.  Layers after
    // the first are chained to their predecessor with programmatic dependent launch (they read nothing but
    // the previous layer's output from it); the first layer only if the caller says so (MOLE_FLAG_CHAIN):
    // whatever precedes it on the stream may be producing ids, tables or router weights.
    const void *src = a->hidden_in;
    for (int l = 0; l < L; ++l) {
        void *dst = ((L - 1 - l) % 2 == 0) ? a->out : a->tmp;
        s.hidden = src;
        s.lut = static_cast<const unsigned char *>(a->lut_base) + static_cast<int64_t>(l) * a->lut_layer_stride_bytes;
        s.w_router = static_cast<const unsigned char *>(a->w_router_base) + static_cast<int64_t>(l) * a->wr_layer_stride_bytes;
        s.norm_weight = a->norm_weight_base
                            ? static_cast<const unsigned char *>(a->norm_weight_base) + static_cast<int64_t>(l) * a->norm_layer_stride_bytes
                            : nullptr;
        s.out = dst;
        s.L = 1;
        s.flags = l > 0 ? MOLE_FLAG_CHAIN : (a->flags & MOLE_FLAG_CHAIN);
        rc = quant ? launch_quant_layer(s, a->lut_format, a->lut_block, current_wait_polls()) : launch_step(s);
        if (rc != MOLE_OK) return rc;
        src = dst;
    }
    return MOLE_OK;
}

int mole_decode_step_ex(const void *hidden_in, const int32_t *ids, const void *lut_base, int64_t lut_layer_stride_bytes,
                        const void *w_router_base, int64_t wr_layer_stride_bytes, void *out, void *tmp, uint32_t *status,
                        int L, int B, int T, int N, int d, int V, int dtype, int mode, int d_split, void *stream)
{
    mole_step_args a;
    memset(&a, 0, sizeof a);
    a.struct_size = sizeof a;
    a.hidden_in = hidden_in;
    a.ids = ids;
    a.lut_base = lut_base;
    a.lut_layer_stride_bytes = lut_layer_stride_bytes;
    a.w_router_base = w_router_base;
    a.wr_layer_stride_bytes = wr_layer_stride_bytes;
    a.out = out;
    a.tmp = tmp;
    a.status = status;
    a.L = L;
    a.B = B;
    a.T = T;
    a.N = N;
    a.d = d;
    a.V = V;
    a.dtype = dtype;
    a.mode = mode;
    a.d_split = d_split;
    a.stream = stream;
    return mole_decode_step_args(&a);
}

int mole_decode_step(const void *hidden_in, const int32_t *ids, const void *lut_base, int64_t lut_layer_stride_bytes,
                     const void *w_router_base, int64_t wr_layer_stride_bytes, void *out, void *tmp, uint32_t *status,
                     int L, int B, int T, int N, int d, int V, int dtype, void *stream)
{
    return mole_decode_step_ex(hidden_in, ids, lut_base, lut_layer_stride_bytes, w_router_base, wr_layer_stride_bytes, out,
                               tmp, status, L, B, T, N, d, V, dtype, MOLE_STEP_AUTO, 0, stream);
}

// Device alias of a host buffer the GPU can address (pinned and mapped: cudaHostAlloc, cudaHostRegister), or
// nullptr for pageable memory.  Asked on every call: a remembered answer would outlive the allocation.
static void *mapped_alias(const void *host)
{
    cudaPointerAttributes attr;
    if (cudaPointerGetAttributes(&attr, host) != cudaSuccess) {
        (void)cudaGetLastError();
        return nullptr;
    }
    return attr.type == cudaMemoryTypeHost ? attr.devicePointer : nullptr;
}

int mole_decode_step_host(const void *hidden_host, const int32_t *ids_host, void *out_host, void *dev_hidden,
                          int32_t *dev_ids, void *dev_out, void *dev_tmp, const void *lut_base,
                          int64_t lut_layer_stride_bytes, const void *w_router_base, int64_t wr_layer_stride_bytes,
                          uint32_t *status, int L, int B, int T, int N, int d, int V, int dtype, void *stream)
{
    // every check the step itself would make, before the first copy is queued
    if (L < 1) return MOLE_ERR_INVALID_ARG;
    int rc = check_common(dev_hidden, dev_ids, lut_base, w_router_base, dev_out, nullptr, B, T, N, d, V, dtype);
    if (rc != MOLE_OK) return rc;
    const long long M = static_cast<long long>(B) * T;
    if (M == 0) return MOLE_OK;
    if (!hidden_host || !ids_host || !out_host) return MOLE_ERR_INVALID_ARG;
    if ((lut_layer_stride_bytes & 15) || (wr_layer_stride_bytes & 15)) return MOLE_ERR_INVALID_ARG;
    if (M * L > 0x3fffffffLL) return MOLE_ERR_TOO_LARGE;
    const bool chained = L > 1 && M > kFusedMaxTokens;
    if (chained && (!dev_tmp || !aligned16(dev_tmp) || dev_out == dev_hidden || dev_tmp == dev_hidden || dev_tmp == dev_out))
        return MOLE_ERR_INVALID_ARG;
    {
        StepPlan plan;
        rc = plan_step(M, chained ? 1 : L, N, d, dtype, 0, &plan);
        if (rc != MOLE_OK) return rc;
    }
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const size_t act_bytes = static_cast<size_t>(M) * d * elem_bytes(dtype);
    // One launch over all layers and host buffers the GPU can address: the launch reads the ids and the hidden
    // state across the link itself and stores the last layer's output across it -- the same bytes cross as with
    // staged copies, without three copy operations and their latencies around the kernel (measured: 60 -> 42 us per
    // step at 256 tokens of the 160M shape).  Every other case stages through the device buffers.
    if (!chained) {
        void *h = mapped_alias(hidden_host), *i = mapped_alias(ids_host), *o = mapped_alias(out_host);
        if (h && i && o && aligned16(h) && aligned16(o) && o != h) {
            mole_step_args a;
            memset(&a, 0, sizeof a);
            a.struct_size = sizeof a;
            a.hidden_in = h;
            a.ids = i;
            a.lut_base = lut_base;
            a.lut_layer_stride_bytes = lut_layer_stride_bytes;
            a.w_router_base = w_router_base;
            a.wr_layer_stride_bytes = wr_layer_stride_bytes;
            a.out = o;
            a.status = status;
            a.L = L;
            a.B = B;
            a.T = T;
            a.N = N;
            a.d = d;
            a.V = V;
            a.dtype = dtype;
            a.mode = MOLE_STEP_FUSED;
            a.stream = stream;
            return mole_decode_step_args(&a);
        }
    }
    MOLE_CUDA_TRY(cudaMemcpyAsync(dev_ids, ids_host, static_cast<size_t>(M) * sizeof(int32_t), cudaMemcpyHostToDevice, st));
    MOLE_CUDA_TRY(cudaMemcpyAsync(dev_hidden, hidden_host, act_bytes, cudaMemcpyHostToDevice, st));
    rc = mole_decode_step(dev_hidden, dev_ids, lut_base, lut_layer_stride_bytes, w_router_base, wr_layer_stride_bytes,
                          dev_out, dev_tmp, status, L, B, T, N, d, V, dtype, stream);
    if (rc != MOLE_OK) return rc;
    MOLE_CUDA_TRY(cudaMemcpyAsync(out_host, dev_out, act_bytes, cudaMemcpyDeviceToHost, st));
    return MOLE_OK;
}

// SM count of the current device if there is one, the nominal B200 figure otherwise (no error is kept)
static int sms_or_nominal()
{
    int sms = kNumSMs;
    if (sm_count(&sms) != MOLE_OK) {
        (void)cudaGetLastError();
        sms = kNumSMs;
    }
    return sms;
}

int mole_prefetch_rows(const void *ids, int M, const void *lut_base, int64_t lut_layer_stride_bytes, int layers, int N, int d, int V,
                       int dtype, uint32_t flags, void *stream)
{
    if (dtype != MOLE_DTYPE_BF16 && dtype != MOLE_DTYPE_F32) return MOLE_ERR_INVALID_ARG;
    if (flags & ~MOLE_FLAG_IDS_INT64) return MOLE_ERR_INVALID_ARG;
    if (M < 0 || layers < 0) return MOLE_ERR_INVALID_ARG;
    const int vec = 16 / elem_bytes(dtype);
    if (N < 1 || N > kMaxN || V < 1 || d < vec || d % vec != 0) return MOLE_ERR_UNSUPPORTED_SHAPE;
    if (M == 0 || layers == 0) return MOLE_OK;
    if (layers > 65535) return MOLE_ERR_TOO_LARGE;
    if (!ids || !lut_base || !aligned16(lut_base) || (lut_layer_stride_bytes & 15)) return MOLE_ERR_INVALID_ARG;
    const long long row_bytes = static_cast<long long>(N) * d * elem_bytes(dtype);
    const int threads = 128;
    dim3 grid(static_cast<unsigned>((M + threads - 1) / threads), static_cast<unsigned>(layers));
    mole_prefetch_rows_kernel<<<grid, threads, 0, static_cast<cudaStream_t>(stream)>>>(
        ids, M, static_cast<const unsigned char *>(lut_base), lut_layer_stride_bytes, row_bytes, V, (flags & MOLE_FLAG_IDS_INT64) ? 1 : 0);
    MOLE_CUDA_TRY(cudaGetLastError());
    return MOLE_OK;
}

int mole_plan(int M, int L, int N, int d, int dtype, int d_split, int *out_d_split, int *out_threads, int *out_smem_bytes,
              int *out_stages, int *out_blocks_per_sm)
{
    StepPlan plan;
    int rc = plan_step(M, L, N, d, dtype, d_split, &plan, false, sms_or_nominal());
    if (rc != MOLE_OK) return rc;
    if (out_d_split) *out_d_split = plan.d_split;
    if (out_threads) *out_threads = plan.threads;
    if (out_smem_bytes) *out_smem_bytes = plan.smem;
    if (out_stages) *out_stages = plan.stages;
    if (out_blocks_per_sm) *out_blocks_per_sm = plan.blocks_per_sm;
    return MOLE_OK;
}

int mole_variant(int M, int L, int N, int d, int dtype, int d_split, int norm, int kernel, int lut_format, int lut_block, char *name,
                 int name_bytes, int *out_threads, int *out_smem_bytes)
{
    if (M < 1 || !name || name_bytes < 1) return MOLE_ERR_INVALID_ARG;
    if (lut_format != MOLE_LUT_PLAIN) {
        if (lut_format != MOLE_LUT_NF4 && lut_format != MOLE_LUT_NF3) return MOLE_ERR_INVALID_ARG;
        if (L != 1 || dtype != MOLE_DTYPE_BF16 || d_split != 0 || kernel == MOLE_KERNEL_RING ||
            !quant_layer_shape_ok(N, d, lut_format, lut_block))
            return MOLE_ERR_UNSUPPORTED_SHAPE;
        snprintf(name, static_cast<size_t>(name_bytes), "%s", quant_variant_name(N, lut_format, norm != 0));
        if (out_threads) *out_threads = d / 4;
        if (out_smem_bytes) *out_smem_bytes = 0;
        return MOLE_OK;
    }
    LaunchChoice c;
    int rc = choose_launch(M, L, N, d, dtype, d_split, norm != 0, kernel, sms_or_nominal(), false, &c);
    if (rc != MOLE_OK) return rc;
    snprintf(name, static_cast<size_t>(name_bytes), "%s", c.name);
    if (out_threads) *out_threads = c.threads;
    if (out_smem_bytes) *out_smem_bytes = c.smem;
    return MOLE_OK;
}

int mole_reload_debug_env(void)
{
    std::lock_guard<std::mutex> lock(g_env_mutex);
    load_env_locked();
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
        case MOLE_ERR_IO: return "table file error";
        default: return "unknown status";
    }
}

const char *mole_last_cuda_error(void) { return g_cuda_error; }

int mole_version(void) { return MOLE_VERSION; }

}  // extern "C"
