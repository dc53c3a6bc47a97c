// Host side of the fused MoLE kernel: launch planning, argument checks and the C entry points
// for a single layer and for a chained L-layer decode step (Eq. 4 and Eq. 8 of arXiv
// 2503.15798).  The kernel itself is in mole_kernel.cuh.
#include <atomic>
#include <string.h>

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

constexpr int kNumSMs = 148;                  // B200; the launch asks the device for its own count
constexpr int kSmemPerBlockMax = 227 * 1024;  // opt-in limit per block
constexpr int kSmemPerSM = 228 * 1024;        // per SM, of which every resident block reserves 1 KB
constexpr long long kFusedMaxTokens = 4096;   // above this a step runs as L chained launches

static int consumers_for(int dc, int vec)
{
    const int groups = dc / vec;
    return round_up(groups < kMaxConsumers ? groups : kMaxConsumers, 32);
}

int plan_step(long long M, int L, int N, int d, int dtype, int d_split, StepPlan *plan)
{
    if (dtype != MOLE_DTYPE_BF16 && dtype != MOLE_DTYPE_F32) return MOLE_ERR_INVALID_ARG;
    if (L < 1 || M < 0) return MOLE_ERR_INVALID_ARG;
    const int eb = elem_bytes(dtype), vec = 16 / eb;
    if (N < 1 || N > kMaxN || d < vec || d % vec != 0) return MOLE_ERR_UNSUPPORTED_SHAPE;
    const int in_ring = L > 1 ? 1 : 0;
    auto fits = [&](int S, int stages) {
        const int dc = d / S;
        return smem_map(N, dc, eb, S, stages, in_ring, consumers_for(dc, vec)).total <=
               static_cast<uint32_t>(kSmemPerBlockMax);
    };
    int S;
    if (d_split != 0) {
        if (d_split != 1 && d_split != 2 && d_split != 4 && d_split != 8) return MOLE_ERR_INVALID_ARG;
        if (d % (d_split * vec) != 0) return MOLE_ERR_UNSUPPORTED_SHAPE;
        S = d_split;
        if (!fits(S, 2)) return MOLE_ERR_UNSUPPORTED_SHAPE;
    } else {
        // Split a token over more blocks while one item (rows + router slice) is too large for a
        // ring of several slots, or while there are too few tokens to give every SM a block;
        // stop when a row piece would drop under 512 bytes.
        S = 1;
        while (S < kMaxSplit && d % (2 * S * vec) == 0 && (d / (2 * S)) * eb >= 512) {
            const long long item = static_cast<long long>(N) * (d / S) * eb * (1 + in_ring);
            if (item > 48 * 1024 || M * S < kNumSMs) S *= 2;
            else break;
        }
        while (!fits(S, 2)) {
            if (S >= kMaxSplit || d % (2 * S * vec) != 0) return MOLE_ERR_UNSUPPORTED_SHAPE;
            S *= 2;
        }
    }
    const int dc = d / S;
    const int consumers = consumers_for(dc, vec);
    const SmemMap one = smem_map(N, dc, eb, S, 1, in_ring, consumers);
    const int fixed = static_cast<int>(one.total - one.slot_bytes);
    const int slot = static_cast<int>(one.slot_bytes);
    // Resident blocks per SM wanted: enough to cover the work (up to 4), each with >= 2 slots.
    long long want = (M * S + kNumSMs - 1) / kNumSMs;
    want = want < 1 ? 1 : (want > 4 ? 4 : want);
    int stages = 2;
    for (; want >= 1; --want) {
        const long long room = kSmemPerSM / want - 1024 - fixed;
        stages = static_cast<int>(room / slot);
        if (stages >= 2) break;
    }
    if (stages < 2) stages = 2;  // fits(S, 2) holds
    if (stages > kMaxStages) stages = kMaxStages;
    // no deeper than the items a block will see
    const long long cap = static_cast<long long>(kNumSMs) * 4;
    const long long blocks = M * S < cap ? M * S : cap;
    const long long items = blocks > 0 ? ((M * S + blocks - 1) / blocks) * L : 1;
    if (stages > items) stages = items < 2 ? 2 : static_cast<int>(items);
    while (stages > 2 && !fits(S, stages)) --stages;
    const SmemMap m = smem_map(N, dc, eb, S, stages, in_ring, consumers);
    plan->d_split = S;
    plan->dc = dc;
    plan->consumers = consumers;
    plan->threads = consumers + 32;
    plan->stages = stages;
    plan->slot_bytes = static_cast<int>(m.slot_bytes);
    plan->wr_in_ring = in_ring;
    plan->smem = static_cast<int>(m.total);
    int per_sm = kSmemPerSM / (plan->smem + 1024);
    if (per_sm > 2048 / plan->threads) per_sm = 2048 / plan->threads;
    if (per_sm > 32) per_sm = 32;
    if (per_sm < 1) per_sm = 1;
    plan->blocks_per_sm = per_sm;
    plan->n_fast = (N == 4 || N == 8 || N == 16 || N == 32 || N == 64) ? N : 0;
    return MOLE_OK;
}

typedef void (*StepKernel)(const StepParams);

template <typename T>
static StepKernel pick_n(int n_fast)
{
    switch (n_fast) {
        case 4: return mole_step_kernel<T, 4>;
        case 8: return mole_step_kernel<T, 8>;
        case 16: return mole_step_kernel<T, 16>;
        case 32: return mole_step_kernel<T, 32>;
        case 64: return mole_step_kernel<T, 64>;
        default: return mole_step_kernel<T, 0>;
    }
}

static StepKernel pick_kernel(int dtype, int n_fast)
{
    return dtype == MOLE_DTYPE_BF16 ? pick_n<__nv_bfloat16>(n_fast) : pick_n<float>(n_fast);
}

// Kernels that need more than 48 KB of dynamic shared memory must opt in once per device.
static int ensure_smem(StepKernel k, int smem)
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

// SM count of the current device, asked once per device.
static int sm_count(int *out)
{
    static std::atomic<int> cache[64];
    int dev = 0;
    MOLE_CUDA_TRY(cudaGetDevice(&dev));
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

int launch_step(const StepLaunch &a)
{
    if (a.M == 0) return MOLE_OK;
    StepPlan plan;
    int rc = plan_step(a.M, a.L, a.N, a.d, a.dtype, a.d_split, &plan);
    if (rc != MOLE_OK) return rc;
    if (a.M * plan.d_split > 0x7fffffffLL) return MOLE_ERR_TOO_LARGE;
    int sms = kNumSMs;
    rc = sm_count(&sms);
    if (rc != MOLE_OK) return rc;
    // a persistent grid: as many blocks as fit at once (whole clusters), never more than the work
    long long grid = static_cast<long long>(plan.blocks_per_sm) * sms / plan.d_split * plan.d_split;
    if (grid < plan.d_split) grid = plan.d_split;
    if (grid > a.M * plan.d_split) grid = a.M * plan.d_split;

    StepParams p;
    p.hidden = a.hidden;
    p.residual = a.residual;
    p.row_index = a.row_index;
    p.lut = a.lut;
    p.w_router = a.w_router;
    p.out = a.out;
    p.gates_out = a.gates_out;
    p.status = a.status;
    p.lut_stride = a.lut_stride;
    p.wr_stride = a.wr_stride;
    p.M = a.M;
    p.rows = a.rows;
    p.N = a.N;
    p.d = a.d;
    p.S = plan.d_split;
    p.dc = plan.dc;
    p.L = a.L;
    p.stages = plan.stages;
    p.slot_bytes = plan.slot_bytes;
    p.wr_in_ring = plan.wr_in_ring;
    p.consumers = plan.consumers;
    p.flags = a.flags;

    StepKernel k = pick_kernel(a.dtype, plan.n_fast);
    rc = ensure_smem(k, plan.smem);
    if (rc != MOLE_OK) return rc;

    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof cfg);
    cfg.gridDim = dim3(static_cast<unsigned>(grid), 1, 1);
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
    if (plan.d_split > 1) {
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

