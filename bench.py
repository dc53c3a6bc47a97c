#!/usr/bin/env python3
"""Benchmark of the fused MoLE layer (arXiv 2503.15798, Eq. 4 + Eq. 8) on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config 160m|410m|1b] [--batch M]
                    [--impl mole|reference] [--no-sweep] [--no-cpu]

A "step" is one decode step of the whole hot path: all L layers of the configuration applied
to one batch of M tokens (router, softmax over all experts, row gather, weighted sum,
residual), chained with programmatic dependent launch and replayed from a CUDA graph.  The
metric is tokens/s for the L-layer step; the roofline block reports the layer kernel's
algorithmic GB/s (gathered rows + hidden in/out + router weights) against the measured HBM
copy bandwidth.  Every step uses a different pre-generated Zipf(1.1) id batch, and the table
(GBs) is far larger than L2.  Beside it, as an extra ("fused_step"), the same step as a single
launch that walks every token through all L layers on chip.

With N > 1 (torchrun) every rank holds its own replica of the tables and its own batches
(tokens are independent, so there is no collective on the data path): weak scaling.

--impl reference times the CPU oracle (oracle/, plain C, fp64) on the host cores instead.
"""
from __future__ import annotations

import argparse
import dataclasses
import json
import os
import statistics
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "MoLE layer tokens/s (L-layer decode step) and achieved HBM GB/s"
UNIT = "tokens/s"
N_BATCHES = 32          # distinct id batches the steps rotate through
OFFLOAD_CONTEXT_TOKENS = 256  # offload mode: the context (staging areas) is sized for this many tokens
FALLBACK_HBM_GBS = 6650.0
# dram__bytes_read.sum + dram__bytes_write.sum of one launch of the dominant kernel, from the ncu
# capture summarised under profiles/ ((config, batch, layers) -> bytes); None until one is taken
TRAFFIC = {
    # profiles/mole_step_kernel_single_layer_160m_batch256.md: mean of three captured launches (one layer each)
    ("160m", 256, 12): 4.43e6,
}
# the same for the fused all-layers launch reported as an extra
FUSED_TRAFFIC = {
    # profiles/mole_step_kernel_fused_160m_batch256.md: 7.59 MB per 2-layer launch, x6 for the 12 layers of a full launch
    ("160m", 256, 12): 45.5e6,
}


def offload_groups(L: int, M: int, row_bytes: int) -> int:
    """Groups of layers mole_offload_decode_step forms on a context of OFFLOAD_CONTEXT_TOKENS tokens (one
    fetch launch and one fused layer launch per group): as many layers as the staging area holds, but at
    least three groups unless the whole step's rows are at most 1 MB."""
    g = min(L, max(1, OFFLOAD_CONTEXT_TOKENS // M))
    if M * row_bytes * L > (1 << 20):
        g = min(g, (L + 2) // 3)
    return -(-L // g)


OFFLOAD_BATCHES = (1, 8, 64)


def timed_launch_shapes():
    """Every launch shape a timed region of this file issues, as dicts (what, M, N, d, L, norm, kernel):
    the parity tests walk this list and require a parity case for the kernel instantiation of each."""
    from paper_2503_15798_b200 import inputs

    shapes = []
    for name in ("160m", "410m", "1b"):
        sh = inputs.SHAPES[name]
        for M in sh.batches:
            for norm in (False, True):
                tag = " norm" if norm else ""
                shapes.append({"what": f"{name} batch {M} chained{tag}", "M": M, "N": sh.N, "d": sh.d, "L": 1, "norm": norm,
                               "kernel": 0})
                if M <= 4096:
                    shapes.append({"what": f"{name} batch {M} fused{tag}", "M": M, "N": sh.N, "d": sh.d, "L": sh.L,
                                   "norm": norm, "kernel": 0})
            shapes.append({"what": f"{name} batch {M} chained, ring kernel", "M": M, "N": sh.N, "d": sh.d, "L": 1,
                           "norm": False, "kernel": 1})
    sh = inputs.SHAPES["410m"]
    for M in OFFLOAD_BATCHES:
        groups = offload_groups(sh.L, M, sh.row_bytes)
        per = -(-sh.L // groups)
        for L in {per, sh.L - per * (groups - 1)}:
            shapes.append({"what": f"410m offload batch {M}, group of {L} layers", "M": M, "N": sh.N, "d": sh.d, "L": L,
                           "norm": False, "kernel": 0})
    return shapes


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=4000)
    ap.add_argument("--warmup", type=int, default=100)
    ap.add_argument("--impl", default="mole", choices=["mole", "reference"])
    ap.add_argument("--config", default="160m", choices=["160m", "410m", "1b"])
    ap.add_argument("--batch", type=int, default=256)
    ap.add_argument("--no-sweep", action="store_true", help="skip the per-batch sweep and the isolated-launch rows")
    ap.add_argument("--no-cpu", action="store_true", help="skip the CPU-oracle baseline leg")
    ap.add_argument("--layers", type=int, default=0, help="override L (debugging; the line then says so)")
    ap.add_argument("--vocab", type=int, default=0,
                    help="override V, the number of table rows (small profiler captures; the line then says so)")
    ap.add_argument("--offload", action="store_true",
                    help="offload mode instead: table in pinned host memory, per-step dedup + row fetch overlapped with "
                         "the previous layer's combine; roofline = measured host-link GB/s")
    return ap.parse_args()


def measured_peak():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(p) as f:
            return float(json.load(f)["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs)"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback (6.65 TB/s, earlier measurement on this pool)"


class ClockSampler:
    """Samples SM clock and throttle reasons through NVML (read-only) while a region runs."""

    def __init__(self, index: int, period_s: float = 0.01):
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self.period, self._stop, self._thread, self.h = period_s, threading.Event(), None, None
        try:
            import pynvml

            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
        except Exception:
            self.nv = None

    def _run(self):
        nv = self.nv
        names = {
            getattr(nv, "nvmlClocksEventReasonHwSlowdown", 0x8): "hw_slowdown",
            getattr(nv, "nvmlClocksEventReasonHwThermalSlowdown", 0x40): "hw_thermal_slowdown",
            getattr(nv, "nvmlClocksEventReasonSwThermalSlowdown", 0x20): "sw_thermal_slowdown",
            getattr(nv, "nvmlClocksEventReasonSwPowerCap", 0x4): "sw_power_cap",
        }
        while not self._stop.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                try:
                    r = nv.nvmlDeviceGetCurrentClocksEventReasons(self.h)
                except Exception:
                    r = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                for bit, name in names.items():
                    if r & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            self._stop.wait(self.period)

    def __enter__(self):
        if self.nv is not None and self.h is not None:
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()
        return self

    def __exit__(self, *exc):
        self._stop.set()
        if self._thread:
            self._thread.join()

    def summary(self):
        return {"sm_mhz": statistics.median(self.samples) if self.samples else None, "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(self.samples)}


def physical_gpu_index(local_rank: int) -> int:
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    if vis:
        try:
            return int(vis.split(",")[local_rank])
        except Exception:
            return local_rank
    return local_rank


def max_over_ranks(ms: float, dist, device) -> float:
    """Step time of the job = the slowest rank's (all-reduce MAX; `dist` None for one process)."""
    if dist is None:
        return ms
    import torch

    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_tokens_per_s(world: int, M: int, steps: int, ms: float) -> float:
    """Replicas only (weak scaling): every rank runs its own M-token steps, so the job's rate is
    world * M * steps over the slowest rank's time."""
    return world * M * steps / (ms * 1e-3)


def rank_seeds(rank: int, layer: int = 0, batch: int = 0, m: int = 0) -> dict:
    """Per-rank seeds: every replica has its own tables, hidden states and id batches."""
    return {"table": 1000 + layer + 100 * rank, "router": 2000 + layer, "hidden": 3000 + rank,
            "ids": 4000 + 1000 * rank + batch + 7 * m}


def reference_arm_runs_here(rank: int) -> bool:
    """--impl reference under torchrun: rank 0 alone runs and prints; the others exit 0 without work."""
    return rank == 0


# ------------------------------------------------------------------------------------------------------
# the CPU oracle leg (only bench.py's baseline leg and --impl reference execute oracle/)
# ------------------------------------------------------------------------------------------------------

def time_oracle(table_bits, wr_bits, hidden_bits, id_batches, L, budget_s, threads):
    """Oracle lookup-form layer (fp64) on host copies; returns tokens/s for the L-layer step
    (= one-layer tokens/s divided by L), the number of timed layer calls and the seconds used."""
    import oracle

    oracle.layer_lookup(hidden_bits, id_batches[0], table_bits, wr_bits, threads=threads)  # warm the pages
    calls, t0 = 0, time.perf_counter()
    while True:
        oracle.layer_lookup(hidden_bits, id_batches[calls % len(id_batches)], table_bits, wr_bits, threads=threads)
        calls += 1
        dt = time.perf_counter() - t0
        if dt >= budget_s or calls >= 1000000:
            break
    M = hidden_bits.shape[0]
    return M * calls / dt / L, calls, dt


def host_bits(t):
    import numpy as np
    import torch

    return t.detach().cpu().contiguous().view(torch.int16).numpy().view(np.uint16)


def run_reference(args):
    """--impl reference: the oracle, as it stands, on the host cores (rank 0 only)."""
    import numpy as np
    import torch

    import oracle
    from paper_2503_15798_b200 import inputs

    if not reference_arm_runs_here(int(os.environ.get("RANK", "0"))):
        return
    sh = inputs.SHAPES[args.config]
    L = args.layers or sh.L
    M = args.batch
    cores = oracle.effective_threads(len(os.sched_getaffinity(0)))
    table = host_bits(inputs.make_table(sh.V, sh.N, sh.d, seed=1000, device="cpu"))
    wr = host_bits(inputs.make_router(sh.d, sh.N, seed=2000, device="cpu"))
    hidden = host_bits(inputs.make_hidden(M, sh.d, seed=3000, device="cpu"))
    batches = [inputs.zipf_ids(M, sh.V, seed=4000 + b).astype(np.int64) for b in range(N_BATCHES)]
    for w in range(max(args.warmup, 1)):
        oracle.layer_lookup(hidden, batches[w % N_BATCHES], table, wr, threads=cores)
    t0 = time.perf_counter()
    for k in range(args.steps):  # each step: ONE layer of the L-layer step (a 1/L sample), scaled below
        oracle.layer_lookup(hidden, batches[k % N_BATCHES], table, wr, threads=cores)
    dt = time.perf_counter() - t0
    value = M * args.steps / dt / L
    sample = (f"each step = the oracle's lookup-form layer on 1 of the {L} layers ({M} tokens, one {sh.name}-shaped "
              f"bf16 table on the host); tokens/s divided by L for the L-layer step")
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": 1e3 * dt / args.steps * L, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": workload_config(sh, L, M, args),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


def workload_config(sh, L, M, args):
    return {
        "workload": f"{sh.name}-shaped decode: V={sh.V}, d={sh.d}, N={sh.N}, L={L}, bf16 table "
                    f"{sh.layer_table_bytes * L / 1e9:.2f} GB, batch {M}x1, ids Zipf(1.1), hidden N(0,1)",
        "V": sh.V, "d": sh.d, "N": sh.N, "L": L, "batch": M, "seq_len": 1,
        "l2": f"inputs larger than L2: {N_BATCHES} rotating id batches over a {sh.layer_table_bytes * L / 1e9:.1f} GB "
              "table; no flush between steps (hot Zipf rows may hit L2, as in the workload)",
        "parallelism": f"replicas x{args.gpus} (tokens independent, no collective)",
    }


# ------------------------------------------------------------------------------------------------------
# the GPU arm
# ------------------------------------------------------------------------------------------------------

class StepGraphs:
    """One CUDA graph per id batch; a graph holds the L chained layer launches of one step."""

    def __init__(self, mole, luts, wrs, hidden, id_batches, mode=0):
        import torch

        self.torch, self.graphs = torch, []
        self.out = torch.empty_like(hidden)
        self.tmp = torch.empty_like(hidden)
        self.status = torch.zeros(1, dtype=torch.int32, device=hidden.device)
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            for ids in id_batches:  # warm-up launches outside capture (sets kernel attributes)
                mole.decode_step(hidden, ids, luts, wrs, self.out, self.tmp, status=self.status, mode=mode)
        torch.cuda.current_stream().wait_stream(side)
        torch.cuda.synchronize()
        for ids in id_batches:
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g):
                mole.decode_step(hidden, ids, luts, wrs, self.out, self.tmp, status=self.status, mode=mode)
            self.graphs.append(g)

    def run(self, k0, k1):
        n = len(self.graphs)
        for k in range(k0, k1):
            self.graphs[k % n].replay()


class NormStepGraphs(StepGraphs):
    """The same chained step with the decoder layer of the paper's App. A.2 listing: every layer's
    router reads RMSNorm(hidden) (fused into the kernel), the residual stays un-normalised."""

    def __init__(self, mole, luts, wrs, gammas, hidden, id_batches, eps=1e-5):
        import torch

        self.torch, self.graphs = torch, []
        self.out = torch.empty_like(hidden)
        self.tmp = torch.empty_like(hidden)
        self.status = torch.zeros(1, dtype=torch.int32, device=hidden.device)
        L = luts.shape[0]

        def step(ids):
            src = hidden
            for l in range(L):
                dst = self.out if (L - 1 - l) % 2 == 0 else self.tmp
                mole.layer_forward(src, ids, luts[l], wrs[l], dst, status=self.status, chain=l > 0,
                                   norm_weight=gammas[l], norm_eps=eps)
                src = dst

        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            for ids in id_batches:
                step(ids)
        torch.cuda.current_stream().wait_stream(side)
        torch.cuda.synchronize()
        for ids in id_batches:
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g):
                step(ids)
            self.graphs.append(g)


def timed_ms(torch, fn):
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record()
    fn()
    b.record()
    b.synchronize()
    return a.elapsed_time(b)


def run_mole(args):
    import numpy as np
    import torch

    from paper_2503_15798_b200 import binding as mole
    from paper_2503_15798_b200 import build as lib_build
    from paper_2503_15798_b200 import inputs

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if rank == 0:
        lib_build.build()
    dist = None
    if world > 1:
        import torch.distributed as dist

        torch.cuda.set_device(local_rank)
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
        dist.barrier()
    else:
        torch.cuda.set_device(local_rank)
    mole.lib()  # fails loudly if the library is missing
    dev = torch.device("cuda", local_rank)
    sh = inputs.SHAPES[args.config]
    if args.vocab > 0:
        sh = dataclasses.replace(sh, V=args.vocab)
    L = args.layers or sh.L
    M = args.batch
    peak, peak_src = measured_peak()

    # ---- resident inputs: L tables, routers, hidden, rotating id batches (per-rank seeds) ----------
    luts = torch.empty((L, sh.V, sh.N, sh.d), dtype=torch.bfloat16, device=dev)
    for l in range(L):
        inputs.make_table(sh.V, sh.N, sh.d, seed=rank_seeds(rank, l)["table"], device=dev, out=luts[l])
    wrs = torch.stack([inputs.make_router(sh.d, sh.N, seed=2000 + l, device=dev) for l in range(L)])
    max_m = max([M] + ([b for b in sh.batches] if not args.no_sweep else []))
    hidden_all = inputs.make_hidden(max_m, sh.d, seed=rank_seeds(rank)["hidden"], device=dev)

    def batches_for(m):
        return [inputs.make_ids(m, sh.V, seed=rank_seeds(rank, 0, b, m)["ids"], device=dev) for b in range(N_BATCHES)]

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    # ---- headline: K steps of the L-layer decode step as a model that runs other work between the layers
    # gets it: one launch per layer, chained with programmatic dependent launch, the layer's output the next
    # layer's hidden state, the L launches of a step replayed from a CUDA graph -----------------------------
    hidden = hidden_all[:M].contiguous()
    fused = False
    graphs = StepGraphs(mole, luts, wrs, hidden, batches_for(M), mode=mole.STEP_CHAINED)
    graphs.run(0, max(args.warmup, 3))
    barrier()
    with ClockSampler(physical_gpu_index(local_rank)) as clocks:
        ms = timed_ms(torch, lambda: graphs.run(0, args.steps))
    barrier()
    assert int(graphs.status.item()) == 0, "a kernel reported a bad id or a timed-out wait"
    ms = max_over_ranks(ms, dist, dev)
    ms_per_step = ms / args.steps
    value = whole_job_tokens_per_s(world, M, args.steps, ms)
    launches = args.steps * (1 if fused else L)
    launch_bytes = sh.step_bytes(M, L) if fused else sh.layer_bytes(M)
    achieved = launch_bytes / (ms * 1e-3 / launches) / 1e9

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
        "data": "synthetic", "config": workload_config(sh, L, M, args),
        "tokens_per_s_per_layer": value * L,
        "gpu_launches": launches,
        "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                     "traffic": TRAFFIC.get((sh.name, M, L)), "kernel": "mole_step_kernel", "peak_source": peak_src,
                     "launch": "one launch per layer (%d per step), chained with programmatic dependent launch" % L,
                     "algorithmic_bytes_per_launch": launch_bytes, "us_per_launch": ms * 1e3 / launches},
        "clocks": clocks.summary(),
    }

    # ---- extra, never the headline: the same step as ONE launch that keeps a token's chain through all L
    # layers on chip (what mole_decode_step picks by itself up to 4096 tokens) ------------------------------
    del graphs
    if L > 1 and M <= 4096:
        g = StepGraphs(mole, luts, wrs, hidden, batches_for(M), mode=mole.STEP_FUSED)
        g.run(0, max(args.warmup, 3))
        barrier()
        ms_f = max_over_ranks(timed_ms(torch, lambda: g.run(0, args.steps)), dist, dev)
        barrier()
        assert int(g.status.item()) == 0, "a kernel reported a bad id or a timed-out wait"
        fb = sh.step_bytes(M, L)
        gbs = fb / (ms_f * 1e-3 / args.steps) / 1e9
        line["fused_step"] = {"what": "all %d layers of a step in one launch (layer-batched), an extra beside the headline" % L,
                              "value": whole_job_tokens_per_s(world, M, args.steps, ms_f), "unit": UNIT,
                              "us_per_step": ms_f * 1e3 / args.steps, "algorithmic_bytes_per_launch": fb,
                              "achieved": gbs, "frac": gbs / peak, "traffic": FUSED_TRAFFIC.get((sh.name, M, L))}
        del g

    # ---- extra: the chained step with RMSNorm fused in front of every layer's router (App. A.2 listing) ----
    if rank == 0:
        gammas = torch.stack([inputs.make_router(sh.d, 1, seed=2500 + l, device=dev).reshape(sh.d) + 1.0 for l in range(L)])
        g = NormStepGraphs(mole, luts, wrs, gammas, hidden, batches_for(M))
        g.run(0, max(args.warmup, 3))
        torch.cuda.synchronize()
        steps_n = min(args.steps, 2000)
        ms_n = timed_ms(torch, lambda: g.run(0, steps_n))
        assert int(g.status.item()) == 0, "a kernel reported a bad id or a timed-out wait"
        us_layer_n = ms_n * 1e3 / (steps_n * L)
        line["norm_router_step"] = {"what": "chained step whose routers read RMSNorm(hidden), fused into the layer kernel",
                                    "us_per_layer": us_layer_n, "value": M / (us_layer_n * L * 1e-6), "unit": UNIT,
                                    "achieved": sh.layer_bytes(M) / us_layer_n / 1e3,
                                    "frac": sh.layer_bytes(M) / us_layer_n / 1e3 / peak}
        del g

    # ---- end to end: host buffers in, host buffer out, through the C ABI, every step ---------------------
    h_host = hidden.cpu().pin_memory()
    out_host = torch.empty_like(h_host).pin_memory()
    ids_host = [b.cpu().pin_memory() for b in batches_for(M)]
    dev_bufs = [torch.empty_like(hidden) for _ in range(3)]
    dev_ids = torch.empty(M, dtype=torch.int32, device=dev)
    e2e_steps = min(args.steps, 2000)

    def e2e_call(k):
        mole.decode_step_host(h_host, ids_host[k % N_BATCHES], out_host, dev_bufs[0], dev_ids, dev_bufs[1],
                              dev_bufs[2], luts, wrs)

    for k in range(3):  # uncaptured calls first (kernel attributes), then one CUDA graph per id batch:
        e2e_call(k)     # two host->device copies, the step, one device->host copy
    torch.cuda.synchronize()
    e2e_graphs = []
    for k in range(N_BATCHES):
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            e2e_call(k)
        e2e_graphs.append(g)

    def e2e_run(n):
        for k in range(n):
            e2e_graphs[k % N_BATCHES].replay()
            torch.cuda.current_stream().synchronize()  # the caller reads out_host after every step

    e2e_run(max(3, min(args.warmup, 50)))
    barrier()
    t0 = time.perf_counter()
    ms_e2e = timed_ms(torch, lambda: e2e_run(e2e_steps))
    wall_e2e = time.perf_counter() - t0
    barrier()
    ms_e2e = max_over_ranks(ms_e2e, dist, dev)
    line["e2e"] = {"value": whole_job_tokens_per_s(world, M, e2e_steps, ms_e2e), "unit": UNIT,
                   "h2d_bytes_per_step": M * sh.d * 2 + M * 4, "d2h_bytes_per_step": M * sh.d * 2,
                   "steps": e2e_steps, "ms_per_step": ms_e2e / e2e_steps,
                   "how": "mole_decode_step_host captured into one CUDA graph per id batch: pinned host hidden+ids -> device, "
                          "the step as mole_decode_step launches it by itself (one fused launch over all layers up to "
                          "4096 tokens), result -> pinned host; one graph launch and one stream synchronisation per step"}

    # ---- sweep over the configuration's batch sizes: chained step + isolated launches -----------------------
    if not args.no_sweep and rank == 0:
        sweep = []
        flush = torch.empty(256 * 1024 * 1024, dtype=torch.uint8, device=dev)
        for m in sh.batches:
            if m * sh.d * 2 > 2**31:
                continue
            hid = hidden_all[:m].contiguous()
            bl = batches_for(m)
            steps_m = max(50, min(args.steps, int(2e6 // max(m, 64))))
            g = StepGraphs(mole, luts, wrs, hid, bl, mode=mole.STEP_CHAINED)
            g.run(0, 20)
            torch.cuda.synchronize()
            ms_m = timed_ms(torch, lambda: g.run(0, steps_m))
            us_layer = ms_m * 1e3 / (steps_m * L)
            del g
            us_fused = None
            if m <= 4096:
                g = StepGraphs(mole, luts, wrs, hid, bl, mode=mole.STEP_FUSED)
                g.run(0, 20)
                torch.cuda.synchronize()
                us_fused = timed_ms(torch, lambda: g.run(0, steps_m)) * 1e3 / steps_m
                del g
            # isolated single launches of layer 0: steady (rotating ids) and cold (L2 flushed before each)
            out = torch.empty_like(hid)
            reps = 200 if m <= 1024 else 20
            iso = []
            for cold in (False, True):
                ts = []
                for r in range(reps):
                    # keep the GPU busy while the host queues the events and the launch, so that the interval
                    # between the events holds the launch alone: an L2 flush (cold) or a spin that touches no memory
                    if cold:
                        flush.fill_(r & 0xFF)
                    else:
                        torch.cuda._sleep(100000)
                    ts.append(timed_ms(torch, lambda: mole.layer_forward(hid, bl[r % N_BATCHES], luts[0], wrs[0], out)))
                iso.append(statistics.median(ts) * 1e3)
            nbytes = sh.layer_bytes(m)
            fb = sh.step_bytes(m, L)
            sweep.append({
                "batch": m,
                "fused_us_per_step": us_fused, "fused_tokens_per_s_all_layers": (m / (us_fused * 1e-6)) if us_fused else None,
                "fused_GBps": (fb / us_fused / 1e3) if us_fused else None,
                "fused_frac_of_peak": (fb / us_fused / 1e3 / peak) if us_fused else None,
                "chained_us_per_layer": us_layer, "tokens_per_s_all_layers": m / (us_layer * L * 1e-6),
                "tokens_per_s_per_layer": m / (us_layer * 1e-6), "chained_GBps": nbytes / us_layer / 1e3,
                "chained_frac_of_peak": nbytes / us_layer / 1e3 / peak,
                "isolated_steady_us": iso[0], "isolated_cold_us": iso[1],
                "isolated_cold_GBps": nbytes / iso[1] / 1e3,
                "plan_layer": mole.plan(m, sh.N, sh.d), "plan_fused": mole.plan(m, sh.N, sh.d, mole.DTYPE_BF16, 0, L),
            })
        line["sweep"] = sweep
        del flush

    # ---- the CPU oracle beside it (rank 0, N = 1 only) ------------------------------------------------------
    if not args.no_cpu and rank == 0 and world == 1:
        import oracle

        cores = oracle.effective_threads(len(os.sched_getaffinity(0)))
        table0 = host_bits(luts[0])
        ids_np = [b.cpu().numpy().astype(np.int64) for b in batches_for(M)]
        v_all, calls, dt = time_oracle(table0, host_bits(wrs[0]), host_bits(hidden), ids_np, L, 12.0, cores)
        v_one, calls1, dt1 = time_oracle(table0, host_bits(wrs[0]), host_bits(hidden), ids_np, L, 5.0, 1)
        line["cpu_baseline"] = {
            "value": v_all, "unit": UNIT, "cores": cores, "kind": "oracle",
            "sample": f"{calls} calls of the oracle's lookup-form layer (fp64) on a host copy of layer 0's table, "
                      f"{M} tokens each, {dt:.1f} s; tokens/s divided by L={L} for the L-layer step",
            "single_thread_value": v_one,
        }

    if rank == 0:
        print(json.dumps(line), flush=True)
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()


# ------------------------------------------------------------------------------------------------------
# offload mode: table in pinned host memory (410M-shaped by default), one JSON line of its own
# ------------------------------------------------------------------------------------------------------

def run_offload(args):
    """Per decode step and layer: dedup the ids on the device, let the GPU fetch the distinct rows
    from the pinned host table into an HBM staging buffer (side stream), combine from staging (main
    stream); layer l+1's fetch overlaps layer l's combine through two buffers (mole_offload_decode_step)."""
    import numpy as np
    import torch

    from paper_2503_15798_b200 import binding as mole
    from paper_2503_15798_b200 import build as lib_build
    from paper_2503_15798_b200 import inputs

    lib_build.build()
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    cfg = args.config if args.config != "160m" else "410m"
    sh = inputs.SHAPES[cfg]
    L = args.layers or sh.L
    row_bytes = sh.row_bytes

    # the host table, layer by layer (generated on the device, copied down once, outside any timed region)
    host = mole.HostTable((L, sh.V, sh.N, sh.d), torch.bfloat16)
    tmp = torch.empty((sh.V, sh.N, sh.d), dtype=torch.bfloat16, device=dev)
    for l in range(L):
        inputs.make_table(sh.V, sh.N, sh.d, seed=1000 + l, device=dev, out=tmp)
        host.tensor[l].copy_(tmp)
    torch.cuda.synchronize()
    wrs = torch.stack([inputs.make_router(sh.d, sh.N, seed=2000 + l, device=dev) for l in range(L)])

    # host link, measured: a large pinned host -> device copy, and the GPU-initiated read of the same bytes
    nrows = 8192
    big = torch.empty((nrows, sh.N, sh.d), dtype=torch.bfloat16, device=dev)
    src = host.tensor[0][:nrows]
    big.copy_(src, non_blocking=True)
    torch.cuda.synchronize()
    ms_copy = min(timed_ms(torch, lambda: big.copy_(src, non_blocking=True)) for _ in range(5))
    link_copy = nrows * row_bytes / ms_copy / 1e6
    uniq_all = torch.arange(nrows, dtype=torch.int32, device=dev)
    cnt_all = torch.tensor([nrows], dtype=torch.int32, device=dev)
    mole.fetch_rows(host.tensor[0], uniq_all, cnt_all, nrows, big)
    torch.cuda.synchronize()
    ms_fetch = min(timed_ms(torch, lambda: mole.fetch_rows(host.tensor[0], uniq_all, cnt_all, nrows, big)) for _ in range(5))
    link_fetch = nrows * row_bytes / ms_fetch / 1e6
    del big

    rows = []
    side = torch.cuda.Stream()
    for M in (1, 8, 64):
        # one context sized for a server's largest batch (256 tokens: two staging areas of 8 MB): at the batches
        # timed here a staging area has room for several layers' rows, fetched in one launch and run as one
        # fused launch
        ctx = mole.OffloadContext(OFFLOAD_CONTEXT_TOKENS, sh.N, sh.d, sh.V, torch.bfloat16, n_buffers=2)
        hidden = inputs.make_hidden(M, sh.d, seed=3000, device=dev)
        bufs = [torch.empty_like(hidden), torch.empty_like(hidden)]
        id_batches = [inputs.make_ids(M, sh.V, seed=4000 + b + 7 * M, device=dev) for b in range(N_BATCHES)]
        status = torch.zeros(1, dtype=torch.int32, device=dev)
        uniq_rows = float(np.mean([len(np.unique(b.cpu().numpy())) for b in id_batches]))

        luts_host = host.tensor  # [L][V][N][d], pinned and device-mapped

        def step(k):  # one call per step: one dedup, layer l+1's fetch under layer l's combine
            ctx.decode_step(hidden, id_batches[k % N_BATCHES], luts_host, wrs, bufs[0], bufs[1], status=status,
                            side_stream=side)

        steps = max(20, min(args.steps, 400))
        for k in range(max(args.warmup, 3)):
            step(k)
        torch.cuda.synchronize()
        ms = timed_ms(torch, lambda: [step(k) for k in range(steps)])
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        us_calls = ms * 1e3 / steps
        # the same steps replayed from CUDA graphs (one per id batch; the side stream joins the capture):
        # at small batches the 2L+1 launches of a step are otherwise bound by the host's launch rate
        graphs = []
        for k in range(N_BATCHES):
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g):
                step(k)
            graphs.append(g)
        for k in range(max(args.warmup, 3)):
            graphs[k % N_BATCHES].replay()
        torch.cuda.synchronize()
        ms = timed_ms(torch, lambda: [graphs[k % N_BATCHES].replay() for k in range(steps)])
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        del graphs
        us_step = ms * 1e3 / steps
        link_bytes = uniq_rows * row_bytes * L  # distinct rows only cross the link
        rows.append({"batch": M, "us_per_step": us_step, "tokens_per_s": M / (us_step * 1e-6),
                     "mean_distinct_ids": uniq_rows, "link_bytes_per_step": link_bytes,
                     "link_GBps": link_bytes / us_step / 1e3, "frac_of_link": link_bytes / us_step / 1e3 / link_fetch,
                     "launches_per_step": 1 + 2 * offload_groups(L, M, row_bytes),  # dedup + (fetch + layers) per group
                     "us_per_step_without_graph": us_calls})
        ctx.destroy()
    top = rows[-1]
    line = {
        "metric": "MoLE offload-mode tokens/s (L-layer decode step) and achieved host-link GB/s", "value": top["tokens_per_s"],
        "unit": UNIT, "n_gpus": 1, "steps": max(20, min(args.steps, 400)), "warmup": max(args.warmup, 3),
        "ms_per_step": top["us_per_step"] / 1e3, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16", "data": "synthetic",
        "config": {"workload": f"{sh.name}-shaped offload decode: table {sh.layer_table_bytes * L / 1e9:.2f} GB in pinned host "
                               f"memory, L={L}, batch 64x1 (sweep 1, 8, 64), ids Zipf(1.1)",
                   "V": sh.V, "d": sh.d, "N": sh.N, "L": L, "batch": 64,
                   "l2": "rows come from host memory; 32 rotating id batches, one CUDA graph per batch"},
        "gpu_launches": top["launches_per_step"] * max(20, min(args.steps, 400)),
        "roofline": {"bound": "host-link", "achieved": top["link_GBps"], "peak": link_fetch, "unit": "GB/s",
                     "frac": top["frac_of_link"], "traffic": None, "kernel": "mole_fetch_kernel",
                     "peak_source": "measured in this run: GPU-initiated read of 8192 rows of the pinned table "
                                    f"({link_fetch:.1f} GB/s; cudaMemcpyAsync of the same bytes {link_copy:.1f} GB/s)"},
        "host_link": {"memcpy_GBps": link_copy, "gpu_read_GBps": link_fetch},
        "sweep": rows,
    }
    host.free()
    print(json.dumps(line), flush=True)


def main():
    args = parse_args()
    if args.offload:
        return run_offload(args)
    if args.impl == "reference":
        run_reference(args)
    else:
        run_mole(args)


if __name__ == "__main__":
    main()
