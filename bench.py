#!/usr/bin/env python3
"""Benchmark of the fused MoLE layer (arXiv 2503.15798, Eq. 4 + Eq. 8) on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config 160m|410m|1b] [--batch M]
                    [--impl mole|reference] [--headline-only] [--no-cpu] [--no-offload] [--offload]

A "step" is one decode step of the whole hot path: all L layers of the configuration applied to
one batch of M tokens (router, softmax over all experts, row gather, weighted sum, residual).
The headline times it as a model that runs other work between the layers gets it: one launch per
layer, chained with programmatic dependent launch, the L launches of a step replayed from a CUDA
graph.  The metric is tokens/s for the L-layer step; the roofline block reports the layer
kernel's algorithmic GB/s (gathered rows + hidden in/out + router weights) against the measured
HBM copy bandwidth.  Every step uses a different pre-generated Zipf(1.1) id batch, and the tables
(GBs) are far larger than L2.  The timed region of exactly K steps is repeated until the repeats
span a quarter of a second; the value is the median repeat.

Beside the headline (one GPU): the same step as a single fused launch ("fused_step"), with
RMSNorm in front of every router, end to end from host buffers through the C ABI ("e2e"), a
sweep over the configuration's batch sizes with isolated-launch times, and a `configs` block with
the chained and fused rows of the other workload shapes, the quantised (NF4 / NF3) tables and the
offload mode.  The CPU oracle is timed on the host cores on a bounded sample of the same
workload, and its outputs are compared with the GPU's for the last timed step.

With N > 1 (torchrun) every rank holds its own replica of the tables and its own batches (tokens
are independent, so there is no collective on the data path): weak scaling; only the headline,
the fused step and the end-to-end number are measured.

--impl reference times the CPU oracle (oracle/, plain C, fp64) on the host cores instead.
"""
from __future__ import annotations

import argparse
import dataclasses
import json
import math
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
N_BATCHES = 32          # distinct id batches the headline's steps rotate through
N_BATCHES_EXTRA = 16    # ... and the rows beside it
MIN_SPAN_S = 0.25       # the timed region is repeated until the repeats span this long
OFFLOAD_CONTEXT_TOKENS = 256  # offload mode: the context (staging areas) is sized for this many tokens
OFFLOAD_BATCHES = (1, 8, 64)
OFFLOAD_HOT_ROWS = 1024       # ids whose rows (all layers) the offload rows "with a hot-row cache" keep in HBM
FALLBACK_HBM_GBS = 6650.0
QUANT_BLOCKS = {"160m": {"nf4": 768, "nf3": 128}, "410m": {"nf4": 1024, "nf3": 128}, "1b": {"nf4": 1024, "nf3": 128}}
# dram__bytes_read.sum + dram__bytes_write.sum of one launch of the dominant kernel, from the ncu
# capture summarised under profiles/ ((config, batch, layers) -> bytes); None until one is taken
# of the kernel as it stands
TRAFFIC = {
    # profiles/mole_step_kernel_single_layer_160m_batch256.md: mean of three captured launches (one layer each)
    ("160m", 256, 12): 4.29e6,
}
FUSED_TRAFFIC = {
    # profiles/mole_step_kernel_fused_160m_batch256.md: 8.1 MB per 2-layer launch, x6 for the 12 layers of a full launch
    ("160m", 256, 12): 48.6e6,
}


def offload_groups(L: int, M: int, row_bytes: int, hot: bool = False) -> int:
    """Groups of layers mole_offload_decode_step forms on a context of OFFLOAD_CONTEXT_TOKENS tokens (one
    fetch launch and one fused layer launch per group): as many layers as the staging area holds, but at
    least three groups unless the whole step's rows are at most 256 KB (1 MB with a hot-row cache)."""
    g = min(L, max(1, OFFLOAD_CONTEXT_TOKENS // M))
    if M * row_bytes * L > ((1 << 20) if hot else (1 << 18)):
        g = min(g, (L + 2) // 3)
    return -(-L // g)


def decode_family_covers(M, sh, L) -> bool:
    """Whether the one-block-per-token family (MOLE_KERNEL_DECODE) has a kernel for this launch."""
    from paper_2503_15798_b200 import binding as mole

    try:
        mole.variant(M, sh.N, sh.d, L=L, kernel=mole.KERNEL_DECODE)
        return True
    except mole.MoleError:
        return False


def timed_launch_shapes():
    """Every launch shape a timed region of this file issues, as dicts (what, M, N, d, L, norm, kernel,
    lut_format, lut_block): the parity tests walk this list and require a parity case for the kernel
    instantiation of each."""
    from paper_2503_15798_b200 import inputs

    shapes = []

    def add(what, M, sh, L, norm=False, kernel=0, fmt=0, block=0):
        shapes.append({"what": what, "M": M, "N": sh.N, "d": sh.d, "L": L, "norm": norm, "kernel": kernel,
                       "lut_format": fmt, "lut_block": block})

    for name in ("160m", "410m", "1b"):
        sh = inputs.SHAPES[name]
        for M in sh.batches:
            for norm in (False, True):
                tag = " norm" if norm else ""
                add(f"{name} batch {M} chained{tag}", M, sh, 1, norm)
                if M <= 4096:
                    add(f"{name} batch {M} fused{tag}", M, sh, sh.L, norm)
            add(f"{name} batch {M} chained, ring kernel", M, sh, 1, kernel=1)
            for L in (1, sh.L):
                if (L == 1 or M <= 4096) and decode_family_covers(M, sh, L):
                    add(f"{name} batch {M} {'chained' if L == 1 else 'fused'}, one block per token", M, sh, L, kernel=2)
            for fmt, tag in ((1, "nf4"), (2, "nf3")):
                add(f"{name} batch {M} chained, {tag} table", M, sh, 1, fmt=fmt, block=QUANT_BLOCKS[name][tag])
    sh = inputs.SHAPES["410m"]
    for M in OFFLOAD_BATCHES:
        for hot in (False, True):
            groups = offload_groups(sh.L, M, sh.row_bytes, hot)
            per = -(-sh.L // groups)
            for L in {per, sh.L - per * (groups - 1)}:
                add(f"410m offload batch {M}, group of {L} layers", M, sh, L, kernel=1)
        for fmt, tag in ((1, "nf4"), (2, "nf3")):
            add(f"410m offload batch {M}, {tag} records", M, sh, 1, fmt=fmt, block=QUANT_BLOCKS["410m"][tag])
    return shapes


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", default="mole", choices=["mole", "reference"])
    ap.add_argument("--config", default="160m", choices=["160m", "410m", "1b"])
    ap.add_argument("--batch", type=int, default=256)
    ap.add_argument("--headline-only", action="store_true",
                    help="only the headline, the fused step and the end-to-end number (what N > 1 runs)")
    ap.add_argument("--no-sweep", action="store_true", help="skip the per-batch sweep and the isolated-launch rows")
    ap.add_argument("--no-configs", action="store_true", help="skip the rows of the other workload shapes")
    ap.add_argument("--no-offload", action="store_true", help="skip the offload-mode rows of the default run")
    ap.add_argument("--no-cpu", action="store_true", help="skip the CPU-oracle baseline leg (and its parity check)")
    ap.add_argument("--layers", type=int, default=0, help="override L (debugging; the line then says so)")
    ap.add_argument("--vocab", type=int, default=0,
                    help="override V, the number of table rows (small profiler captures; the line then says so)")
    ap.add_argument("--min-span-s", type=float, default=MIN_SPAN_S,
                    help="repeat every timed region until the repeats span this long (0: three repeats; profiler captures)")
    ap.add_argument("--builder", action="store_true",
                    help="the table builder alone (Eq. 6-7 on the tensor cores), one 160M-shaped layer; --vocab shrinks it")
    ap.add_argument("--offload", action="store_true",
                    help="offload mode alone: table in pinned host memory, per-step dedup + row fetch overlapped with "
                         "the previous layers' combine; roofline = measured host-link GB/s")
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

    def __init__(self, index: int, period_s: float = 0.005):
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


def repeats_for(ms_one: float, min_span_s: float = None) -> int:
    """How often a timed region of ms_one milliseconds is repeated to span min_span_s (at least 3, at most 4000)."""
    span = MIN_SPAN_S if min_span_s is None else min_span_s
    return max(3, min(4000, int(math.ceil(span * 1e3 / max(ms_one, 1e-6)))))


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


def oracle_chain_check(luts, wrs, hidden, ids, got, threads):
    """Part of the CPU-baseline leg: the oracle's L-layer chain (each layer fed the bf16 rounding of the
    previous one) on the rows this batch references, compared element by element with `got`, the GPU's
    output for the same step.  Returns (max |err| / bound, seconds), bound = L * 2^-7 * max(1, |ref|): one
    bf16 ulp per layer."""
    import numpy as np
    import torch

    import oracle

    t0 = time.perf_counter()
    L = luts.shape[0]
    ids_np = ids.cpu().numpy()
    uniq, inv = np.unique(ids_np, return_inverse=True)
    sel = torch.from_numpy(uniq).long().to(luts.device)
    h = hidden.cpu()
    ref = None
    for l in range(L):
        rows = luts[l][sel].cpu()  # plain torch index: the bytes the kernel gathered
        ref, _, bad = oracle.layer_lookup(host_bits(h), inv, host_bits(rows), host_bits(wrs[l]), threads=threads)
        assert bad == 0
        h = torch.from_numpy(ref).to(torch.bfloat16)
    err = np.abs(got.cpu().to(torch.float64).numpy() - ref)
    bound = L * 2.0 ** -7 * np.maximum(1.0, np.abs(ref))
    return float((err / bound).max()), time.perf_counter() - t0


def run_reference(args):
    """--impl reference: the oracle, as it stands, on the host cores (rank 0 only)."""
    import numpy as np

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
    """One CUDA graph per id batch; a graph holds the launches of one step.  `step(ids, out, tmp, status)`
    issues them."""

    def __init__(self, torch, step, hidden, id_batches):
        self.torch, self.graphs = torch, []
        self.out = torch.empty_like(hidden)
        self.tmp = torch.empty_like(hidden)
        self.status = torch.zeros(1, dtype=torch.int32, device=hidden.device)
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            for ids in id_batches[:4]:  # launches outside capture first (they set kernel attributes)
                step(ids, self.out, self.tmp, self.status)
        torch.cuda.current_stream().wait_stream(side)
        torch.cuda.synchronize()
        for ids in id_batches:
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g):
                step(ids, self.out, self.tmp, self.status)
            self.graphs.append(g)
        self.id_batches = id_batches

    def run(self, k0, k1):
        n = len(self.graphs)
        for k in range(k0, k1):
            self.graphs[k % n].replay()

    def ok(self):
        return int(self.status.item()) == 0


def event_ms(torch, fn):
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record()
    fn()
    b.record()
    b.synchronize()
    return a.elapsed_time(b)


class _Null:
    def __enter__(self):
        return self

    def __exit__(self, *exc):
        return False


def timed_steps(torch, run, steps, warmup, barrier=None, dist=None, dev=None, sampler=None):
    """Warm-up, then the timed region of exactly `steps` steps (barrier + synchronise on both sides, CUDA
    events on the launching stream), repeated until the repeats span MIN_SPAN_S; every repeat's time is
    the maximum over ranks.  Returns (median ms of a repeat, dict with min / max / repeats)."""
    sync = barrier if barrier else torch.cuda.synchronize
    run(0, max(warmup, 3))
    sync()
    first = event_ms(torch, lambda: run(0, steps))
    reps = repeats_for(max_over_ranks(first, dist, dev))
    times = []
    with (sampler if sampler is not None else _Null()):
        for _ in range(reps):
            sync()
            times.append(event_ms(torch, lambda: run(0, steps)))
    sync()
    if dist is not None:
        t = torch.tensor(times, dtype=torch.float64, device=dev)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        times = [float(x) for x in t.cpu()]
    med = statistics.median(times)
    return med, {"repeats": reps, "ms_min": min(times), "ms_max": max(times), "span_s": sum(times) * 1e-3}


def make_tables(torch, inputs, sh, L, rank, dev):
    luts = torch.empty((L, sh.V, sh.N, sh.d), dtype=torch.bfloat16, device=dev)
    for l in range(L):
        inputs.make_table(sh.V, sh.N, sh.d, seed=rank_seeds(rank, l)["table"], device=dev, out=luts[l])
    wrs = torch.stack([inputs.make_router(sh.d, sh.N, seed=2000 + l, device=dev) for l in range(L)])
    return luts, wrs


def config_rows(torch, mole, inputs, sh, L, luts, wrs, batches, steps, warmup, peak, dev, quant=True):
    """Chained and fused rows of one workload shape (and, with `quant`, the chained step over its tables
    quantised to NF4 and NF3): per batch the step time, tokens/s, algorithmic bytes and fraction of peak."""
    rows = []
    hidden_all = inputs.make_hidden(max(batches), sh.d, seed=3000, device=dev)
    qtables = {}
    if quant:
        for tag, fmt in (("nf4", mole.LUT_NF4), ("nf3", mole.LUT_NF3)):
            block = QUANT_BLOCKS[sh.name][tag]
            rb = mole.quant_record_bytes(sh.N, sh.d, fmt, block)
            packed = torch.zeros((L, sh.V, rb), dtype=torch.uint8, device=dev)
            for l in range(L):
                mole.QuantTable.quantize(luts[l], fmt, block, out=packed[l])
            qtables[tag] = mole.QuantTable(packed, sh.N, sh.d, fmt, block)
        torch.cuda.synchronize()
    for m in batches:
        hid = hidden_all[:m].contiguous()
        bl = [inputs.make_ids(m, sh.V, seed=4000 + b + 7 * m, device=dev) for b in range(N_BATCHES_EXTRA)]
        k = max(10, min(steps, int(2e6 // max(m * L, 64))))
        row = {"batch": m, "steps": k}
        modes = [("chained", mole.STEP_CHAINED, mole.KERNEL_AUTO, None)]
        if decode_family_covers(m, sh, 1):
            modes.append(("chained_one_block_per_token", mole.STEP_CHAINED, mole.KERNEL_DECODE, None))
        if not mole.variant(m, sh.N, sh.d)[0].startswith("step"):  # the library's own choice is not the ring kernel: time that too
            modes.append(("chained_ring", mole.STEP_CHAINED, mole.KERNEL_RING, None))
        if m <= 4096:
            modes.append(("fused", mole.STEP_FUSED, mole.KERNEL_AUTO, None))
            if decode_family_covers(m, sh, L):
                modes.append(("fused_one_block_per_token", mole.STEP_FUSED, mole.KERNEL_DECODE, None))
        for tag in qtables:
            modes.append(("chained_" + tag, mole.STEP_CHAINED, mole.KERNEL_AUTO, qtables[tag]))
        for name, mode, kernel, qt in modes:
            table = qt if qt is not None else luts

            def step(ids, out, tmp, status, table=table, mode=mode, kernel=kernel):
                mole.decode_step_args(hid, ids, table, wrs, out, tmp, status=status, mode=mode, kernel=kernel)

            g = StepGraphs(torch, step, hid, bl)
            ms, spread = timed_steps(torch, g.run, k, min(warmup, 20))
            assert g.ok(), "a kernel reported a bad id or a timed-out wait"
            us = ms * 1e3 / k
            if qt is not None:
                nbytes = L * (m * qt.record_bytes + 2 * m * sh.d * 2 + sh.d * sh.N * 2)
            elif mode == mole.STEP_FUSED:
                nbytes = sh.step_bytes(m, L)
            else:
                nbytes = L * sh.layer_bytes(m)
            row[name] = {"us_per_step": us, "us_per_layer": us / L, "tokens_per_s": m / (us * 1e-6),
                         "algorithmic_bytes_per_step": nbytes, "GBps": nbytes / us / 1e3, "frac_of_peak": nbytes / us / 1e3 / peak,
                         "repeats": spread["repeats"],
                         "kernel": mole.variant(m, sh.N, sh.d, L=L if mode == mole.STEP_FUSED else 1, kernel=kernel,
                                                lut_format=qt.fmt if qt else 0, lut_block=qt.block if qt else 0)[0]}
            del g
        rows.append(row)
    return rows


def isolated_rows(torch, mole, inputs, sh, luts, wrs, batches, peak, dev):
    """One layer alone (no chaining): `reps` launches inside one event pair, each preceded by a kernel that
    keeps the GPU busy while the host queues the launch -- an L2 flush (cold) or a short spin (steady) --
    minus the same region without the launches."""
    flush = torch.empty(256 * 1024 * 1024, dtype=torch.uint8, device=dev)
    rows = []
    for m in batches:
        if m * sh.d * 2 > 2**31:
            continue
        hid = inputs.make_hidden(m, sh.d, seed=3000, device=dev)
        bl = [inputs.make_ids(m, sh.V, seed=4000 + b + 7 * m, device=dev) for b in range(N_BATCHES_EXTRA)]
        out = torch.empty_like(hid)
        reps = 100 if m <= 1024 else 20
        res = {}
        for mode in ("steady", "cold", "prefetched"):
            cold = mode != "steady"

            def filler(r, mode=mode):
                if mode == "steady":
                    torch.cuda._sleep(20000)
                    return
                flush.fill_(r & 0xFF)
                if mode == "prefetched":  # the step's rows asked for ahead of the layer, then other work (a spin) in between
                    mole.prefetch_rows(bl[r % N_BATCHES_EXTRA], luts, layers=1)
                    torch.cuda._sleep(20000)

            def with_launches():
                for r in range(reps):
                    filler(r)
                    mole.layer_forward(hid, bl[r % N_BATCHES_EXTRA], luts[0], wrs[0], out)

            def without():
                for r in range(reps):
                    filler(r)

            with_launches()
            torch.cuda.synchronize()
            t1 = min(event_ms(torch, with_launches) for _ in range(3))
            t0 = min(event_ms(torch, without) for _ in range(3))
            res[mode] = max(t1 - t0, 0.0) * 1e3 / reps
        nbytes = sh.layer_bytes(m)
        rows.append({"batch": m, "isolated_steady_us": res["steady"], "isolated_cold_us": res["cold"],
                     "isolated_cold_prefetched_us": res["prefetched"],
                     "isolated_cold_GBps": nbytes / max(res["cold"], 1e-3) / 1e3,
                     "isolated_cold_frac_of_peak": nbytes / max(res["cold"], 1e-3) / 1e3 / peak,
                     "how": f"{reps} launches, each after an L2 flush (cold), a spin (steady), or an L2 flush followed by "
                            "mole_prefetch_rows for the launch's ids and a spin (prefetched), inside one event pair, minus the "
                            "same region without the launches"})
    del flush
    return rows


def measured_tensor_peak():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(p) as f:
            return float(json.load(f)["bf16_tflops"]), "measured (MEASURED_PEAKS.json bf16_tflops, burst: each build is timed by itself)"
    except Exception:
        return 1590.0, "fallback (1.59 PFLOP/s, earlier measurement on this pool)"


def measured_tensor_peak_sustained():
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            return float(json.load(f)["bf16_tflops_sustained"])
    except Exception:
        return 1400.0


def oracle_build_check(E, W1, W2, lut):
    """Part of the CPU-baseline leg: six sampled ids' rows of the table the timed builds left behind against the
    oracle's builder (fp64) run on those embedding rows.  Returns max |err| / bound, the bound being the bf16
    materialisation of the hidden activations and of the result (half an ulp of every |h_k w2_k| term, the final
    rounding of the entry, 1e-6 absolute)."""
    import numpy as np
    import torch

    import oracle

    V = E.shape[0]
    sample = torch.tensor([0, 1, V // 3, V // 2, V - 2, V - 1], device=E.device)
    f64 = lambda t: t.detach().cpu().to(torch.float64).numpy()
    E64, W1_64, W2_64 = f64(E[sample]), f64(W1), f64(W2)
    ref = oracle.build_lut(E64, W1_64, W2_64)
    absum = np.empty_like(ref)
    for j in range(W1_64.shape[0]):
        pre = E64 @ W1_64[j].T
        h = np.vectorize(oracle.gelu)(pre)
        absum[:, j, :] = np.abs(h) @ np.abs(W2_64[j]).T
    bound = 2.0 ** -8 * absum + 2.0 ** -8 * np.abs(ref) + 1e-6
    return float((np.abs(f64(lut[sample]) - ref) / bound).max())


def builder_row(torch, mole, inputs, dev, vocab=0, check=False):
    """The re-parameterisation of one 160M-shaped layer (Eq. 6-7): V = 50304 embedding rows through N = 16 experts
    of width D = 4 d = 3072 (Table 2), two tensor-core GEMMs; TFLOP/s against the measured bf16 GEMM rate."""
    sh = inputs.SHAPES["160m"]
    if vocab > 0:
        sh = dataclasses.replace(sh, V=vocab)
    D = 4 * sh.d
    g = torch.Generator(device=dev)
    g.manual_seed(77)
    E = torch.empty((sh.V, sh.d), dtype=torch.bfloat16, device=dev).normal_(0, 1, generator=g)
    W1 = torch.empty((sh.N, D, sh.d), dtype=torch.bfloat16, device=dev).normal_(0, sh.d ** -0.5, generator=g)
    W2 = torch.empty((sh.N, sh.d, D), dtype=torch.bfloat16, device=dev).normal_(0, D ** -0.5, generator=g)
    lut = torch.empty((sh.V, sh.N, sh.d), dtype=torch.bfloat16, device=dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    mole.build_lut(E, W1, W2, out=lut, status=status)  # allocates its scratch buffer through torch; synchronises
    times = []
    clocks = ClockSampler(physical_gpu_index(int(os.environ.get("LOCAL_RANK", "0"))), period_s=0.002)
    with clocks:
        for _ in range(20):  # each build timed by itself (a burst, like the GEMM rate it is compared with)
            torch.cuda.synchronize()
            times.append(event_ms(torch, lambda: mole.build_lut(E, W1, W2, out=lut, status=status)))
    assert int(status.item()) == 0
    ms = statistics.median(times)
    parity = oracle_build_check(E, W1, W2, lut) if check else None
    flops = 2 * 2.0 * sh.V * sh.d * D * sh.N
    peak, src = measured_tensor_peak()
    tf = flops / (ms * 1e-3) / 1e12
    return {"V": sh.V, "d": sh.d, "D": D, "N": sh.N, "ms_per_layer": ms, "flops_per_layer": flops, "TFLOPps": tf,
            "roofline": {"bound": "tensor", "achieved": tf, "peak": peak, "unit": "TFLOP/s", "frac": tf / peak, "traffic": None,
                         "kernel": "mole_gemm_tn_kernel", "peak_source": src},
            "frac_of_sustained_peak": tf / measured_tensor_peak_sustained(),  # context: after a long run the GPU is at its power cap
            "table_rows_per_s": sh.V / (ms * 1e-3), "ms_min": min(times), "ms_max": max(times), "builds_timed": len(times),
            "clocks": clocks.summary(),
            "parity_of_the_timed_build": None if parity is None else {
                "max_err_over_bound": parity, "ok": parity <= 1.0,
                "what": "six ids' rows (16 experts x 768 columns each) of the table the timed builds wrote against the oracle's "
                        "builder on those embedding rows (part of the CPU-baseline leg)"}}


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
    extras = world == 1 and not args.headline_only
    t_start = time.perf_counter()

    luts, wrs = make_tables(torch, inputs, sh, L, rank, dev)
    hidden = inputs.make_hidden(M, sh.d, seed=rank_seeds(rank)["hidden"], device=dev)

    def batches_for(m, n=N_BATCHES):
        return [inputs.make_ids(m, sh.V, seed=rank_seeds(rank, 0, b, m)["ids"], device=dev) for b in range(n)]

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    def plain_step(mode, kernel=mole.KERNEL_AUTO):
        def step(ids, out, tmp, status):
            mole.decode_step_args(hidden, ids, luts, wrs, out, tmp, status=status, mode=mode, kernel=kernel)
        return step

    # ---- headline: K steps of the L-layer decode step as a model that runs other work between the layers
    # gets it: one launch per layer, chained with programmatic dependent launch, the layer's output the next
    # layer's hidden state, the L launches of a step replayed from a CUDA graph -----------------------------
    graphs = StepGraphs(torch, plain_step(mole.STEP_CHAINED), hidden, batches_for(M))
    clocks = ClockSampler(physical_gpu_index(local_rank))
    ms, spread = timed_steps(torch, graphs.run, args.steps, args.warmup, barrier, dist, dev, sampler=clocks)
    assert graphs.ok(), "a kernel reported a bad id or a timed-out wait"
    last_ids = graphs.id_batches[(args.steps - 1) % N_BATCHES]
    headline_out = graphs.out.clone()  # the last timed step's result (every repeat ends on the same id batch)
    ms_per_step = ms / args.steps
    value = whole_job_tokens_per_s(world, M, args.steps, ms)
    launches = args.steps * L
    launch_bytes = sh.layer_bytes(M)
    achieved = launch_bytes / (ms * 1e-3 / launches) / 1e9
    kernel_name = mole.variant(M, sh.N, sh.d)[0]

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
        "data": "synthetic", "config": workload_config(sh, L, M, args),
        "timing": dict(spread, what=f"the timed region of {args.steps} steps repeated {spread['repeats']} times "
                                    "(barrier + synchronise around each); value from the median repeat"),
        "tokens_per_s_per_layer": value * L,
        "gpu_launches": launches,
        "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                     "traffic": TRAFFIC.get((sh.name, M, L)), "kernel": kernel_name, "peak_source": peak_src,
                     "launch": "one launch per layer (%d per step), chained with programmatic dependent launch" % L,
                     "algorithmic_bytes_per_launch": launch_bytes, "us_per_launch": ms * 1e3 / launches},
        "clocks": clocks.summary(),
    }
    if extras:
        # the same chained step issued from the host every step (no CUDA graph): what the library's launch path costs
        ids_all, out_h, tmp_h, st_h = graphs.id_batches, graphs.out, graphs.tmp, graphs.status
        step_fn = plain_step(mole.STEP_CHAINED)

        def host_run(k0, k1):
            for k in range(k0, k1):
                step_fn(ids_all[k % N_BATCHES], out_h, tmp_h, st_h)

        ms_h, _ = timed_steps(torch, host_run, args.steps, args.warmup)
        line["chained_step_host_issued"] = {"what": "the headline's step without a CUDA graph: one mole_decode_step_args call per step, "
                                                    "L launches issued by the library from the host",
                                            "us_per_step": ms_h * 1e3 / args.steps, "value": M * args.steps / (ms_h * 1e-3), "unit": UNIT,
                                            "ratio_to_graph_replay": ms_h / ms}
    del graphs

    # ---- extra, never the headline: the same step as ONE launch that keeps a token's chain through all L
    # layers on chip (what mole_decode_step picks by itself up to 4096 tokens) ------------------------------
    fused_out = None
    if L > 1 and M <= 4096:
        g = StepGraphs(torch, plain_step(mole.STEP_FUSED), hidden, batches_for(M))
        ms_f, spread_f = timed_steps(torch, g.run, args.steps, args.warmup, barrier, dist, dev)
        assert g.ok(), "a kernel reported a bad id or a timed-out wait"
        fb = sh.step_bytes(M, L)
        gbs = fb / (ms_f * 1e-3 / args.steps) / 1e9
        line["fused_step"] = {"what": "all %d layers of a step in one launch (layer-batched), an extra beside the headline" % L,
                              "value": whole_job_tokens_per_s(world, M, args.steps, ms_f), "unit": UNIT,
                              "us_per_step": ms_f * 1e3 / args.steps, "algorithmic_bytes_per_launch": fb,
                              "achieved": gbs, "frac": gbs / peak, "traffic": FUSED_TRAFFIC.get((sh.name, M, L)),
                              "kernel": mole.variant(M, sh.N, sh.d, L=L)[0], "repeats": spread_f["repeats"]}
        fused_out = g.out.clone()
        del g

    # ---- extra: the chained and the fused step with RMSNorm in front of every layer's router (App. A.2
    # listing), through the same C entry point ---------------------------------------------------------------
    if extras:
        gammas = torch.stack([inputs.make_router(sh.d, 1, seed=2500 + l, device=dev).reshape(sh.d) + 1.0 for l in range(L)])
        norm = {}
        for name, mode in (("chained", mole.STEP_CHAINED), ("fused", mole.STEP_FUSED)):
            if mode == mole.STEP_FUSED and not (L > 1 and M <= 4096):
                continue

            def step(ids, out, tmp, status, mode=mode):
                mole.decode_step_args(hidden, ids, luts, wrs, out, tmp, status=status, mode=mode, norm_weights=gammas,
                                      norm_eps=1e-5)

            g = StepGraphs(torch, step, hidden, batches_for(M, N_BATCHES_EXTRA))
            k = min(args.steps, 500)
            ms_n, _ = timed_steps(torch, g.run, k, min(args.warmup, 20))
            assert g.ok(), "a kernel reported a bad id or a timed-out wait"
            us = ms_n * 1e3 / k
            nbytes = L * sh.layer_bytes(M) if mode == mole.STEP_CHAINED else sh.step_bytes(M, L)
            norm[name] = {"us_per_step": us, "us_per_layer": us / L, "value": M / (us * 1e-6), "unit": UNIT,
                          "achieved": nbytes / us / 1e3, "frac": nbytes / us / 1e3 / peak,
                          "kernel": mole.variant(M, sh.N, sh.d, L=L if mode == mole.STEP_FUSED else 1, norm=True)[0]}
            del g
        line["norm_router_step"] = dict(norm, what="the step with every router reading RMSNorm(hidden), fused into the layer "
                                                   "kernels (mole_decode_step_args with norm weights)")

    # ---- end to end: host buffers in, host buffer out, through the C ABI, every step ---------------------
    h_host = hidden.cpu().pin_memory()
    out_host = torch.empty_like(h_host).pin_memory()
    ids_host = [b.cpu().pin_memory() for b in batches_for(M)]
    dev_bufs = [torch.empty_like(hidden) for _ in range(3)]
    dev_ids = torch.empty(M, dtype=torch.int32, device=dev)
    e2e_steps = min(args.steps, 1000)

    def e2e_call(k):
        mole.decode_step_host(h_host, ids_host[k % N_BATCHES], out_host, dev_bufs[0], dev_ids, dev_bufs[1],
                              dev_bufs[2], luts, wrs)

    for k in range(3):  # uncaptured calls first (kernel attributes), then one CUDA graph per id batch
        e2e_call(k)
    torch.cuda.synchronize()
    e2e_graphs = []
    for k in range(N_BATCHES):
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            e2e_call(k)
        e2e_graphs.append(g)

    def e2e_run(k0, k1):
        for k in range(k0, k1):
            e2e_graphs[k % N_BATCHES].replay()
            torch.cuda.current_stream().synchronize()  # the caller reads out_host after every step

    ms_e2e, spread_e = timed_steps(torch, e2e_run, e2e_steps, min(args.warmup, 50), barrier, dist, dev)
    line["e2e"] = {"value": whole_job_tokens_per_s(world, M, e2e_steps, ms_e2e), "unit": UNIT,
                   "h2d_bytes_per_step": M * sh.d * 2 + M * 4, "d2h_bytes_per_step": M * sh.d * 2,
                   "steps": e2e_steps, "ms_per_step": ms_e2e / e2e_steps, "repeats": spread_e["repeats"],
                   "how": "mole_decode_step_host captured into one CUDA graph per id batch; the host buffers are pinned and "
                          "mapped, so the step's one fused launch reads hidden + ids across the host link itself and stores "
                          "the last layer's output into the host buffer (the same bytes as with staged copies, no copy "
                          "operations around the kernel); one graph launch and one stream synchronisation per step"}
    e2e_out = out_host.clone()
    del e2e_graphs

    # ---- sweep over the configuration's batch sizes: chained + fused steps, isolated launches ---------------
    if extras and not args.no_sweep:
        rows = config_rows(torch, mole, inputs, sh, L, luts, wrs, sh.batches, args.steps, args.warmup, peak, dev)
        iso = {r["batch"]: r for r in isolated_rows(torch, mole, inputs, sh, luts, wrs, sh.batches, peak, dev)}
        for r in rows:
            r.update({k: v for k, v in iso.get(r["batch"], {}).items() if k != "batch"})
        line["sweep"] = rows

    # ---- the CPU oracle beside it (rank 0, N = 1 only): timed on a bounded sample of the same workload, and
    # its outputs compared with the GPU's for the last timed step ----------------------------------------------
    if not args.no_cpu and rank == 0 and world == 1:
        import oracle

        cores = oracle.effective_threads(len(os.sched_getaffinity(0)))
        table0 = host_bits(luts[0])
        ids_np = [b.cpu().numpy().astype(np.int64) for b in batches_for(M)]
        v_all, calls, dt = time_oracle(table0, host_bits(wrs[0]), host_bits(hidden), ids_np, L, 10.0, cores)
        v_one, calls1, dt1 = time_oracle(table0, host_bits(wrs[0]), host_bits(hidden), ids_np, L, 4.0, 1)
        del table0
        parity = {}
        ratio, secs = oracle_chain_check(luts, wrs, hidden, last_ids, headline_out, cores)
        parity["chained_step"] = {"max_err_over_bound": ratio, "ok": ratio <= 1.0}
        if fused_out is not None:
            ratio_f, _ = oracle_chain_check(luts, wrs, hidden, last_ids, fused_out, cores)
            parity["fused_step"] = {"max_err_over_bound": ratio_f, "ok": ratio_f <= 1.0}
        e2e_ids = ids_host[(e2e_steps - 1) % N_BATCHES].to(dev)
        ratio_e, _ = oracle_chain_check(luts, wrs, hidden, e2e_ids, e2e_out.to(dev), cores)
        parity["e2e_step"] = {"max_err_over_bound": ratio_e, "ok": ratio_e <= 1.0}
        line["cpu_baseline"] = {
            "value": v_all, "unit": UNIT, "cores": cores, "kind": "oracle",
            "sample": f"{calls} calls of the oracle's lookup-form layer (fp64) on a host copy of layer 0's table, "
                      f"{M} tokens each, {dt:.1f} s; tokens/s divided by L={L} for the L-layer step",
            "single_thread_value": v_one,
            "parity_of_the_last_timed_step": dict(parity, what=f"the oracle's {L}-layer chain on all {M} tokens of the last timed "
                                                  "step's id batch against the GPU's output, element by element; bound "
                                                  f"{L} x 2^-7 x max(1, |ref|)"),
        }
        assert all(v["ok"] for v in parity.values() if isinstance(v, dict)), parity

    del luts, wrs
    torch.cuda.empty_cache()

    # ---- the other workload shapes, their quantised tables, the offload mode (one GPU only) ------------------
    if extras and not args.no_configs:
        configs = {}
        # the table builder first: each build is timed by itself against the burst GEMM rate, so it runs while the
        # GPU is as cool as the CPU leg has left it, not after a minute of sustained load
        try:
            configs["builder_160m_layer"] = builder_row(torch, mole, inputs, dev, check=not args.no_cpu and rank == 0 and world == 1)
        except Exception as e:
            configs["builder_160m_layer"] = {"error": f"{type(e).__name__}: {e}"}
        torch.cuda.empty_cache()
        for name in ("160m", "410m", "1b"):
            if name == sh.name:
                continue
            osh = inputs.SHAPES[name]
            try:
                oluts, owrs = make_tables(torch, inputs, osh, osh.L, rank, dev)
                rows = config_rows(torch, mole, inputs, osh, osh.L, oluts, owrs, osh.batches, args.steps, args.warmup, peak, dev)
                configs[name] = {"V": osh.V, "d": osh.d, "N": osh.N, "L": osh.L,
                                 "table_GB": osh.layer_table_bytes * osh.L / 1e9, "rows": rows}
                del oluts, owrs
            except Exception as e:  # e.g. not enough device memory for the 105 GB table on a smaller part
                configs[name] = {"error": f"{type(e).__name__}: {e}"}
            torch.cuda.empty_cache()
        if not args.no_offload:
            try:
                configs["410m_offload"] = offload_rows(args, torch, mole, inputs, dev)
            except Exception as e:
                configs["410m_offload"] = {"error": f"{type(e).__name__}: {e}"}
        line["configs"] = configs
    line["bench_wall_s"] = time.perf_counter() - t_start

    if rank == 0:
        print(json.dumps(line), flush=True)
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()


# ------------------------------------------------------------------------------------------------------
# offload mode: table in pinned host memory (410M-shaped)
# ------------------------------------------------------------------------------------------------------

def offload_rows(args, torch, mole, inputs, dev, formats=("bf16", "nf4", "nf3")):
    """Per decode step: dedup the ids on the device, let the GPU fetch the distinct rows from the pinned host
    table into an HBM staging buffer (side stream), combine from staging (main stream); the next layers'
    fetch overlaps the current layers' combine through two buffers (mole_offload_decode_step).  Rows for the
    bf16 host table and for the host table quantised to NF4 / NF3 (packed records cross the link)."""
    import numpy as np

    sh = inputs.SHAPES["410m"]
    L = args.layers or sh.L
    result = {"V": sh.V, "d": sh.d, "N": sh.N, "L": L, "context_tokens": OFFLOAD_CONTEXT_TOKENS}
    tmp = torch.empty((sh.V, sh.N, sh.d), dtype=torch.bfloat16, device=dev)
    wrs = torch.stack([inputs.make_router(sh.d, sh.N, seed=2000 + l, device=dev) for l in range(L)])
    side = torch.cuda.Stream()
    link = None
    for tag in formats:
        fmt = {"bf16": mole.LUT_PLAIN, "nf4": mole.LUT_NF4, "nf3": mole.LUT_NF3}[tag]
        block = QUANT_BLOCKS["410m"].get(tag, 0)
        row_bytes = sh.row_bytes if fmt == mole.LUT_PLAIN else mole.quant_record_bytes(sh.N, sh.d, fmt, block)
        # the host table, layer by layer (generated on the device, copied down once, outside any timed region)
        packed = None
        if fmt == mole.LUT_PLAIN:
            host = mole.HostTable((L, sh.V, sh.N, sh.d), torch.bfloat16)
        else:
            host = mole.HostTable((L, sh.V, row_bytes), torch.uint8)
            packed = torch.zeros((sh.V, row_bytes), dtype=torch.uint8, device=dev)
        for l in range(L):
            inputs.make_table(sh.V, sh.N, sh.d, seed=1000 + l, device=dev, out=tmp)
            if fmt == mole.LUT_PLAIN:
                host.tensor[l].copy_(tmp)
            else:
                mole.QuantTable.quantize(tmp, fmt, block, out=packed)
                host.tensor[l].copy_(packed)
        torch.cuda.synchronize()
        if link is None:
            # host link, measured: a large pinned host -> device copy, and the GPU-initiated read of the same bytes
            nrows = 8192
            big = torch.empty((nrows, sh.N, sh.d), dtype=torch.bfloat16, device=dev)
            src = host.tensor[0][:nrows]
            big.copy_(src, non_blocking=True)
            torch.cuda.synchronize()
            ms_copy = min(event_ms(torch, lambda: big.copy_(src, non_blocking=True)) for _ in range(5))
            uniq_all = torch.arange(nrows, dtype=torch.int32, device=dev)
            cnt_all = torch.tensor([nrows], dtype=torch.int32, device=dev)
            mole.fetch_rows(host.tensor[0], uniq_all, cnt_all, nrows, big)
            torch.cuda.synchronize()
            ms_fetch = min(event_ms(torch, lambda: mole.fetch_rows(host.tensor[0], uniq_all, cnt_all, nrows, big)) for _ in range(5))
            link = {"memcpy_GBps": nrows * sh.row_bytes / ms_copy / 1e6, "gpu_read_GBps": nrows * sh.row_bytes / ms_fetch / 1e6}
            link["peak_GBps"] = max(link["memcpy_GBps"], link["gpu_read_GBps"])
            link["peak_source"] = ("measured in this run: the faster of cudaMemcpyAsync and a GPU-initiated read of 8192 rows "
                                   "of the pinned table")
            del big
        rows = []
        hot_ids = inputs.zipf_hot_ids(sh.V, OFFLOAD_HOT_ROWS)
        for M, hot in [(m, False) for m in OFFLOAD_BATCHES] + ([(m, True) for m in OFFLOAD_BATCHES] if fmt == mole.LUT_PLAIN else []):
            # one context sized for a server's largest batch (256 tokens: two staging areas): at the batches timed
            # here a staging area has room for several layers' rows, fetched in one launch
            ctx = mole.OffloadContext(OFFLOAD_CONTEXT_TOKENS, sh.N, sh.d, sh.V, torch.bfloat16, n_buffers=2, lut_format=fmt,
                                      lut_block=block)
            if hot:  # the rows of the most probable ids of all layers kept in HBM: they never cross the link again
                ctx.set_hot_rows(hot_ids, host.tensor)
            hidden = inputs.make_hidden(M, sh.d, seed=3000, device=dev)
            bufs = [torch.empty_like(hidden), torch.empty_like(hidden)]
            id_batches = [inputs.make_ids(M, sh.V, seed=4000 + b + 7 * M, device=dev) for b in range(N_BATCHES)]
            status = torch.zeros(1, dtype=torch.int32, device=dev)
            uniq_rows = float(np.mean([len(np.unique(b.cpu().numpy())) for b in id_batches]))

            def step(k):  # one call per step: one dedup, the next layers' fetch under the current layers' combine
                ctx.decode_step(hidden, id_batches[k % N_BATCHES], host.tensor, wrs, bufs[0], bufs[1], status=status,
                                side_stream=side)

            steps = max(20, min(args.steps, 200))
            for k in range(max(min(args.warmup, 10), 3)):
                step(k)
            torch.cuda.synchronize()
            us_calls = event_ms(torch, lambda: [step(k) for k in range(steps)]) * 1e3 / steps
            torch.cuda.synchronize()
            # the same steps replayed from CUDA graphs (one per id batch; the side stream joins the capture)
            graphs = []
            for k in range(N_BATCHES):
                g = torch.cuda.CUDAGraph()
                with torch.cuda.graph(g):
                    step(k)
                graphs.append(g)

            def run(k0, k1):
                for k in range(k0, k1):
                    graphs[k % N_BATCHES].replay()

            ms, spread = timed_steps(torch, run, steps, 5)
            assert int(status.item()) == 0
            us_step = ms * 1e3 / steps
            link_bytes = uniq_rows * row_bytes * L  # distinct rows only cross the link
            hits_per_step = None
            if hot:  # ... and of those, not the ones the hot-row cache serves (counted by the fetch kernel)
                ctx.hot_hits(reset=True)
                run(0, N_BATCHES)
                hits_per_step = ctx.hot_hits() / N_BATCHES
                link_bytes -= hits_per_step * row_bytes
            rows.append({"batch": M, "hot_rows_cached": OFFLOAD_HOT_ROWS if hot else 0, "rows_from_cache_per_step": hits_per_step,
                         "us_per_step": us_step, "tokens_per_s": M / (us_step * 1e-6),
                         "mean_distinct_ids": uniq_rows, "link_bytes_per_step": link_bytes,
                         "link_GBps": link_bytes / us_step / 1e3, "frac_of_link": link_bytes / us_step / 1e3 / link["peak_GBps"],
                         "us_per_step_without_graph": us_calls, "repeats": spread["repeats"]})
            del graphs
            ctx.destroy()
        result[tag] = {"row_bytes": row_bytes, "host_table_GB": row_bytes * sh.V * L / 1e9, "rows": rows}
        host.free()
        del packed
    result["host_link"] = link
    return result


def run_offload(args):
    """--offload: the offload mode alone, one JSON line of its own."""
    import torch

    from paper_2503_15798_b200 import binding as mole
    from paper_2503_15798_b200 import build as lib_build
    from paper_2503_15798_b200 import inputs

    lib_build.build()
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    res = offload_rows(args, torch, mole, inputs, dev)
    top = [r for r in res["bf16"]["rows"] if r["batch"] == OFFLOAD_BATCHES[-1] and not r["hot_rows_cached"]][0]
    steps = max(20, min(args.steps, 200))
    line = {
        "metric": "MoLE offload-mode tokens/s (L-layer decode step) and achieved host-link GB/s", "value": top["tokens_per_s"],
        "unit": UNIT, "n_gpus": 1, "steps": steps, "warmup": max(min(args.warmup, 10), 3),
        "ms_per_step": top["us_per_step"] / 1e3, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16", "data": "synthetic",
        "config": {"workload": f"410m-shaped offload decode: table {res['bf16']['host_table_GB']:.2f} GB in pinned host "
                               f"memory, L={res['L']}, batch 64x1 (sweep 1, 8, 64), ids Zipf(1.1)",
                   "V": res["V"], "d": res["d"], "N": res["N"], "L": res["L"], "batch": 64,
                   "l2": "rows come from host memory; 32 rotating id batches, one CUDA graph per batch"},
        "gpu_launches": (1 + 2 * offload_groups(res["L"], 64, res["bf16"]["row_bytes"])) * steps,
        "roofline": {"bound": "host-link", "achieved": top["link_GBps"], "peak": res["host_link"]["peak_GBps"], "unit": "GB/s",
                     "frac": top["frac_of_link"], "traffic": None, "kernel": "mole_fetch_kernel",
                     "peak_source": res["host_link"]["peak_source"]},
        "offload": res,
    }
    print(json.dumps(line), flush=True)


def run_builder(args):
    """--builder: the table builder alone, one JSON line of its own."""
    import torch

    from paper_2503_15798_b200 import binding as mole
    from paper_2503_15798_b200 import build as lib_build
    from paper_2503_15798_b200 import inputs

    lib_build.build()
    torch.cuda.set_device(0)
    row = builder_row(torch, mole, inputs, torch.device("cuda", 0), args.vocab)
    line = {"metric": "MoLE table builder (Eq. 6-7) TFLOP/s, one 160M-shaped layer", "value": row["TFLOPps"], "unit": "TFLOP/s",
            "n_gpus": 1, "steps": row["builds_timed"], "warmup": 1, "ms_per_step": row["ms_per_layer"], "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": f"re-parameterisation of one layer: V={row['V']}, d={row['d']}, D={row['D']}, N={row['N']}"},
            "gpu_launches": 2 * row["builds_timed"], "roofline": row["roofline"], "clocks": row["clocks"], "builder": row}
    print(json.dumps(line), flush=True)


def main():
    global MIN_SPAN_S
    args = parse_args()
    MIN_SPAN_S = args.min_span_s
    if args.builder:
        return run_builder(args)
    if args.offload:
        return run_offload(args)
    if args.impl == "reference":
        run_reference(args)
    else:
        run_mole(args)


if __name__ == "__main__":
    main()
