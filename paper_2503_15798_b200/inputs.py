"""Seeded synthetic inputs for the MoLE layer: shapes, id streams, tables, hidden states.

This module holds no arithmetic of the method (no router, no softmax, no combine, no FFN):
it only draws random inputs with the shapes and distributions of the workloads, so both
the CUDA path and the CPU oracle can be fed the same bytes.

Workload shapes follow Table 2 of the paper (L, d per model size; N routed experts) with a
Pythia-sized vocabulary (the paper's "50k" tokenizer, padded to 50304 embedding rows).
The paper's text corpus is replaced by a bounded Zipf(1.1) id stream; table values are
i.i.d. N(0, 0.05) (values do not affect speed, the id distribution does).
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np

try:  # torch is only needed for the tensor-producing helpers
    import torch
except Exception:  # pragma: no cover
    torch = None


@dataclass(frozen=True)
class Shape:
    name: str
    V: int
    d: int
    N: int
    L: int
    dtype: str  # "bf16" or "f32"
    batches: tuple
    D: int = 0  # expert FFN width (only the tiny config builds its table from FFNs)

    @property
    def elem_bytes(self) -> int:
        return 2 if self.dtype == "bf16" else 4

    @property
    def row_bytes(self) -> int:
        """Bytes gathered per token per layer: N*d elements (Eq. 14)."""
        return self.N * self.d * self.elem_bytes

    @property
    def layer_table_bytes(self) -> int:
        return self.V * self.row_bytes

    def layer_bytes(self, M: int) -> int:
        """Algorithmic bytes of one layer call: gathered rows + hidden in/out + router weights."""
        e = self.elem_bytes
        return M * self.N * self.d * e + 2 * M * self.d * e + self.d * self.N * e

    def step_bytes(self, M: int, L: int) -> int:
        """Algorithmic bytes of L chained layers run as ONE launch: per layer the gathered rows
        and the router weights, plus hidden in and out once (between layers the hidden state
        never leaves the chip)."""
        e = self.elem_bytes
        return L * (M * self.N * self.d * e + self.d * self.N * e) + 2 * M * self.d * e


SHAPES = {
    "tiny": Shape("tiny", V=512, d=64, N=4, L=2, dtype="f32", batches=(64,), D=256),
    "160m": Shape("160m", V=50304, d=768, N=16, L=12, dtype="bf16", batches=(1, 8, 64, 256)),
    "410m": Shape("410m", V=50304, d=1024, N=16, L=24, dtype="bf16", batches=(1, 64, 256, 16384)),
    "1b": Shape("1b", V=50304, d=2048, N=32, L=16, dtype="bf16", batches=(1, 16, 64, 256)),
}


# ---- id streams ---------------------------------------------------------------------------

def zipf_probs(V: int, s: float = 1.1) -> np.ndarray:
    """Bounded Zipf: P(rank k) = k^-s / H, k = 1..V, H = sum_k k^-s (fp64)."""
    w = np.arange(1, V + 1, dtype=np.float64) ** (-s)
    return w / w.sum()


def zipf_ids(M: int, V: int, s: float = 1.1, seed: int = 0, permute: bool = True) -> np.ndarray:
    """M ids drawn from the bounded Zipf(s) over V ranks by inverse CDF on the finite table.

    With ``permute`` the rank -> id map is a seeded permutation of [0, V), so hot rows are
    scattered over the table instead of sitting at its start.
    """
    rng = np.random.default_rng(seed)
    cdf = np.cumsum(zipf_probs(V, s))
    cdf[-1] = 1.0
    ranks = np.searchsorted(cdf, rng.random(M), side="right")
    ranks = np.minimum(ranks, V - 1)
    if permute:
        perm = np.random.default_rng(0x5EED + V).permutation(V)
        return perm[ranks].astype(np.int32)
    return ranks.astype(np.int32)


def zipf_hot_ids(V: int, K: int, permute: bool = True) -> np.ndarray:
    """The ids of the K most probable ranks of zipf_ids' distribution (what a cache of hot rows holds)."""
    K = min(K, V)
    if permute:
        return np.random.default_rng(0x5EED + V).permutation(V)[:K].astype(np.int32)
    return np.arange(K, dtype=np.int32)


def uniform_ids(M: int, V: int, seed: int = 0) -> np.ndarray:
    return np.random.default_rng(seed).integers(0, V, size=M, dtype=np.int64).astype(np.int32)


# ---- the tiny FFN-built configuration -------------------------------------------------------

def tiny_model(seed: int = 0, shape: Shape = SHAPES["tiny"], B: int = 4, T: int = 16) -> dict:
    """fp32 inputs of the tiny configuration: embeddings N(0,1), FFN and router weights
    N(0,0.02), ids uniform over V, hidden N(0,1).  Per layer: W1 [N][D][d], W2 [N][d][D],
    Wr [d][N].  The tables are NOT built here (that is the method's Eq. 6)."""
    rng = np.random.default_rng(seed)
    V, d, N, L, D = shape.V, shape.d, shape.N, shape.L, shape.D
    f = np.float32
    out = {
        "shape": shape,
        "E": rng.standard_normal((V, d)).astype(f),
        "W1": [(0.02 * rng.standard_normal((N, D, d))).astype(f) for _ in range(L)],
        "W2": [(0.02 * rng.standard_normal((N, d, D))).astype(f) for _ in range(L)],
        "Wr": [(0.02 * rng.standard_normal((d, N))).astype(f) for _ in range(L)],
        "hidden": rng.standard_normal((B * T, d)).astype(f),
        "ids": rng.integers(0, V, size=B * T, dtype=np.int64).astype(np.int32),
        "B": B,
        "T": T,
    }
    return out


# ---- tensors for the large shapes (torch; generated on the target device) ---------------------

def _tdtype(name: str):
    return torch.bfloat16 if name == "bf16" else torch.float32


def make_table(V: int, N: int, d: int, seed: int, device, dtype: str = "bf16", std: float = 0.05,
               out=None):
    """One layer's table [V][N][d], i.i.d. N(0, std), drawn in place on ``device``."""
    g = torch.Generator(device=device)
    g.manual_seed(seed)
    if out is None:
        out = torch.empty((V, N, d), dtype=_tdtype(dtype), device=device)
    # fill in slabs: normal_ on bf16 draws through fp32 temporaries only inside the kernel
    out.view(-1).normal_(0.0, std, generator=g)
    return out


def make_router(d: int, N: int, seed: int, device, dtype: str = "bf16", std: float = 0.02):
    g = torch.Generator(device="cpu")
    g.manual_seed(seed)
    w = torch.empty((d, N), dtype=torch.float32).normal_(0.0, std, generator=g)
    return w.to(_tdtype(dtype)).to(device)


def make_hidden(M: int, d: int, seed: int, device, dtype: str = "bf16"):
    g = torch.Generator(device="cpu")
    g.manual_seed(seed)
    h = torch.empty((M, d), dtype=torch.float32).normal_(0.0, 1.0, generator=g)
    return h.to(_tdtype(dtype)).to(device)


def make_ids(M: int, V: int, seed: int, device, kind: str = "zipf"):
    ids = zipf_ids(M, V, seed=seed) if kind == "zipf" else uniform_ids(M, V, seed=seed)
    return torch.from_numpy(ids).to(device)
