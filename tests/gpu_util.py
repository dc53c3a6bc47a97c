"""Helpers shared by the GPU parity tests: seeded inputs on the device, the same bytes on the
host for the oracle, and the two error bounds."""
import numpy as np
import torch

import oracle
from paper_2503_15798_b200 import build

build.build()


def bits(t: torch.Tensor) -> np.ndarray:
    """Raw bf16 bit patterns of a tensor (uint16), or the float32 / int values unchanged."""
    t = t.detach().cpu().contiguous()
    if t.dtype == torch.bfloat16:
        return t.view(torch.int16).numpy().view(np.uint16)
    return t.numpy()


def as_f64(t: torch.Tensor) -> np.ndarray:
    return t.detach().cpu().to(torch.float64).numpy()


def rand_case(M, N, d, V, seed, dtype=torch.bfloat16, ids_kind="uniform", lut_std=0.05, wr_std=0.02):
    g = torch.Generator(device="cpu")
    g.manual_seed(seed)
    hidden = torch.empty(M, d).normal_(0, 1, generator=g).to(dtype)
    lut = torch.empty(V, N, d).normal_(0, lut_std, generator=g).to(dtype)
    wr = torch.empty(d, N).normal_(0, wr_std, generator=g).to(dtype)
    if ids_kind == "uniform":
        ids = torch.randint(0, V, (M,), generator=g, dtype=torch.int32)
    else:
        from paper_2503_15798_b200 import inputs

        ids = torch.from_numpy(inputs.zipf_ids(M, V, seed=seed))
    return hidden, ids, lut, wr


def oracle_layer(hidden, ids, lut, wr, residual=None):
    """fp64 oracle on exactly the bytes the GPU sees."""
    r = None if residual is None else bits(residual)
    out, gates, bad = oracle.layer_lookup(bits(hidden), ids.cpu().numpy(), bits(lut), bits(wr), residual=r)
    return out, gates, bad


def check_out(got: torch.Tensor, ref: np.ndarray, dtype=torch.bfloat16):
    """The stated bound max|err| <= 1e-2 * max(1, |ref|), and the tight one the arithmetic
    supports: one rounding of the fp64 value to the storage type plus fp32 accumulation noise."""
    got64 = as_f64(got)
    err = np.abs(got64 - ref)
    scale = np.maximum(1.0, np.abs(ref))
    assert (err <= 1e-2 * scale).all(), float((err / scale).max())
    if dtype == torch.bfloat16:
        tight = 2.0 ** -8 * np.abs(ref) + 2e-5  # <= 1 bf16 ulp of |ref| (half an ulp of rounding + slack)
    else:
        tight = 4e-6 * scale
    assert (err <= tight).all(), float((err - tight).max())


def check_gates(gates: torch.Tensor, ref: np.ndarray):
    g = gates.detach().cpu().to(torch.float64).numpy()
    assert np.abs(g - ref).max() <= 1e-5, float(np.abs(g - ref).max())
    assert np.abs(g.sum(axis=1) - 1.0).max() <= 1e-6


def near_tie_slack(normed: np.ndarray, wr: torch.Tensor, dtype=torch.bfloat16) -> np.ndarray:
    """Per token, how far the gates may move because the normalised state is rounded to the storage type
    in fp32 on the GPU and in fp64 by the oracle.  Only an element whose exact (fp64) value lies within fp32
    noise (2^-20 relative) of a rounding tie can land on the other neighbour; that moves logit j by one
    storage-type ulp of THAT element times W_r[c][j], and a softmax moves by at most half of its largest
    logit change.  A token without such an element gets no slack at all."""
    if dtype != torch.bfloat16:
        return np.zeros(normed.shape[0])  # fp32 storage: a last-place difference moves a logit by ~1e-7
    a = np.abs(normed)
    ulp = 2.0 ** (np.floor(np.log2(np.maximum(a, 1e-300))) - 7)  # bf16: 8 significant bits
    frac = (a / ulp) % 1.0
    near = np.abs(frac - 0.5) * ulp <= 2.0 ** -20 * a
    wmax = np.abs(wr.detach().cpu().to(torch.float64).numpy()).max(axis=1)  # [d]
    return 0.5 * (near * ulp * wmax[None, :]).sum(axis=1)


def check_gates_normed_router(gates: torch.Tensor, ref: np.ndarray, normed: np.ndarray, wr: torch.Tensor, dtype=torch.bfloat16):
    """Gates of the layer whose router reads RMSNorm(hidden) rounded to the storage type: within 1e-5 of
    the oracle's, plus -- only for tokens that have an element on a rounding tie -- what those elements'
    flips can move (near_tie_slack).  `normed`: the oracle's normalised state in fp64, before rounding."""
    g = gates.detach().cpu().to(torch.float64).numpy()
    err = np.abs(g - ref)
    slack = near_tie_slack(normed, wr, dtype)
    assert (err <= 1e-5 + slack[:, None]).all(), (float(err.max()), float(slack.max()), int((slack > 0).sum()))
    assert np.abs(g.sum(axis=1) - 1.0).max() <= 1e-6
