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


def check_gates_normed_router(gates: torch.Tensor, ref: np.ndarray, normed: np.ndarray, wr: torch.Tensor, dtype=torch.bfloat16):
    """Gates of the layer whose router reads RMSNorm(hidden) rounded to the storage type.  That rounding
    is a decision taken in fp32 on the GPU and in fp64 by the oracle: an element within fp32 noise of a
    tie (about one in ten thousand) lands on the neighbouring value, which moves a logit by one
    storage-type ulp of that element times a router weight and a gate by at most a quarter of that.
    So: every gate within two such flips of the oracle's, and all but a few within the plain 1e-5."""
    g = gates.detach().cpu().to(torch.float64).numpy()
    err = np.abs(g - ref)
    ulp = 2.0 ** -8 if dtype == torch.bfloat16 else 2.0 ** -24
    flip = 0.25 * ulp * float(np.abs(normed).max()) * float(wr.abs().max())
    assert err.max() <= 1e-5 + 2 * flip, (float(err.max()), flip)
    assert (err <= 1e-5).mean() >= 0.97, float((err <= 1e-5).mean())
    assert np.abs(g.sum(axis=1) - 1.0).max() <= 1e-6
