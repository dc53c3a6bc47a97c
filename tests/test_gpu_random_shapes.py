"""Seeded random sweep over shapes, chunk counts, storage types and entry points: every case is
compared with the fp64 oracle element by element.  The fixed cases elsewhere pin the shapes of the
paper's Table 2; this file walks the combinations in between (odd N, d that is no power of two, ragged
token counts, forced chunk counts that do and do not divide N, the normalised router)."""
import numpy as np
import pytest
import torch

import oracle
from gpu_util import as_f64, bits, check_gates, check_gates_normed_router, check_out, oracle_layer
from paper_2503_15798_b200 import binding as mole

pytestmark = pytest.mark.gpu
DEV = "cuda"


def draw(seed):
    r = np.random.default_rng(seed)
    dtype = torch.float32 if r.random() < 0.25 else torch.bfloat16
    vec = 4 if dtype == torch.float32 else 8
    N = int(r.choice([1, 2, 3, 4, 5, 7, 8, 12, 16, 16, 24, 32, 33, 48, 64]))
    d = vec * int(r.choice([1, 2, 3, 8, 12, 16, 24, 40, 64, 96, 128, 160, 256, 320]))
    M = int(r.choice([1, 2, 3, 17, 31, 32, 33, 64, 100, 150, 299, 700]))
    if M * N * d > 6e6:
        M = max(1, int(6e6 // (N * d)))
    V = int(r.integers(1, 200))
    split = int(r.choice([0, 0, 0, 1, 2, 4, 8, 16]))
    L = int(r.choice([1, 1, 2, 3, 5]))
    norm = bool(r.random() < 0.3)
    return dtype, N, d, M, V, split, L, norm


@pytest.mark.parametrize("seed", range(48))
def test_random_case_against_the_oracle(seed):
    dtype, N, d, M, V, split, L, norm = draw(seed)
    g = torch.Generator().manual_seed(1000 + seed)
    luts = torch.empty(L, V, N, d).normal_(0, 0.05, generator=g).to(dtype)
    wrs = torch.empty(L, d, N).normal_(0, 0.05, generator=g).to(dtype)
    hidden = torch.empty(M, d).normal_(0, 1, generator=g).to(dtype)
    ids = torch.randint(0, V, (M,), generator=g, dtype=torch.int32)
    try:
        mole.plan(M, N, d, mole.DTYPE_F32 if dtype == torch.float32 else mole.DTYPE_BF16, split, L)
    except mole.MoleError as e:
        assert e.code == mole.ERR_UNSUPPORTED_SHAPE  # a chunk count this shape cannot take (host check, nothing launched)
        pytest.skip("shape / chunk count rejected by the plan")
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    if L == 1:
        gates = torch.zeros(M, N, dtype=torch.float32, device=DEV)
        if norm:
            gamma = (1.0 + 0.2 * torch.empty(d).normal_(0, 1, generator=g)).to(dtype)
            normed = np.stack([oracle.rmsnorm(as_f64(hidden)[t], as_f64(gamma), 1e-5) for t in range(M)])
            normed_t = torch.from_numpy(normed).to(dtype)
            ref, gref, _ = oracle.layer_lookup(bits(normed_t), ids.numpy(), bits(luts[0]), bits(wrs[0]), residual=bits(hidden))
            out = mole.layer_forward(hidden.to(DEV), ids.to(DEV), luts[0].to(DEV), wrs[0].to(DEV), gates_out=gates, status=status,
                                     d_split=split, norm_weight=gamma.to(DEV), norm_eps=1e-5)
            torch.cuda.synchronize()
            assert int(status.item()) == 0
            check_gates_normed_router(gates, gref, normed, wrs[0], dtype)
            dg = np.abs(gates.cpu().to(torch.float64).numpy() - gref).sum(axis=1, keepdims=True)
            err = np.abs(as_f64(out) - ref)
            unit = 2.0 ** -8 if dtype == torch.bfloat16 else 4e-6
            assert (err <= unit * np.maximum(1.0, np.abs(ref)) + 2e-5 + dg * float(luts[0].abs().max())).all()
            return
        else:
            ref, gref, _ = oracle_layer(hidden, ids, luts[0], wrs[0])
            out = mole.layer_forward(hidden.to(DEV), ids.to(DEV), luts[0].to(DEV), wrs[0].to(DEV), gates_out=gates, status=status,
                                     d_split=split)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        check_out(out, ref, dtype)
        check_gates(gates, gref)
        return
    # several layers: fused and chained against the oracle's chain (each layer fed the storage-type rounding)
    h = hidden
    for l in range(L):
        ref, _, _ = oracle_layer(h, ids, luts[l], wrs[l])
        h = torch.from_numpy(ref).to(dtype)
    hd, idd, ld, wd = hidden.to(DEV), ids.to(DEV), luts.to(DEV), wrs.to(DEV)
    for mode in (mole.STEP_FUSED, mole.STEP_CHAINED):
        out = mole.decode_step(hd, idd, ld, wd, torch.empty_like(hd), torch.empty_like(hd), status=status, mode=mode, d_split=split)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        err = np.abs(as_f64(out) - as_f64(h))
        unit = 2.0 ** -7 if dtype == torch.bfloat16 else 1e-5
        assert (err <= L * unit * np.maximum(1.0, np.abs(as_f64(h)))).all(), (mode, float(err.max()))
