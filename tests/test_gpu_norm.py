"""GPU parity of the decoder-layer form of the paper's App. A.2 listing: the router reads
RMSNorm(hidden), the residual stays un-normalised.  The expected values are composed from the
oracle's own pieces: its RMSNorm (pinned by a closed form), one rounding to the storage type (the
listing materialises the normalised activations in the model's type), then its lookup-form layer
with the un-normalised hidden state as residual."""
import numpy as np
import pytest
import torch

import oracle
from gpu_util import as_f64, bits, check_gates_normed_router, check_out, rand_case
from paper_2503_15798_b200 import binding as mole

pytestmark = pytest.mark.gpu
DEV = "cuda"


def oracle_norm_layer(hidden, ids, lut, wr, gamma, eps, residual=None):
    h64, g64 = as_f64(hidden), as_f64(gamma)
    normed = np.stack([oracle.rmsnorm(h64[t], g64, eps) for t in range(h64.shape[0])])
    normed_t = torch.from_numpy(normed).to(hidden.dtype)  # round to nearest even, once
    res = hidden if residual is None else residual
    out, gates, bad = oracle.layer_lookup(bits(normed_t), ids.cpu().numpy(), bits(lut), bits(wr), residual=bits(res))
    return out, gates, normed


def check_out_after_flips(out, ref, gates, gref, lut):
    """check_out, with room for the gate differences that check_gates_normed_router allows: the routed term
    moves by at most sum_j |dg_j| max|row|."""
    dg = np.abs(gates.detach().cpu().to(torch.float64).numpy() - gref).sum(axis=1, keepdims=True)
    slack = dg * float(lut.abs().max())
    err = np.abs(as_f64(out) - ref)
    assert (err <= 2.0 ** -8 * np.abs(ref) + 2e-5 + slack).all(), float((err - slack).max())


def run(hidden, ids, lut, wr, gamma, eps, **kw):
    M, N = hidden.shape[0], lut.shape[1]
    gates = torch.zeros(M, N, dtype=torch.float32, device=DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    res = kw.pop("residual", None)
    out = mole.layer_forward(hidden.to(DEV), ids.to(DEV), lut.to(DEV), wr.to(DEV), gates_out=gates, status=status,
                             residual=None if res is None else res.to(DEV), norm_weight=gamma.to(DEV), norm_eps=eps, **kw)
    torch.cuda.synchronize()
    return out, gates, int(status.item())


@pytest.mark.parametrize("M,N,d,V,split", [(7, 16, 768, 50, 0), (300, 16, 1024, 200, 0), (33, 32, 2048, 60, 0),
                                           (33, 32, 2048, 60, 8), (11, 5, 512, 30, 2), (1500, 16, 768, 400, 0),
                                           (9, 64, 4096, 12, 0), (5, 4, 64, 20, 1)])
def test_bf16_norm_parity(M, N, d, V, split):
    hidden, ids, lut, wr = rand_case(M, N, d, V, seed=7 * M + N)
    g = torch.Generator().manual_seed(M)
    gamma = (1.0 + 0.2 * torch.empty(d).normal_(0, 1, generator=g)).to(torch.bfloat16)
    hidden = (hidden.float() * 3.0).to(torch.bfloat16)  # RMS far from 1: the scale must really be divided out
    ref, gref, normed = oracle_norm_layer(hidden, ids, lut, wr, gamma, 1e-5)
    out, gates, status = run(hidden, ids, lut, wr, gamma, 1e-5, d_split=split)
    assert status == 0
    check_gates_normed_router(gates, gref, normed, wr)
    check_out_after_flips(out, ref, gates, gref, lut)
    # and it is not the un-normalised router
    plain = mole.layer_forward(hidden.to(DEV), ids.to(DEV), lut.to(DEV), wr.to(DEV))
    assert not torch.equal(plain, out)


def test_fp32_norm_parity_and_separate_residual():
    M, N, d, V = 40, 4, 64, 32
    hidden, ids, lut, wr = rand_case(M, N, d, V, seed=3, dtype=torch.float32)
    g = torch.Generator().manual_seed(5)
    gamma = 1.0 + 0.3 * torch.empty(d).normal_(0, 1, generator=g)
    residual = torch.empty(M, d).normal_(0, 1, generator=g)
    ref, gref, normed = oracle_norm_layer(hidden, ids, lut, wr, gamma, 1e-6, residual=residual)
    out, gates, status = run(hidden, ids, lut, wr, gamma, 1e-6, residual=residual)
    assert status == 0
    check_out(out, ref, torch.float32)
    check_gates_normed_router(gates, gref, normed, wr, torch.float32)


def test_norm_is_invariant_to_a_power_of_two_scale_when_eps_is_zero():
    """RMSNorm(2^k x) == RMSNorm(x) exactly for eps = 0 (every operation scales exactly): the gates must
    not change by a single bit, while the residual -- which is not normalised -- does scale."""
    M, N, d, V = 64, 16, 768, 100
    hidden, ids, lut, wr = rand_case(M, N, d, V, seed=21)
    gamma = torch.ones(d, dtype=torch.bfloat16)
    out1, gates1, _ = run(hidden, ids, lut, wr, gamma, 0.0)
    out4, gates4, _ = run((hidden.float() * 4.0).to(torch.bfloat16), ids, lut, wr, gamma, 0.0)
    assert torch.equal(gates1, gates4)
    # the same routed term on a residual four times as large: each output rounded once at its own magnitude
    routed1 = as_f64(out1) - as_f64(hidden.to(DEV))
    routed4 = as_f64(out4) - 4.0 * as_f64(hidden.to(DEV))
    bound = 2.0 ** -8 * (np.abs(as_f64(out1)) + np.abs(as_f64(out4))) + 1e-6  # half a bf16 ulp each
    assert (np.abs(routed1 - routed4) <= bound).all()


def test_unit_weight_and_unit_rms_rows_match_the_plain_router():
    """Rows of +-1 have mean square 1: with weight 1 and eps 0 the normalised state equals the state,
    so the norm kernel must reproduce the plain kernel's gates (same router arithmetic)."""
    M, N, d, V = 32, 16, 1024, 64
    _, ids, lut, wr = rand_case(M, N, d, V, seed=9)
    g = torch.Generator().manual_seed(1)
    hidden = (torch.randint(0, 2, (M, d), generator=g).float() * 2 - 1).to(torch.bfloat16)
    gamma = torch.ones(d, dtype=torch.bfloat16)
    out_n, gates_n, _ = run(hidden, ids, lut, wr, gamma, 0.0)
    gates_p = torch.zeros(M, N, dtype=torch.float32, device=DEV)
    out_p = mole.layer_forward(hidden.to(DEV), ids.to(DEV), lut.to(DEV), wr.to(DEV), gates_out=gates_p)
    torch.cuda.synchronize()
    assert np.abs(as_f64(gates_n) - as_f64(gates_p)).max() <= 1e-6
    assert np.abs(as_f64(out_n) - as_f64(out_p)).max() <= 2.0 ** -7


@pytest.mark.parametrize("norm", [False, True])
def test_cluster_kernel_with_a_separate_residual(norm):
    """d = 2048: the one-token-per-cluster kernel with a residual that is not the hidden state (the App. A.2 layer
    adds the shared expert's output to it), with and without the RMSNorm in front of the router, gates included."""
    M, N, d, V = 19, 32, 2048, 45
    hidden, ids, lut, wr = rand_case(M, N, d, V, seed=77)
    g = torch.Generator().manual_seed(3)
    residual = torch.empty(M, d).normal_(0, 1, generator=g).to(torch.bfloat16)
    assert mole.variant(M, N, d, norm=norm)[0] == f"cdecode<32,4,{int(norm)}>"
    if norm:
        gamma = (1.0 + 0.2 * torch.empty(d).normal_(0, 1, generator=g)).to(torch.bfloat16)
        ref, gref, normed = oracle_norm_layer(hidden, ids, lut, wr, gamma, 1e-5, residual=residual)
        out, gates, status = run(hidden, ids, lut, wr, gamma, 1e-5, residual=residual)
        assert status == 0
        check_gates_normed_router(gates, gref, normed, wr)
        check_out_after_flips(out, ref, gates, gref, lut)
    else:
        ref, gref, bad = oracle.layer_lookup(bits(hidden), ids.cpu().numpy(), bits(lut), bits(wr), residual=bits(residual))
        gates = torch.zeros(M, N, dtype=torch.float32, device=DEV)
        status = torch.zeros(1, dtype=torch.int32, device=DEV)
        out = mole.layer_forward(hidden.to(DEV), ids.to(DEV), lut.to(DEV), wr.to(DEV), gates_out=gates, status=status,
                                 residual=residual.to(DEV))
        torch.cuda.synchronize()
        assert bad == 0 and int(status.item()) == 0
        assert np.abs(as_f64(gates) - gref).max() <= 1e-5
        err = np.abs(as_f64(out) - ref)
        assert (err <= 2.0 ** -8 * np.abs(ref) + 2e-5).all(), float(err.max())
