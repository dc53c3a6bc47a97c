"""GPU parity of the re-parameterisation (Eq. 6-7): the tensor-core table builder against the oracle's
builder (plain fp64 loops over every id, expert and column, pinned by its own tests), and the paper's
defining identity on the GPU path: the lookup layer over a GPU-built table equals the experts run on the fly."""
import numpy as np
import pytest
import torch

import oracle
from gpu_util import as_f64, bits
from paper_2503_15798_b200 import binding as mole
from paper_2503_15798_b200 import inputs

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _weights(V, N, d, D, seed, scale1=None, scale2=None):
    g = torch.Generator().manual_seed(seed)
    E = torch.empty(V, d).normal_(0, 1, generator=g).to(torch.bfloat16)
    W1 = torch.empty(N, D, d).normal_(0, scale1 or d ** -0.5, generator=g).to(torch.bfloat16)
    W2 = torch.empty(N, d, D).normal_(0, scale2 or D ** -0.5, generator=g).to(torch.bfloat16)
    return E, W1, W2


def _bound(E64, W1, W2, ref):
    """What the bf16 materialisation of the hidden activations and of the result can move an entry by: half a
    bf16 ulp (2^-9) of every |h_k w2_k| term, fp32 accumulation noise, and the final rounding of the entry."""
    W1_64, W2_64 = as_f64(W1), as_f64(W2)
    out = np.empty_like(ref)
    from scipy.special import erf
    for j in range(W1_64.shape[0]):
        pre = E64 @ W1_64[j].T
        h = 0.5 * pre * (1.0 + erf(pre / np.sqrt(2.0)))
        out[:, j, :] = np.abs(h) @ np.abs(W2_64[j]).T
    return 2.0 ** -8 * out + 2.0 ** -8 * np.abs(ref) + 1e-6


@pytest.mark.parametrize("V,N,d,D,norm", [(512, 4, 64, 256, False), (300, 3, 64, 128, True), (130, 16, 768, 256, False),
                                          (257, 2, 1024, 520, True), (128, 1, 8, 8, False), (1000, 5, 136, 72, False)])
def test_built_table_matches_the_oracle_builder(V, N, d, D, norm):
    E, W1, W2 = _weights(V, N, d, D, seed=V + d)
    gamma = None
    if norm:
        gamma = (1.0 + 0.2 * torch.empty(d).normal_(0, 1, generator=torch.Generator().manual_seed(1))).to(torch.bfloat16)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    lut = mole.build_lut(E.to(DEV), W1.to(DEV), W2.to(DEV), None if gamma is None else gamma.to(DEV), 1e-5, status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    E64 = as_f64(E)
    if norm:  # the normalised rows are materialised in bf16 before the experts see them
        normed = np.stack([oracle.rmsnorm(E64[i], as_f64(gamma), 1e-5) for i in range(V)])
        E64 = as_f64(torch.from_numpy(normed).to(torch.bfloat16))
    ref = oracle.build_lut(E64, as_f64(W1), as_f64(W2))
    err = np.abs(as_f64(lut) - ref)
    bound = _bound(E64, W1, W2, ref)
    if norm:  # an element of the normalised row on a rounding tie may land on the other neighbour
        bound = bound + 2.0 ** -7 * np.abs(ref) + 2.0 ** -6
    assert (err <= bound).all(), float((err / bound).max())
    assert np.abs(as_f64(lut)).max() > 0.05  # not a table of zeros


def test_tiny_config_lookup_over_a_gpu_built_table_equals_experts_on_the_fly():
    """Eq. 5 with Eq. 6 substituted is Eq. 8: the fused lookup layer over the table the GPU builder made, against
    the oracle running the expert FFNs on the embedding rows of the batch's ids."""
    m = inputs.tiny_model(seed=0)
    sh = m["shape"]
    E = torch.from_numpy(m["E"]).to(torch.bfloat16)
    hidden = torch.from_numpy(m["hidden"]).to(torch.bfloat16)
    ids = torch.from_numpy(m["ids"])
    for l in range(sh.L):
        W1 = torch.from_numpy(m["W1"][l] * 20).to(torch.bfloat16)  # larger weights: a routed term that shows in bf16
        W2 = torch.from_numpy(m["W2"][l] * 20).to(torch.bfloat16)
        Wr = torch.from_numpy(m["Wr"][l]).to(torch.bfloat16)
        lut = mole.build_lut(E.to(DEV), W1.to(DEV), W2.to(DEV))
        out = mole.layer_forward(hidden.to(DEV), ids.to(DEV), lut, Wr.to(DEV))
        torch.cuda.synchronize()
        fly, bad = oracle.layer_onthefly(as_f64(hidden), m["ids"], as_f64(E), as_f64(W1), as_f64(W2), as_f64(Wr))
        assert bad == 0
        routed = fly - as_f64(hidden)
        assert np.abs(routed).max() > 0.05
        err = np.abs(as_f64(out) - fly)
        assert (err <= 2.0 ** -7 * np.abs(fly) + 2.0 ** -6 * np.abs(routed).max() + 1e-4).all(), float(err.max())


def test_builder_argument_checks():
    E, W1, W2 = _weights(128, 2, 64, 64, seed=1)
    with pytest.raises(mole.MoleError) as e:  # d not a multiple of 8
        mole.build_lut(E[:, :60].contiguous().to(DEV), W1[:, :, :60].contiguous().to(DEV), W2[:, :60].contiguous().to(DEV))
    assert e.value.code in (mole.ERR_INVALID_ARG, mole.ERR_UNSUPPORTED_SHAPE)


@pytest.mark.parametrize("V,N,d,D,norm", [(4096, 8, 256, 1024, False), (3000, 4, 768, 3072, True)])
def test_many_tiles_per_block_sampled_rows(V, N, d, D, norm):
    """Shapes with several hundred output tiles per GEMM, so that every persistent block walks many tiles (both
    accumulators in tensor memory and the operand ring reused again and again, ragged last tile rows): sampled
    ids' rows of the table against the oracle's builder run on those embedding rows alone."""
    E, W1, W2 = _weights(V, N, d, D, seed=V + D)
    gamma = None
    if norm:
        gamma = (1.0 + 0.2 * torch.empty(d).normal_(0, 1, generator=torch.Generator().manual_seed(2))).to(torch.bfloat16)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    lut = mole.build_lut(E.to(DEV), W1.to(DEV), W2.to(DEV), None if gamma is None else gamma.to(DEV), 1e-5, status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    rng = np.random.default_rng(V)
    sample = np.unique(np.concatenate([rng.integers(0, V, 48), [0, 127, 128, V - 129, V - 1]]))
    E64 = as_f64(E[sample])
    if norm:
        normed = np.stack([oracle.rmsnorm(E64[i], as_f64(gamma), 1e-5) for i in range(len(sample))])
        E64 = as_f64(torch.from_numpy(normed).to(torch.bfloat16))
    ref = oracle.build_lut(E64, as_f64(W1), as_f64(W2))
    got = as_f64(lut[torch.from_numpy(sample).to(DEV)])
    err = np.abs(got - ref)
    bound = _bound(E64, W1, W2, ref)
    if norm:
        bound = bound + 2.0 ** -7 * np.abs(ref) + 2.0 ** -6
    assert (err <= bound).all(), float((err / bound).max())
    # every row was written: no tile skipped (rows of a zero-filled output would be exactly zero)
    assert bool((lut.abs().amax(dim=(1, 2)) > 0).all())
