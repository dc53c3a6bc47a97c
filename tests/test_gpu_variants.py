"""Every kernel instantiation that bench.py times has a parity case here, element by element against the
fp64 oracle, at the token count, width and expert count the bench uses (the table itself is small: the
instantiation does not depend on the number of table rows).  The CPU half of the file walks the launch
shapes bench.py declares and fails if one of them resolves to an instantiation without a case below."""
import numpy as np
import pytest
import torch

import bench
import oracle
from gpu_util import as_f64, bits, check_gates, check_gates_normed_router, check_out, oracle_layer
from paper_2503_15798_b200 import binding as mole

DEV = "cuda"
RING, DECODE, AUTO = mole.KERNEL_RING, mole.KERNEL_DECODE, mole.KERNEL_AUTO
DEC = DECODE

# instantiation -> launches that reach it: (M, N, d, L, norm, kernel)
CASES = {
    # single-layer launches of the chained step
    "decode<16,0>": [(256, 16, 768, 1, False, DEC), (64, 16, 1024, 1, False, DEC), (1, 16, 768, 1, False, DEC),
                     (2048, 16, 1024, 1, False, DEC)],
    "decode<16,1>": [(256, 16, 768, 1, True, DEC), (256, 16, 1024, 1, True, DEC), (8, 16, 768, 1, True, DEC)],
    "decode<32,0>": [(70, 32, 1024, 1, False, DEC)],
    "decode<32,1>": [(70, 32, 512, 1, True, DEC)],
    "decode<8,0>": [(33, 8, 256, 1, False, DEC)],
    "decode<8,1>": [(33, 8, 384, 1, True, DEC)],
    "decode<4,0>": [(19, 4, 128, 1, False, DEC)],
    "decode<4,1>": [(19, 4, 2048, 1, True, DEC)],
    # one token per cluster of four blocks (d = 2048)
    "cdecode<32,4,0>": [(256, 32, 2048, 1, False, DEC), (16, 32, 2048, 1, False, DEC), (1, 32, 2048, 1, False, DEC),
                        (333, 32, 2048, 1, False, DEC)],
    "cdecode<32,4,1>": [(256, 32, 2048, 1, True, DEC), (16, 32, 2048, 1, True, AUTO), (1, 32, 2048, 1, True, DEC)],
    "cdecode<16,4,0>": [(40, 16, 2048, 1, False, DEC)],
    "cdecode<16,4,1>": [(40, 16, 2048, 1, True, DEC)],
    "step<bf16,16,1,2,1,1,0>": [(256, 16, 768, 1, False, AUTO), (500, 16, 768, 1, False, AUTO)],  # the second: a one-slot ring
    "step<bf16,16,1,2,1,0,0>": [(64, 16, 768, 1, False, AUTO), (3000, 16, 768, 1, False, AUTO)],
    "step<bf16,16,1,2,2,1,0>": [(256, 16, 1024, 1, False, AUTO), (400, 16, 1024, 1, False, AUTO)],
    "step<bf16,16,1,2,2,0,0>": [(64, 16, 1024, 1, False, AUTO), (2500, 16, 1024, 1, False, AUTO)],
    "step<bf16,16,1,2,1,1,1>": [(256, 16, 768, 1, True, AUTO), (400, 16, 768, 1, True, AUTO)],  # the second: a one-slot ring
    "step<bf16,16,1,2,1,0,1>": [(700, 16, 768, 1, True, AUTO)],
    "step<bf16,16,1,2,2,1,1>": [(256, 16, 1024, 1, True, AUTO)],
    "step<bf16,16,1,2,2,0,1>": [(2500, 16, 1024, 1, True, AUTO)],
    # fused steps: the decode arithmetic with a ring (default) ...
    "fstep<16,1,0>": [(256, 16, 768, 3, False, DEC), (64, 16, 768, 12, False, DEC), (256, 16, 1024, 3, False, DEC),
                      (8, 16, 1024, 8, False, DEC), (1, 16, 768, 12, False, DEC), (700, 16, 768, 2, False, DEC)],
    "fstep<16,1,1>": [(256, 16, 768, 3, True, DEC), (64, 16, 1024, 2, True, DEC)],
    "fstep<32,2,0>": [(256, 32, 2048, 3, False, DEC), (64, 32, 2048, 3, False, DEC), (16, 32, 2048, 2, False, DEC)],
    "fstep<32,2,1>": [(256, 32, 2048, 2, True, DEC), (16, 32, 2048, 2, True, DEC)],
    "fstep<32,1,0>": [(40, 32, 1024, 2, False, DEC)],
    "fstep<32,0,1>": [(40, 32, 512, 3, True, DEC)],
    "fstep<16,2,0>": [(40, 16, 2048, 2, False, DEC)],
    "fstep<8,0,0>": [(33, 8, 256, 5, False, DEC)],
    "fstep<4,0,1>": [(33, 4, 128, 3, True, DEC)],
    # ... and the ring kernel's own fused form (on request; the offload step's groups)
    "step<bf16,16,1,1,1,0,0>": [(256, 16, 768, 3, False, AUTO), (64, 16, 768, 12, False, AUTO)],
    "step<bf16,16,1,1,2,0,0>": [(256, 16, 1024, 3, False, AUTO), (64, 16, 1024, 4, False, AUTO), (8, 16, 1024, 8, False, AUTO)],
    "step<bf16,16,1,1,1,0,1>": [(256, 16, 768, 3, True, AUTO), (8, 16, 768, 12, True, AUTO)],
    "step<bf16,16,1,1,2,0,1>": [(256, 16, 1024, 3, True, AUTO), (64, 16, 1024, 2, True, AUTO)],
    "step<bf16,16,1,0,0,0,1>": [(256, 16, 1536, 3, True, AUTO), (64, 16, 1536, 2, True, AUTO)],
    "step<bf16,32,2,3,3,0,0>": [(256, 32, 2048, 1, False, AUTO), (256, 32, 2048, 3, False, AUTO)],
    "step<bf16,32,2,3,4,0,0>": [(64, 32, 2048, 1, False, RING), (140, 32, 2048, 1, False, AUTO), (64, 32, 2048, 3, False, AUTO), (148, 32, 2048, 2, False, AUTO)],
    "step<bf16,32,2,3,3,0,1>": [(256, 32, 2048, 1, True, AUTO), (256, 32, 2048, 2, True, AUTO)],
    "step<bf16,32,2,3,4,0,1>": [(16, 32, 2048, 1, True, RING), (64, 32, 2048, 2, True, AUTO)],
    "step<bf16,32,1,0,0,0,1>": [(16, 32, 1024, 2, True, AUTO)],
    "step<bf16,32,2,0,0,0,1>": [(256, 32, 4096, 2, True, AUTO)],
}
FLAT = [(name,) + c for name, cs in CASES.items() for c in cs]


def test_every_launch_shape_the_bench_times_has_a_parity_case():
    import test_gpu_quant

    covered = set(CASES) | test_gpu_quant.covered_variants()
    missing = {}
    for sh in bench.timed_launch_shapes():
        name = mole.variant(sh["M"], sh["N"], sh["d"], L=sh["L"], norm=sh["norm"], kernel=sh["kernel"],
                            lut_format=sh["lut_format"], lut_block=sh["lut_block"])[0]
        if name not in covered:
            missing.setdefault(name, []).append(sh["what"])
    assert not missing, missing


def decode_exists(M, N, d, norm):
    try:
        return mole.variant(M, N, d, norm=norm, kernel=DECODE)[0].startswith("decode")
    except mole.MoleError:
        return False


def _oracle_chain(hidden, ids, luts, wrs, gammas, eps):
    """The oracle layer after layer, each fed the storage-type rounding of the previous one; with gammas the
    router of every layer reads the rounded RMSNorm of its input.  Returns the last layer's fp64 output, its
    gates, the (fp64) normalised state of the last layer."""
    h = hidden
    for l in range(luts.shape[0]):
        if gammas is None:
            ref, gref, _ = oracle_layer(h, ids, luts[l], wrs[l])
            normed = None
        else:
            h64, g64 = as_f64(h), as_f64(gammas[l])
            normed = np.stack([oracle.rmsnorm(h64[t], g64, eps) for t in range(h64.shape[0])])
            ref, gref, _ = oracle.layer_lookup(bits(torch.from_numpy(normed).to(torch.bfloat16)), ids.cpu().numpy(),
                                               bits(luts[l]), bits(wrs[l]), residual=bits(h))
        h = torch.from_numpy(ref).to(torch.bfloat16)
    return ref, gref, normed


@pytest.mark.gpu
@pytest.mark.parametrize("name,M,N,d,L,norm,kernel", FLAT)
def test_variant_against_the_oracle(name, M, N, d, L, norm, kernel):
    assert mole.variant(M, N, d, L=L, norm=norm, kernel=kernel)[0] == name
    V = 97
    g = torch.Generator().manual_seed(M + 7 * d + L)
    luts = torch.empty(L, V, N, d).normal_(0, 0.05, generator=g).to(torch.bfloat16)
    wrs = torch.empty(L, d, N).normal_(0, 0.02, generator=g).to(torch.bfloat16)
    hidden = (1.5 * torch.empty(M, d).normal_(0, 1, generator=g)).to(torch.bfloat16)
    ids = torch.randint(0, V, (M,), generator=g, dtype=torch.int32)
    gammas = (1.0 + 0.2 * torch.empty(L, d).normal_(0, 1, generator=g)).to(torch.bfloat16) if norm else None
    eps = 1e-5
    ref, gref, normed = _oracle_chain(hidden, ids, luts, wrs, gammas, eps)
    hd, idd, ld, wd = hidden.to(DEV), ids.to(DEV), luts.to(DEV), wrs.to(DEV)
    gd = gammas.to(DEV) if norm else None
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    if L == 1:
        gates = torch.zeros(M, N, dtype=torch.float32, device=DEV)
        out = mole.layer_forward(hd, idd, ld[0], wd[0], gates_out=gates, status=status, kernel=kernel, chain=True,
                                 norm_weight=None if gd is None else gd[0], norm_eps=eps)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        if norm:
            check_gates_normed_router(gates, gref, normed, wrs[0])
            dg = np.abs(as_f64(gates) - gref).sum(axis=1, keepdims=True)
            err = np.abs(as_f64(out) - ref)
            assert (err <= 2.0 ** -8 * np.abs(ref) + 2e-5 + dg * float(luts.abs().max())).all()
        else:
            check_gates(gates, gref)
            check_out(out, ref)
        return
    outs = []
    for mode in (mole.STEP_FUSED, mole.STEP_CHAINED):
        # the family asked for runs the fused launch; the chained launches too where it has a single-layer kernel
        k = kernel if (mode == mole.STEP_FUSED or kernel != DECODE or decode_exists(M, N, d, norm)) else AUTO
        out = mole.decode_step_args(hd, idd, ld, wd, torch.empty_like(hd), torch.empty_like(hd), status=status, mode=mode,
                                    norm_weights=gd, norm_eps=eps, kernel=k)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        err = np.abs(as_f64(out) - ref)
        slack = 0.0
        if norm:  # a rounding tie in a normalised element moves a gate (see gpu_util.near_tie_slack): per layer, a few 1e-4
            slack = L * 1e-3 * float(luts.abs().max()) * N
        assert (err <= L * 2.0 ** -7 * np.maximum(1.0, np.abs(ref)) + slack).all(), (mode, float(err.max()))
        outs.append(out)
    if not norm:
        # the two ways of launching a step differ at most in the order of fp32 sums
        assert (np.abs(as_f64(outs[0]) - as_f64(outs[1])) <= L * 2.0 ** -7 * np.maximum(1.0, np.abs(ref))).all()
    if name.startswith("fstep") and decode_exists(M, N, d, norm):
        # the fused step adds in the order of the one-block-per-token kernel: the bits of L chained launches of it
        assert torch.equal(outs[0], outs[1])


@pytest.mark.gpu
@pytest.mark.parametrize("M,N,norm", [(64, 32, False), (5, 16, False), (9, 32, True)])
def test_cluster_kernel_chained_step(M, N, norm):
    """L chained launches of the one-token-per-cluster kernel (programmatic dependent launch between them)
    against the oracle's chain."""
    d, L, V = 2048, 3, 61
    assert mole.variant(M, N, d, kernel=DECODE, norm=norm)[0] == f"cdecode<{N},4,{int(norm)}>"
    g = torch.Generator().manual_seed(11 * M + N)
    luts = torch.empty(L, V, N, d).normal_(0, 0.05, generator=g).to(torch.bfloat16)
    wrs = torch.empty(L, d, N).normal_(0, 0.02, generator=g).to(torch.bfloat16)
    hidden = (1.5 * torch.empty(M, d).normal_(0, 1, generator=g)).to(torch.bfloat16)
    ids = torch.randint(0, V, (M,), generator=g, dtype=torch.int32)
    gammas = (1.0 + 0.2 * torch.empty(L, d).normal_(0, 1, generator=g)).to(torch.bfloat16) if norm else None
    ref, _, _ = _oracle_chain(hidden, ids, luts, wrs, gammas, 1e-5)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    hd = hidden.to(DEV)
    out = mole.decode_step_args(hd, ids.to(DEV), luts.to(DEV), wrs.to(DEV), torch.empty_like(hd), torch.empty_like(hd),
                                status=status, mode=mole.STEP_CHAINED, kernel=DECODE, norm_weights=gammas.to(DEV) if norm else None,
                                norm_eps=1e-5)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    err = np.abs(as_f64(out) - ref)
    slack = L * 1e-3 * float(luts.abs().max()) * N if norm else 0.0  # a rounding tie in a normalised element moves a gate
    assert (err <= L * 2.0 ** -7 * np.maximum(1.0, np.abs(ref)) + slack).all(), float(err.max())


@pytest.mark.gpu
@pytest.mark.parametrize("with_tmp", [True, False])
def test_step_auto_on_the_widest_layers_at_few_tokens(with_tmp):
    """mole_decode_step's own choice (MOLE_STEP_AUTO) for d = 2048 at up to 16 tokens: chained launches of the
    cluster kernel when the caller gave a second buffer, the fused ring launch when not; both against the oracle."""
    M, N, d, L, V = 8, 32, 2048, 3, 41
    g = torch.Generator().manual_seed(5)
    luts = torch.empty(L, V, N, d).normal_(0, 0.05, generator=g).to(torch.bfloat16)
    wrs = torch.empty(L, d, N).normal_(0, 0.02, generator=g).to(torch.bfloat16)
    hidden = (1.5 * torch.empty(M, d).normal_(0, 1, generator=g)).to(torch.bfloat16)
    ids = torch.randint(0, V, (M,), generator=g, dtype=torch.int32)
    ref, _, _ = _oracle_chain(hidden, ids, luts, wrs, None, 0.0)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    hd = hidden.to(DEV)
    out = mole.decode_step_args(hd, ids.to(DEV), luts.to(DEV), wrs.to(DEV), torch.empty_like(hd),
                                torch.empty_like(hd) if with_tmp else None, status=status, mode=mole.STEP_AUTO)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    err = np.abs(as_f64(out) - ref)
    assert (err <= L * 2.0 ** -7 * np.maximum(1.0, np.abs(ref))).all(), float(err.max())
