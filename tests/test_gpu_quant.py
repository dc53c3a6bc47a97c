"""GPU parity of the quantised tables (Sec. 4.5 / Table 8): the library's codebooks against the oracle's
derivation, the GPU quantiser against the oracle's packed records bit for bit, and the fused layer over
packed records against the oracle's lookup layer over the de-quantised table, element by element."""
import numpy as np
import pytest
import torch

import oracle
from oracle import quant
from gpu_util import as_f64, bits, rand_case
from paper_2503_15798_b200 import binding as mole

DEV = "cuda"
FMT = {4: mole.LUT_NF4, 3: mole.LUT_NF3}


@pytest.mark.parametrize("nbits", [4, 3])
def test_library_codebook_equals_the_oracles_derivation(nbits):
    # host arithmetic on both sides (bisection on erfc in the library, scipy's quantile function in the oracle)
    got = np.array(mole.nf_codebook(FMT[nbits]), dtype=np.float32)
    assert np.array_equal(got, quant.nf_codebook_f32(nbits))


def test_record_sizes_and_argument_checks():
    assert mole.quant_record_bytes(4, 768, mole.LUT_NF4, 768) == 4 * 388        # Table 8: 388 bytes per 768 elements
    assert mole.quant_record_bytes(4, 768, mole.LUT_NF3, 128) == 4 * 6 * 50     # 50 bytes per 128 elements
    for N, d, nbits, block in ((16, 768, 4, 768), (16, 1024, 3, 128), (32, 2048, 4, 1024), (4, 128, 3, 32)):
        assert mole.quant_record_bytes(N, d, FMT[nbits], block) == quant.record_bytes(N, d, nbits, block)
    for args in ((16, 768, 7, 128), (16, 768, mole.LUT_NF4, 100), (16, 768, mole.LUT_NF4, 512), (0, 768, mole.LUT_NF4, 768)):
        with pytest.raises(mole.MoleError):
            mole.quant_record_bytes(*args)


def _table(V, N, d, seed):
    g = torch.Generator().manual_seed(seed)
    lut = torch.empty(V, N, d).normal_(0, 0.05, generator=g).to(torch.bfloat16)
    lut[0, 0, :] = 0                       # an all-zero block
    lut[1, 1, :] = lut[1, 1, 0]            # an all-equal block
    lut[2, 0, 5] = 3.0                     # one element far above the rest
    return lut


@pytest.mark.gpu
@pytest.mark.parametrize("nbits,block,V,N,d", [(4, 768, 70, 16, 768), (3, 128, 70, 16, 768), (4, 1024, 33, 16, 1024),
                                                (3, 128, 33, 16, 1024), (4, 512, 9, 32, 2048), (3, 128, 9, 32, 2048),
                                                (4, 32, 40, 4, 128), (3, 32, 40, 5, 96), (4, 64, 21, 64, 256)])
def test_gpu_quantiser_writes_the_oracles_records_bit_for_bit(nbits, block, V, N, d):
    lut = _table(V, N, d, seed=V + d)
    want = quant.quantize_table(as_f64(lut).astype(np.float32), nbits, block)
    q = mole.QuantTable.quantize(lut.to(DEV), FMT[nbits], block)
    torch.cuda.synchronize()
    got = q.packed.cpu().numpy()
    assert got.shape == want.shape
    assert np.array_equal(got, want)


# (code bits, block, tokens, experts, width, normalised router): the quantised-layer launches with a parity case
LAYER_CASES = [
    (4, 768, 256, 16, 768, False), (3, 128, 256, 16, 768, False), (4, 1024, 64, 16, 1024, False), (3, 128, 64, 16, 1024, False),
    (4, 1024, 256, 32, 2048, False), (3, 128, 70, 32, 2048, False), (4, 128, 19, 4, 128, False), (3, 32, 19, 8, 384, False),
    (4, 768, 33, 16, 768, True), (3, 128, 33, 16, 1024, True), (4, 256, 1, 16, 768, False), (3, 128, 3000, 16, 768, False),
    (4, 1024, 16384, 16, 1024, False)]


def covered_variants():
    return {mole.variant(M, N, d, norm=norm, lut_format=FMT[nbits], lut_block=block)[0] for nbits, block, M, N, d, norm in LAYER_CASES}


@pytest.mark.gpu
@pytest.mark.parametrize("nbits,block,M,N,d,norm", LAYER_CASES)
def test_quantised_layer_against_the_oracle_on_the_dequantised_table(nbits, block, M, N, d, norm):
    V = 61
    hidden, ids, _, wr = rand_case(M, N, d, V, seed=M + N + nbits)
    lut = _table(V, N, d, seed=7)
    ids[0] = 0
    if M > 2:
        ids[1], ids[2] = 1, 2
    q = mole.QuantTable.quantize(lut.to(DEV), FMT[nbits], block)
    torch.cuda.synchronize()
    # the oracle's own quantiser and de-quantiser give the table the layer is defined over
    deq = quant.dequantize_table(quant.quantize_table(as_f64(lut).astype(np.float32), nbits, block), N, d, nbits, block)
    h64, w64 = as_f64(hidden), as_f64(wr)
    gamma = None
    router_in = h64
    if norm:
        gamma = (1.0 + 0.2 * torch.empty(d).normal_(0, 1, generator=torch.Generator().manual_seed(2))).to(torch.bfloat16)
        normed = np.stack([oracle.rmsnorm(h64[t], as_f64(gamma), 1e-5) for t in range(M)])
        router_in = as_f64(torch.from_numpy(normed).to(torch.bfloat16))
    ref, gref, bad = oracle.layer_lookup(router_in, ids.numpy(), deq, w64, residual=h64)
    assert bad == 0
    gates = torch.zeros(M, N, dtype=torch.float32, device=DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    out = mole.layer_forward(hidden.to(DEV), ids.to(DEV), q, wr.to(DEV), gates_out=gates, status=status, chain=True,
                             norm_weight=None if gamma is None else gamma.to(DEV), norm_eps=1e-5)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    gerr = np.abs(as_f64(gates) - gref)
    if norm:
        from gpu_util import near_tie_slack
        assert (gerr <= 1e-5 + near_tie_slack(normed, wr)[:, None]).all()
        slack = gerr.sum(axis=1, keepdims=True) * float(np.abs(deq).max())
    else:
        assert gerr.max() <= 1e-5
        slack = 0.0
    err = np.abs(as_f64(out) - ref)
    assert (err <= 1e-2 * np.maximum(1.0, np.abs(ref))).all()
    assert (err <= 2.0 ** -8 * np.abs(ref) + 2e-5 + slack).all(), float(err.max())


@pytest.mark.gpu
def test_quantised_layer_bad_ids_residual_and_step():
    nbits, block, M, N, d, V, L = 4, 768, 40, 16, 768, 50, 3
    g = torch.Generator().manual_seed(11)
    luts = torch.empty(L, V, N, d).normal_(0, 0.05, generator=g).to(torch.bfloat16)
    wrs = torch.empty(L, d, N).normal_(0, 0.02, generator=g).to(torch.bfloat16)
    hidden = torch.empty(M, d).normal_(0, 1, generator=g).to(torch.bfloat16)
    res = torch.empty(M, d).normal_(0, 1, generator=g).to(torch.bfloat16)
    ids = torch.randint(0, V, (M,), generator=g, dtype=torch.int32)
    ids[3], ids[9] = -1, V
    q = mole.QuantTable.quantize(luts.to(DEV), FMT[nbits], block)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    out = mole.layer_forward(hidden.to(DEV), ids.to(DEV), q.layer(0), wrs[0].to(DEV), residual=res.to(DEV), status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == mole.STATUS_BAD_ID
    assert np.array_equal(bits(out)[3], bits(res)[3]) and np.array_equal(bits(out)[9], bits(res)[9])
    deq0 = quant.dequantize_table(quant.quantize_table(as_f64(luts[0]).astype(np.float32), nbits, block), N, d, nbits, block)
    ref, _, bad = oracle.layer_lookup(as_f64(hidden), ids.numpy(), deq0, as_f64(wrs[0]), residual=as_f64(res))
    assert bad == 2
    err = np.abs(as_f64(out) - ref)
    assert (err <= 2.0 ** -8 * np.abs(ref) + 2e-5).all()
    # an L-layer step over quantised tables equals the single layers, one after the other
    ids2 = torch.randint(0, V, (M,), generator=g, dtype=torch.int32).to(DEV)
    status.zero_()
    hd = hidden.to(DEV)
    step = mole.decode_step_args(hd, ids2, q, wrs.to(DEV), torch.empty_like(hd), torch.empty_like(hd), status=status)
    h = hd
    for l in range(L):
        h = mole.layer_forward(h, ids2, q.layer(l), wrs[l].to(DEV))
    torch.cuda.synchronize()
    assert int(status.item()) == 0 and torch.equal(step, h)
    with pytest.raises(mole.MoleError) as e:  # quantised tables run layer by layer
        mole.decode_step_args(hd, ids2, q, wrs.to(DEV), torch.empty_like(hd), None, mode=mole.STEP_FUSED)
    assert e.value.code == mole.ERR_UNSUPPORTED_SHAPE


@pytest.mark.gpu
@pytest.mark.parametrize("nbits,block,M,cap", [(4, 1024, 8, 64), (3, 128, 8, 64), (4, 1024, 64, 64), (3, 128, 1, 256)])
def test_offload_over_quantised_host_tables_equals_the_resident_quantised_step(nbits, block, M, cap):
    """Offload mode with the host table quantised: only the distinct ids' packed records cross the host link,
    the layers de-quantise from the staging area.  Bitwise equal to the resident step over the same records."""
    from paper_2503_15798_b200 import inputs

    N, d, V, L = 16, 1024, 900, 5
    g = torch.Generator().manual_seed(3 + M)
    luts = torch.empty(L, V, N, d).normal_(0, 0.05, generator=g).to(torch.bfloat16).to(DEV)
    wrs = torch.empty(L, d, N).normal_(0, 0.02, generator=g).to(torch.bfloat16).to(DEV)
    hidden = torch.empty(M, d).normal_(0, 1, generator=g).to(torch.bfloat16).to(DEV)
    q = mole.QuantTable.quantize(luts, FMT[nbits], block)
    torch.cuda.synchronize()
    host = mole.HostTable(tuple(q.packed.shape), torch.uint8)
    ctx = mole.OffloadContext(max_tokens=cap, N=N, d=d, V=V, n_buffers=2, lut_format=FMT[nbits], lut_block=block)
    side = torch.cuda.Stream()
    try:
        host.tensor.copy_(q.packed)
        torch.cuda.synchronize()
        status = torch.zeros(1, dtype=torch.int32, device=DEV)
        for step in range(2):
            ids = torch.from_numpy(inputs.zipf_ids(M, V, seed=step)).to(DEV)
            if step == 1 and M > 2:
                ids[1] = V + 1
            out, tmp = torch.empty_like(hidden), torch.empty_like(hidden)
            ctx.decode_step(hidden, ids, host.tensor, wrs, out, tmp, status=status, side_stream=side)
            want = mole.decode_step_args(hidden, ids, q, wrs, torch.empty_like(hidden), torch.empty_like(hidden))
            torch.cuda.synchronize()
            assert torch.equal(out, want)
            # single layer through prefetch + forward
            one = torch.empty_like(hidden)
            ctx.prefetch(0, ids, host.tensor[2], side_stream=side)
            ctx.forward(0, hidden, wrs[2], one)
            torch.cuda.synchronize()
            assert torch.equal(one, mole.layer_forward(hidden, ids, q.layer(2), wrs[2]))
        assert int(status.item()) == (mole.STATUS_BAD_ID if M > 2 else 0)
    finally:
        ctx.destroy()
        host.free()
