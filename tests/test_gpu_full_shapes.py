"""Parity at the full workload shapes (160M / 410M / 1B-shaped tables, Zipf ids), in the launch
configuration the bench times.  One layer's table is generated on the device; the rows the batch
references are copied back with a plain index and handed to the oracle as a compact table, so the
oracle sees exactly the bytes the kernel gathered."""
import numpy as np
import pytest
import torch

import oracle
from gpu_util import bits, check_gates, check_out
from paper_2503_15798_b200 import binding as mole
from paper_2503_15798_b200 import inputs

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _oracle_on_compact_rows(hidden, ids, lut, wr, sample):
    ids_s = ids[sample].cpu().numpy()
    uniq, inv = np.unique(ids_s, return_inverse=True)
    rows = lut[torch.from_numpy(uniq).long().to(lut.device)].cpu()  # plain torch index, shares nothing with the kernel
    out, gates, bad = oracle.layer_lookup(bits(hidden[sample]), inv, bits(rows), bits(wr))
    assert bad == 0
    return out, gates


@pytest.mark.parametrize("name,batches,n_sample", [
    ("160m", (1, 8, 64, 256), 256),
    ("410m", (1, 64, 256, 16384), 256),
    ("1b", (1, 16, 64, 256), 64),
])
def test_full_shape_layer_against_oracle(name, batches, n_sample):
    sh = inputs.SHAPES[name]
    lut = inputs.make_table(sh.V, sh.N, sh.d, seed=7, device=DEV)
    wr = inputs.make_router(sh.d, sh.N, seed=8, device=DEV)
    for M in batches:
        hidden = inputs.make_hidden(M, sh.d, seed=M, device=DEV)
        ids = inputs.make_ids(M, sh.V, seed=M + 1, device=DEV)
        gates = torch.empty(M, sh.N, dtype=torch.float32, device=DEV)
        status = torch.zeros(1, dtype=torch.int32, device=DEV)
        out = mole.layer_forward(hidden, ids, lut, wr, gates_out=gates, status=status, chain=True)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        sample = torch.from_numpy(np.sort(np.random.default_rng(M).permutation(M)[:n_sample])).to(DEV)
        ref, gref = _oracle_on_compact_rows(hidden, ids, lut, wr, sample)
        check_out(out[sample], ref)
        check_gates(gates[sample], gref)
        # token independence at full size: the sampled tokens alone give the same bytes
        if M > 1:  # ... in the same kernel family and launch shape
            if mole.variant(M, sh.N, sh.d)[0].startswith("decode"):
                how = {"kernel": mole.KERNEL_DECODE}
            else:
                how = {"kernel": mole.KERNEL_RING, "d_split": mole.plan(M, sh.N, sh.d)[0]}
            alone = mole.layer_forward(hidden[sample].contiguous(), ids[sample].contiguous(), lut, wr, **how)
            assert torch.equal(alone, out[sample])
    del lut


def test_last_row_of_a_table_beyond_4GiB_is_addressed_correctly():
    # 1B-shaped layer: 6.6 GB, row offsets overflow 32 bits
    sh = inputs.SHAPES["1b"]
    lut = torch.zeros(sh.V, sh.N, sh.d, dtype=torch.bfloat16, device=DEV)
    marks = {0: 1.0, 32767: 2.0, 32768: 3.0, sh.V - 1: 4.0}  # 32768 * 131072 B = 4 GiB exactly
    for row, v in marks.items():
        lut[row] = v
    ids = torch.tensor(list(marks), dtype=torch.int32, device=DEV)
    hidden = torch.zeros(len(marks), sh.d, dtype=torch.bfloat16, device=DEV)
    wr = torch.zeros(sh.d, sh.N, dtype=torch.bfloat16, device=DEV)
    out = mole.layer_forward(hidden, ids, lut, wr)
    torch.cuda.synchronize()
    for k, v in enumerate(marks.values()):  # uniform gates over equal rows: out == the mark exactly
        assert (out[k].float() == v).all()


@pytest.mark.parametrize("name,M,n_sample", [("160m", 256, 96), ("410m", 256, 64), ("1b", 256, 48), ("1b", 64, 32)])
def test_full_shape_decode_step_chained_and_fused(name, M, n_sample):
    """Three layers of the full-size tables as the bench launches them (chained with programmatic
    dependent launch, and the single fused launch): sampled tokens against the oracle's chain on the
    rows they reference."""
    sh = inputs.SHAPES[name]
    L = 3
    luts = torch.empty((L, sh.V, sh.N, sh.d), dtype=torch.bfloat16, device=DEV)
    for l in range(L):
        inputs.make_table(sh.V, sh.N, sh.d, seed=20 + l, device=DEV, out=luts[l])
    wrs = torch.stack([inputs.make_router(sh.d, sh.N, seed=30 + l, device=DEV) for l in range(L)])
    hidden = inputs.make_hidden(M, sh.d, seed=5, device=DEV)
    ids = inputs.make_ids(M, sh.V, seed=6, device=DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    sample = torch.from_numpy(np.sort(np.random.default_rng(1).permutation(M)[:n_sample])).to(DEV)
    h = hidden[sample].contiguous()
    ids_s = ids[sample].contiguous()
    everyone = torch.arange(n_sample, device=DEV)
    for l in range(L):  # the oracle's chain, each layer fed the storage-type rounding of the previous one
        ref, _ = _oracle_on_compact_rows(h, ids_s, luts[l], wrs[l], everyone)
        h = torch.from_numpy(ref).to(torch.bfloat16).to(DEV)
    want = h.cpu().to(torch.float64).numpy()
    for mode in (mole.STEP_CHAINED, mole.STEP_FUSED):
        out = mole.decode_step(hidden, ids, luts, wrs, torch.empty_like(hidden), torch.empty_like(hidden), status=status, mode=mode)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        got = out[sample].cpu().to(torch.float64).numpy()
        assert (np.abs(got - want) <= L * 2.0 ** -7 * np.maximum(1.0, np.abs(want))).all(), mode
    del luts
