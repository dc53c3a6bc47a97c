"""GPU parity: the fused sm_100a layer, through the C ABI, against the fp64 CPU oracle on the
same seeded inputs, element by element."""
import os

import numpy as np
import pytest
import torch

import oracle
from gpu_util import as_f64, bits, check_gates, check_out, oracle_layer, rand_case
from paper_2503_15798_b200 import binding as mole
from paper_2503_15798_b200 import inputs

pytestmark = pytest.mark.gpu
DEV = "cuda"


def run_gpu(hidden, ids, lut, wr, **kw):
    M, N = hidden.shape[0], lut.shape[1]
    gates = torch.zeros(M, N, dtype=torch.float32, device=DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    res = kw.pop("residual", None)
    out = mole.layer_forward(hidden.to(DEV), ids.to(DEV), lut.to(DEV), wr.to(DEV),
                             residual=None if res is None else res.to(DEV), gates_out=gates, status=status, **kw)
    torch.cuda.synchronize()
    return out, gates, int(status.item())


# ---- the tiny FFN-built configuration, fp32, both layers, every element ------------------------

def test_tiny_config_fp32_two_layers_every_element():
    m = inputs.tiny_model(seed=0)
    sh = m["shape"]
    h_gpu = torch.from_numpy(m["hidden"]).to(DEV)
    ids = torch.from_numpy(m["ids"])
    h_ref = m["hidden"]
    for l in range(sh.L):
        lut32 = oracle.build_lut(m["E"], m["W1"][l], m["W2"][l]).astype(np.float32)  # Eq. 6-7 on the CPU
        wr = m["Wr"][l]
        ref, gref, bad = oracle.layer_lookup(h_ref, m["ids"], lut32, wr)
        fly, _ = oracle.layer_onthefly(h_ref, m["ids"], m["E"], m["W1"][l], m["W2"][l], wr)
        out, gates, status = run_gpu(h_gpu, ids, torch.from_numpy(lut32), torch.from_numpy(wr), B=m["B"], T=m["T"])
        assert bad == 0 and status == 0
        check_out(out, ref, torch.float32)
        check_gates(gates, gref)
        # the lookup output equals the on-the-fly expert computation (Eq. 5 == Eq. 8)
        assert np.abs(as_f64(out) - fly).max() <= 1e-5
        h_gpu = out
        h_ref = out.cpu().numpy()  # feed the oracle the bytes the next GPU layer sees


# ---- bf16 parity over shapes and splits ---------------------------------------------------------------

CASES = [
    # M, N, d, V
    (1, 16, 768, 50),
    (7, 16, 768, 300),
    (64, 16, 768, 1000),
    (300, 16, 1024, 777),   # more tokens than 2 x 148 blocks: no split
    (33, 32, 2048, 129),    # 128 KB of rows per token: split 8
    (5, 4, 64, 20),
    (19, 8, 256, 64),
    (3, 64, 512, 10),
    (11, 3, 128, 40),       # N without an unrolled router: generic path
    (9, 33, 256, 30),
    (4, 1, 64, 8),
    (6, 12, 2560, 16),      # d-groups (320) beyond 256 threads: strided loops
    (1500, 16, 768, 900),   # more tokens than resident blocks: every block loops over several tokens
    (2100, 8, 256, 64),
]


@pytest.mark.parametrize("M,N,d,V", CASES)
def test_bf16_parity_auto_plan(M, N, d, V):
    hidden, ids, lut, wr = rand_case(M, N, d, V, seed=M * 1000 + N)
    ref, gref, _ = oracle_layer(hidden, ids, lut, wr)
    out, gates, status = run_gpu(hidden, ids, lut, wr)
    assert status == 0
    check_out(out, ref)
    check_gates(gates, gref)


@pytest.mark.parametrize("split", [1, 2, 4, 8, 16])
@pytest.mark.parametrize("N,d", [(16, 768), (32, 2048), (5, 512), (4, 64), (8, 256), (64, 512)])
def test_bf16_parity_every_split(split, N, d):
    if d % (split * 8) != 0:
        pytest.skip("column slice would not be a whole number of 16-byte vectors")
    M, V = 37, 211
    try:
        mole.plan(M, N, d, mole.DTYPE_BF16, split)
    except mole.MoleError as e:  # two ring slots of this split do not fit in shared memory
        assert e.code == mole.ERR_UNSUPPORTED_SHAPE and N * (d // split) * 2 * 2 + d * N * 2 > 200 * 1024
        pytest.skip("this split does not fit")
    hidden, ids, lut, wr = rand_case(M, N, d, V, seed=d + N + split)
    ref, gref, _ = oracle_layer(hidden, ids, lut, wr)
    out, gates, status = run_gpu(hidden, ids, lut, wr, d_split=split)
    assert status == 0
    check_out(out, ref)
    check_gates(gates, gref)


def test_fp32_parity_splits():
    M, N, d, V = 21, 8, 256, 50
    hidden, ids, lut, wr = rand_case(M, N, d, V, seed=5, dtype=torch.float32)
    ref, gref, _ = oracle.layer_lookup(hidden.numpy(), ids.numpy(), lut.numpy(), wr.numpy())
    for split in (0, 1, 2, 4, 8):
        out, gates, status = run_gpu(hidden, ids, lut, wr, d_split=split)
        assert status == 0
        check_out(out, ref, torch.float32)
        check_gates(gates, gref)


def test_larger_router_logits_keep_gate_accuracy():
    # router weights 10x the workload's: logits of order 5-10, sharply peaked softmax
    M, N, d, V = 50, 16, 768, 64
    hidden, ids, lut, wr = rand_case(M, N, d, V, seed=77, wr_std=0.2)
    ref, gref, _ = oracle_layer(hidden, ids, lut, wr)
    out, gates, _ = run_gpu(hidden, ids, lut, wr)
    check_out(out, ref)
    check_gates(gates, gref)
    assert gref.max() > 0.9


# ---- the gather is bit-exact ---------------------------------------------------------------------

def _one_hot_inputs(M, N, d, jstar, c0):
    hidden = torch.zeros(M, d, dtype=torch.bfloat16)
    hidden[:, c0] = 1.0
    wr = torch.zeros(d, N, dtype=torch.bfloat16)
    wr[c0, jstar] = 256.0  # logit gap 256: exp underflows to 0 in fp32, gates are exactly one-hot
    return hidden, wr


def _encoded_table_bits(V, N, d, kind):
    i = np.arange(V, dtype=np.int64)[:, None, None]
    j = np.arange(N, dtype=np.int64)[None, :, None]
    c = np.arange(d, dtype=np.int64)[None, None, :]
    if kind == "hash":
        x = (i * 0x9E3779B1 + j * 0x85EBCA6B + c * 0xC2B2AE35 + 0x27D4EB2F) & 0xFFFFFFFF
        x ^= x >> 15
        x = (x * 0x2C1B3C6D) & 0xFFFFFFFF
        x ^= x >> 12
        b = (x & 0xFFFF).astype(np.uint16)
        expo = ((b >> 7) & 0xFF).astype(np.int64)
        expo = 1 + expo % 254  # finite, normal: no zero / denormal / inf / nan patterns
        return ((b & 0x807F) | (expo.astype(np.uint16) << 7)).astype(np.uint16)
    vals = {"id_lo": i % 256, "id_hi": i // 256, "expert": j, "col_lo": c % 256, "col_hi": c // 256}[kind]
    vals = np.broadcast_to(vals, (V, N, d)).astype(np.float32) + 1.0  # 1..257, exact in bf16
    return (np.ascontiguousarray(vals).view(np.uint32) >> 16).astype(np.uint16)


@pytest.mark.parametrize("kind", ["hash", "id_lo", "id_hi", "expert", "col_lo", "col_hi"])
@pytest.mark.parametrize("N,d,split", [(16, 768, 0), (16, 768, 4), (16, 768, 1), (32, 2048, 0), (5, 512, 2)])
def test_gather_bit_exact_with_one_hot_gates(kind, N, d, split):
    V, M = 300, 40
    tb = _encoded_table_bits(V, N, d, kind)
    lut = torch.from_numpy(tb.view(np.int16)).view(torch.bfloat16)
    ids = torch.from_numpy(np.random.default_rng(1).integers(0, V, M).astype(np.int32))
    ids[0], ids[1] = 0, V - 1
    zeros = torch.zeros(M, d, dtype=torch.bfloat16)
    for jstar in sorted({0, N // 2, N - 1}):
        hidden, wr = _one_hot_inputs(M, N, d, jstar, c0=(3 * jstar + 1) % d)
        out, gates, status = run_gpu(hidden, ids, lut, wr, residual=zeros, d_split=split)
        want_g = np.zeros((M, N), dtype=np.float32)
        want_g[:, jstar] = 1.0
        assert np.array_equal(gates.cpu().numpy(), want_g)
        assert np.array_equal(bits(out), tb[ids.numpy(), jstar, :])  # raw uint16 equality, every column


def test_gather_bit_exact_fp32_table_encoding_id_expert_column():
    sh = inputs.SHAPES["tiny"]
    V, N, d, M = sh.V, sh.N, sh.d, 64
    table = ((np.arange(V)[:, None, None] * N + np.arange(N)[None, :, None]) * d + np.arange(d)[None, None, :])
    assert table.max() < 2 ** 24
    lut = torch.from_numpy(table.astype(np.float32))
    ids = torch.from_numpy(inputs.uniform_ids(M, V, seed=3))
    for jstar in range(N):
        hidden = torch.zeros(M, d)
        hidden[:, 7] = 1.0
        wr = torch.zeros(d, N)
        wr[7, jstar] = 256.0
        out, gates, _ = run_gpu(hidden, ids, lut, wr, residual=torch.zeros(M, d))
        assert np.array_equal(out.cpu().numpy(), table[ids.numpy(), jstar, :].astype(np.float32))


# ---- properties that hold at any size -----------------------------------------------------------------

def test_zero_table_returns_hidden_bitwise_and_equal_rows_ignore_router():
    M, N, d, V = 30, 16, 768, 40
    hidden, ids, lut, wr = rand_case(M, N, d, V, seed=9)
    out, _, _ = run_gpu(hidden, ids, torch.zeros_like(lut), wr)
    assert np.array_equal(bits(out), bits(hidden))
    same = lut[:, :1, :].expand(V, N, d).contiguous()
    ref, _, _ = oracle_layer(hidden, ids, same, wr)
    out, _, _ = run_gpu(hidden, ids, same, wr)
    check_out(out, ref)
    check_out(out, as_f64(hidden) + as_f64(same[ids.long(), 0, :]))


def test_zero_router_gives_uniform_gates_exactly():
    M, N, d, V = 10, 16, 768, 20
    hidden, ids, lut, wr = rand_case(M, N, d, V, seed=10)
    out, gates, _ = run_gpu(hidden, ids, lut, torch.zeros_like(wr))
    assert np.array_equal(gates.cpu().numpy(), np.full((M, N), 1.0 / N, dtype=np.float32))
    check_out(out, as_f64(hidden) + as_f64(lut[ids.long()]).mean(axis=1))


def test_token_permutation_and_batch_size_do_not_change_a_token():
    M, N, d, V = 96, 16, 768, 500
    hidden, ids, lut, wr = rand_case(M, N, d, V, seed=11, ids_kind="zipf")
    lut_d, wr_d = lut.to(DEV), wr.to(DEV)
    base = mole.layer_forward(hidden.to(DEV), ids.to(DEV), lut_d, wr_d, d_split=2)
    perm = torch.randperm(M, generator=torch.Generator().manual_seed(1))
    permuted = mole.layer_forward(hidden[perm].to(DEV), ids[perm].to(DEV), lut_d, wr_d, d_split=2)
    assert torch.equal(permuted, base[perm.to(DEV)])
    for t in (0, 17, 95):  # the same token alone, same launch shape
        one = mole.layer_forward(hidden[t:t + 1].to(DEV), ids[t:t + 1].to(DEV), lut_d, wr_d,
                                 d_split=2)
        assert torch.equal(one[0], base[t])
    again = mole.layer_forward(hidden.to(DEV), ids.to(DEV), lut_d, wr_d, d_split=2)
    assert torch.equal(again, base)  # run-to-run deterministic


def test_expert_permutation_changes_nothing_beyond_rounding():
    M, N, d, V = 20, 16, 768, 64
    hidden, ids, lut, wr = rand_case(M, N, d, V, seed=12)
    perm = torch.randperm(N, generator=torch.Generator().manual_seed(2))
    ref, _, _ = oracle_layer(hidden, ids, lut, wr)
    out, _, _ = run_gpu(hidden, ids, lut[:, perm, :].contiguous(), wr[:, perm].contiguous())
    check_out(out, ref)


def test_in_place_output_and_separate_residual():
    M, N, d, V = 70, 16, 768, 90
    hidden, ids, lut, wr = rand_case(M, N, d, V, seed=13)
    ref, _, _ = oracle_layer(hidden, ids, lut, wr)
    for split in (0, 1, 2, 4):
        h = hidden.to(DEV).clone()
        out = mole.layer_forward(h, ids.to(DEV), lut.to(DEV), wr.to(DEV), out=h, d_split=split)
        torch.cuda.synchronize()
        assert out.data_ptr() == h.data_ptr()
        check_out(h, ref)
    res = torch.empty(M, d).normal_(0, 1, generator=torch.Generator().manual_seed(3)).to(torch.bfloat16)
    ref_r, _, _ = oracle_layer(hidden, ids, lut, wr, residual=res)
    out, _, _ = run_gpu(hidden, ids, lut, wr, residual=res)
    check_out(out, ref_r)


def test_int64_ids_and_basic_entry_point_agree():
    M, N, d, V = 40, 16, 768, 1000
    hidden, ids, lut, wr = rand_case(M, N, d, V, seed=14)
    a = mole.layer_forward(hidden.to(DEV), ids.to(DEV), lut.to(DEV), wr.to(DEV))
    b = mole.layer_forward(hidden.to(DEV), ids.to(DEV).long(), lut.to(DEV), wr.to(DEV))
    c = torch.empty_like(a)
    mole.layer_forward_basic(hidden.to(DEV), ids.to(DEV), lut.to(DEV), wr.to(DEV), c)
    torch.cuda.synchronize()
    assert torch.equal(a, b) and torch.equal(a, c)


def test_bad_ids_leave_the_residual_and_raise_the_status_bit():
    M, N, d, V = 12, 16, 768, 30
    hidden, ids, lut, wr = rand_case(M, N, d, V, seed=15)
    ids[3], ids[8] = -1, V
    ref, gref, bad = oracle_layer(hidden, ids, lut, wr)
    assert bad == 2
    for split in (0, 1, 2):
        out, gates, status = run_gpu(hidden, ids, lut, wr, d_split=split)
        assert status & mole.STATUS_BAD_ID and not status & mole.STATUS_TIMEOUT
        check_out(out, ref)
        assert np.array_equal(bits(out)[3], bits(hidden)[3]) and np.array_equal(bits(out)[8], bits(hidden)[8])
        check_gates(gates, gref)


def test_zero_tokens_is_a_no_op():
    N, d, V = 16, 768, 10
    _, _, lut, wr = rand_case(1, N, d, V, seed=16)
    hidden = torch.empty(0, d, dtype=torch.bfloat16, device=DEV)
    ids = torch.empty(0, dtype=torch.int32, device=DEV)
    out = mole.layer_forward(hidden, ids, lut.to(DEV), wr.to(DEV))
    assert out.shape == (0, d)


def test_maximum_sizes_N64_and_wide_d():
    M, N, d, V = 9, 64, 4096, 12  # 512 KB of rows per token: only fits when split
    hidden, ids, lut, wr = rand_case(M, N, d, V, seed=17)
    ref, gref, _ = oracle_layer(hidden, ids, lut, wr)
    out, gates, status = run_gpu(hidden, ids, lut, wr)
    assert status == 0
    check_out(out, ref)
    check_gates(gates, gref)


@pytest.mark.parametrize("M,N,d,split", [(37, 64, 1024, 4), (37, 64, 1024, 16), (21, 64, 4096, 8), (21, 64, 4096, 16),
                                         (70, 32, 2048, 2), (301, 32, 2048, 4)])
def test_rows_cut_by_experts_single_layer(M, N, d, split):
    """Router matrices too large to stay resident travel through the ring; with several chunks per
    item the rows then arrive as whole rows of N / split experts: one, two and four column groups
    per lane, chunks of more and of fewer experts than one load batch."""
    hidden, ids, lut, wr = rand_case(M, N, d, 50, seed=M + N + split)
    ref, gref, _ = oracle_layer(hidden, ids, lut, wr)
    out, gates, status = run_gpu(hidden, ids, lut, wr, d_split=split)
    assert status == 0
    check_out(out, ref)
    check_gates(gates, gref)
    with mole.debug_env(MOLE_FORCE_COLUMN_CHUNKS=1):  # the same launch with the rows cut by columns
        out2, gates2, status2 = run_gpu(hidden, ids, lut, wr, d_split=split)
    assert status2 == 0
    check_out(out2, ref)
    check_gates(gates2, gref)


# ---- chained layers ------------------------------------------------------------------------------

def _step_case(M, N, d, L, V=400):
    g = torch.Generator().manual_seed(M + L)
    luts = torch.empty(L, V, N, d).normal_(0, 0.05, generator=g).to(torch.bfloat16).to(DEV)
    wrs = torch.empty(L, d, N).normal_(0, 0.02, generator=g).to(torch.bfloat16).to(DEV)
    hidden = torch.empty(M, d).normal_(0, 1, generator=g).to(torch.bfloat16).to(DEV)
    ids = torch.from_numpy(inputs.zipf_ids(M, V, seed=4)).to(DEV)
    return luts, wrs, hidden, ids


@pytest.mark.parametrize("M,N,d,L,split", [(64, 16, 768, 5, 1), (64, 16, 768, 5, 2), (3, 16, 1024, 4, 4), (40, 32, 2048, 3, 8),
                                           (300, 16, 768, 2, 1), (8, 4, 64, 1, 1), (9, 5, 512, 3, 2), (700, 8, 256, 3, 1),
                                           (1300, 16, 768, 2, 2)])
def test_decode_step_fused_and_chained_equal_layer_after_layer(M, N, d, L, split):
    luts, wrs, hidden, ids = _step_case(M, N, d, L)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    keep = hidden.clone()
    fused = mole.decode_step(hidden, ids, luts, wrs, torch.empty_like(hidden), None, status=status,
                             mode=mole.STEP_FUSED, d_split=split)
    chained = mole.decode_step(hidden, ids, luts, wrs, torch.empty_like(hidden), torch.empty_like(hidden), status=status,
                               mode=mole.STEP_CHAINED, d_split=split)
    h = hidden
    for l in range(L):  # single layers, each checked against the oracle
        ref, _, _ = oracle_layer(h, ids, luts[l], wrs[l])
        h = mole.layer_forward(h, ids, luts[l], wrs[l], d_split=split)
        check_out(h, ref)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    assert torch.equal(chained, h)  # one launch per layer, chained or not: the same bits
    # The fused launch sums an item's experts in the same order as the single layers when the rows
    # arrive cut by columns (always with one chunk); cut by experts (several chunks, bf16, K | N) the
    # order of the fp32 sum differs, and with it now and then a rounding decision.
    with mole.debug_env(MOLE_FORCE_COLUMN_CHUNKS=1):
        by_columns = mole.decode_step(hidden, ids, luts, wrs, torch.empty_like(hidden), None, status=status,
                                      mode=mole.STEP_FUSED, d_split=split)
        torch.cuda.synchronize()
    assert torch.equal(by_columns, h)
    if split == 1:
        assert torch.equal(fused, h)
    else:
        err = np.abs(as_f64(fused) - as_f64(h))
        assert (err <= L * 2.0 ** -7 * np.maximum(1.0, np.abs(as_f64(h)))).all(), float(err.max())
    assert int(status.item()) == 0
    assert torch.equal(hidden, keep)  # the input is never written


@pytest.mark.parametrize("M,N,d,L", [(64, 16, 768, 12), (256, 16, 1024, 6), (16, 32, 2048, 4), (1, 16, 768, 12)])
def test_decode_step_auto_plan_against_the_oracle_chain(M, N, d, L):
    luts, wrs, hidden, ids = _step_case(M, N, d, L, V=300)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    out = mole.decode_step_basic(hidden, ids, luts, wrs, torch.empty_like(hidden), torch.empty_like(hidden), status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    # the oracle, layer after layer, each layer fed the storage-type rounding of the previous one
    h = hidden
    for l in range(L):
        ref, _, _ = oracle_layer(h, ids, luts[l], wrs[l])
        h = torch.from_numpy(ref).to(torch.bfloat16)
    # rounding decisions may differ from the oracle's by one ulp per layer and then propagate
    err = np.abs(as_f64(out) - as_f64(h))
    assert (err <= L * 2.0 ** -7 * np.maximum(1.0, np.abs(as_f64(h)))).all(), float(err.max())


def test_decode_step_fused_in_place_and_bad_ids():
    M, N, d, L = 50, 16, 768, 4
    luts, wrs, hidden, ids = _step_case(M, N, d, L)
    ids[7], ids[31] = -2, 400
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    want = mole.decode_step(hidden, ids, luts, wrs, torch.empty_like(hidden), torch.empty_like(hidden), status=status,
                            mode=mole.STEP_CHAINED, d_split=1)
    h = hidden.clone()
    mole.decode_step(h, ids, luts, wrs, h, None, status=status, mode=mole.STEP_FUSED, d_split=1)
    torch.cuda.synchronize()
    assert int(status.item()) == mole.STATUS_BAD_ID
    assert torch.equal(h, want)
    assert torch.equal(h[7], hidden[7]) and torch.equal(h[31], hidden[31])  # no routed term in any layer


@pytest.mark.parametrize("pinned", [True, False])
def test_decode_step_host_round_trip(pinned):
    """Pinned, mapped host buffers: the launch reads and writes them itself and leaves the device buffers alone;
    pageable ones: staged through the device buffers.  The same bits either way."""
    M, N, d, L, V = 64, 16, 768, 4, 300
    g = torch.Generator().manual_seed(5)
    luts = torch.empty(L, V, N, d).normal_(0, 0.05, generator=g).to(torch.bfloat16).to(DEV)
    wrs = torch.empty(L, d, N).normal_(0, 0.02, generator=g).to(torch.bfloat16).to(DEV)
    h_host = torch.empty(M, d).normal_(0, 1, generator=g).to(torch.bfloat16)
    ids_host = torch.from_numpy(inputs.zipf_ids(M, V, seed=6))
    out_host = torch.empty_like(h_host)
    if pinned:
        h_host, ids_host, out_host = h_host.pin_memory(), ids_host.pin_memory(), out_host.pin_memory()
    dev = [torch.full((M, d), 777.0, dtype=torch.bfloat16, device=DEV) for _ in range(3)]
    dev_ids = torch.full((M,), -5, dtype=torch.int32, device=DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    mole.decode_step_host(h_host, ids_host, out_host, dev[0], dev_ids, dev[1], dev[2], luts, wrs, status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    want = torch.empty(M, d, dtype=torch.bfloat16, device=DEV)
    mole.decode_step(h_host.to(DEV), ids_host.to(DEV), luts, wrs, want, torch.empty_like(want))
    torch.cuda.synchronize()
    assert torch.equal(out_host, want.cpu())
    untouched = bool((dev[0] == 777.0).all()) and bool((dev_ids == -5).all())
    assert untouched == pinned


@pytest.mark.parametrize("wide", [False, True])
def test_prefetch_rows_is_a_hint(wide):
    """mole_prefetch_rows before a step: the same bits as without it; ids outside the table are skipped (the
    layer reports them as before); int64 ids."""
    M, N, d, L, V = (40, 32, 2048, 2, 50) if wide else (70, 16, 768, 3, 300)
    g = torch.Generator().manual_seed(9)
    luts = torch.empty(L, V, N, d).normal_(0, 0.05, generator=g).to(torch.bfloat16).to(DEV)
    wrs = torch.empty(L, d, N).normal_(0, 0.02, generator=g).to(torch.bfloat16).to(DEV)
    hidden = torch.empty(M, d).normal_(0, 1, generator=g).to(torch.bfloat16).to(DEV)
    ids = torch.randint(0, V, (M,), generator=g, dtype=torch.int32)
    ids[3], ids[M - 1] = -1, V + 5
    ids = ids.to(DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    want = mole.decode_step(hidden, ids, luts, wrs, torch.empty_like(hidden), torch.empty_like(hidden), status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == mole.STATUS_BAD_ID
    mole.prefetch_rows(ids, luts)
    mole.prefetch_rows(ids.to(torch.int64), luts, layers=1, first_layer=L - 1)
    got = mole.decode_step(hidden, ids, luts, wrs, torch.empty_like(hidden), torch.empty_like(hidden), status=status)
    torch.cuda.synchronize()
    assert torch.equal(got, want)
