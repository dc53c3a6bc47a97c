"""Pins for the CPU oracle: facts fixed by the paper or by mathematics, none of them
computed by the oracle itself.  Each pin is a function that raises AssertionError when the
oracle (``import oracle``) violates it.  ``test_oracle_pins.py`` runs them on the real
oracle; ``test_oracle_mutants.py`` runs them on deliberately broken copies and requires a
failure, which shows that a dropped term, a wrong sign or a transposed operand is caught.
"""
from __future__ import annotations

import math
import os

import numpy as np

import oracle

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")


def _golden_rows(name):
    rows = []
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            line = line.strip()
            if line and not line.startswith("#"):
                rows.append([c.strip() for c in line.split("|")])
    return rows


def _phi(x):
    """Standard normal CDF from scipy (a routine the oracle does not call)."""
    from scipy.stats import norm

    return float(norm.cdf(x))


# ---- FFN (Sec. 3.2 experts; Table 1 parameter / FLOP counts) -------------------------------

def pin_gelu_is_x_times_normal_cdf():
    for x in (-3.0, -1.0, -0.25, 0.0, 0.5, 1.0, 2.5):
        assert abs(oracle.gelu(x) - x * _phi(x)) < 1e-15, x
    # textbook values: Phi(1) = 0.8413447460685429
    assert abs(oracle.gelu(1.0) - 0.8413447460685429) < 1e-15
    assert abs(oracle.gelu(-1.0) + 0.15865525393145707) < 1e-15
    assert oracle.gelu(0.0) == 0.0
    # gelu(x) - gelu(-x) = x
    assert abs(oracle.gelu(1.7) - oracle.gelu(-1.7) - 1.7) < 1e-15


def pin_ffn_hand_worked():
    # d = 2, D = 3.  W1 rows pick x0, x1 and x0 + x1; W2 is not symmetric in any sense.
    x = np.array([1.0, -1.0])
    W1 = np.array([[1.0, 0.0], [0.0, 1.0], [1.0, 1.0]])  # [D][d] -> pre-activations (1, -1, 0)
    W2 = np.array([[1.0, 2.0, 5.0], [3.0, 4.0, 7.0]])  # [d][D]
    a0, a1 = 1.0 * _phi(1.0), -1.0 * _phi(-1.0)  # gelu(1), gelu(-1); gelu(0) = 0
    want = np.array([1.0 * a0 + 2.0 * a1, 3.0 * a0 + 4.0 * a1])
    got = oracle.ffn(x, W1, W2)
    assert np.allclose(got, want, rtol=0, atol=1e-15), (got, want)


def pin_ffn_linear_regime_matches_matmul():
    # for large positive pre-activations gelu(s) == s to fp64, so FFN(x) == W2 @ (W1 @ x)
    rng = np.random.default_rng(1)
    d, D = 5, 7
    W1 = rng.uniform(20.0, 30.0, size=(D, d))
    W2 = rng.standard_normal((d, D))
    x = rng.uniform(1.0, 2.0, size=d)
    want = W2 @ (W1 @ x)
    assert np.allclose(oracle.ffn(x, W1, W2), want, rtol=1e-13, atol=0)


def pin_rmsnorm_closed_form():
    x = np.array([3.0, 4.0])  # mean square 12.5
    w = np.array([2.0, 0.5])
    got = oracle.rmsnorm(x, w, 0.0)
    assert np.allclose(got, [3.0 / math.sqrt(12.5) * 2.0, 4.0 / math.sqrt(12.5) * 0.5], atol=1e-15)
    got = oracle.rmsnorm(x, w, 3.5)  # 12.5 + 3.5 = 16
    assert np.allclose(got, [3.0 / 4.0 * 2.0, 4.0 / 4.0 * 0.5], atol=1e-15)


# ---- router (Eq. 4) --------------------------------------------------------------------------

def pin_worked_example_gates_and_output():
    rows = {r[0]: [float(v) for v in r[1:]] for r in _golden_rows("worked_layer_example.txt")}
    h = np.array([[1.0, 2.0], [1.0, 2.0]])
    Wr = np.array([[math.log(3.0), math.log(2.0)], [math.log(2.0) / 2.0, 0.0]])
    lut = np.zeros((3, 2, 2))
    lut[1] = [[10.0, 20.0], [30.0, 40.0]]
    lut[2] = [[-4.0, 8.0], [12.0, -16.0]]
    out, gates, bad = oracle.layer_lookup(h, np.array([1, 2]), lut, Wr)
    assert bad == 0
    assert np.allclose(gates[0], rows["gates"], atol=1e-15)
    assert np.allclose(oracle.router_gates(h[0], Wr), rows["gates"], atol=1e-15)
    assert np.allclose(out[0], rows["out_id1"], atol=1e-13)
    assert np.allclose(out[1], rows["out_id2"], atol=1e-13)


def pin_softmax_invariants():
    rng = np.random.default_rng(2)
    d, N = 12, 7
    h = rng.standard_normal(d)
    Wr = rng.standard_normal((d, N))
    g = oracle.router_gates(h, Wr)
    assert abs(g.sum() - 1.0) < 1e-15 and (g > 0).all()
    # adding the same vector u to every router column shifts all logits equally
    u = rng.standard_normal(d)
    g2 = oracle.router_gates(h, Wr + u[:, None])
    assert np.allclose(g, g2, atol=1e-14)
    # large logits must not overflow
    g3 = oracle.router_gates(h * 1e4, Wr)
    assert np.isfinite(g3).all() and abs(g3.sum() - 1.0) < 1e-15
    # all experts stay active: no top-k truncation
    assert (oracle.router_gates(h, 0.01 * Wr) > 0.5 / N).all()


def pin_router_matches_library_softmax_of_matmul():
    from scipy.special import softmax

    rng = np.random.default_rng(3)
    d, N = 16, 5
    h = rng.standard_normal(d)
    Wr = rng.standard_normal((d, N))  # [d][N]: logits = h @ Wr
    assert np.allclose(oracle.router_gates(h, Wr), softmax(h @ Wr), atol=1e-14)


def pin_zero_router_gives_mean_of_rows():
    rng = np.random.default_rng(4)
    M, d, N, V = 5, 6, 4, 9
    h = rng.standard_normal((M, d))
    lut = rng.standard_normal((V, N, d))
    ids = rng.integers(0, V, M)
    out, gates, _ = oracle.layer_lookup(h, ids, lut, np.zeros((d, N)))
    assert np.array_equal(gates, np.full((M, N), 1.0 / N))
    assert np.allclose(out, h + lut[ids].mean(axis=1), atol=1e-14)


def pin_single_expert_is_plain_lookup_plus_residual():
    rng = np.random.default_rng(5)
    M, d, V = 4, 3, 6
    h = rng.standard_normal((M, d))
    lut = rng.standard_normal((V, 1, d))
    ids = np.array([5, 0, 3, 3])
    out, gates, _ = oracle.layer_lookup(h, ids, lut, rng.standard_normal((d, 1)))
    assert np.array_equal(gates, np.ones((M, 1)))
    assert np.array_equal(out, h + lut[ids, 0])


# ---- gather (Eq. 6-7 layout [V][N][d]; Eq. 14 rows per token) ------------------------------------

def pin_one_hot_gather_is_exact():
    # hidden has one non-zero column c0; W_r[c0][j*] is huge, so exp() of every other logit
    # underflows to 0 and g == e_{j*} exactly: out[c] == LUT[id][j*][c] bit for bit for c != c0.
    M, d, N, V = 6, 8, 5, 11
    lut = np.empty((V, N, d))
    for i in range(V):
        for j in range(N):
            for c in range(d):
                lut[i, j, c] = (i * N + j) * d + c  # encodes (id, expert, column)
    ids = np.array([10, 0, 3, 7, 7, 1])
    for jstar in range(N):
        for c0 in (0, 5):
            h = np.zeros((M, d))
            h[:, c0] = 1.0
            Wr = np.zeros((d, N))
            Wr[c0, jstar] = 2000.0
            out, gates, _ = oracle.layer_lookup(h, ids, lut, Wr)
            onehot = np.zeros(N)
            onehot[jstar] = 1.0
            assert np.array_equal(gates, np.tile(onehot, (M, 1)))
            cols = [c for c in range(d) if c != c0]
            assert np.array_equal(out[:, cols], lut[ids, jstar][:, cols])


def pin_combine_matches_embedding_bag():
    # Eq. 8's routed term is a per-sample-weighted embedding bag over the table viewed as
    # [V*N][d] with indices id*N + j; torch's CPU routine is an independent implementation.
    import torch
    from scipy.special import softmax

    rng = np.random.default_rng(6)
    M, d, N, V = 7, 10, 6, 13
    h = rng.standard_normal((M, d))
    Wr = rng.standard_normal((d, N))
    lut = rng.standard_normal((V, N, d))
    ids = rng.integers(0, V, M)
    g = softmax(h @ Wr, axis=1)
    idx = torch.from_numpy(ids[:, None] * N + np.arange(N)[None, :])
    bag = torch.nn.functional.embedding_bag(idx, torch.from_numpy(lut.reshape(V * N, d)),
                                            per_sample_weights=torch.from_numpy(g), mode="sum")
    out, gates, _ = oracle.layer_lookup(h, ids, lut, Wr)
    assert np.allclose(gates, g, atol=1e-14)
    assert np.allclose(out, h + bag.numpy(), atol=1e-13)


def pin_separate_residual_and_zero_table():
    rng = np.random.default_rng(7)
    M, d, N, V = 3, 4, 3, 5
    h = rng.standard_normal((M, d))
    r = rng.standard_normal((M, d))
    Wr = rng.standard_normal((d, N))
    ids = np.array([0, 4, 2])
    out, _, _ = oracle.layer_lookup(h, ids, np.zeros((V, N, d)), Wr)
    assert np.array_equal(out, h)  # zero table: out == hidden exactly
    lut = rng.standard_normal((V, N, d))
    out_h, _, _ = oracle.layer_lookup(h, ids, lut, Wr)
    out_r, _, _ = oracle.layer_lookup(h, ids, lut, Wr, residual=r)
    assert np.allclose(out_r - r, out_h - h, atol=1e-14)  # router still reads hidden


def pin_equal_rows_make_router_irrelevant():
    rng = np.random.default_rng(8)
    M, d, N, V = 4, 5, 6, 3
    base = rng.standard_normal((V, 1, d))
    lut = np.repeat(base, N, axis=1)
    h = rng.standard_normal((M, d))
    ids = np.array([2, 1, 0, 2])
    out, _, _ = oracle.layer_lookup(h, ids, lut, rng.standard_normal((d, N)))
    assert np.allclose(out, h + base[ids, 0], atol=1e-14)


def pin_bad_ids_leave_the_residual():
    rng = np.random.default_rng(9)
    M, d, N, V = 4, 3, 2, 5
    h = rng.standard_normal((M, d))
    lut = rng.standard_normal((V, N, d))
    out, _, bad = oracle.layer_lookup(h, np.array([0, -1, 5, 4]), lut, rng.standard_normal((d, N)))
    assert bad == 2
    assert np.array_equal(out[1], h[1]) and np.array_equal(out[2], h[2])
    assert not np.array_equal(out[0], h[0])


def pin_storage_types_widen_exactly():
    rng = np.random.default_rng(10)
    M, d, N, V = 3, 8, 2, 4
    # values exactly representable in bf16 (8 significant bits)
    def q(a):
        return np.round(a * 16.0) / 16.0

    h, lut, Wr = q(rng.uniform(-4, 4, (M, d))), q(rng.uniform(-4, 4, (V, N, d))), q(rng.uniform(-1, 1, (d, N)))
    ids = np.array([3, 0, 1])
    ref, _, _ = oracle.layer_lookup(h, ids, lut, Wr)
    f32, _, _ = oracle.layer_lookup(h.astype(np.float32), ids, lut.astype(np.float32), Wr.astype(np.float32))
    bits = lambda a: (a.astype(np.float32).view(np.uint32) >> 16).astype(np.uint16)
    b16, _, _ = oracle.layer_lookup(bits(h), ids, bits(lut), bits(Wr))
    assert np.array_equal(ref, f32) and np.array_equal(ref, b16)


# ---- the defining identity: Eq. 5 with Eq. 6 substituted equals Eq. 8 ----------------------------

def pin_lookup_equals_onthefly_small():
    rng = np.random.default_rng(11)
    V, d, D, N, M = 17, 6, 9, 3, 10
    E = rng.standard_normal((V, d))
    W1 = rng.standard_normal((N, D, d))
    W2 = rng.standard_normal((N, d, D))
    Wr = rng.standard_normal((d, N))
    h = rng.standard_normal((M, d))
    ids = rng.integers(0, V, M)
    lut = oracle.build_lut(E, W1, W2)
    a, _, _ = oracle.layer_lookup(h, ids, lut, Wr)
    b, _ = oracle.layer_onthefly(h, ids, E, W1, W2, Wr)
    assert np.allclose(a, b, rtol=0, atol=1e-12)
    # with the expert norm folded into the table
    nw = rng.uniform(0.5, 1.5, d)
    lut_n = oracle.build_lut(E, W1, W2, norm_w=nw, eps=1e-6)
    a, _, _ = oracle.layer_lookup(h, ids, lut_n, Wr)
    b, _ = oracle.layer_onthefly(h, ids, E, W1, W2, Wr, norm_w=nw, eps=1e-6)
    assert np.allclose(a, b, rtol=0, atol=1e-12)
    assert not np.allclose(lut, lut_n)


def pin_lut_entry_is_ffn_of_embedding_row():
    # Eq. 6 entry by entry, against numpy + scipy's normal CDF
    from scipy.stats import norm

    rng = np.random.default_rng(12)
    V, d, D, N = 5, 4, 6, 3
    E = rng.standard_normal((V, d))
    W1 = rng.standard_normal((N, D, d))
    W2 = rng.standard_normal((N, d, D))
    lut = oracle.build_lut(E, W1, W2)
    assert lut.shape == (V, N, d)
    for i in range(V):
        for j in range(N):
            s = W1[j] @ E[i]
            want = W2[j] @ (s * norm.cdf(s))
            assert np.allclose(lut[i, j], want, atol=1e-13), (i, j)


# ---- sizes (Eq. 13, Eq. 14; Tables 3, 6, 8) --------------------------------------------------------

def pin_paper_parameter_counts():
    V_paper = 50000
    for src, d, N, L, off_b, load_m in _golden_rows("paper_param_counts.txt"):
        d, N, L = int(d), int(N), int(L)
        digits = len(off_b.split(".")[1])
        got = oracle.offloaded_params(d, N, V_paper, L) / 1e9
        assert abs(got - float(off_b)) <= 0.5 * 10 ** (-digits) + 1e-9, (src, got, off_b)
        if load_m != "-":
            digits = len(load_m.split(".")[1])
            got = oracle.loaded_params_per_token(d, N, L) / 1e6
            assert abs(got - float(load_m)) <= 0.5 * 10 ** (-digits) + 1e-9, (src, got, load_m)
    for prec, d, N, L, eb, kb in (r for r in _golden_rows("paper_table8_bytes.txt") if len(r) == 6):  # the FP16 row
        assert oracle.loaded_params_per_token(int(d), int(N), int(L)) * int(eb) == int(kb) * 1024


# ---- dedup -----------------------------------------------------------------------------------

def pin_dedup_against_numpy_unique():
    rng = np.random.default_rng(13)
    for M in (1, 2, 17, 300):
        ids = rng.integers(0, 40, M)
        uniq, slot = oracle.dedup(ids)
        assert np.array_equal(np.sort(uniq), np.unique(ids))
        assert np.array_equal(uniq[slot], ids)
        # first-occurrence order
        _, first = np.unique(ids, return_index=True)
        assert np.array_equal(uniq, ids[np.sort(first)])
    uniq, slot = oracle.dedup(np.array([], dtype=np.int64))
    assert uniq.size == 0 and slot.size == 0


PINS = [v for k, v in sorted(globals().items()) if k.startswith("pin_") and callable(v)]
