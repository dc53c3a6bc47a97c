"""The tiny FFN-built configuration (V=512, d=64, N=4, D=256, 2 layers, batch 4x16):
the table built by Eq. 6-7 makes the lookup form (Eq. 8) equal the on-the-fly form (Eq. 5),
layer after layer, and the router weights of every token sum to one."""
import numpy as np

import oracle
from paper_2503_15798_b200 import inputs


def test_identity_on_tiny_config_two_layers():
    m = inputs.tiny_model(seed=0)
    sh = m["shape"]
    h_lookup = m["hidden"].astype(np.float64)
    h_fly = h_lookup.copy()
    for l in range(sh.L):
        lut = oracle.build_lut(m["E"], m["W1"][l], m["W2"][l])  # fp64 table
        assert lut.shape == (sh.V, sh.N, sh.d)
        Wr = m["Wr"][l].astype(np.float64)
        h_lookup, gates, bad = oracle.layer_lookup(h_lookup, m["ids"], lut, Wr)
        h_fly, bad2 = oracle.layer_onthefly(h_fly, m["ids"], m["E"], m["W1"][l], m["W2"][l], Wr)
        assert bad == 0 and bad2 == 0
        assert np.allclose(gates.sum(axis=1), 1.0, atol=1e-15)
        assert (gates > 0).all()
        assert np.allclose(h_lookup, h_fly, rtol=0, atol=1e-12)
    assert not np.allclose(h_lookup, m["hidden"])  # the layers did something


def test_identity_survives_fp32_table_storage():
    m = inputs.tiny_model(seed=0)
    l = 0
    lut64 = oracle.build_lut(m["E"], m["W1"][l], m["W2"][l])
    lut32 = lut64.astype(np.float32)
    a, _, _ = oracle.layer_lookup(m["hidden"], m["ids"], lut32, m["Wr"][l])
    b, _ = oracle.layer_onthefly(m["hidden"], m["ids"], m["E"], m["W1"][l], m["W2"][l], m["Wr"][l])
    scale = np.maximum(1.0, np.abs(b))
    assert (np.abs(a - b) / scale).max() < 1e-6


def test_threads_do_not_change_the_result():
    m = inputs.tiny_model(seed=0)
    lut = oracle.build_lut(m["E"][:64], m["W1"][0], m["W2"][0]).astype(np.float32)
    ids = m["ids"] % 64
    a, ga, _ = oracle.layer_lookup(m["hidden"], ids, lut, m["Wr"][0], threads=1)
    b, gb, _ = oracle.layer_lookup(m["hidden"], ids, lut, m["Wr"][0], threads=4)
    assert np.array_equal(a, b) and np.array_equal(ga, gb)
