"""Seeded input generators: the bounded Zipf(1.1) id stream and the workload shapes."""
import numpy as np

from paper_2503_15798_b200 import inputs


def test_zipf_table_closed_form_values():
    V, s = 50304, 1.1
    p = inputs.zipf_probs(V, s)
    H = sum(k ** -s for k in range(1, V + 1))  # plain Python sum, independent of numpy
    assert abs(H - 7.19726) < 1e-4
    assert abs(p[0] - 1.0 / H) < 1e-12 and abs(p[0] - 0.1389) < 1e-4
    assert abs(p.sum() - 1.0) < 1e-12
    assert abs(p[:10].sum() - 0.372) < 2e-3
    assert abs(p[:100].sum() - 0.594) < 2e-3
    assert abs(p[:1000].sum() - 0.774) < 2e-3
    assert np.all(np.diff(p) < 0)


def test_zipf_ids_follow_the_table_and_are_seeded():
    V = 50304
    a = inputs.zipf_ids(200000, V, seed=3, permute=False)
    b = inputs.zipf_ids(200000, V, seed=3, permute=False)
    assert np.array_equal(a, b)
    assert a.min() >= 0 and a.max() < V
    p = inputs.zipf_probs(V)
    freq0 = (a == 0).mean()
    assert abs(freq0 - p[0]) < 4 * np.sqrt(p[0] * (1 - p[0]) / a.size)
    top100 = (a < 100).mean()
    assert abs(top100 - p[:100].sum()) < 0.01
    c = inputs.zipf_ids(200000, V, seed=3, permute=True)
    assert c.min() >= 0 and c.max() < V and not np.array_equal(a, c)
    # the permutation is a bijection applied to the same ranks
    assert len(np.unique(c)) == len(np.unique(a))


def test_expected_unique_ids_per_step():
    # E[U] = sum_k 1 - (1 - p_k)^M ; the sampled mean must sit on it
    V = 50304
    p = inputs.zipf_probs(V)
    for M, want in ((8, 7.3), (64, 46.0), (256, 149.0)):
        exact = float(np.sum(1.0 - (1.0 - p) ** M))
        assert abs(exact - want) < 0.02 * want + 0.1
        got = np.mean([len(np.unique(inputs.zipf_ids(M, V, seed=s))) for s in range(200)])
        assert abs(got - exact) < 0.05 * exact + 0.5


def test_shapes_reproduce_table_sizes():
    sh = inputs.SHAPES
    assert abs(sh["160m"].layer_table_bytes * sh["160m"].L / 1e9 - 14.84) < 0.01
    assert abs(sh["410m"].layer_table_bytes * sh["410m"].L / 1e9 - 39.56) < 0.01
    assert abs(sh["1b"].layer_table_bytes * sh["1b"].L / 1e9 - 105.5) < 0.1
    assert sh["160m"].row_bytes == 24576 and sh["410m"].row_bytes == 32768 and sh["1b"].row_bytes == 131072
    assert sh["tiny"].row_bytes == 1024
    # gathered rows + hidden in/out + router weights
    assert sh["160m"].layer_bytes(64) == 64 * 24576 + 2 * 64 * 768 * 2 + 768 * 16 * 2


def test_tiny_model_is_seeded_and_shaped():
    a, b = inputs.tiny_model(0), inputs.tiny_model(0)
    assert np.array_equal(a["E"], b["E"]) and np.array_equal(a["ids"], b["ids"])
    assert a["E"].shape == (512, 64) and a["W1"][0].shape == (4, 256, 64) and a["W2"][1].shape == (4, 64, 256)
    assert a["Wr"][0].shape == (64, 4) and a["hidden"].shape == (64, 64) and a["ids"].shape == (64,)
    assert abs(a["W1"][0].std() - 0.02) < 1e-3 and abs(a["E"].std() - 1.0) < 0.02
    assert a["E"].dtype == np.float32
