"""Pins of the quantisation oracle (oracle/quant.py) against what the papers and the mathematics fix:
the NF4 values the QLoRA paper prints, the sizes Table 8 of the MoLE paper prints, the definition
"nearest codebook value of the block divided by its absolute maximum" by brute force, and the closed
forms of degenerate blocks.  No GPU."""
import os

import numpy as np
import pytest
from scipy.stats import norm

from oracle import quant

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")


def _rows(name):
    with open(os.path.join(GOLDEN, name)) as f:
        return [[c.strip() for c in ln.split("|")] for ln in f if ln.strip() and not ln.startswith("#")]


def test_nf4_codebook_reproduces_the_values_printed_in_the_qlora_paper():
    printed = np.array([float(r[0]) for r in _rows("qlora_nf4_values.txt")])
    assert printed.shape == (16,)
    got = quant.nf_codebook(4)
    # the printed values are float32 roundings of a float32 computation: agreement to a few 1e-7
    assert np.abs(got - printed).max() <= 5e-7
    assert np.array_equal(quant.nf_codebook_f32(4) == 0, printed == 0)


@pytest.mark.parametrize("bits", [3, 4])
def test_codebook_structure(bits):
    cb = quant.nf_codebook(bits)
    n = 2 ** bits
    assert cb.shape == (n,) and np.all(np.diff(cb) > 0)          # 2^k distinct values, ascending
    assert cb[0] == -1.0 and cb[-1] == 1.0                       # normalised to [-1, 1]
    assert cb[n // 2 - 1] == 0.0 and (cb == 0).sum() == 1        # zero exactly representable, once
    assert (cb < 0).sum() == n // 2 - 1 and (cb > 0).sum() == n // 2   # the positive half has one value more
    # every value is a quantile of N(0,1) at evenly spaced probabilities, divided by the largest one
    top = norm.ppf(1 - 0.5 * (1 / (2 * (n - 1)) + 1 / (2 * n)))
    p_pos = norm.cdf(cb[n // 2 - 1:] * top)
    assert np.allclose(np.diff(p_pos), np.diff(p_pos)[0], rtol=0, atol=1e-12)
    p_neg = norm.cdf(cb[: n // 2] * top)
    assert np.allclose(np.diff(p_neg), np.diff(p_neg)[0], rtol=0, atol=1e-12)
    assert abs(p_pos[-1] + p_neg[0] - 1.0) <= 1e-12              # the same tail mass on both sides


def test_storage_sizes_match_table_8():
    fp16_kb = None
    for r in _rows("paper_table8_bytes.txt"):
        if len(r) == 6:
            fp16_kb = int(r[5])
            continue
        prec, d, N, L, block, bits, scale_bytes, kb, pct, gb = r
        d, N, L, block, bits, scale_bytes = (int(v) for v in (d, N, L, block, bits, scale_bytes))
        assert np.dtype(quant.SCALE_DTYPE[bits]).itemsize == scale_bytes
        per_block = block * bits // 8 + scale_bytes
        assert per_block == {4: 388, 3: 50}[bits]
        assert round(100.0 * per_block / (block * 2), 1) == float(pct)             # 25.3 % / 19.5 % of FP16
        rec = quant.record_bytes(N, d, bits, block)
        assert rec == N * (d // block) * per_block                                  # no padding at this shape
        assert round(rec * L / 1024) == int(kb)                                     # 18 KB / 14 KB per token
        assert round(3.5 * per_block / (block * 2), 1) == float(gb)                 # 0.9 GB / 0.7 GB of 3.5 GB
    assert fp16_kb == 72


@pytest.mark.parametrize("bits,block", [(4, 768), (3, 128), (4, 64), (3, 32)])
def test_codes_are_the_nearest_codebook_value_of_the_normalised_block(bits, block):
    rng = np.random.default_rng(bits * 100 + block)
    x = (0.05 * rng.standard_normal((40, 3 * block))).astype(np.float32)
    codes, scales = quant.quantize(x, bits, block)
    cb = quant.nf_codebook(bits)
    s = np.repeat(scales.astype(np.float64), block, axis=1)
    y = x.astype(np.float64) / s
    dist = np.abs(y[..., None] - cb)                      # brute force over the whole codebook, in float64
    best = dist.min(axis=-1)
    chosen = np.take_along_axis(dist, codes[..., None].astype(np.int64), axis=-1)[..., 0]
    assert (chosen <= best + 1e-6).all()                  # the chosen value is a nearest one (float32 decision noise)
    assert (np.abs(codes.astype(int) - dist.argmin(axis=-1)) <= 1).all()
    assert (codes.astype(int) != dist.argmin(axis=-1)).mean() < 1e-3
    # absmax scaling: the scale is the block's largest magnitude, and that element maps to +-1 exactly
    want_scale = np.abs(x.reshape(40, 3, block)).max(axis=2).astype(quant.SCALE_DTYPE[bits])
    assert np.array_equal(scales, want_scale)
    deq = quant.dequantize(codes, scales, bits, block)
    gaps = np.diff(cb).max() / 2
    assert (np.abs(deq - x) <= s * gaps * (1 + 1e-3) + 1e-12).all()   # error at most half the widest gap times the scale


@pytest.mark.parametrize("bits,block", [(4, 768), (3, 128)])
def test_quantising_twice_changes_nothing_and_power_of_two_scaling_commutes(bits, block):
    rng = np.random.default_rng(5)
    x = (0.05 * rng.standard_normal((16, 768))).astype(np.float32)
    codes, scales = quant.quantize(x, bits, block)
    deq = quant.dequantize(codes, scales, bits, block)
    codes2, scales2 = quant.quantize(deq.astype(np.float32), bits, block)
    assert np.array_equal(scales2, scales) and np.array_equal(codes2, codes)
    codes8, scales8 = quant.quantize(x * 8, bits, block)
    assert np.array_equal(codes8, codes) and np.array_equal(scales8.astype(np.float64), scales.astype(np.float64) * 8)
    codes_n, scales_n = quant.quantize(-x, bits, block)    # not symmetric: the codebook has one more positive value
    assert np.array_equal(scales_n, scales)
    at_min = x == -scales.astype(np.float32).repeat(block, axis=1)
    assert (codes[at_min] == 0).all() and (codes_n[at_min] == 2 ** bits - 1).all()
    at_max = x == scales.astype(np.float32).repeat(block, axis=1)
    if bits == 4:  # a float32 scale is the block's maximum itself (a float16 one is its rounding)
        assert (at_min | at_max).reshape(16, -1, block).any(axis=2).all()


@pytest.mark.parametrize("bits,block", [(4, 768), (3, 128)])
def test_degenerate_blocks_round_trip_exactly(bits, block):
    d = 768
    x = np.zeros((5, d), dtype=np.float32)
    x[0, :] = 0.375                       # all equal: every element is the maximum -> +1 * scale
    x[1, :] = -0.375                      # -> -1 * scale
    x[2, 5] = 0.09375                     # one non-zero per block: +-1 * scale there, the zero code elsewhere
    x[4, d - 1] = -3.0
    codes, scales = quant.quantize(x, bits, block)
    assert np.array_equal(quant.dequantize(codes, scales, bits, block), x.astype(np.float64))
    assert (codes[0] == 2 ** bits - 1).all() and (codes[1] == 0).all() and (codes[3] == 2 ** (bits - 1) - 1).all()
    assert (scales[3] == 0).all()         # an all-zero block: scale 0, the zero code, value 0


@pytest.mark.parametrize("bits,block,N,d", [(4, 768, 16, 768), (3, 128, 16, 768), (4, 1024, 4, 1024), (3, 128, 4, 128),
                                            (4, 128, 32, 2048), (3, 128, 32, 2048)])
def test_packed_records_round_trip_and_put_every_code_where_the_layout_says(bits, block, N, d):
    rng = np.random.default_rng(N + d)
    V = 5
    codes = rng.integers(0, 2 ** bits, (V, N, d)).astype(np.uint8)
    scales = rng.random((V, N, d // block)).astype(quant.SCALE_DTYPE[bits])
    rec = quant.pack_rows(codes, scales, bits)
    assert rec.shape == (V, quant.record_bytes(N, d, bits, block)) and rec.shape[1] % 16 == 0
    c2, s2 = quant.unpack_rows(rec, N, d, bits, block)
    assert np.array_equal(c2, codes) and np.array_equal(s2, scales)
    # spot checks of single codes, by the stated bit positions
    for (v, j, c) in ((0, 0, 0), (1, N - 1, d - 1), (4, N // 2, 37), (2, 1, 130 % d)):
        k = int(codes[v, j, c])
        if bits == 4:
            byte = rec[v, j * (d // 2) + c // 2]
            assert (byte >> (4 * (c % 2))) & 15 == k
        else:
            a = rec[v, j * (d // 4) + c // 4]
            b = rec[v, N * (d // 4) + j * (d // 8) + c // 8]
            assert ((a >> (2 * (c % 4))) & 3) | (((b >> (c % 8)) & 1) << 2) == k


def test_layer_over_a_quantised_table_is_the_layer_over_its_dequantised_values():
    """The quantised layer has no definition of its own: it is Eq. 8 over the table that de-quantisation
    gives back.  Zero quantisation error (values that are codebook multiples) must reproduce the plain
    layer exactly."""
    import oracle

    rng = np.random.default_rng(3)
    V, N, d, M = 12, 4, 128, 9
    for bits, block in ((4, 128), (3, 128)):
        cb = quant.nf_codebook_f32(bits)
        codes = rng.integers(0, 2 ** bits, (V * N, d))
        codes[:, 0] = 2 ** bits - 1                     # every block holds its own maximum: scale survives
        lut = (cb[codes] * np.float32(0.25)).astype(np.float64).reshape(V, N, d)
        rec = quant.quantize_table(lut.astype(np.float32), bits, block)
        assert np.array_equal(quant.dequantize_table(rec, N, d, bits, block), lut)
        hidden = rng.standard_normal((M, d))
        wr = 0.1 * rng.standard_normal((d, N))
        ids = rng.integers(0, V, M)
        want, _, _ = oracle.layer_lookup(hidden, ids, lut, wr)
        got, _, _ = oracle.layer_lookup(hidden, ids, quant.dequantize_table(rec, N, d, bits, block), wr)
        assert np.array_equal(got, want)
