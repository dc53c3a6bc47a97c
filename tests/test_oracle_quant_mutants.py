"""Planted mistakes in the quantisation oracle: each one must make at least one pin of
tests/test_oracle_quant.py fail (the pins are called directly, with the mistake patched into
oracle.quant).  Shows that the pins can tell a wrong quantiser from a right one."""
import numpy as np
import pytest

import test_oracle_quant as pins
from oracle import quant

PIN_CALLS = [
    (pins.test_nf4_codebook_reproduces_the_values_printed_in_the_qlora_paper, ()),
    (pins.test_codebook_structure, (3,)), (pins.test_codebook_structure, (4,)),
    (pins.test_storage_sizes_match_table_8, ()),
    (pins.test_codes_are_the_nearest_codebook_value_of_the_normalised_block, (4, 768)),
    (pins.test_codes_are_the_nearest_codebook_value_of_the_normalised_block, (3, 128)),
    (pins.test_quantising_twice_changes_nothing_and_power_of_two_scaling_commutes, (4, 768)),
    (pins.test_degenerate_blocks_round_trip_exactly, (4, 768)), (pins.test_degenerate_blocks_round_trip_exactly, (3, 128)),
    (pins.test_packed_records_round_trip_and_put_every_code_where_the_layout_says, (4, 768, 16, 768)),
    (pins.test_packed_records_round_trip_and_put_every_code_where_the_layout_says, (3, 128, 16, 768)),
    (pins.test_layer_over_a_quantised_table_is_the_layer_over_its_dequantised_values, ()),
]


def some_pin_fails():
    for fn, args in PIN_CALLS:
        try:
            fn(*args)
        except Exception:  # an assertion, or a shape error the mistake causes
            return True
    return False


def test_the_unmodified_oracle_passes_every_pin():
    assert not some_pin_fails()


def _uniform_codebook(bits):
    return np.linspace(-1.0, 1.0, 2 ** bits)


def _symmetric_halves(bits):  # the same number of quantiles on both sides: zero appears twice, one value short
    cb = quant_orig["nf_codebook"](bits)
    out = cb.copy()
    out[2 ** (bits - 1):] = -cb[: 2 ** (bits - 1)][::-1]
    return out


def _unnormalised(bits):
    from scipy.stats import norm

    cb = quant_orig["nf_codebook"](bits)
    return cb * norm.ppf(1 - 0.5 * (1 / (2 * (2 ** bits - 1)) + 1 / (2 * 2 ** bits)))


def _floor_instead_of_nearest(bits):  # thresholds at the codebook values themselves
    return quant_orig["nf_codebook_f32"](bits)[1:]


def _quantize_with_mean_scale(x, bits, block):
    x = np.ascontiguousarray(x, dtype=np.float32)
    rows, d = x.shape
    xb = x.reshape(rows, d // block, block)
    scales = np.abs(xb).mean(axis=2).astype(quant.SCALE_DTYPE[bits])
    s = np.maximum(scales.astype(np.float32), 1e-30)[:, :, None]
    y = (xb / s).astype(np.float32)
    codes = (y[..., None] > quant.midpoints_f32(bits)).sum(axis=-1).astype(np.uint8)
    return codes.reshape(rows, d), scales


def _dequantize_without_scale(codes, scales, bits, block):
    return quant_orig["nf_codebook_f32"](bits).astype(np.float64)[codes]


def _pack_nibbles_swapped(codes, scales, bits):
    c = codes.copy()
    if bits == 4:
        c[:, :, 0::2], c[:, :, 1::2] = codes[:, :, 1::2], codes[:, :, 0::2]
    else:
        c = codes ^ 4  # high bit inverted
    return quant_orig["pack_rows"](c, scales, bits)


quant_orig = {}
MUTANTS = {
    "uniform grid instead of normal quantiles": ("nf_codebook", _uniform_codebook),
    "no extra positive value": ("nf_codebook", _symmetric_halves),
    "codebook not normalised to [-1, 1]": ("nf_codebook", _unnormalised),
    "largest value not above, instead of nearest": ("midpoints_f32", _floor_instead_of_nearest),
    "mean instead of absolute maximum as scale": ("quantize", _quantize_with_mean_scale),
    "scale dropped at de-quantisation": ("dequantize", _dequantize_without_scale),
    "codes packed in the wrong place": ("pack_rows", _pack_nibbles_swapped),
    "NF3 scale stored as float32": ("SCALE_DTYPE", {4: np.float32, 3: np.float32}),
    "NF4 scale stored as float16": ("SCALE_DTYPE", {4: np.float16, 3: np.float16}),
}


@pytest.mark.parametrize("name", sorted(MUTANTS))
def test_planted_mistake_is_caught(name, monkeypatch):
    for k in ("nf_codebook", "nf_codebook_f32", "pack_rows"):
        quant_orig[k] = getattr(quant, k)
    attr, replacement = MUTANTS[name]
    monkeypatch.setattr(quant, attr, replacement)
    assert some_pin_fails(), name
