"""Plant one mistake at a time in a copy of the oracle's C source and require that the pin
suite notices.  The mistakes are the plausible ones: a transposed router weight, a table
indexed [V][d][N], a dropped residual, a missing max-subtraction partner, a tanh GELU, a
transposed second FFN matrix, experts summed over the wrong range, softmax without the
normalisation, a top-1 router."""
import ctypes
import os
import subprocess

import pytest

import oracle
import oracle_pins

SRC = os.path.join(os.path.dirname(oracle.__file__), "mole_oracle.c")

MUTANTS = {
    "router_weight_transposed": ("z += h[c] * Wr[(size_t)c * N + j];", "z += h[c] * Wr[(size_t)j * d + c];"),
    "table_indexed_V_d_N": ("widen(lut, (id * N + j) * (int64_t)d + c, dtype)",
                            "widen(lut, (id * (int64_t)d + c) * N + j, dtype)"),
    "residual_dropped": ("out[t * d + c] = r + s;", "out[t * d + c] = s;"),
    "residual_sign": ("out[t * d + c] = r + s;", "out[t * d + c] = r - s;"),
    "softmax_not_normalised": ("for (int j = 0; j < N; ++j) g[j] /= sum;", ""),
    "softmax_of_negated_logits": ("g[j] = exp(g[j] - zmax);", "g[j] = exp(zmax - g[j]);"),
    "gelu_tanh_approximation": ("return 0.5 * x * (1.0 + erf(x / sqrt(2.0)));",
                                "return 0.5 * x * (1.0 + tanh(0.7978845608028654 * (x + 0.044715 * x * x * x)));"),
    "ffn_second_matrix_transposed": ("s += W2[(size_t)c * D + k] * a[k];", "s += W2[(size_t)k * d + c] * a[k];"),
    "ffn_first_matrix_transposed": ("s += W1[(size_t)k * d + c] * x[c];", "s += W1[(size_t)c * D + k] * x[c];"),
    "last_expert_skipped": ("for (int j = 0; j < N; ++j)\n                    s += g[j] * widen(",
                            "for (int j = 0; j + 1 < N; ++j)\n                    s += g[j] * widen("),
    "gates_ignored_plain_sum": ("s += g[j] * widen(lut", "s += widen(lut"),
    "residual_pointer_ignored": ("double r = residual ? widen(residual, t * d + c, dtype) : h[c];", "double r = h[c];"),
    "wrong_token_id": ("int64_t id = ids[t];\n        int ok", "int64_t id = ids[(t + 1) % M];\n        int ok"),
    "lut_built_from_wrong_expert": ("oracle_ffn(e, W1 + (size_t)j * D * d, W2 + (size_t)j * d * D, d, D,\n                       lut",
                                    "oracle_ffn(e, W1 + (size_t)j * D * d, W2 + (size_t)((j + 1) % N) * d * D, d, D,\n                       lut"),
    "rmsnorm_eps_outside_sqrt": ("double r = 1.0 / sqrt(ms + eps);", "double r = 1.0 / (sqrt(ms) + eps);"),
    "dedup_slot_off": ("slot[t] = u;", "slot[t] = (u > 0) ? u - 1 : 0;"),
    "bf16_widened_from_low_half": ("uint32_t bits = ((uint32_t)((const uint16_t *)p)[i]) << 16;",
                                   "uint32_t bits = ((uint32_t)((const uint16_t *)p)[i]);"),
}


@pytest.mark.parametrize("name", sorted(MUTANTS))
def test_pins_catch_mutant(name, tmp_path, monkeypatch):
    old, new = MUTANTS[name]
    src = open(SRC).read()
    assert src.count(old) >= 1, f"mutation site for {name} not found"
    c_path = tmp_path / "mutant.c"
    so_path = tmp_path / "libmutant.so"
    c_path.write_text(src.replace(old, new))
    subprocess.check_call(["gcc", "-O1", "-std=c11", "-fopenmp", "-shared", "-fPIC", str(c_path), "-o",
                           str(so_path), "-lm"])
    oracle._load()
    monkeypatch.setattr(oracle, "_lib", oracle._configure(ctypes.CDLL(str(so_path))))
    failed = []
    for pin in oracle_pins.PINS:
        try:
            pin()
        except AssertionError:
            failed.append(pin.__name__)
    assert failed, f"no pin noticed the planted mistake '{name}'"
