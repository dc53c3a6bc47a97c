"""CPU oracle for the MoLE inference layer (arXiv 2503.15798) -- TEST INFRASTRUCTURE ONLY.

A ctypes wrapper around ``oracle/mole_oracle.c`` (plain C, fp64 arithmetic).  Nothing on
the product path may import this package: it exists so that the tests, the smoke check and
the bench's CPU-baseline leg can compare the CUDA library against an independent statement
of Eq. 4 (router softmax over all experts), Eq. 6-7 (table construction) and Eq. 8 (the
lookup-form layer).  It imports nothing from the CUDA package.

Arrays are numpy; storage types are float64, float32 or uint16 (raw bf16 bit patterns).
CPU torch tensors are accepted and converted without changing a bit.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "mole_oracle.c")
_LIB = os.path.join(_HERE, "libmole_oracle.so")
_lock = threading.Lock()
_lib = None

F64, F32, BF16 = 0, 1, 2


def build(force: bool = False) -> str:
    """Compile the C oracle with gcc (OpenMP over tokens only) and return the .so path."""
    with _lock:
        stale = (not os.path.exists(_LIB)) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC)
        if force or stale:
            tmp = _LIB + f".tmp{os.getpid()}"
            subprocess.check_call(
                ["gcc", "-O2", "-std=c11", "-fopenmp", "-shared", "-fPIC", _SRC, "-o", tmp, "-lm"]
            )
            os.replace(tmp, _LIB)
    return _LIB


def _configure(lib):
    """Declare the C signatures on a loaded library (also used for deliberately broken
    copies that the tests build to show that the pins catch mistakes)."""
    c = ctypes
    dp, ip, vp = c.POINTER(c.c_double), c.POINTER(c.c_int64), c.c_void_p
    lib.oracle_gelu.restype = c.c_double
    lib.oracle_gelu.argtypes = [c.c_double]
    lib.oracle_ffn.restype = None
    lib.oracle_ffn.argtypes = [dp, dp, dp, c.c_int, c.c_int, dp]
    lib.oracle_rmsnorm.restype = None
    lib.oracle_rmsnorm.argtypes = [dp, dp, c.c_double, c.c_int, dp]
    lib.oracle_build_lut.restype = None
    lib.oracle_build_lut.argtypes = [dp, dp, dp, dp, c.c_double, c.c_int, c.c_int, c.c_int, c.c_int, dp]
    lib.oracle_router_gates.restype = None
    lib.oracle_router_gates.argtypes = [dp, dp, c.c_int, c.c_int, dp]
    lib.oracle_layer_lookup.restype = c.c_int64
    lib.oracle_layer_lookup.argtypes = [vp, ip, vp, vp, vp, c.c_int, c.c_int64, c.c_int, c.c_int,
                                        c.c_int64, dp, dp, c.c_int]
    lib.oracle_layer_onthefly.restype = c.c_int64
    lib.oracle_layer_onthefly.argtypes = [dp, ip, dp, dp, dp, dp, dp, c.c_double, c.c_int64, c.c_int,
                                          c.c_int, c.c_int, c.c_int64, dp]
    lib.oracle_dedup.restype = c.c_int64
    lib.oracle_dedup.argtypes = [ip, c.c_int64, ip, ip]
    lib.oracle_effective_threads.restype = c.c_int
    lib.oracle_effective_threads.argtypes = [c.c_int]
    return lib


def _load():
    global _lib
    if _lib is None:
        _lib = _configure(ctypes.CDLL(build()))
    return _lib


def _np(x):
    """numpy view of a numpy array or a CPU torch tensor; bf16 tensors become uint16 bits."""
    if isinstance(x, np.ndarray):
        return x
    import torch  # only to unwrap tensors handed in by the tests

    assert isinstance(x, torch.Tensor) and x.device.type == "cpu"
    if x.dtype == torch.bfloat16:
        return x.contiguous().view(torch.int16).numpy().view(np.uint16)
    return x.contiguous().numpy()


def _dtype_tag(a: np.ndarray) -> int:
    if a.dtype == np.float64:
        return F64
    if a.dtype == np.float32:
        return F32
    if a.dtype == np.uint16:
        return BF16
    raise TypeError(f"oracle: unsupported storage type {a.dtype}")


def _d(a):
    return a.ctypes.data_as(ctypes.POINTER(ctypes.c_double))


def _i(a):
    return a.ctypes.data_as(ctypes.POINTER(ctypes.c_int64))


def _f64(x):
    return np.ascontiguousarray(_np(x), dtype=np.float64)


def bf16_bits_to_f64(bits: np.ndarray) -> np.ndarray:
    """Exact widening of raw bf16 bit patterns (uint16) to float64."""
    return (bits.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def gelu(x: float) -> float:
    return float(_load().oracle_gelu(float(x)))


def ffn(x, W1, W2) -> np.ndarray:
    """FFN(x) = W2 . gelu(W1 . x); W1 [D][d], W2 [d][D]."""
    x, W1, W2 = _f64(x), _f64(W1), _f64(W2)
    D, d = W1.shape
    assert W2.shape == (d, D) and x.shape == (d,)
    y = np.empty(d, dtype=np.float64)
    _load().oracle_ffn(_d(x), _d(W1), _d(W2), d, D, _d(y))
    return y


def rmsnorm(x, w, eps: float) -> np.ndarray:
    x, w = _f64(x), _f64(w)
    y = np.empty_like(x)
    _load().oracle_rmsnorm(_d(x), _d(w), float(eps), x.shape[0], _d(y))
    return y


def build_lut(E, W1, W2, norm_w=None, eps: float = 1e-6) -> np.ndarray:
    """Eq. 6-7: LUT[i][j] = FFN_j(E[i]).  E [V][d], W1 [N][D][d], W2 [N][d][D] -> [V][N][d] fp64."""
    E, W1, W2 = _f64(E), _f64(W1), _f64(W2)
    V, d = E.shape
    N, D, d1 = W1.shape
    assert d1 == d and W2.shape == (N, d, D)
    lut = np.empty((V, N, d), dtype=np.float64)
    nw = None if norm_w is None else _f64(norm_w)
    _load().oracle_build_lut(_d(E), _d(W1), _d(W2), None if nw is None else _d(nw), float(eps),
                             V, d, D, N, _d(lut))
    return lut


def router_gates(h, Wr) -> np.ndarray:
    """Eq. 4 for one token: softmax over all N logits; Wr is [d][N]."""
    h, Wr = _f64(h), _f64(Wr)
    d, N = Wr.shape
    assert h.shape == (d,)
    g = np.empty(N, dtype=np.float64)
    _load().oracle_router_gates(_d(h), _d(Wr), d, N, _d(g))
    return g


def layer_lookup(hidden, ids, lut, w_router, residual=None, threads: int = 1):
    """Eq. 8 (lookup form).  Returns (out [M][d] fp64, gates [M][N] fp64, n_bad_ids).

    hidden [M][d], lut [V][N][d], w_router [d][N] and residual (optional, [M][d]) must share
    one storage type: float64, float32 or uint16 (bf16 bits).
    """
    hidden, lut, w_router = (np.ascontiguousarray(_np(a)) for a in (hidden, lut, w_router))
    tag = _dtype_tag(hidden)
    assert _dtype_tag(lut) == tag and _dtype_tag(w_router) == tag
    M, d = hidden.shape
    V, N, d1 = lut.shape
    assert d1 == d and w_router.shape == (d, N)
    res_p = None
    if residual is not None:
        residual = np.ascontiguousarray(_np(residual))
        assert _dtype_tag(residual) == tag and residual.shape == (M, d)
        res_p = residual.ctypes.data
    ids64 = np.ascontiguousarray(_np(ids), dtype=np.int64).reshape(-1)
    assert ids64.shape[0] == M
    out = np.empty((M, d), dtype=np.float64)
    gates = np.empty((M, N), dtype=np.float64)
    bad = _load().oracle_layer_lookup(hidden.ctypes.data, _i(ids64), lut.ctypes.data,
                                      w_router.ctypes.data, res_p, tag, M, N, d, V, _d(out), _d(gates),
                                      int(threads))
    return out, gates, int(bad)


def layer_onthefly(hidden, ids, E, W1, W2, Wr, norm_w=None, eps: float = 1e-6):
    """Eq. 5 (experts run on the embedding row).  All fp64.  Returns (out, n_bad_ids)."""
    hidden, E, W1, W2, Wr = _f64(hidden), _f64(E), _f64(W1), _f64(W2), _f64(Wr)
    M, d = hidden.shape
    V = E.shape[0]
    N, D, _ = W1.shape
    ids64 = np.ascontiguousarray(_np(ids), dtype=np.int64).reshape(-1)
    out = np.empty((M, d), dtype=np.float64)
    nw = None if norm_w is None else _f64(norm_w)
    bad = _load().oracle_layer_onthefly(_d(hidden), _i(ids64), _d(E), _d(W1), _d(W2), _d(Wr),
                                        None if nw is None else _d(nw), float(eps), M, N, d, D, V, _d(out))
    return out, int(bad)


def dedup(ids):
    """Distinct ids in order of first occurrence and slot[t] with uniq[slot[t]] == ids[t]."""
    ids64 = np.ascontiguousarray(_np(ids), dtype=np.int64).reshape(-1)
    M = ids64.shape[0]
    uniq = np.empty(max(M, 1), dtype=np.int64)
    slot = np.empty(max(M, 1), dtype=np.int64)
    U = int(_load().oracle_dedup(_i(ids64), M, _i(uniq), _i(slot)))
    return uniq[:U].copy(), slot[:M].copy()


def effective_threads(threads: int) -> int:
    return int(_load().oracle_effective_threads(int(threads)))


# ---- size formulas of Sec. 3.4 (Eq. 13, Eq. 14; Table 1 last row) -------------------------

def offloaded_params(d: int, N: int, V: int, L: int = 1) -> int:
    """Eq. 13 per layer (d*N*|V|), times L layers."""
    return d * N * V * L


def loaded_params_per_token(d: int, N: int, L: int = 1) -> int:
    """Eq. 14 per layer (d*N), times L layers."""
    return d * N * L
