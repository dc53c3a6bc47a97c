"""CPU oracle for the quantised lookup tables of Sec. 4.5 / Table 8 (arXiv 2503.15798) -- TEST
INFRASTRUCTURE ONLY, like the rest of this package: nothing on the product path imports it, and it
imports nothing from the CUDA package.

The paper compresses the FP16 tables after training to the NF4 and NF3 data types of the QLoRA paper
(Dettmers et al. 2023), with "token-wise" blocks of 768 (NF4) and 128 (NF3) elements, and prints the
resulting sizes: 25.3 % and 19.5 % of FP16.  Those two ratios fix the storage of a block:

    NF4: 768 codes of 4 bits + one 4-byte scale = 388 bytes per 768 elements = 25.3 % of 1536
    NF3: 128 codes of 3 bits + one 2-byte scale =  50 bytes per 128 elements = 19.5 % of 256

so the scale (the block's absolute maximum) is a float32 for NF4 and a float16 for NF3.

What follows is the plain definition, in the order the QLoRA paper gives it:
  1. the k-bit NormalFloat codebook: quantiles of N(0, 1) -- 2^(k-1) evenly spaced probabilities for
     the negative half and 2^(k-1) + 1 for the positive half, both including the median, so that zero
     is exactly representable; one of the two zeros dropped; values divided by the largest magnitude
     so that they span [-1, 1] (QLoRA Sec. 3 "4-bit NormalFloat Quantization" and its appendix on the
     data type's exact values);
  2. block-wise absmax quantisation: every block is divided by its absolute maximum and each element
     takes the code of the NEAREST codebook value; de-quantisation multiplies the code's value by the
     block's scale.
The nearest-value decision is taken in float32 (the precision the GPU quantiser uses): normalised value
y = x / scale in IEEE float32, compared against the float32 midpoints of adjacent codebook values; a
value exactly on a midpoint takes the lower code.

Readings where the papers are silent (listed in the design doc): NF3 follows the same construction with
k = 3 (the QLoRA paper prints only the 4-bit values); the outermost probability is 1 - delta with
delta = (1/(2(2^k - 1)) + 1/(2 * 2^k)) / 2, the offset that reproduces QLoRA's printed NF4 values;
a block never straddles two (id, expert) rows; the packed byte layout is this library's own.
"""
from __future__ import annotations

import numpy as np
from scipy.stats import norm

SCALE_DTYPE = {4: np.float32, 3: np.float16}


def nf_codebook(bits: int) -> np.ndarray:
    """The 2^bits NormalFloat values in ascending order, float64."""
    half = 2 ** (bits - 1)
    delta = 0.5 * (1.0 / (2 * (2 ** bits - 1)) + 1.0 / (2 * 2 ** bits))
    positive = norm.ppf(np.linspace(0.5, 1.0 - delta, half + 1))  # half + 1 quantiles, the first is the median 0
    negative = -norm.ppf(np.linspace(0.5, 1.0 - delta, half))     # half quantiles, the first is the median 0
    values = np.concatenate([negative[1:][::-1], positive])       # one zero only: 2^bits values
    values[half - 1] = 0.0
    return values / np.abs(values).max()


def nf_codebook_f32(bits: int) -> np.ndarray:
    return nf_codebook(bits).astype(np.float32)


def midpoints_f32(bits: int) -> np.ndarray:
    cb = nf_codebook_f32(bits)
    return (np.float32(0.5) * (cb[:-1] + cb[1:])).astype(np.float32)


def quantize(x: np.ndarray, bits: int, block: int):
    """x [rows][d] (any float type; values are taken as float32) -> (codes uint8 [rows][d],
    scales [rows][d / block] in the stored type: float32 for NF4, float16 for NF3)."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    rows, d = x.shape
    assert d % block == 0
    xb = x.reshape(rows, d // block, block)
    absmax = np.abs(xb).max(axis=2)                                   # float32, exact
    if bits == 3:
        absmax = np.minimum(absmax, np.float32(65504.0))              # the largest float16
    scales = absmax.astype(SCALE_DTYPE[bits])                         # round to nearest even when stored
    s_eff = scales.astype(np.float32)[:, :, None]
    with np.errstate(divide="ignore", invalid="ignore"):
        y = np.where(s_eff > 0, xb / s_eff, np.float32(0.0)).astype(np.float32)   # IEEE float32 division
    mid = midpoints_f32(bits)
    codes = (y[..., None] > mid).sum(axis=-1).astype(np.uint8)        # number of midpoints below y
    return codes.reshape(rows, d), scales


def dequantize(codes: np.ndarray, scales: np.ndarray, bits: int, block: int) -> np.ndarray:
    """float64 values: codebook value (as float32) times the stored scale, exactly."""
    rows, d = codes.shape
    cb = nf_codebook_f32(bits).astype(np.float64)
    s = np.repeat(scales.astype(np.float64), block, axis=1)
    return cb[codes] * s


# ---- the packed record of one id: what the library stores and gathers -----------------------------

def record_bytes(N: int, d: int, bits: int, block: int) -> int:
    code_bytes = N * d // 2 if bits == 4 else N * (d // 4 + d // 8)
    scale_bytes = N * (d // block) * np.dtype(SCALE_DTYPE[bits]).itemsize
    return (code_bytes + scale_bytes + 15) // 16 * 16


def pack_rows(codes: np.ndarray, scales: np.ndarray, bits: int) -> np.ndarray:
    """codes [V][N][d] uint8, scales [V][N][d / block] -> uint8 [V][record_bytes].

    NF4: N rows of d/2 bytes, byte i of a row = code[2i] | code[2i+1] << 4; then the N * d/block scales.
    NF3: N rows of d/4 bytes holding the two low bits of every code (byte i = codes 4i .. 4i+3, code
    4i+k at bits 2k, 2k+1); then N rows of d/8 bytes holding the high bits (byte i = codes 8i .. 8i+7,
    code 8i+k at bit k); then the scales.  Zero padding up to a multiple of 16 bytes."""
    V, N, d = codes.shape
    nblk = scales.shape[2]
    block = d // nblk
    rec = np.zeros((V, record_bytes(N, d, bits, block)), dtype=np.uint8)
    c = codes.astype(np.uint8)
    if bits == 4:
        body = (c[:, :, 0::2] | (c[:, :, 1::2] << 4)).reshape(V, N * d // 2)
    else:
        lo = c & 3
        plane_a = lo[:, :, 0::4] | (lo[:, :, 1::4] << 2) | (lo[:, :, 2::4] << 4) | (lo[:, :, 3::4] << 6)
        hi = (c >> 2) & 1
        plane_b = np.zeros((V, N, d // 8), dtype=np.uint8)
        for k in range(8):
            plane_b |= hi[:, :, k::8] << k
        body = np.concatenate([plane_a.reshape(V, -1), plane_b.reshape(V, -1)], axis=1)
    sc = np.ascontiguousarray(scales.astype(SCALE_DTYPE[bits])).view(np.uint8).reshape(V, -1)
    rec[:, : body.shape[1]] = body
    rec[:, body.shape[1]: body.shape[1] + sc.shape[1]] = sc
    return rec


def unpack_rows(rec: np.ndarray, N: int, d: int, bits: int, block: int):
    """Inverse of pack_rows: (codes [V][N][d], scales [V][N][d / block])."""
    V = rec.shape[0]
    if bits == 4:
        nb = N * d // 2
        body = rec[:, :nb].reshape(V, N, d // 2)
        codes = np.empty((V, N, d), dtype=np.uint8)
        codes[:, :, 0::2] = body & 15
        codes[:, :, 1::2] = body >> 4
    else:
        na, nbp = N * d // 4, N * d // 8
        plane_a = rec[:, :na].reshape(V, N, d // 4)
        plane_b = rec[:, na: na + nbp].reshape(V, N, d // 8)
        codes = np.empty((V, N, d), dtype=np.uint8)
        for k in range(4):
            codes[:, :, k::4] = (plane_a >> (2 * k)) & 3
        for k in range(8):
            codes[:, :, k::8] |= ((plane_b >> k) & 1) << 2
        nb = na + nbp
    st = SCALE_DTYPE[bits]
    ns = N * (d // block) * np.dtype(st).itemsize
    scales = np.ascontiguousarray(rec[:, nb: nb + ns]).view(st).reshape(V, N, d // block)
    return codes, scales


def quantize_table(lut: np.ndarray, bits: int, block: int) -> np.ndarray:
    """lut [V][N][d] -> packed records uint8 [V][record_bytes]."""
    V, N, d = lut.shape
    codes, scales = quantize(lut.reshape(V * N, d), bits, block)
    return pack_rows(codes.reshape(V, N, d), scales.reshape(V, N, d // block), bits)


def dequantize_table(rec: np.ndarray, N: int, d: int, bits: int, block: int) -> np.ndarray:
    """packed records -> float64 table [V][N][d]: what a layer over the quantised table looks up."""
    codes, scales = unpack_rows(rec, N, d, bits, block)
    V = rec.shape[0]
    return dequantize(codes.reshape(V * N, d), scales.reshape(V * N, d // block), bits, block).reshape(V, N, d)
