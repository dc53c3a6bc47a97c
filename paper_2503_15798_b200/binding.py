"""Python face of the C-ABI library declared in ``include/mole.h``.

Argument marshalling only: every function takes torch tensors (used for device memory and
streams, nothing else), checks shapes and dtypes, and passes raw pointers and sizes to the
entry point of the same name.  No arithmetic of the layer happens here, and there is no
fallback: if ``libmole_b200.so`` has not been built, the first call raises.
"""
from __future__ import annotations

import ctypes
import os
from ctypes import POINTER, c_char_p, c_int, c_int32, c_int64, c_size_t, c_uint32, c_void_p

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libmole_b200.so")

OK, ERR_INVALID_ARG, ERR_UNSUPPORTED_SHAPE, ERR_CUDA, ERR_NOMEM, ERR_TOO_LARGE, ERR_IO = range(7)
STATUS_BAD_ID, STATUS_TIMEOUT = 1, 2
DTYPE_BF16, DTYPE_F32 = 0, 1
FLAG_IDS_INT64, FLAG_CHAIN = 1, 2
STEP_AUTO, STEP_FUSED, STEP_CHAINED = 0, 1, 2
KERNEL_AUTO, KERNEL_RING, KERNEL_DECODE = 0, 1, 2
LUT_PLAIN, LUT_NF4, LUT_NF3 = 0, 1, 2

# every symbol include/mole.h declares
EXPORTS = (
    "mole_layer_forward", "mole_layer_forward_ex", "mole_decode_step", "mole_decode_step_ex", "mole_decode_step_host",
    "mole_dedup_ids", "mole_dedup_ids_static", "mole_fetch_rows", "mole_host_alloc", "mole_host_free", "mole_offload_create",
    "mole_offload_destroy", "mole_offload_prefetch", "mole_layer_forward_offload", "mole_offload_decode_step",
    "mole_offload_buffers",
    "mole_status_string", "mole_last_cuda_error", "mole_version", "mole_plan", "mole_variant", "mole_reload_debug_env",
    "mole_build_lut", "mole_build_lut_scratch_bytes", "mole_table_file_write", "mole_table_file_info", "mole_table_file_read", "mole_table_file_read_rows",
    "mole_decode_step_args", "mole_offload_create_ex", "mole_offload_set_hot_rows", "mole_offload_hot_hits", "mole_nf_codebook", "mole_quant_record_bytes", "mole_quantize_lut",
    "mole_prefetch_rows",
)


class MoleArgs(ctypes.Structure):
    _fields_ = [
        ("struct_size", c_uint32), ("flags", c_uint32),
        ("hidden", c_void_p), ("ids", c_void_p), ("lut", c_void_p), ("w_router", c_void_p), ("out", c_void_p),
        ("residual", c_void_p), ("gates_out", c_void_p), ("status", c_void_p),
        ("B", c_int32), ("T", c_int32), ("N", c_int32), ("d", c_int32), ("V", c_int32),
        ("dtype", c_int32), ("kernel", c_int32), ("d_split", c_int32),
        ("stream", c_void_p),
        ("norm_weight", c_void_p), ("norm_eps", ctypes.c_float), ("lut_format", c_int32), ("lut_block", c_int32),
        ("reserved2", c_int32),
    ]


class MoleStepArgs(ctypes.Structure):
    _fields_ = [
        ("struct_size", c_uint32), ("flags", c_uint32),
        ("hidden_in", c_void_p), ("ids", c_void_p), ("lut_base", c_void_p), ("lut_layer_stride_bytes", c_int64),
        ("w_router_base", c_void_p), ("wr_layer_stride_bytes", c_int64),
        ("norm_weight_base", c_void_p), ("norm_layer_stride_bytes", c_int64),
        ("out", c_void_p), ("tmp", c_void_p), ("status", c_void_p),
        ("L", c_int32), ("B", c_int32), ("T", c_int32), ("N", c_int32), ("d", c_int32), ("V", c_int32),
        ("dtype", c_int32), ("mode", c_int32), ("d_split", c_int32), ("kernel", c_int32),
        ("norm_eps", ctypes.c_float), ("lut_format", c_int32), ("lut_block", c_int32), ("reserved", c_int32),
        ("stream", c_void_p),
    ]


class MoleTableInfo(ctypes.Structure):
    _fields_ = [("L", c_int64), ("V", c_int64), ("N", c_int32), ("d", c_int32), ("dtype", c_int32), ("lut_format", c_int32),
                ("lut_block", c_int32), ("reserved", c_int32), ("row_bytes", c_int64)]


class MoleError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        msg = lib().mole_status_string(code).decode()
        if code == ERR_CUDA:
            msg += ": " + lib().mole_last_cuda_error().decode()
        super().__init__(f"{where}: {msg} (code {code})")


_lib = None


def lib() -> ctypes.CDLL:
    """The loaded library.  Raises if it is missing -- there is no other implementation."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(
                f"{LIB_PATH} is missing: build it with `python -m paper_2503_15798_b200.build` "
                "(nvcc, sm_100a); this package has no fallback path")
        L = ctypes.CDLL(LIB_PATH)
        vp, ip = c_void_p, c_void_p
        L.mole_layer_forward.argtypes = [vp, ip, vp, vp, vp, c_int, c_int, c_int, c_int, c_int, vp]
        L.mole_layer_forward_ex.argtypes = [POINTER(MoleArgs)]
        L.mole_decode_step.argtypes = [vp, ip, vp, c_int64, vp, c_int64, vp, vp, vp, c_int, c_int, c_int, c_int,
                                       c_int, c_int, c_int, vp]
        L.mole_decode_step_ex.argtypes = [vp, ip, vp, c_int64, vp, c_int64, vp, vp, vp, c_int, c_int, c_int, c_int,
                                          c_int, c_int, c_int, c_int, c_int, vp]
        L.mole_decode_step_host.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp, c_int64, vp, c_int64, vp, c_int, c_int,
                                            c_int, c_int, c_int, c_int, c_int, vp]
        L.mole_dedup_ids.argtypes = [ip, c_int, c_int, ip, ip, ip, ip, vp, vp]
        L.mole_dedup_ids_static.argtypes = [ip, c_int, c_int, ip, ip, ip, vp, vp]
        L.mole_fetch_rows.argtypes = [vp, ip, ip, c_int, c_int64, vp, vp]
        L.mole_host_alloc.argtypes = [POINTER(c_void_p), c_size_t]
        L.mole_host_free.argtypes = [vp]
        L.mole_offload_create.argtypes = [POINTER(c_void_p), c_int, c_int, c_int, c_int, c_int, c_int]
        L.mole_offload_create_ex.argtypes = [POINTER(c_void_p), c_int, c_int, c_int, c_int, c_int, c_int, c_int, c_int]
        L.mole_build_lut_scratch_bytes.argtypes = [c_int, c_int, c_int, c_int, c_int, POINTER(c_int64)]
        L.mole_build_lut.argtypes = [vp, vp, vp, vp, ctypes.c_float, vp, vp, c_int, c_int, c_int, c_int, vp, vp]
        L.mole_table_file_write.argtypes = [c_char_p, vp, c_int64, c_int, c_int, c_int, c_int, c_int, c_int, c_int]
        L.mole_table_file_info.argtypes = [c_char_p, POINTER(MoleTableInfo)]
        L.mole_table_file_read.argtypes = [c_char_p, vp, c_int64, c_int, c_int]
        L.mole_table_file_read_rows.argtypes = [c_char_p, c_int, vp, c_int, vp]
        L.mole_offload_set_hot_rows.argtypes = [vp, vp, c_int, vp, c_int64, c_int]
        L.mole_offload_hot_hits.argtypes = [vp, POINTER(ctypes.c_uint64), c_int]
        L.mole_offload_destroy.argtypes = [vp]
        L.mole_offload_prefetch.argtypes = [vp, c_int, ip, c_int, vp, vp]
        L.mole_layer_forward_offload.argtypes = [vp, c_int, vp, vp, vp, vp, c_int, c_int, vp]
        L.mole_offload_decode_step.argtypes = [vp, vp, ip, vp, c_int64, vp, c_int64, vp, vp, vp, c_int, c_int, c_int, vp, vp]
        L.mole_offload_buffers.argtypes = [vp, c_int, POINTER(c_void_p), POINTER(c_void_p), POINTER(c_void_p),
                                           POINTER(c_void_p)]
        L.mole_status_string.argtypes = [c_int]
        L.mole_status_string.restype = c_char_p
        L.mole_last_cuda_error.argtypes = []
        L.mole_last_cuda_error.restype = c_char_p
        L.mole_version.argtypes = []
        L.mole_plan.argtypes = [c_int, c_int, c_int, c_int, c_int, c_int, POINTER(c_int), POINTER(c_int),
                                POINTER(c_int), POINTER(c_int), POINTER(c_int)]
        L.mole_variant.argtypes = [c_int, c_int, c_int, c_int, c_int, c_int, c_int, c_int, c_int, c_int, ctypes.c_char_p,
                                   c_int, POINTER(c_int), POINTER(c_int)]
        L.mole_reload_debug_env.argtypes = []
        L.mole_decode_step_args.argtypes = [POINTER(MoleStepArgs)]
        L.mole_nf_codebook.argtypes = [c_int, POINTER(ctypes.c_float)]
        L.mole_quant_record_bytes.argtypes = [c_int, c_int, c_int, c_int, POINTER(c_int64)]
        L.mole_quantize_lut.argtypes = [vp, vp, c_int64, c_int, c_int, c_int, c_int, vp]
        L.mole_prefetch_rows.argtypes = [vp, c_int, vp, c_int64, c_int, c_int, c_int, c_int, c_int, ctypes.c_uint32, vp]
        for name in EXPORTS:
            fn = getattr(L, name)
            if fn.restype is not c_char_p:
                fn.restype = c_int
        _lib = L
    return _lib


def _check(code: int, where: str):
    if code != OK:
        raise MoleError(code, where)


def _dtype_tag(t: torch.Tensor) -> int:
    if t.dtype == torch.bfloat16:
        return DTYPE_BF16
    if t.dtype == torch.float32:
        return DTYPE_F32
    raise TypeError(f"unsupported element type {t.dtype}")


def _ptr(t):
    return None if t is None else t.data_ptr()


def _stream(stream) -> int:
    if stream is None:
        return torch.cuda.current_stream().cuda_stream
    if isinstance(stream, int):
        return stream
    return stream.cuda_stream


def _dev(t: torch.Tensor, name: str):
    if not (t.is_cuda and t.is_contiguous()):
        raise ValueError(f"{name} must be a contiguous CUDA tensor")


class QuantTable:
    """A table quantised to NF4 / NF3 (Sec. 4.5 of the paper): `packed` is a uint8 device (or pinned host)
    tensor [V][record_bytes] -- or [L][V][record_bytes] for the tables of L layers -- of the records
    mole_quantize_lut writes."""

    def __init__(self, packed, N: int, d: int, fmt: int, block: int):
        self.packed, self.N, self.d, self.fmt, self.block = packed, N, d, fmt, block
        self.record_bytes = quant_record_bytes(N, d, fmt, block)
        if packed.dtype != torch.uint8 or packed.shape[-1] != self.record_bytes:
            raise ValueError("packed must be uint8 [..., V, record_bytes]")
        self.V = packed.shape[-2]

    def layer(self, l: int) -> "QuantTable":
        return QuantTable(self.packed[l], self.N, self.d, self.fmt, self.block)

    @staticmethod
    def quantize(lut, fmt: int, block: int, out=None, stream=None) -> "QuantTable":
        """mole_quantize_lut: lut bf16 [V][N][d] (or [L][V][N][d]) on the device."""
        _dev(lut, "lut")
        if lut.dtype != torch.bfloat16:
            raise TypeError("mole_quantize_lut takes a bf16 table")
        N, d = lut.shape[-2], lut.shape[-1]
        rb = quant_record_bytes(N, d, fmt, block)
        lead = tuple(lut.shape[:-2])
        if out is None:
            out = torch.zeros(lead + (rb,), dtype=torch.uint8, device=lut.device)
        rows = 1
        for n in lead:
            rows *= n
        _check(lib().mole_quantize_lut(_ptr(lut), _ptr(out), rows, N, d, fmt, block, _stream(stream)), "mole_quantize_lut")
        return QuantTable(out, N, d, fmt, block)


def nf_codebook(fmt: int):
    """mole_nf_codebook: the codebook values (16 for NF4, 8 for NF3) as Python floats (exact float32 values)."""
    buf = (ctypes.c_float * 16)()
    _check(lib().mole_nf_codebook(fmt, buf), "mole_nf_codebook")
    return [float(buf[i]) for i in range(16 if fmt == LUT_NF4 else 8)]


def quant_record_bytes(N: int, d: int, fmt: int, block: int) -> int:
    b = c_int64()
    _check(lib().mole_quant_record_bytes(N, d, fmt, block, ctypes.byref(b)), "mole_quant_record_bytes")
    return b.value


def layer_forward(hidden, ids, lut, w_router, out=None, *, residual=None, gates_out=None, status=None,
                  d_split: int = 0, chain: bool = False, stream=None, B=None, T=None, norm_weight=None,
                  norm_eps: float = 1e-6, kernel: int = KERNEL_AUTO):
    """mole_layer_forward_ex.  hidden [M][d] (or [B][T][d]), ids [M] int32/int64, lut [V][N][d] or a
    QuantTable, w_router [d][N]; returns out (allocated like hidden if not given).  norm_weight [d]: the
    router reads RMSNorm(hidden) with that scale and norm_eps, the residual stays un-normalised."""
    quant = lut if isinstance(lut, QuantTable) else None
    lut_t = quant.packed if quant else lut
    for name, t in (("hidden", hidden), ("ids", ids), ("lut", lut_t), ("w_router", w_router)):
        _dev(t, name)
    if quant:
        V, N, d = quant.V, quant.N, quant.d
        if quant.packed.dim() != 2:
            raise ValueError("a single layer takes one table: use QuantTable.layer(l)")
    else:
        V, N, d = lut.shape
    M = hidden.numel() // d if d else 0
    if hidden.shape[-1] != d or tuple(w_router.shape) != (d, N) or ids.numel() != M:
        raise ValueError("shape mismatch between hidden, ids, lut and w_router")
    tag = _dtype_tag(hidden)
    if not ((quant or lut.dtype == hidden.dtype) and w_router.dtype == hidden.dtype):
        raise TypeError("hidden, lut and w_router must share one element type")
    if out is None:
        out = torch.empty_like(hidden)
    _dev(out, "out")
    flags = 0
    if ids.dtype == torch.int64:
        flags |= FLAG_IDS_INT64
    elif ids.dtype != torch.int32:
        raise TypeError("ids must be int32 or int64")
    if chain:
        flags |= FLAG_CHAIN
    if B is None:
        B, T = M, 1
    a = MoleArgs()
    a.struct_size = ctypes.sizeof(MoleArgs)
    a.flags = flags
    a.hidden, a.ids, a.lut, a.w_router, a.out = _ptr(hidden), _ptr(ids), _ptr(lut_t), _ptr(w_router), _ptr(out)
    a.residual, a.gates_out, a.status = _ptr(residual), _ptr(gates_out), _ptr(status)
    a.B, a.T, a.N, a.d, a.V = B, T, N, d, V
    a.dtype, a.kernel, a.d_split = tag, kernel, d_split
    a.stream = _stream(stream)
    if norm_weight is not None:
        _dev(norm_weight, "norm_weight")
        if norm_weight.dtype != hidden.dtype or norm_weight.numel() != d:
            raise ValueError("norm_weight must be [d] of the element type of hidden")
    a.norm_weight, a.norm_eps, a.reserved2 = _ptr(norm_weight), float(norm_eps), 0
    a.lut_format, a.lut_block = (quant.fmt, quant.block) if quant else (LUT_PLAIN, 0)
    _check(lib().mole_layer_forward_ex(ctypes.byref(a)), "mole_layer_forward_ex")
    return out


def layer_forward_basic(hidden, ids, lut, w_router, out, stream=None):
    """mole_layer_forward (bf16, int32 ids), the plain entry point."""
    V, N, d = lut.shape
    M = ids.numel()
    _check(lib().mole_layer_forward(_ptr(hidden), _ptr(ids), _ptr(lut), _ptr(w_router), _ptr(out), M, 1, N, d, V,
                                    _stream(stream)), "mole_layer_forward")
    return out


def decode_step(hidden_in, ids, luts, w_routers, out, tmp=None, status=None, stream=None, mode: int = STEP_AUTO,
                d_split: int = 0):
    """mole_decode_step_ex: luts [L][V][N][d], w_routers [L][d][N]; returns out.  mode: STEP_AUTO,
    STEP_FUSED (one launch over all layers) or STEP_CHAINED (L launches, needs tmp when L > 1)."""
    L, V, N, d = luts.shape
    M = ids.numel()
    tag = _dtype_tag(hidden_in)
    _check(lib().mole_decode_step_ex(_ptr(hidden_in), _ptr(ids), _ptr(luts), luts.stride(0) * luts.element_size(),
                                     _ptr(w_routers), w_routers.stride(0) * w_routers.element_size(), _ptr(out),
                                     _ptr(tmp), _ptr(status), L, M, 1, N, d, V, tag, mode, d_split, _stream(stream)),
           "mole_decode_step_ex")
    return out


def decode_step_args(hidden_in, ids, luts, w_routers, out, tmp=None, status=None, stream=None, mode: int = STEP_AUTO,
                     d_split: int = 0, norm_weights=None, norm_eps: float = 1e-6, kernel: int = KERNEL_AUTO,
                     chain_first: bool = False):
    """mole_decode_step_args: decode_step with every option; luts [L][V][N][d] or a QuantTable with packed
    [L][V][record_bytes]; norm_weights [L][d] puts RMSNorm(hidden) in front of every layer's router."""
    quant = luts if isinstance(luts, QuantTable) else None
    if quant:
        lut_t = quant.packed
        L, V, N, d = lut_t.shape[0], quant.V, quant.N, quant.d
    else:
        lut_t = luts
        L, V, N, d = luts.shape
    a = MoleStepArgs()
    a.struct_size = ctypes.sizeof(MoleStepArgs)
    a.flags = FLAG_CHAIN if chain_first else 0
    a.hidden_in, a.ids, a.lut_base = _ptr(hidden_in), _ptr(ids), _ptr(lut_t)
    a.lut_layer_stride_bytes = lut_t.stride(0) * lut_t.element_size()
    a.w_router_base, a.wr_layer_stride_bytes = _ptr(w_routers), w_routers.stride(0) * w_routers.element_size()
    if norm_weights is not None:
        _dev(norm_weights, "norm_weights")
        if norm_weights.dtype != hidden_in.dtype or tuple(norm_weights.shape) != (L, d):
            raise ValueError("norm_weights must be [L][d] of the element type of hidden")
        a.norm_weight_base, a.norm_layer_stride_bytes = _ptr(norm_weights), norm_weights.stride(0) * norm_weights.element_size()
    a.out, a.tmp, a.status = _ptr(out), _ptr(tmp), _ptr(status)
    a.L, a.B, a.T, a.N, a.d, a.V = L, ids.numel(), 1, N, d, V
    a.dtype, a.mode, a.d_split, a.kernel = _dtype_tag(hidden_in), mode, d_split, kernel
    a.norm_eps, a.reserved = float(norm_eps), 0
    a.lut_format, a.lut_block = (quant.fmt, quant.block) if quant else (LUT_PLAIN, 0)
    a.stream = _stream(stream)
    _check(lib().mole_decode_step_args(ctypes.byref(a)), "mole_decode_step_args")
    return out


def decode_step_basic(hidden_in, ids, luts, w_routers, out, tmp=None, status=None, stream=None):
    """mole_decode_step, the plain entry point (mode and split chosen by the library)."""
    L, V, N, d = luts.shape
    M = ids.numel()
    tag = _dtype_tag(hidden_in)
    _check(lib().mole_decode_step(_ptr(hidden_in), _ptr(ids), _ptr(luts), luts.stride(0) * luts.element_size(),
                                  _ptr(w_routers), w_routers.stride(0) * w_routers.element_size(), _ptr(out),
                                  _ptr(tmp), _ptr(status), L, M, 1, N, d, V, tag, _stream(stream)),
           "mole_decode_step")
    return out


def decode_step_host(hidden_host, ids_host, out_host, dev_hidden, dev_ids, dev_out, dev_tmp, luts, w_routers,
                     status=None, stream=None):
    """mole_decode_step_host: activations in (pinned) host tensors, tables on the device."""
    L, V, N, d = luts.shape
    M = ids_host.numel()
    tag = _dtype_tag(dev_hidden)
    _check(lib().mole_decode_step_host(_ptr(hidden_host), _ptr(ids_host), _ptr(out_host), _ptr(dev_hidden),
                                       _ptr(dev_ids), _ptr(dev_out), _ptr(dev_tmp), _ptr(luts),
                                       luts.stride(0) * luts.element_size(), _ptr(w_routers),
                                       w_routers.stride(0) * w_routers.element_size(), _ptr(status), L, M, 1, N, d,
                                       V, tag, _stream(stream)), "mole_decode_step_host")
    return out_host


def prefetch_rows(ids, luts, layers: int = 0, first_layer: int = 0, stream=None):
    """mole_prefetch_rows: an L2 prefetch of the rows of `ids` in `layers` tables of luts [L][V][N][d] from
    first_layer on (all of them by default).  A hint; no result changes."""
    L, V, N, d = luts.shape
    n = layers if layers > 0 else L - first_layer
    flags = FLAG_IDS_INT64 if ids.dtype == torch.int64 else 0
    _check(lib().mole_prefetch_rows(_ptr(ids), ids.numel(), ctypes.c_void_p(luts.data_ptr() + first_layer * luts.stride(0) * luts.element_size()),
                                    luts.stride(0) * luts.element_size(), n, N, d, V, _dtype_tag(luts), flags, _stream(stream)),
           "mole_prefetch_rows")


def dedup_ids(ids, V: int, scratch, uniq, slot, count, status=None, stream=None):
    """mole_dedup_ids: all tensors int32 on the device; scratch [V] must be zero on entry."""
    _check(lib().mole_dedup_ids(_ptr(ids), ids.numel(), V, _ptr(scratch), _ptr(uniq), _ptr(slot), _ptr(count),
                                _ptr(status), _stream(stream)), "mole_dedup_ids")


STATIC_DEDUP_MAX_V = 65536


def dedup_ids_static(ids, V: int, uniq, slot, count, status=None, stream=None):
    """mole_dedup_ids_static: dedup_ids without a caller-supplied scratch table, for callers that
    cannot allocate device memory; the table is a fixed 256 KB array inside the library, shared by
    all calls on a device (so calls must not overlap on the GPU).  V <= STATIC_DEDUP_MAX_V."""
    _check(lib().mole_dedup_ids_static(_ptr(ids), ids.numel(), V, _ptr(uniq), _ptr(slot), _ptr(count),
                                       _ptr(status), _stream(stream)), "mole_dedup_ids_static")


def fetch_rows(lut_host, uniq, count, max_rows: int, staging, stream=None):
    """mole_fetch_rows: lut_host is a pinned host tensor [V][N][d]; staging a device tensor."""
    row_bytes = lut_host[0].numel() * lut_host.element_size()
    _check(lib().mole_fetch_rows(_ptr(lut_host), _ptr(uniq), _ptr(count), max_rows, row_bytes, _ptr(staging),
                                 _stream(stream)), "mole_fetch_rows")


class _DevicePointer:
    """Lets torch view memory the library owns (CUDA array interface, no copy)."""

    def __init__(self, ptr: int, shape, typestr: str):
        self.__cuda_array_interface__ = {"shape": tuple(shape), "typestr": typestr, "data": (ptr, False),
                                         "version": 2}


def _wrap_device(ptr: int, shape, typestr: str) -> torch.Tensor:
    return torch.as_tensor(_DevicePointer(ptr, shape, typestr), device="cuda")


class HostTable:
    """A pinned, device-mapped host allocation from mole_host_alloc, viewed as a torch tensor."""

    def __init__(self, shape, dtype=torch.bfloat16):
        n = 1
        for s in shape:
            n *= s
        self.nbytes = n * torch.empty((), dtype=dtype).element_size()
        p = c_void_p()
        _check(lib().mole_host_alloc(ctypes.byref(p), self.nbytes), "mole_host_alloc")
        self.ptr = p.value
        buf = (ctypes.c_uint8 * self.nbytes).from_address(self.ptr)
        self.tensor = torch.frombuffer(buf, dtype=torch.uint8).view(dtype).view(*shape)

    def free(self):
        if self.ptr:
            self.tensor = None
            _check(lib().mole_host_free(self.ptr), "mole_host_free")
            self.ptr = None


class OffloadContext:
    """mole_offload_create / prefetch / forward / destroy."""

    def __init__(self, max_tokens: int, N: int, d: int, V: int, dtype=torch.bfloat16, n_buffers: int = 2,
                 lut_format: int = LUT_PLAIN, lut_block: int = 0):
        self.max_tokens, self.N, self.d, self.V, self.dtype, self.n_buffers = max_tokens, N, d, V, dtype, n_buffers
        tag = DTYPE_BF16 if dtype == torch.bfloat16 else DTYPE_F32
        h = c_void_p()
        _check(lib().mole_offload_create_ex(ctypes.byref(h), max_tokens, N, d, V, tag, n_buffers, lut_format, lut_block),
               "mole_offload_create_ex")
        self.handle = h.value

    def prefetch(self, buf: int, ids, lut_host_layer, side_stream=None):
        _check(lib().mole_offload_prefetch(self.handle, buf, _ptr(ids), ids.numel(), _ptr(lut_host_layer),
                                           _stream(side_stream)), "mole_offload_prefetch")

    def forward(self, buf: int, hidden, w_router, out, status=None, stream=None):
        M = hidden.numel() // self.d
        _check(lib().mole_layer_forward_offload(self.handle, buf, _ptr(hidden), _ptr(w_router), _ptr(out),
                                                _ptr(status), M, 1, _stream(stream)), "mole_layer_forward_offload")
        return out

    def decode_step(self, hidden_in, ids, luts_host, w_routers, out, tmp=None, status=None, stream=None, side_stream=None):
        """mole_offload_decode_step: luts_host [L][V][N][d] pinned host tensor, w_routers [L][d][N] device."""
        L = luts_host.shape[0]
        M = ids.numel()
        _check(lib().mole_offload_decode_step(self.handle, _ptr(hidden_in), _ptr(ids), _ptr(luts_host),
                                              luts_host.stride(0) * luts_host.element_size(), _ptr(w_routers),
                                              w_routers.stride(0) * w_routers.element_size(), _ptr(out), _ptr(tmp),
                                              _ptr(status), L, M, 1, _stream(stream), _stream(side_stream)),
               "mole_offload_decode_step")
        return out

    def set_hot_rows(self, hot_ids, luts_host):
        """mole_offload_set_hot_rows: keep the rows of hot_ids (host int32 tensor / array, distinct) of every layer of
        luts_host ([L][V][...] pinned host tensor) in device memory; an empty list frees the cache."""
        ids = torch.as_tensor(hot_ids, dtype=torch.int32).contiguous().cpu()
        L = luts_host.shape[0]
        _check(lib().mole_offload_set_hot_rows(self.handle, _ptr(ids) if ids.numel() else None, ids.numel(), _ptr(luts_host),
                                               luts_host.stride(0) * luts_host.element_size(), L), "mole_offload_set_hot_rows")

    def hot_hits(self, reset: bool = False) -> int:
        h = ctypes.c_uint64()
        _check(lib().mole_offload_hot_hits(self.handle, ctypes.byref(h), int(reset)), "mole_offload_hot_hits")
        return h.value

    def buffers(self, buf: int):
        """(uniq, slot, count, staging) device pointers of a buffer, as ints."""
        u, s, c, g = c_void_p(), c_void_p(), c_void_p(), c_void_p()
        _check(lib().mole_offload_buffers(self.handle, buf, ctypes.byref(u), ctypes.byref(s), ctypes.byref(c),
                                          ctypes.byref(g)), "mole_offload_buffers")
        return u.value, s.value, c.value, g.value

    def read_buffer(self, buf: int):
        """Host copies of a buffer's (uniq[:count], slot[:max_tokens], count); synchronises."""
        u, s, c, _ = self.buffers(buf)
        torch.cuda.synchronize()
        n = int(_wrap_device(c, (1,), "<i4").cpu().item())
        uniq = _wrap_device(u, (self.max_tokens,), "<i4").cpu()
        slot = _wrap_device(s, (self.max_tokens,), "<i4").cpu()
        return uniq[:n].clone(), slot, n

    def destroy(self):
        if self.handle:
            _check(lib().mole_offload_destroy(self.handle), "mole_offload_destroy")
            self.handle = None

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass


def plan(M: int, N: int, d: int, dtype: int = DTYPE_BF16, d_split: int = 0, L: int = 1):
    """mole_plan: (d_split, threads, smem_bytes, stages, blocks_per_sm) of a launch over M tokens
    and L layers (L = 1: a single layer)."""
    a, b, c, e, f = c_int(), c_int(), c_int(), c_int(), c_int()
    _check(lib().mole_plan(M, L, N, d, dtype, d_split, ctypes.byref(a), ctypes.byref(b), ctypes.byref(c),
                           ctypes.byref(e), ctypes.byref(f)), "mole_plan")
    return a.value, b.value, c.value, e.value, f.value


def variant(M: int, N: int, d: int, dtype: int = DTYPE_BF16, d_split: int = 0, L: int = 1, norm: bool = False,
            kernel: int = KERNEL_AUTO, lut_format: int = LUT_PLAIN, lut_block: int = 0):
    """mole_variant: (name, threads, smem_bytes) of the kernel instantiation a launch of this shape runs."""
    buf = ctypes.create_string_buffer(96)
    th, sm = c_int(), c_int()
    _check(lib().mole_variant(M, L, N, d, dtype, d_split, int(norm), kernel, lut_format, lut_block, buf, len(buf),
                              ctypes.byref(th), ctypes.byref(sm)), "mole_variant")
    return buf.value.decode(), th.value, sm.value


class debug_env:
    """Context manager: set MOLE_FORCE_* / MOLE_DEBUG_* variables, make the library read them, and put
    the environment back (and make the library read it again) on exit."""

    def __init__(self, **variables):
        self.variables = {k: str(v) for k, v in variables.items()}
        self.saved = {}

    def __enter__(self):
        for k, v in self.variables.items():
            self.saved[k] = os.environ.get(k)
            os.environ[k] = v
        _check(lib().mole_reload_debug_env(), "mole_reload_debug_env")
        return self

    def __exit__(self, *exc):
        for k, old in self.saved.items():
            if old is None:
                os.environ.pop(k, None)
            else:
                os.environ[k] = old
        _check(lib().mole_reload_debug_env(), "mole_reload_debug_env")


def build_lut(embedding, w1, w2, norm_weight=None, norm_eps: float = 1e-6, out=None, status=None, stream=None):
    """mole_build_lut (Eq. 6-7 on the tensor cores): embedding [V][d], w1 [N][D][d], w2 [N][d][D], all bf16 on the
    device; returns the table [V][N][d] bf16.  The scratch buffer is allocated here (torch) and freed on return."""
    for name, t in (("embedding", embedding), ("w1", w1), ("w2", w2)):
        _dev(t, name)
        if t.dtype != torch.bfloat16:
            raise TypeError("mole_build_lut takes bf16 inputs")
    V, d = embedding.shape
    N, D, d1 = w1.shape
    if d1 != d or tuple(w2.shape) != (N, d, D):
        raise ValueError("shape mismatch between embedding, w1 and w2")
    if out is None:
        out = torch.empty((V, N, d), dtype=torch.bfloat16, device=embedding.device)
    b = c_int64()
    _check(lib().mole_build_lut_scratch_bytes(V, N, d, D, int(norm_weight is not None), ctypes.byref(b)), "mole_build_lut_scratch_bytes")
    scratch = torch.empty(b.value, dtype=torch.uint8, device=embedding.device)
    _check(lib().mole_build_lut(_ptr(embedding), _ptr(w1), _ptr(w2), _ptr(norm_weight), float(norm_eps), _ptr(out), _ptr(scratch),
                                V, N, d, D, _ptr(status), _stream(stream)), "mole_build_lut")
    torch.cuda.current_stream().synchronize() if stream is None else None  # the scratch buffer dies with this frame
    return out


def table_file_write(path: str, tables, N: int, d: int, lut_format: int = LUT_PLAIN, lut_block: int = 0):
    """mole_table_file_write: tables is a CPU tensor [L][V][N][d] (plain) or uint8 [L][V][record_bytes] (quantised)."""
    t = tables.contiguous()
    dtype = DTYPE_BF16 if lut_format != LUT_PLAIN else _dtype_tag(t)
    _check(lib().mole_table_file_write(path.encode(), _ptr(t), t.stride(0) * t.element_size(), t.shape[0], t.shape[1], N, d, dtype,
                                       lut_format, lut_block), "mole_table_file_write")


def table_file_info(path: str) -> MoleTableInfo:
    info = MoleTableInfo()
    _check(lib().mole_table_file_info(path.encode(), ctypes.byref(info)), "mole_table_file_info")
    return info


def table_file_read(path: str, dst, layer0: int = 0, n_layers: int = None):
    """mole_table_file_read into a CPU (ideally pinned) tensor whose first axis is the layer."""
    n = dst.shape[0] if n_layers is None else n_layers
    _check(lib().mole_table_file_read(path.encode(), _ptr(dst), dst.stride(0) * dst.element_size(), layer0, n), "mole_table_file_read")
    return dst


def table_file_read_rows(path: str, layer: int, ids, dst):
    ids = torch.as_tensor(ids, dtype=torch.int32).contiguous().cpu()
    _check(lib().mole_table_file_read_rows(path.encode(), layer, _ptr(ids), ids.numel(), _ptr(dst)), "mole_table_file_read_rows")
    return dst


def version() -> int:
    return lib().mole_version()
