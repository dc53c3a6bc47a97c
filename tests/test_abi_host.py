"""Host-side checks of the C-ABI library that need no GPU: it loads, exports every symbol
the header declares, names its status codes, plans launches, and rejects bad arguments
before touching CUDA."""
import ctypes
import os
import re

import pytest

from paper_2503_15798_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
HEADER = os.path.join(ROOT, "include", "mole.h")


@pytest.fixture(scope="module")
def lib():
    build.build()
    return binding.lib()


def declared_symbols():
    text = open(HEADER).read()
    return sorted(set(re.findall(r"MOLE_API\s+(?:const\s+char\s*\*|int)\s*(mole_\w+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = declared_symbols()
    assert len(names) >= 17
    for n in names:
        assert hasattr(lib, n), n
    assert set(names) == set(binding.EXPORTS)


def test_version_and_status_strings(lib):
    assert lib.mole_version() == 300
    seen = {lib.mole_status_string(c).decode() for c in range(7)}
    assert len(seen) == 7 and "ok" in seen
    assert lib.mole_status_string(99).decode() == "unknown status"


def test_variant_names_and_kernel_choice(lib):
    V = binding.variant
    D, R = binding.KERNEL_DECODE, binding.KERNEL_RING
    # the library's own choice: the ring kernel, single layers and fused steps alike
    assert V(256, 16, 768)[0] == "step<bf16,16,1,2,1,1,0>" == V(256, 16, 768, kernel=R)[0]
    assert V(16384, 16, 1024)[0] == "step<bf16,16,1,2,2,0,0>" and V(256, 16, 768, L=12)[0] == "step<bf16,16,1,1,1,0,0>"
    assert V(256, 32, 2048)[0] == "step<bf16,32,2,3,3,0,0>" and V(64, 32, 2048, L=16)[0] == "step<bf16,32,2,3,4,0,0>"
    # on request: one block per token (d / 4 threads), and the fused step built on it
    assert V(256, 16, 768, kernel=D) == ("decode<16,0>", 192, V(256, 16, 768, kernel=D)[2]) and V(64, 16, 1024, kernel=D)[:2] == ("decode<16,0>", 256)
    assert V(256, 16, 768, norm=True, kernel=D)[0] == "decode<16,1>" and V(64, 32, 1024, kernel=D)[0] == "decode<32,0>"
    assert V(256, 16, 768, L=12, kernel=D)[0] == "fstep<16,1,0>" and V(64, 32, 2048, L=16, kernel=D)[0] == "fstep<32,2,0>"
    # the widest layers: one token per cluster of four blocks, the library's own choice up to 128 tokens
    assert V(256, 32, 2048, kernel=D)[:2] == ("cdecode<32,4,0>", 128) == V(128, 32, 2048)[:2] and V(16, 16, 2048, kernel=D)[0] == "cdecode<16,4,0>"
    assert V(136, 32, 2048)[0].startswith("step<") and V(16, 16, 2048)[0].startswith("step<") and V(16, 32, 2048, kernel=R)[0].startswith("step<")
    assert V(64, 32, 2048, norm=True)[0] == "cdecode<32,4,1>"
    for args, kw in (((256, 32, 4096), {}), ((64, 5, 768), {}), ((64, 16, 768), {"d_split": 2}), ((64, 4, 64, binding.DTYPE_F32), {})):
        with pytest.raises(binding.MoleError) as e:  # shapes the family does not cover
            V(*args, kernel=D, **kw)
        assert e.value.code == binding.ERR_UNSUPPORTED_SHAPE
    assert V(64, 5, 768)[0].startswith("step<bf16,0,") and V(64, 4, 64, binding.DTYPE_F32)[0].startswith("step<f32,4,")
    # quantised tables
    assert V(256, 16, 768, lut_format=binding.LUT_NF4, lut_block=768)[0] == "qdecode<16,nf4,0>"


def test_plan_shapes():
    P = binding.plan
    # rows of up to 32 KB per token travel as one chunk; a ring of slots and one producer warp
    for d in (768, 1024):
        k, threads, smem, stages, per_sm = P(16384, 16, d)
        assert k == 1 and 2 <= stages <= 8 and smem <= 227 * 1024 and threads == d // 8 + 32  # one lane per column group
        assert per_sm >= 2 and per_sm * (smem + 1024) <= 228 * 1024
    # the 1B-shaped rows (128 KB per token) are cut into column chunks of at most 32 KB
    k, threads, smem, stages, per_sm = P(256, 32, 2048)
    assert k == 4 and stages >= 2 and smem <= 227 * 1024
    # few tokens: one block per SM may use all of its shared memory for a deep ring
    B = binding.DTYPE_BF16
    assert P(64, 16, 768, B, 0, 12)[3] > P(16384, 16, 768, B, 0, 12)[3] and P(64, 16, 768, B, 0, 12)[4] == 1
    # at most one token per SM and a streaming router: chunks of up to 64 KB in a ring of three
    assert P(64, 32, 2048, B, 0, 16)[0] == 2 and P(64, 32, 2048, B, 0, 16)[3] >= 3 and P(148, 32, 2048, B, 0, 1)[0] == 2
    assert P(149, 32, 2048, B, 0, 16)[0] == 4 and P(64, 16, 1024, B, 0, 24)[0] == 1
    # an explicit number of chunks is honoured
    assert P(64, 16, 768, binding.DTYPE_BF16, 4)[0] == 4 and P(64, 16, 768, binding.DTYPE_BF16, 1)[0] == 1
    # never a deeper ring than the chunks a block will see
    assert P(1, 16, 768, binding.DTYPE_BF16, 1, 1)[3] == 2 and P(1, 16, 768, binding.DTYPE_BF16, 1, 3)[3] == 6
    # fp32 tiny shape
    k, threads, smem, stages, per_sm = P(64, 4, 64, binding.DTYPE_F32)
    assert k == 1 and threads == 96 and smem >= 2 * 4 * 64 * 4  # 16 groups x 4 lanes + the producer warp


def test_plan_rejects_bad_shapes():
    for args in ((64, 0, 768), (64, 65, 768), (64, 16, 772), (64, 16, 4)):
        with pytest.raises(binding.MoleError) as e:
            binding.plan(*args)
        assert e.value.code == binding.ERR_UNSUPPORTED_SHAPE
    with pytest.raises(binding.MoleError) as e:
        binding.plan(64, 16, 768, 7)
    assert e.value.code == binding.ERR_INVALID_ARG
    with pytest.raises(binding.MoleError) as e:
        binding.plan(64, 16, 768, binding.DTYPE_BF16, 3)
    assert e.value.code == binding.ERR_INVALID_ARG
    with pytest.raises(binding.MoleError) as e:
        binding.plan(64, 16, 768, binding.DTYPE_BF16, 0, 0)  # zero layers
    assert e.value.code == binding.ERR_INVALID_ARG
    with pytest.raises(binding.MoleError) as e:  # 768 / 16 columns is not a whole number of vectors
        binding.plan(64, 16, 40, binding.DTYPE_BF16, 8)
    assert e.value.code == binding.ERR_UNSUPPORTED_SHAPE


def test_forward_rejects_bad_arguments_without_launching(lib):
    good = 0x10000  # an aligned, non-null address that is never dereferenced: every call below fails validation
    f = lib.mole_layer_forward
    assert f(None, good, good, good, good, 4, 1, 16, 768, 100, None) == binding.ERR_INVALID_ARG
    assert f(good, None, good, good, good, 4, 1, 16, 768, 100, None) == binding.ERR_INVALID_ARG
    assert f(good, good, good + 8, good, good, 4, 1, 16, 768, 100, None) == binding.ERR_INVALID_ARG  # misaligned table
    assert f(good, good, good, good, good, -1, 1, 16, 768, 100, None) == binding.ERR_INVALID_ARG
    assert f(good, good, good, good, good, 4, 1, 65, 768, 100, None) == binding.ERR_UNSUPPORTED_SHAPE
    assert f(good, good, good, good, good, 4, 1, 16, 772, 100, None) == binding.ERR_UNSUPPORTED_SHAPE
    assert f(good, good, good, good, good, 4, 1, 16, 768, 0, None) == binding.ERR_UNSUPPORTED_SHAPE
    # zero tokens: success, nothing launched, pointers not even looked at
    assert f(None, None, None, None, None, 0, 7, 16, 768, 100, None) == binding.OK
    assert f(None, None, None, None, None, 3, 0, 16, 768, 100, None) == binding.OK


def test_ex_rejects_bad_struct(lib):
    a = binding.MoleArgs()
    assert lib.mole_layer_forward_ex(None) == binding.ERR_INVALID_ARG
    a.struct_size = 12
    assert lib.mole_layer_forward_ex(ctypes.byref(a)) == binding.ERR_INVALID_ARG
    a.struct_size = ctypes.sizeof(binding.MoleArgs)
    a.flags = 0x80
    assert lib.mole_layer_forward_ex(ctypes.byref(a)) == binding.ERR_INVALID_ARG
    a.flags = 0
    a.B, a.T, a.N, a.d, a.V, a.dtype = 2, 2, 16, 768, 10, 5
    assert lib.mole_layer_forward_ex(ctypes.byref(a)) == binding.ERR_INVALID_ARG
    a.dtype = binding.DTYPE_BF16
    good = 0x10000
    a.hidden = a.lut = a.w_router = a.out = good
    a.ids = good + 2  # misaligned ids
    assert lib.mole_layer_forward_ex(ctypes.byref(a)) == binding.ERR_INVALID_ARG
    a.ids = good
    a.residual = good  # residual aliasing out while not being hidden ... here it IS hidden: allowed, so poison out
    a.out = good + 0x100
    a.residual = good + 0x100
    assert lib.mole_layer_forward_ex(ctypes.byref(a)) == binding.ERR_INVALID_ARG
    a.residual = None
    a.kernel = 9
    assert lib.mole_layer_forward_ex(ctypes.byref(a)) == binding.ERR_INVALID_ARG
    a.kernel = 0
    a.reserved2 = 1
    assert lib.mole_layer_forward_ex(ctypes.byref(a)) == binding.ERR_INVALID_ARG
    a.reserved2 = 0
    a.norm_weight = good + 4  # misaligned scale of the RMSNorm in front of the router
    assert lib.mole_layer_forward_ex(ctypes.byref(a)) == binding.ERR_INVALID_ARG
    a.norm_weight = good
    for eps in (-1.0, float("nan"), float("inf")):
        a.norm_eps = eps
        assert lib.mole_layer_forward_ex(ctypes.byref(a)) == binding.ERR_INVALID_ARG


def test_decode_step_and_offload_argument_checks(lib):
    good = 0x10000
    ds = lib.mole_decode_step
    assert ds(good, good, good, 16, good, 16, good + 0x100, None, None, 0, 4, 1, 16, 768, 100, 0, None) == binding.ERR_INVALID_ARG
    assert ds(good, good, good, 8, good, 16, good + 0x100, good + 0x200, None, 2, 4, 1, 16, 768, 100, 0, None) == binding.ERR_INVALID_ARG
    assert ds(None, None, None, 16, None, 16, None, None, None, 2, 0, 1, 16, 768, 100, 0, None) == binding.OK
    dx = lib.mole_decode_step_ex
    CH = binding.STEP_CHAINED
    # chained launches need a scratch buffer and cannot run in place
    assert dx(good, good, good, 16, good, 16, good + 0x100, None, None, 2, 4, 1, 16, 768, 100, 0, CH, 0, None) == binding.ERR_INVALID_ARG
    assert dx(good, good, good, 16, good, 16, good, good + 0x200, None, 2, 4, 1, 16, 768, 100, 0, CH, 0, None) == binding.ERR_INVALID_ARG
    assert dx(good, good, good, 16, good, 16, good + 0x100, good + 0x200, None, 2, 4, 1, 16, 768, 100, 0, 7, 0, None) == binding.ERR_INVALID_ARG
    # the host-buffer form validates everything before it queues its first copy
    dh = lib.mole_decode_step_host
    assert dh(good, good, good, good, good, good + 0x100, good + 0x200, good, 16, good, 16, None, 2, 4, 1, 16, 772, 100, 0,
              None) == binding.ERR_UNSUPPORTED_SHAPE
    assert dh(good, good, good, good, good, good + 0x100, good + 0x200, good, 16, good, 16, None, 2, 4, 1, 16, -8, 100, 0,
              None) == binding.ERR_UNSUPPORTED_SHAPE
    assert dh(good, good, good, good, good, good + 0x100, good + 0x200, good, 8, good, 16, None, 2, 4, 1, 16, 768, 100, 0,
              None) == binding.ERR_INVALID_ARG
    assert dh(None, good, good, good, good, good + 0x100, good + 0x200, good, 16, good, 16, None, 2, 4, 1, 16, 768, 100, 0,
              None) == binding.ERR_INVALID_ARG
    sa = binding.MoleStepArgs()
    assert lib.mole_decode_step_args(None) == binding.ERR_INVALID_ARG
    assert lib.mole_decode_step_args(ctypes.byref(sa)) == binding.ERR_INVALID_ARG  # struct_size 0
    sa.struct_size = ctypes.sizeof(binding.MoleStepArgs)
    sa.hidden_in = sa.ids = sa.lut_base = sa.w_router_base = good
    sa.out, sa.tmp = good + 0x100, good + 0x200
    sa.L, sa.B, sa.T, sa.N, sa.d, sa.V = 2, 4, 1, 16, 768, 100
    sa.norm_weight_base, sa.norm_eps = good + 8, 1e-5  # misaligned scale vectors
    assert lib.mole_decode_step_args(ctypes.byref(sa)) == binding.ERR_INVALID_ARG
    sa.norm_weight_base, sa.norm_eps = good, -1.0
    assert lib.mole_decode_step_args(ctypes.byref(sa)) == binding.ERR_INVALID_ARG
    sa.norm_eps, sa.flags = 1e-5, 1  # only MOLE_FLAG_CHAIN is a flag of a step
    assert lib.mole_decode_step_args(ctypes.byref(sa)) == binding.ERR_INVALID_ARG
    pf = lib.mole_prefetch_rows  # the L2 hint validates like the layer it serves
    assert pf(good, 4, good, 16, 2, 16, 768, 100, 0, 4, None) == binding.ERR_INVALID_ARG        # unknown flag
    assert pf(good, 4, good + 8, 16, 2, 16, 768, 100, 0, 0, None) == binding.ERR_INVALID_ARG    # table not 16-byte aligned
    assert pf(good, 4, good, 24, 2, 16, 768, 100, 0, 0, None) == binding.ERR_INVALID_ARG        # layer stride not a multiple of 16
    assert pf(good, 4, good, 16, 2, 16, 772, 100, 0, 0, None) == binding.ERR_UNSUPPORTED_SHAPE
    assert pf(good, 4, good, 16, 70000, 16, 768, 100, 0, 0, None) == binding.ERR_TOO_LARGE
    assert pf(None, 0, None, 0, 2, 16, 768, 100, 0, 0, None) == binding.OK                      # nothing to do
    dd = lib.mole_dedup_ids
    assert dd(good, -1, 10, good, good, good, good, None, None) == binding.ERR_INVALID_ARG
    assert dd(good, (1 << 20) + 1, 10, good, good, good, good, None, None) == binding.ERR_TOO_LARGE
    assert dd(good, 4, 10, None, good, good, good, None, None) == binding.ERR_INVALID_ARG
    fr = lib.mole_fetch_rows
    assert fr(good, good, good, 4, 24, good, None) == binding.ERR_INVALID_ARG  # row not a multiple of 16 bytes
    assert fr(good, good, good, 70000, 32, good, None) == binding.ERR_TOO_LARGE
    assert fr(None, None, None, 0, 32, None, None) == binding.OK
    h = ctypes.c_void_p()
    assert lib.mole_offload_create(None, 4, 16, 768, 100, 0, 2) == binding.ERR_INVALID_ARG
    assert lib.mole_offload_create(ctypes.byref(h), 0, 16, 768, 100, 0, 2) == binding.ERR_INVALID_ARG
    assert lib.mole_offload_create(ctypes.byref(h), 4, 65, 768, 100, 0, 2) == binding.ERR_UNSUPPORTED_SHAPE
    assert lib.mole_offload_create(ctypes.byref(h), 70000, 16, 768, 100, 0, 2) == binding.ERR_TOO_LARGE
    assert lib.mole_offload_destroy(None) == binding.OK
    assert lib.mole_host_alloc(None, 16) == binding.ERR_INVALID_ARG
    assert lib.mole_host_free(None) == binding.OK


def test_binding_fails_loudly_without_the_library(monkeypatch, tmp_path):
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "LIB_PATH", str(tmp_path / "nope.so"))
    with pytest.raises(RuntimeError, match="no fallback"):
        binding.lib()


def test_offload_decode_step_argument_checks(lib):
    good = 0x10000
    f = lib.mole_offload_decode_step
    # no context; zero layers; the same stream for both roles
    assert f(None, good, good, good, 16, good, 16, good, good, None, 2, 4, 1, None, good) == binding.ERR_INVALID_ARG
