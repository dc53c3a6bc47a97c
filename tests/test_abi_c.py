"""The header as a C compiler sees it: include/mole.h must compile as plain C, a C program linked
against the library must be able to call it, and the ctypes mirror of every struct in binding.py must
have the size and field offsets that the C compiler gives the header's struct."""
import ctypes
import os
import subprocess

import pytest

from paper_2503_15798_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
INCLUDE = os.path.join(ROOT, "include")

PROGRAM = r"""
#include <stddef.h>
#include <stdio.h>
#include "mole.h"
#define FIELD(S, f) printf(#S "." #f " %zu\n", offsetof(S, f))
int main(void)
{
    int k = 0, threads = 0, smem = 0, stages = 0, per_sm = 0;
    printf("version %d\n", mole_version());
    printf("plan_rc %d\n", mole_plan(256, 1, 32, 2048, MOLE_DTYPE_BF16, 0, &k, &threads, &smem, &stages, &per_sm));
    printf("plan %d %d %d %d %d\n", k, threads, smem, stages, per_sm);
    printf("string %s\n", mole_status_string(MOLE_ERR_TOO_LARGE));
    printf("sizeof.mole_args %zu\n", sizeof(mole_args));
    FIELD(mole_args, struct_size); FIELD(mole_args, flags); FIELD(mole_args, hidden); FIELD(mole_args, ids);
    FIELD(mole_args, lut); FIELD(mole_args, w_router); FIELD(mole_args, out); FIELD(mole_args, residual);
    FIELD(mole_args, gates_out); FIELD(mole_args, status); FIELD(mole_args, B); FIELD(mole_args, T); FIELD(mole_args, N);
    FIELD(mole_args, d); FIELD(mole_args, V); FIELD(mole_args, dtype); FIELD(mole_args, kernel); FIELD(mole_args, d_split);
    FIELD(mole_args, stream); FIELD(mole_args, norm_weight); FIELD(mole_args, norm_eps); FIELD(mole_args, lut_format);
    FIELD(mole_args, lut_block); FIELD(mole_args, reserved2);
    printf("sizeof.mole_step_args %zu\n", sizeof(mole_step_args));
    FIELD(mole_step_args, struct_size); FIELD(mole_step_args, flags); FIELD(mole_step_args, hidden_in); FIELD(mole_step_args, ids);
    FIELD(mole_step_args, lut_base); FIELD(mole_step_args, lut_layer_stride_bytes); FIELD(mole_step_args, w_router_base);
    FIELD(mole_step_args, wr_layer_stride_bytes); FIELD(mole_step_args, norm_weight_base);
    FIELD(mole_step_args, norm_layer_stride_bytes); FIELD(mole_step_args, out); FIELD(mole_step_args, tmp);
    FIELD(mole_step_args, status); FIELD(mole_step_args, L); FIELD(mole_step_args, B); FIELD(mole_step_args, T);
    FIELD(mole_step_args, N); FIELD(mole_step_args, d); FIELD(mole_step_args, V); FIELD(mole_step_args, dtype);
    FIELD(mole_step_args, mode); FIELD(mole_step_args, d_split); FIELD(mole_step_args, kernel); FIELD(mole_step_args, norm_eps);
    FIELD(mole_step_args, lut_format); FIELD(mole_step_args, lut_block);
    FIELD(mole_step_args, reserved); FIELD(mole_step_args, stream);
    return 0;
}
"""


def test_header_is_valid_c99():
    for std in ("c99", "c11"):
        r = subprocess.run(["gcc", f"-std={std}", "-pedantic", "-Wall", "-Werror", "-fsyntax-only", "-x", "c",
                            os.path.join(INCLUDE, "mole.h")], capture_output=True, text=True)
        assert r.returncode == 0, r.stderr


@pytest.fixture(scope="module")
def c_report(tmp_path_factory):
    build.build()
    tmp = tmp_path_factory.mktemp("abi_c")
    src, exe = tmp / "abi.c", tmp / "abi"
    src.write_text(PROGRAM)
    libdir = os.path.dirname(binding.LIB_PATH)
    r = subprocess.run(["gcc", "-std=c99", "-Wall", "-Werror", "-I", INCLUDE, str(src), "-o", str(exe), "-L", libdir,
                        "-l:libmole_b200.so", f"-Wl,-rpath,{libdir}"], capture_output=True, text=True)
    assert r.returncode == 0, r.stderr
    r = subprocess.run([str(exe)], capture_output=True, text=True)
    assert r.returncode == 0, r.stderr
    rep = {}
    for line in r.stdout.splitlines():
        key, _, val = line.partition(" ")
        rep[key] = val
    return rep


def test_c_program_links_and_calls_the_library(c_report):
    assert int(c_report["version"]) == binding.version()
    assert int(c_report["plan_rc"]) == 0
    assert tuple(int(x) for x in c_report["plan"].split()) == binding.plan(256, 32, 2048)
    assert c_report["string"] == "size beyond the stated maximum"


@pytest.mark.parametrize("cname,mirror", [("mole_args", binding.MoleArgs), ("mole_step_args", binding.MoleStepArgs)])
def test_ctypes_mirror_has_the_c_compilers_layout(c_report, cname, mirror):
    assert int(c_report[f"sizeof.{cname}"]) == ctypes.sizeof(mirror)
    fields = [k.split(".", 1)[1] for k in c_report if k.startswith(cname + ".")]
    assert fields == [f[0] for f in mirror._fields_]  # the same fields in the same order
    for f in fields:
        assert int(c_report[f"{cname}.{f}"]) == getattr(mirror, f).offset, f
