"""mole_dedup_ids_static: the dedup entry point for callers that cannot allocate device memory
(a plug-in whose host server owns all of HBM, or a loop that must never meet cudaMalloc's
device-wide synchronisation).  Its scratch table is a fixed array inside the library, so the
same array serves every call: the test runs it twice in a row, on different id batches, and
requires the integer outputs to equal those of mole_dedup_ids (caller-supplied scratch) exactly.

Collected last on purpose (file name), so that a run that stops at the first failure has already
run every other test; it passes alone in a fresh process as well as after the others."""
import ctypes

import numpy as np
import pytest
import torch

from paper_2503_15798_b200 import binding as mole
from paper_2503_15798_b200 import build, inputs

build.build()
DEV = "cuda"


def _outputs(M):
    return (torch.full((M,), -3, dtype=torch.int32, device=DEV), torch.full((M,), -3, dtype=torch.int32, device=DEV),
            torch.full((1,), -3, dtype=torch.int32, device=DEV))


@pytest.mark.gpu
def test_static_scratch_dedup_equals_caller_scratch_dedup_twice_in_a_row():
    V = 50304  # the workloads' vocabulary fits the built-in table
    assert V <= mole.STATIC_DEDUP_MAX_V
    scratch = torch.zeros(V, dtype=torch.int32, device=DEV)
    for call, (M, seed) in enumerate(((256, 11), (4096, 12), (64, 13))):
        ids_np = inputs.zipf_ids(M, V, seed=seed)
        if call == 1:
            ids_np[5], ids_np[77] = -4, V  # ids outside the vocabulary
        ids = torch.from_numpy(ids_np).to(DEV)
        u0, s0, c0 = _outputs(M)
        st0 = torch.zeros(1, dtype=torch.int32, device=DEV)
        mole.dedup_ids(ids, V, scratch, u0, s0, c0, status=st0)
        u1, s1, c1 = _outputs(M)
        st1 = torch.zeros(1, dtype=torch.int32, device=DEV)
        mole.dedup_ids_static(ids, V, u1, s1, c1, status=st1)
        torch.cuda.synchronize()
        n = int(c0.item())
        assert int(c1.item()) == n and n == len(np.unique(ids_np[(ids_np >= 0) & (ids_np < V)]))
        assert torch.equal(u1[:n], u0[:n]) and torch.equal(s1, s0)
        assert int(st1.item()) == int(st0.item()) == (mole.STATUS_BAD_ID if call == 1 else 0)


@pytest.mark.gpu
def test_static_scratch_dedup_rejects_a_vocabulary_beyond_its_table():
    M = 8
    ids = torch.zeros(M, dtype=torch.int32, device=DEV)
    u, s, c = _outputs(M)
    with pytest.raises(mole.MoleError) as e:
        mole.dedup_ids_static(ids, mole.STATIC_DEDUP_MAX_V + 1, u, s, c)
    assert e.value.code == mole.ERR_TOO_LARGE
    torch.cuda.synchronize()
    assert int(c.item()) == -3  # nothing was launched
    mole.dedup_ids_static(ids, mole.STATIC_DEDUP_MAX_V, u, s, c)  # the maximum itself is accepted
    torch.cuda.synchronize()
    assert int(c.item()) == 1 and int(u[0].item()) == 0 and int(s.abs().sum().item()) == 0


def test_static_scratch_dedup_argument_checks_need_no_gpu():
    lib = mole.lib()
    good = 0x10000
    f = lib.mole_dedup_ids_static
    assert f(good, 4, mole.STATIC_DEDUP_MAX_V + 1, good, good, good, None, None) == mole.ERR_TOO_LARGE
    assert f(good, -1, 10, good, good, good, None, None) == mole.ERR_INVALID_ARG
    assert f(good, 4, 0, good, good, good, None, None) == mole.ERR_INVALID_ARG
    assert f(good, 4, 10, good, good, None, None, None) == mole.ERR_INVALID_ARG
    assert f(None, 4, 10, good, good, good, None, None) == mole.ERR_INVALID_ARG
