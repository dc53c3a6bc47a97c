"""A bounded device-side wait that runs out.  Every wait inside the kernels has a poll limit; here the
limit is set to zero polls through the debugging variable MOLE_DEBUG_WAIT_LIMIT, so a wait that is not
satisfied on the spot gives up while its copy is still on its way.  Nothing faults and nothing hangs: the
launch must return, report MOLE_STATUS_TIMEOUT, stay inside its own output rows, and leave the stream
usable for a correct launch right after."""
import numpy as np
import pytest
import torch

from gpu_util import check_gates, check_out, oracle_layer, rand_case
from paper_2503_15798_b200 import binding as mole

pytestmark = pytest.mark.gpu
DEV = "cuda"
GUARD = 3  # rows of sentinel before and after the output rows


def _padded_out(M, d):
    buf = torch.full((M + 2 * GUARD, d), 12345.0, dtype=torch.bfloat16, device=DEV)
    return buf, buf[GUARD:GUARD + M]


@pytest.mark.parametrize("kernel,M,N,d", [
    (mole.KERNEL_RING, 4, 4, 64),      # router matrix resident: the consumers' wait for it runs out
    (mole.KERNEL_RING, 5, 16, 768),
    (mole.KERNEL_DECODE, 4, 4, 128),   # one block per token: the wait for the router matrix runs out
    (mole.KERNEL_DECODE, 7, 16, 768),
    (mole.KERNEL_DECODE, 6, 32, 2048),  # one token per cluster: the waits for the router slice and for the peers' partial logits run out
])
def test_a_wait_that_runs_out_reports_timeout_and_the_stream_stays_usable(kernel, M, N, d):
    hidden, ids, lut, wr = rand_case(M, N, d, 40, seed=M + d)
    hidden, ids, lut, wr = hidden.to(DEV), ids.to(DEV), lut.to(DEV), wr.to(DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    buf, out = _padded_out(M, d)
    name = mole.variant(M, N, d, kernel=kernel)[0]
    assert name.startswith(("decode", "cdecode") if kernel == mole.KERNEL_DECODE else "step")
    with mole.debug_env(MOLE_DEBUG_WAIT_LIMIT=-1):
        mole.layer_forward(hidden, ids, lut, wr, out, status=status, kernel=kernel)
        torch.cuda.synchronize()  # the launch returns
    assert int(status.item()) & mole.STATUS_TIMEOUT
    assert (buf[:GUARD] == 12345.0).all() and (buf[GUARD + M:] == 12345.0).all()  # nothing written outside the output rows
    # the limit is back to its default: the same buffers, the same stream, a correct result
    status.zero_()
    gates = torch.zeros(M, N, dtype=torch.float32, device=DEV)
    mole.layer_forward(hidden, ids, lut, wr, out, status=status, gates_out=gates, kernel=kernel)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    ref, gref, _ = oracle_layer(hidden, ids, lut, wr)
    check_out(out, ref)
    check_gates(gates, gref)
    assert (buf[:GUARD] == 12345.0).all() and (buf[GUARD + M:] == 12345.0).all()


@pytest.mark.parametrize("kernel", [mole.KERNEL_DECODE, mole.KERNEL_RING])
def test_the_producer_of_the_ring_gives_up_when_no_slot_comes_back(kernel):
    """More chunks per block than ring slots: with a limit of zero polls the producer's first wait for a free
    slot runs out, it stops issuing, and the consumers, told so, stop waiting too."""
    M, N, d, L = 6, 8, 256, 12  # one block per token, 24 chunks each, at most 8 slots
    g = torch.Generator().manual_seed(3)
    luts = torch.empty(L, 30, N, d).normal_(0, 0.05, generator=g).to(torch.bfloat16).to(DEV)
    wrs = torch.empty(L, d, N).normal_(0, 0.02, generator=g).to(torch.bfloat16).to(DEV)
    hidden = torch.empty(M, d).normal_(0, 1, generator=g).to(torch.bfloat16).to(DEV)
    ids = torch.randint(0, 30, (M,), generator=g, dtype=torch.int32).to(DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    buf, out = _padded_out(M, d)
    assert mole.plan(M, N, d, mole.DTYPE_BF16, 0, L)[3] < 2 * L
    assert mole.variant(M, N, d, L=L, kernel=kernel)[0].startswith("fstep" if kernel == mole.KERNEL_DECODE else "step")
    with mole.debug_env(MOLE_DEBUG_WAIT_LIMIT=-1):
        mole.decode_step_args(hidden, ids, luts, wrs, out, None, status=status, mode=mole.STEP_FUSED, kernel=kernel)
        torch.cuda.synchronize()
    assert int(status.item()) & mole.STATUS_TIMEOUT
    assert (buf[:GUARD] == 12345.0).all() and (buf[GUARD + M:] == 12345.0).all()
    status.zero_()
    want = mole.decode_step(hidden, ids, luts, wrs, torch.empty_like(hidden), torch.empty_like(hidden), status=status,
                            mode=mole.STEP_CHAINED, d_split=1)
    mole.decode_step(hidden, ids, luts, wrs, out, None, status=status, mode=mole.STEP_FUSED, d_split=1)
    torch.cuda.synchronize()
    assert int(status.item()) == 0 and torch.equal(out, want)
