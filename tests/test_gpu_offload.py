"""GPU parity of the offload mode: device-side dedup, GPU-initiated row fetch from pinned host
memory, and the fused layer gathering from the staging buffer -- bit-identical to resident mode."""
import numpy as np
import pytest
import torch

import oracle
from gpu_util import bits, check_out, oracle_layer, rand_case
from paper_2503_15798_b200 import binding as mole
from paper_2503_15798_b200 import inputs

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _dedup(ids_np, V):
    M = len(ids_np)
    ids = torch.from_numpy(ids_np.astype(np.int32)).to(DEV)
    scratch = torch.zeros(V, dtype=torch.int32, device=DEV)
    uniq = torch.full((max(M, 1),), -7, dtype=torch.int32, device=DEV)
    slot = torch.full((max(M, 1),), -7, dtype=torch.int32, device=DEV)
    count = torch.full((1,), -7, dtype=torch.int32, device=DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    mole.dedup_ids(ids, V, scratch, uniq, slot, count, status=status)
    torch.cuda.synchronize()
    n = int(count.item())
    return uniq[:n].cpu().numpy(), slot[:M].cpu().numpy(), n, scratch, int(status.item())


@pytest.mark.parametrize("M", [1, 2, 8, 64, 256, 1000, 1024, 1025, 16384, 40000])
def test_dedup_matches_the_oracle(M):
    V = 50304
    ids = inputs.zipf_ids(M, V, seed=M)
    uniq, slot, n, scratch, status = _dedup(ids, V)
    want_uniq, want_slot = oracle.dedup(ids)
    assert n == len(want_uniq) and status == 0
    assert np.array_equal(np.sort(uniq), np.sort(want_uniq))  # the set is what is unique
    assert np.array_equal(uniq[slot], ids)                      # and the map must be valid
    assert np.array_equal(uniq, want_uniq) and np.array_equal(slot, want_slot)  # first-occurrence order
    assert int(scratch.abs().sum().item()) == 0                 # scratch left clean for the next call


def test_dedup_degenerate_cases():
    V = 100
    uniq, slot, n, scratch, status = _dedup(np.full(500, 42), V)  # one id only
    assert n == 1 and uniq[0] == 42 and (slot == 0).all()
    uniq, slot, n, scratch, status = _dedup(np.arange(100)[::-1].copy(), V)  # all distinct, whole vocabulary
    assert n == 100 and np.array_equal(uniq, np.arange(100)[::-1]) and np.array_equal(slot, np.arange(100))
    uniq, slot, n, scratch, status = _dedup(np.array([5, -1, 5, 100, 7, 2 ** 31 - 1]), V)  # ids outside [0, V)
    assert n == 2 and list(uniq) == [5, 7] and list(slot) == [0, -1, 0, -1, 1, -1]
    assert status & mole.STATUS_BAD_ID and int(scratch.abs().sum().item()) == 0
    uniq, slot, n, scratch, status = _dedup(np.array([], dtype=np.int64), V)
    assert n == 0
    # back-to-back calls on one scratch table
    ids_a, ids_b = inputs.zipf_ids(300, V, seed=1), inputs.zipf_ids(300, V, seed=2)
    scratch = torch.zeros(V, dtype=torch.int32, device=DEV)
    for ids in (ids_a, ids_b, ids_a):
        u = torch.empty(300, dtype=torch.int32, device=DEV)
        s = torch.empty(300, dtype=torch.int32, device=DEV)
        c = torch.empty(1, dtype=torch.int32, device=DEV)
        mole.dedup_ids(torch.from_numpy(ids).to(DEV), V, scratch, u, s, c)
        torch.cuda.synchronize()
        wu, ws = oracle.dedup(ids)
        assert int(c.item()) == len(wu) and np.array_equal(u[:len(wu)].cpu().numpy(), wu)


def test_fetch_rows_copies_exactly_the_selected_rows():
    V, N, d = 1000, 16, 1024  # 32 KB rows: two 16 KB chunks
    host = mole.HostTable((V, N, d), torch.bfloat16)
    try:
        g = torch.Generator().manual_seed(1)
        host.tensor.copy_(torch.empty(V, N, d).normal_(0, 0.05, generator=g).to(torch.bfloat16))
        for row_elems, U, maxr in ((N * d, 37, 64), (N * d, 64, 64), (N * d, 0, 8)):
            uniq_np = np.random.default_rng(U).permutation(V)[:maxr].astype(np.int32)
            uniq = torch.from_numpy(uniq_np).to(DEV)
            count = torch.tensor([U], dtype=torch.int32, device=DEV)
            staging = torch.full((maxr, N, d), 7.0, dtype=torch.bfloat16, device=DEV)
            mole.fetch_rows(host.tensor, uniq, count, maxr, staging)
            torch.cuda.synchronize()
            got = bits(staging)
            assert np.array_equal(got[:U], bits(host.tensor)[uniq_np[:U]])
            assert (staging[U:].float() == 7.0).all()  # rows beyond count are untouched
    finally:
        host.free()


def test_fetch_rows_ragged_row_size():
    V, N, d = 50, 5, 520  # 5200-byte rows: one partial 16 KB chunk; and 3 x 16 KB + tail below
    for N, d in ((5, 520), (25, 1000)):
        host = mole.HostTable((V, N, d), torch.bfloat16)
        try:
            host.tensor.copy_(torch.arange(V * N * d).remainder(251).view(V, N, d).to(torch.bfloat16))
            uniq = torch.tensor([49, 0, 17], dtype=torch.int32, device=DEV)
            count = torch.tensor([3], dtype=torch.int32, device=DEV)
            staging = torch.zeros(4, N, d, dtype=torch.bfloat16, device=DEV)
            mole.fetch_rows(host.tensor, uniq, count, 4, staging)
            torch.cuda.synchronize()
            assert torch.equal(staging[:3].cpu(), host.tensor[[49, 0, 17]])
            assert (staging[3] == 0).all()
        finally:
            host.free()


@pytest.mark.parametrize("M,N,d", [(1, 16, 1024), (8, 16, 1024), (64, 16, 1024), (200, 16, 768), (33, 32, 2048)])
def test_offload_layer_is_bit_identical_to_resident(M, N, d):
    V = 2000
    hidden, ids, lut, wr = rand_case(M, N, d, V, seed=M + d, ids_kind="zipf")
    ids[M // 2] = ids[0]  # at least one duplicate when M > 1
    host = mole.HostTable((V, N, d), torch.bfloat16)
    ctx = mole.OffloadContext(max_tokens=256, N=N, d=d, V=V, n_buffers=2)
    side = torch.cuda.Stream()
    try:
        host.tensor.copy_(lut)
        h, i, w = hidden.to(DEV), ids.to(DEV), wr.to(DEV)
        resident = mole.layer_forward(h, i, lut.to(DEV), w)
        ref, _, _ = oracle_layer(hidden, ids, lut, wr)
        check_out(resident, ref)
        torch.cuda.synchronize()
        for buf in (0, 1, 0):
            out = torch.empty_like(h)
            ctx.prefetch(buf, i, host.tensor, side_stream=side)
            ctx.forward(buf, h, w, out)
            torch.cuda.synchronize()
            assert torch.equal(out, resident)
            uniq, slot, n = ctx.read_buffer(buf)
            want_uniq, want_slot = oracle.dedup(ids.numpy())
            assert n == len(want_uniq) and np.array_equal(uniq.numpy(), want_uniq)
            assert np.array_equal(slot[:M].numpy(), want_slot)
    finally:
        ctx.destroy()
        host.free()


def test_offload_pipeline_over_layers_double_buffered():
    # layer l+1's fetch is issued on the side stream before layer l's combine is enqueued
    M, N, d, V, L = 64, 16, 1024, 3000, 6
    g = torch.Generator().manual_seed(3)
    hosts = [mole.HostTable((V, N, d), torch.bfloat16) for _ in range(L)]
    ctx = mole.OffloadContext(max_tokens=M, N=N, d=d, V=V, n_buffers=2)
    side = torch.cuda.Stream()
    try:
        for t in hosts:
            t.tensor.copy_(torch.empty(V, N, d).normal_(0, 0.05, generator=g).to(torch.bfloat16))
        wrs = torch.empty(L, d, N).normal_(0, 0.02, generator=g).to(torch.bfloat16).to(DEV)
        hidden = torch.empty(M, d).normal_(0, 1, generator=g).to(torch.bfloat16).to(DEV)
        ids = torch.from_numpy(inputs.zipf_ids(M, V, seed=8)).to(DEV)
        # resident reference, layer after layer
        h = hidden
        for l in range(L):
            h = mole.layer_forward(h, ids, hosts[l].tensor.to(DEV), wrs[l])
        torch.cuda.synchronize()
        bufs = [torch.empty_like(hidden), torch.empty_like(hidden)]
        ctx.prefetch(0, ids, hosts[0].tensor, side_stream=side)
        cur = hidden
        for l in range(L):
            if l + 1 < L:
                ctx.prefetch((l + 1) % 2, ids, hosts[l + 1].tensor, side_stream=side)
            nxt = bufs[l % 2]
            ctx.forward(l % 2, cur, wrs[l], nxt)
            cur = nxt
        torch.cuda.synchronize()
        assert torch.equal(cur, h)
    finally:
        ctx.destroy()
        for t in hosts:
            t.free()


def test_offload_bad_ids_and_size_checks():
    M, N, d, V = 6, 16, 768, 50
    hidden, ids, lut, wr = rand_case(M, N, d, V, seed=21)
    ids[2] = V + 3
    host = mole.HostTable((V, N, d), torch.bfloat16)
    ctx = mole.OffloadContext(max_tokens=8, N=N, d=d, V=V, n_buffers=1)
    try:
        host.tensor.copy_(lut)
        h, i, w = hidden.to(DEV), ids.to(DEV), wr.to(DEV)
        status = torch.zeros(1, dtype=torch.int32, device=DEV)
        out = torch.empty_like(h)
        ctx.prefetch(0, i, host.tensor)
        ctx.forward(0, h, w, out, status=status)
        torch.cuda.synchronize()
        assert int(status.item()) & mole.STATUS_BAD_ID
        ref, _, _ = oracle_layer(hidden, ids, lut, wr)
        check_out(out, ref)
        assert np.array_equal(bits(out)[2], bits(hidden)[2])
        with pytest.raises(mole.MoleError) as e:  # more tokens than the context was made for
            ctx.prefetch(0, torch.zeros(9, dtype=torch.int32, device=DEV), host.tensor)
        assert e.value.code == mole.ERR_TOO_LARGE
        with pytest.raises(mole.MoleError) as e:  # forward with a token count that does not match the prefetch
            ctx.forward(0, h[:3], w, out[:3])
        assert e.value.code == mole.ERR_INVALID_ARG
    finally:
        ctx.destroy()
        host.free()


@pytest.mark.parametrize("M,L,cap", [(1, 3, 1), (8, 5, 8), (64, 4, 64), (300, 2, 300), (5, 1, 5),
                                     (1, 7, 64), (5, 7, 64), (24, 5, 64), (9, 6, 20), (33, 3, 64)])
def test_offload_decode_step_equals_resident_layers(M, L, cap):
    """The whole offload step in one call (one dedup, the next fetch under the current layers' combine)
    gives the bytes of L resident single-layer calls; repeated steps on one context stay correct.
    `cap` = the context's max_tokens: with room for cap / M layers' rows in a staging area, one fetch
    launch brings several layers (all 7, groups of 2 + 2 + 1, 2 + 2 + 2, or one at a time)."""
    N, d, V = 16, 1024, 700
    g = torch.Generator().manual_seed(100 + M)
    host = mole.HostTable((L, V, N, d), torch.bfloat16)
    ctx = mole.OffloadContext(max_tokens=cap, N=N, d=d, V=V, n_buffers=2)
    side = torch.cuda.Stream()
    try:
        host.tensor.copy_(torch.empty(L, V, N, d).normal_(0, 0.05, generator=g).to(torch.bfloat16))
        wrs = torch.empty(L, d, N).normal_(0, 0.02, generator=g).to(torch.bfloat16).to(DEV)
        hidden = torch.empty(M, d).normal_(0, 1, generator=g).to(torch.bfloat16).to(DEV)
        luts_dev = host.tensor.to(DEV)
        status = torch.zeros(1, dtype=torch.int32, device=DEV)
        for step in range(3):  # back-to-back steps reuse the slot map and both staging areas
            ids_np = inputs.zipf_ids(M, V, seed=step)
            if step == 2 and M > 2:
                ids_np[1] = V + 5  # an id outside the table: no routed term in any layer
            ids = torch.from_numpy(ids_np).to(DEV)
            out, tmp = torch.empty_like(hidden), torch.empty_like(hidden)
            ctx.decode_step(hidden, ids, host.tensor, wrs, out, tmp, status=status, side_stream=side)
            h = hidden
            for l in range(L):
                h = mole.layer_forward(h, ids, luts_dev[l], wrs[l], kernel=mole.KERNEL_RING)
            torch.cuda.synchronize()
            assert torch.equal(out, h)
            if step == 2 and M > 2:
                assert torch.equal(out[1], hidden[1])
        assert int(status.item()) == (mole.STATUS_BAD_ID if M > 2 else 0)
    finally:
        ctx.destroy()
        host.free()


def test_offload_decode_step_replayed_from_cuda_graphs():
    """The offload step captured into CUDA graphs (the side stream joins the capture and is joined
    back): replays, with other steps' replays in between, give the bytes of the uncaptured call."""
    M, L, N, d, V = 24, 5, 16, 768, 500
    g = torch.Generator().manual_seed(77)
    host = mole.HostTable((L, V, N, d), torch.bfloat16)
    ctx = mole.OffloadContext(max_tokens=M, N=N, d=d, V=V, n_buffers=2)
    side = torch.cuda.Stream()
    try:
        host.tensor.copy_(torch.empty(L, V, N, d).normal_(0, 0.05, generator=g).to(torch.bfloat16))
        wrs = torch.empty(L, d, N).normal_(0, 0.02, generator=g).to(torch.bfloat16).to(DEV)
        hidden = torch.empty(M, d).normal_(0, 1, generator=g).to(torch.bfloat16).to(DEV)
        status = torch.zeros(1, dtype=torch.int32, device=DEV)
        out, tmp = torch.empty_like(hidden), torch.empty_like(hidden)
        batches = [torch.from_numpy(inputs.zipf_ids(M, V, seed=40 + b)).to(DEV) for b in range(3)]
        want = []
        for ids in batches:  # uncaptured calls first (they also set the kernels' attributes)
            ctx.decode_step(hidden, ids, host.tensor, wrs, out, tmp, status=status, side_stream=side)
            torch.cuda.synchronize()
            want.append(out.clone())
        graphs = []
        for ids in batches:
            gr = torch.cuda.CUDAGraph()
            with torch.cuda.graph(gr):
                ctx.decode_step(hidden, ids, host.tensor, wrs, out, tmp, status=status, side_stream=side)
            graphs.append(gr)
        for k in (0, 1, 2, 1, 0, 2, 2):
            out.zero_()
            graphs[k].replay()
            torch.cuda.synchronize()
            assert torch.equal(out, want[k])
        for k in range(30):  # back to back, no synchronisation in between
            graphs[k % 3].replay()
        torch.cuda.synchronize()
        assert torch.equal(out, want[29 % 3]) and int(status.item()) == 0
    finally:
        ctx.destroy()
        host.free()


@pytest.mark.parametrize("M", [1, 8, 64])
def test_offload_decode_step_at_the_benchmarked_shape(M):
    """The offload configuration as bench.py times it: 410M-shaped host tables (V = 50304, 32 KB rows; three
    layers, 4.9 GB pinned, a layer stride of 1.65 GB), a context of 256 tokens (so one fetch launch brings
    several layers' rows), Zipf ids.  Bitwise equal to resident ring-kernel layers on a device copy of the
    same tables, and element by element within the chain bound of the oracle on the referenced rows."""
    sh = inputs.SHAPES["410m"]
    L, N, d, V = 3, sh.N, sh.d, sh.V
    host = mole.HostTable((L, V, N, d), torch.bfloat16)
    ctx = mole.OffloadContext(max_tokens=256, N=N, d=d, V=V, n_buffers=2)
    side = torch.cuda.Stream()
    try:
        dev_tables = torch.empty((L, V, N, d), dtype=torch.bfloat16, device=DEV)
        for l in range(L):
            inputs.make_table(V, N, d, seed=50 + l, device=DEV, out=dev_tables[l])
            host.tensor[l].copy_(dev_tables[l])
        torch.cuda.synchronize()
        wrs = torch.stack([inputs.make_router(d, N, seed=60 + l, device=DEV) for l in range(L)])
        hidden = inputs.make_hidden(M, d, seed=M, device=DEV)
        status = torch.zeros(1, dtype=torch.int32, device=DEV)
        for step in range(2):
            ids = inputs.make_ids(M, V, seed=70 + step + M, device=DEV)
            out, tmp = torch.empty_like(hidden), torch.empty_like(hidden)
            ctx.decode_step(hidden, ids, host.tensor, wrs, out, tmp, status=status, side_stream=side)
            h = hidden
            for l in range(L):
                h = mole.layer_forward(h, ids, dev_tables[l], wrs[l], kernel=mole.KERNEL_RING)
            torch.cuda.synchronize()
            assert int(status.item()) == 0
            assert torch.equal(out, h)
            # the oracle's chain on the rows this batch references (plain torch index on the pinned host table)
            ids_np = ids.cpu().numpy()
            uniq, inv = np.unique(ids_np, return_inverse=True)
            ho = hidden.cpu()
            for l in range(L):
                rows = host.tensor[l][torch.from_numpy(uniq).long()]
                ref, _, bad = oracle.layer_lookup(bits(ho), inv, bits(rows), bits(wrs[l]))
                assert bad == 0
                ho = torch.from_numpy(ref).to(torch.bfloat16)
            err = np.abs(out.cpu().double().numpy() - ref)
            assert (err <= L * 2.0 ** -7 * np.maximum(1.0, np.abs(ref))).all(), float(err.max())
        del dev_tables
    finally:
        ctx.destroy()
        host.free()


@pytest.mark.parametrize("M,cap", [(48, 64), (5, 64), (64, 64)])
def test_hot_rows_cache_serves_the_listed_ids_and_changes_no_bit(M, cap):
    """A cache of hot rows in device memory in front of the host link: ids on the list are served from it
    (shown by overwriting their rows in the host table after they were cached -- the output must not notice),
    the hit counter counts exactly the (distinct id, layer) pairs on the list, and dropping the cache goes
    back to the host rows."""
    N, d, V, L = 16, 1024, 700, 4
    g = torch.Generator().manual_seed(9)
    host = mole.HostTable((L, V, N, d), torch.bfloat16)
    ctx = mole.OffloadContext(max_tokens=cap, N=N, d=d, V=V, n_buffers=2)
    side = torch.cuda.Stream()
    try:
        host.tensor.copy_(torch.empty(L, V, N, d).normal_(0, 0.05, generator=g).to(torch.bfloat16))
        wrs = torch.empty(L, d, N).normal_(0, 0.02, generator=g).to(torch.bfloat16).to(DEV)
        hidden = torch.empty(M, d).normal_(0, 1, generator=g).to(torch.bfloat16).to(DEV)
        ids_np = inputs.zipf_ids(M, V, seed=3)
        ids = torch.from_numpy(ids_np).to(DEV)
        out, tmp = torch.empty_like(hidden), torch.empty_like(hidden)
        want = ctx.decode_step(hidden, ids, host.tensor, wrs, out, tmp, side_stream=side).clone()
        torch.cuda.synchronize()
        hot = inputs.zipf_hot_ids(V, 40)
        assert len(set(hot.tolist()) & set(ids_np.tolist())) >= 1
        ctx.set_hot_rows(hot, host.tensor)
        assert ctx.hot_hits(reset=True) == 0
        keep = host.tensor[:, torch.from_numpy(hot).long()].clone()
        host.tensor[:, torch.from_numpy(hot).long()] = 7.0   # the host copies of the cached rows are never read again
        got = ctx.decode_step(hidden, ids, host.tensor, wrs, out, tmp, side_stream=side)
        torch.cuda.synchronize()
        assert torch.equal(got, want)
        assert ctx.hot_hits() == len(set(hot.tolist()) & set(ids_np.tolist())) * L
        # the single-layer path finds the cache through the layer's host address
        one = torch.empty_like(hidden)
        ctx.prefetch(0, ids, host.tensor[2], side_stream=side)
        ctx.forward(0, hidden, wrs[2], one)
        torch.cuda.synchronize()
        host.tensor[:, torch.from_numpy(hot).long()] = keep
        plain = torch.empty_like(hidden)
        ctx.set_hot_rows([], host.tensor)
        ctx.prefetch(0, ids, host.tensor[2], side_stream=side)
        ctx.forward(0, hidden, wrs[2], plain)
        assert torch.equal(ctx.decode_step(hidden, ids, host.tensor, wrs, out, tmp, side_stream=side), want)
        torch.cuda.synchronize()
        assert torch.equal(one, plain)
        with pytest.raises(mole.MoleError):  # an id listed twice
            ctx.set_hot_rows([1, 2, 1], host.tensor)
        with pytest.raises(mole.MoleError):
            ctx.set_hot_rows([V], host.tensor)
    finally:
        ctx.destroy()
        host.free()


def test_tables_from_a_file_feed_the_offload_mode(tmp_path):
    """Disk -> pinned host memory -> offload step: tables written to a table file, read back into a pinned
    host allocation, served by the offload step; equal to the step over the tables they were written from."""
    N, d, V, L, M = 16, 768, 300, 3, 20
    g = torch.Generator().manual_seed(4)
    tables = torch.empty(L, V, N, d).normal_(0, 0.05, generator=g).to(torch.bfloat16)
    path = str(tmp_path / "tables.mole")
    mole.table_file_write(path, tables, N, d)
    host = mole.HostTable((L, V, N, d), torch.bfloat16)
    ctx = mole.OffloadContext(max_tokens=32, N=N, d=d, V=V, n_buffers=2)
    side = torch.cuda.Stream()
    try:
        mole.table_file_read(path, host.tensor)
        assert torch.equal(host.tensor.view(torch.int16), tables.view(torch.int16))
        wrs = torch.empty(L, d, N).normal_(0, 0.02, generator=g).to(torch.bfloat16).to(DEV)
        hidden = torch.empty(M, d).normal_(0, 1, generator=g).to(torch.bfloat16).to(DEV)
        ids = torch.from_numpy(inputs.zipf_ids(M, V, seed=1)).to(DEV)
        out = ctx.decode_step(hidden, ids, host.tensor, wrs, torch.empty_like(hidden), torch.empty_like(hidden), side_stream=side)
        h = hidden
        dev_tables = tables.to(DEV)
        for l in range(L):
            h = mole.layer_forward(h, ids, dev_tables[l], wrs[l], kernel=mole.KERNEL_RING)
        torch.cuda.synchronize()
        assert torch.equal(out, h)
    finally:
        ctx.destroy()
        host.free()
