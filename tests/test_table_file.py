"""Table files (the tier below host memory): written from host memory, header read back, whole layers and
single rows read back bit for bit, plain and quantised; every file error is an error code, never a crash.
Host code only -- no GPU."""
import os

import numpy as np
import pytest
import torch

from oracle import quant
from paper_2503_15798_b200 import binding as mole
from paper_2503_15798_b200 import build

build.build()


def test_plain_table_round_trip(tmp_path):
    L, V, N, d = 3, 37, 4, 64
    g = torch.Generator().manual_seed(1)
    tables = torch.empty(L, V, N, d).normal_(0, 0.05, generator=g).to(torch.bfloat16)
    path = str(tmp_path / "t.mole")
    mole.table_file_write(path, tables, N, d)
    info = mole.table_file_info(path)
    assert (info.L, info.V, info.N, info.d, info.dtype, info.lut_format, info.lut_block, info.row_bytes) == (L, V, N, d, mole.DTYPE_BF16, 0, 0, N * d * 2)
    assert os.path.getsize(path) == 4096 + L * V * N * d * 2
    back = torch.zeros_like(tables)
    mole.table_file_read(path, back)
    assert torch.equal(back.view(torch.int16), tables.view(torch.int16))
    # layers 1..2 into a destination with a wider layer stride
    wide = torch.zeros(2, V + 5, N, d, dtype=torch.bfloat16)
    mole.table_file_read(path, wide, layer0=1, n_layers=2)
    assert torch.equal(wide[:, :V].view(torch.int16), tables[1:].view(torch.int16)) and (wide[:, V:] == 0).all()
    # single rows by id: the tier that leaves the file on disk
    ids = [36, 0, 7, 7]
    rows = torch.zeros(len(ids), N, d, dtype=torch.bfloat16)
    mole.table_file_read_rows(path, 2, ids, rows)
    assert torch.equal(rows.view(torch.int16), tables[2][ids].view(torch.int16))
    # fp32 tables too
    t32 = torch.empty(1, 5, 4, 8).normal_(0, 1, generator=g)
    mole.table_file_write(path, t32, 4, 8)
    assert mole.table_file_info(path).dtype == mole.DTYPE_F32
    assert torch.equal(mole.table_file_read(path, torch.zeros_like(t32)), t32)


@pytest.mark.parametrize("nbits,block", [(4, 64), (3, 32)])
def test_quantised_table_round_trip(tmp_path, nbits, block):
    L, V, N, d = 2, 19, 4, 128
    fmt = {4: mole.LUT_NF4, 3: mole.LUT_NF3}[nbits]
    rng = np.random.default_rng(nbits)
    packed = np.stack([quant.quantize_table((0.05 * rng.standard_normal((V, N, d))).astype(np.float32), nbits, block) for _ in range(L)])
    t = torch.from_numpy(packed)
    path = str(tmp_path / "q.mole")
    mole.table_file_write(path, t, N, d, fmt, block)
    info = mole.table_file_info(path)
    assert (info.lut_format, info.lut_block, info.row_bytes) == (fmt, block, quant.record_bytes(N, d, nbits, block))
    back = mole.table_file_read(path, torch.zeros_like(t))
    assert torch.equal(back, t)
    rows = torch.zeros(2, info.row_bytes, dtype=torch.uint8)
    mole.table_file_read_rows(path, 1, [18, 3], rows)
    assert torch.equal(rows, t[1][[18, 3]])


def test_file_errors_are_error_codes(tmp_path):
    L, V, N, d = 2, 9, 4, 64
    tables = torch.zeros(L, V, N, d, dtype=torch.bfloat16)
    path = str(tmp_path / "t.mole")
    for fn in (lambda: mole.table_file_info(str(tmp_path / "missing")), lambda: mole.table_file_read(str(tmp_path / "missing"), tables)):
        with pytest.raises(mole.MoleError) as e:
            fn()
        assert e.value.code == mole.ERR_IO
    with pytest.raises(mole.MoleError) as e:
        mole.table_file_write(str(tmp_path / "no_such_dir" / "t"), tables, N, d)
    assert e.value.code == mole.ERR_IO
    (tmp_path / "junk").write_bytes(b"not a table file" * 400)
    with pytest.raises(mole.MoleError) as e:
        mole.table_file_info(str(tmp_path / "junk"))
    assert e.value.code == mole.ERR_IO
    mole.table_file_write(path, tables, N, d)
    with open(path, "r+b") as f:  # cut the last row off
        f.truncate(os.path.getsize(path) - 100)
    with pytest.raises(mole.MoleError) as e:
        mole.table_file_info(path)
    assert e.value.code == mole.ERR_IO
    with pytest.raises(mole.MoleError) as e:
        mole.table_file_read(path, tables)
    assert e.value.code == mole.ERR_IO
    mole.table_file_write(path, tables, N, d)
    with pytest.raises(mole.MoleError) as e:  # more layers than the file holds
        mole.table_file_read(path, torch.zeros(3, V, N, d, dtype=torch.bfloat16))
    assert e.value.code == mole.ERR_INVALID_ARG
    with pytest.raises(mole.MoleError) as e:  # an id outside the table
        mole.table_file_read_rows(path, 0, [V], torch.zeros(1, N, d, dtype=torch.bfloat16))
    assert e.value.code == mole.ERR_INVALID_ARG
    with pytest.raises(mole.MoleError) as e:  # a destination too narrow for a layer
        mole.table_file_read(path, torch.zeros(L, V - 1, N, d, dtype=torch.bfloat16))
    assert e.value.code == mole.ERR_INVALID_ARG
