"""Host logic of the row-sharded GEMV on CPU: the band plan, slicing a ROWWISE stream into bands, and the path with
two ranks (gloo): each rank works on its band alone, the handles travel through the process group, and the
assembled vector is the unsharded product (the per-band products come from the oracle here: the device kernels
are covered by the GPU tests)."""
import os
import sys

import numpy as np
import pytest
import torch.multiprocessing as mp

import llvq_inputs as gen
from paper_2603_11021_b200.rowshard import band_of_stream, row_bands

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.mark.parametrize("n_out,world,align", [(4096, 8, 8), (11008, 8, 64), (11008, 3, 8), (67, 4, 8), (5, 8, 8), (0, 2, 8),
                                               (28672, 7, 128), (1000, 1, 8)])
def test_row_bands_cover_align_balance(n_out, world, align):
    bands = row_bands(n_out, world, align)
    assert len(bands) == world
    nxt = 0
    for row0, n in bands:
        assert row0 == nxt and n >= 0
        assert row0 % align == 0 or row0 == n_out
        nxt = row0 + n
    assert nxt == n_out
    groups = [(n + align - 1) // align for _, n in bands]
    assert max(groups) - min(groups) <= 1
    assert groups == sorted(groups, reverse=True)              # the extra groups go to the first ranks


def test_row_bands_rejects_nonsense():
    for args in [(-1, 2, 8), (8, 0, 8), (8, 2, 0)]:
        with pytest.raises(ValueError):
            row_bands(*args)


@pytest.mark.parametrize("code,n_out,k_in,world", [((2, 13), 67, 500, 3), ((2, 2), 40, 768, 2), ((3, 3), 24, 100, 4),
                                                   ((2, 2), 5, 24, 3)])          # the last one: empty bands that start at row 5
def test_bands_of_a_stream_give_the_bands_of_y(oracle_mod, code, n_out, k_in, world):
    o = oracle_mod.Code(*code)
    stream, gain, _ = gen.make_layer(o.N, o.W, n_out, k_in, 1, seed=12)
    x = gen.normal_bf16(k_in, seed=12)
    want = o.gemv(stream, gain, n_out, k_in, x)
    parts = []
    for row0, n in row_bands(n_out, world):
        s, g = band_of_stream(stream, gain, k_in, o.W, row0, n)
        assert s.size % 16 == 0 and g.size == n * ((k_in + 23) // 24)
        parts.append(o.gemv(s, g, n, k_in, x) if n else np.zeros(0))
    assert np.array_equal(np.concatenate(parts), want)         # the same arithmetic row by row: identical, not close


def test_band_must_start_on_a_byte():
    with pytest.raises(ValueError):
        band_of_stream(np.zeros(64, np.uint8), np.zeros(16, np.uint16), 24, 18, 1, 2)


def _rank_main(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import torch
    import torch.distributed as dist
    import oracle
    from paper_2603_11021_b200.rowshard import band_of_stream, exchange_handles, row_bands
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    o = oracle.Code(2, 13)
    n_out, k_in = 83, 600
    stream, gain, _ = gen.make_layer(o.N, o.W, n_out, k_in, 1, seed=21)
    x = gen.normal_bf16(k_in, seed=21)
    handles = exchange_handles(bytes([rank]) * 64)
    bands = row_bands(n_out, world)
    row0, n = bands[rank]
    s, g = band_of_stream(stream, gain, k_in, o.W, row0, n)
    mine = torch.from_numpy(o.gemv(s, g, n, k_in, x))
    pieces = [None] * world
    dist.all_gather_object(pieces, mine)                       # the bands differ in length
    y = torch.cat(pieces).numpy()
    out[rank] = (handles, bool(np.array_equal(y, o.gemv(stream, gain, n_out, k_in, x))), (row0, n))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_assemble_the_unsharded_product():
    ctx = mp.get_context("spawn")
    with ctx.Manager() as m:
        out = m.dict()
        procs = [ctx.Process(target=_rank_main, args=(r, 2, 29541, out)) for r in range(2)]
        for p in procs:
            p.start()
        for p in procs:
            p.join(180)
            assert p.exitcode == 0
        res = dict(out)
    for r in range(2):
        handles, same, band = res[r]
        assert handles == [bytes([0]) * 64, bytes([1]) * 64]    # every rank holds every handle, in rank order
        assert same
    assert res[0][2] == (0, 48) and res[1][2] == (48, 35)
