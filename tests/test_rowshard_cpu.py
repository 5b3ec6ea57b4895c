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


def _protocol_rank(rank, world, port, out):
    """The order and the arguments of the device calls of RowShardedGemv, with the library calls replaced by recorders."""
    sys.path.insert(0, ROOT)
    from types import SimpleNamespace
    import torch
    import torch.distributed as dist
    import paper_2603_11021_b200.rowshard as rs
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    log = []
    own = 0x10000000 * (rank + 1)
    mapped = lambda r: 0x10000000 * (r + 1) + 0x5000000              # where this process "maps" rank r's buffer
    rs.llvq_exchange_create = lambda ctx, nbytes: (log.append(("create", nbytes)), (own, bytes([rank]) * 64))[1]
    rs.llvq_exchange_open = lambda ctx, handle: mapped(handle[0])
    rs.llvq_exchange_close = lambda ctx, p: log.append(("close", p))
    rs.llvq_exchange_destroy = lambda ctx, p: log.append(("destroy", p))
    rs.llvq_gemv_rowshard = lambda ctx, s, g, n, k, x, y_all, slot, row0, dt, words, epoch, stream: \
        log.append(("gemv", n, k, x, tuple(y_all), slot, row0, tuple(words), epoch))
    rs.llvq_signal_ranks = lambda ctx, words, epoch, stream=None: log.append(("signal", tuple(words), epoch))
    rs.llvq_wait_ranks = lambda ctx, flags, w, skip, epoch, spins=0, stream=None: log.append(("wait", flags, w, skip, epoch))

    class Recorded(rs.RowShardedGemv):
        def _wrap(self, ptr):
            return ptr

        def _synchronize(self):
            pass

    n_out, k_in = 12, 600                                             # two row groups: ranks 0 and 1 get 8 and 4 rows, rank 2 none
    op = Recorded(SimpleNamespace(device=0), n_out, k_in, "stream", "gain", torch.float32)
    y1 = op(d_x="x1")
    y2 = op(d_x="x2")
    op.close()
    out[rank] = (log, y1, y2, own, [mapped(r) for r in range(world)])
    dist.barrier()
    dist.destroy_process_group()


def test_three_ranks_step_protocol():
    world = 3
    ctx = mp.get_context("spawn")
    with ctx.Manager() as m:
        out = m.dict()
        procs = [ctx.Process(target=_protocol_rank, args=(r, world, 29553, out)) for r in range(world)]
        for p in procs:
            p.start()
        for p in procs:
            p.join(180)
            assert p.exitcode == 0
        res = dict(out)
    y_bytes = 256                                                     # 12 floats, padded to 256 bytes
    bands = [(0, 8), (8, 4), (12, 0)]
    for r in range(world):
        log, y1, y2, own, mapped = res[r]
        bufs = [own if q == r else mapped[q] for q in range(world)]
        words = tuple(b + 4 * r for b in bufs)                        # this rank's flag word in every buffer
        y_at = lambda parity: tuple(b + 256 + parity * y_bytes for b in bufs)
        assert log[0] == ("create", 256 + 2 * y_bytes)
        row0, n = bands[r]
        if n:
            step1 = ("gemv", n, 600, "x1", y_at(1), r, row0, words, 1)
            step2 = ("gemv", n, 600, "x2", y_at(0), r, row0, words, 2)
        else:                                                         # no rows: the flags still go out
            peers = tuple(w for q, w in enumerate(words) if q != r)
            step1, step2 = ("signal", peers, 1), ("signal", peers, 2)
        assert log[1:5] == [step1, ("wait", own, world, r, 1), step2, ("wait", own, world, r, 2)]
        assert (y1, y2) == (own + 256 + y_bytes, own + 256)           # the two y buffers alternate with the epoch
        assert log[5:] == [("close", mapped[q]) for q in range(world) if q != r] + [("destroy", own)]
