"""Row-sharded fused GEMV through the C ABI, on one GPU: the ranks' launches run one after another (none of them
waits on another), each writing its band into every rank's copy of y; all copies must then hold the oracle's
product.  The flag words, the bounded wait and its expiry, and the inter-process exchange buffers (two processes on
the same device, stepped by host barriers) are covered too."""
import os
import sys

import numpy as np
import pytest
import torch
import torch.multiprocessing as mp

import llvq_inputs as gen
from gpu_util import gemv_error, to_dev_bf16, to_dev_f16, to_dev_u8

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
TOL = 1e-3
TOL_BF16_OUT = 1e-3 + 2.0 ** -8


@pytest.fixture(scope="module")
def lib():
    import paper_2603_11021_b200 as P
    assert torch.cuda.is_available(), "these tests need a CUDA device; there is no CPU path"
    return P


@pytest.fixture(scope="module")
def ctx(lib):
    return lib.Context(2, 13, device=0)


@pytest.fixture(scope="module")
def code(oracle_mod):
    return oracle_mod.Code(2, 13)


def _bands_on_device(lib, ctx, o, stream, gain, n_out, k_in, world, sorted_layout):
    from paper_2603_11021_b200.rowshard import band_of_stream, row_bands
    out = []
    for row0, n in row_bands(n_out, world):
        s, g = band_of_stream(stream, gain, k_in, o.W, row0, n)
        ds, dg = to_dev_u8(s), to_dev_f16(g)
        if sorted_layout and n:
            ds = lib.llvq_sort_blocks(ctx, ds, n, k_in)
        out.append((row0, n, ds, dg))
    return out


@pytest.mark.parametrize("sorted_layout", [False, True])
@pytest.mark.parametrize("n_out,k_in,world,dtype", [(1000, 2000, 2, torch.float32), (4096, 4096, 8, torch.bfloat16),
                                                   (67, 500, 3, torch.bfloat16), (20, 480, 8, torch.float32)])
def test_every_copy_of_y_holds_the_product(lib, ctx, code, n_out, k_in, world, dtype, sorted_layout):
    o = code
    stream, gain, _ = gen.make_layer(o.N, o.W, n_out, k_in, 1, seed=31)
    x = gen.normal_bf16(k_in, seed=31)
    want = o.gemv(stream, gain, n_out, k_in, x, threads=4)
    dx = to_dev_bf16(x)
    copies = [torch.full((n_out + 8,), float("nan"), dtype=dtype, device="cuda") for _ in range(world)]
    flags = [torch.zeros(world, dtype=torch.int32, device="cuda") for _ in range(world)]
    call = lib.llvq_gemv_sorted_rowshard if sorted_layout else lib.llvq_gemv_rowshard
    for r, (row0, n, ds, dg) in enumerate(_bands_on_device(lib, ctx, o, stream, gain, n_out, k_in, world, sorted_layout)):
        words = [flags[p].data_ptr() + 4 * r for p in range(world)]      # rank r's word at every rank
        if r % 2:                                                         # the kernel raises the flags itself ...
            call(ctx, ds, dg, n, k_in, dx, copies, r, row0, dtype, flag_words=words, epoch=1)
        else:                                                             # ... or a launch of its own does
            if n:
                call(ctx, ds, dg, n, k_in, dx, copies, r, row0, dtype)
            lib.llvq_signal_ranks(ctx, [w for p, w in enumerate(words) if p != r], 1)
    for r in range(world):                         # every flag is up already: the waits return at their first look
        lib.llvq_wait_ranks(ctx, flags[r], world, r, 1)
    torch.cuda.synchronize()
    assert lib.llvq_last_error(ctx) == (0, 0)
    tol = TOL if dtype == torch.float32 else TOL_BF16_OUT
    for r in range(world):
        f = flags[r].cpu().numpy()
        assert all(f[p] == (0 if p == r else 1) for p in range(world))
        y = copies[r].float().cpu().numpy()
        assert np.isnan(y[n_out:]).all()           # nothing written past the vector
        assert gemv_error(y[:n_out], want) <= tol
    # a band's rows do not depend on which copy they were written to
    for r in range(1, world):
        assert torch.equal(copies[r][:n_out], copies[0][:n_out])


@pytest.mark.parametrize("sorted_layout", [False, True])
@pytest.mark.parametrize("n_out,k_in,world,batch", [(1000, 2000, 2, 16), (520, 1536, 4, 5), (300, 4096, 3, 64)])
def test_every_copy_of_the_batched_product(lib, ctx, code, n_out, k_in, world, batch, sorted_layout):
    from paper_2603_11021_b200.rowshard import band_of_stream, row_bands
    o = code
    stream, gain, _ = gen.make_layer(o.N, o.W, n_out, k_in, 1, seed=33)
    x = gen.normal_bf16((batch, k_in), seed=33)
    want = o.gemm(stream, gain, n_out, k_in, x, threads=4)
    dx = to_dev_bf16(x)
    copies = [torch.full((batch + 1, n_out), float("nan"), dtype=torch.bfloat16, device="cuda") for _ in range(world)]
    flags = [torch.zeros(world, dtype=torch.int32, device="cuda") for _ in range(world)]
    for r, (row0, n) in enumerate(row_bands(n_out, world, align=128 if sorted_layout else 8)):
        s, g = band_of_stream(stream, gain, k_in, o.W, row0, n)
        ds, dg = to_dev_u8(s), to_dev_f16(g)
        if sorted_layout and n:
            ds = lib.llvq_sort_blocks_gemm(ctx, ds, n, k_in)
        words = [flags[p].data_ptr() + 4 * r for p in range(world)]
        lib.llvq_gemm_small_batch_rowshard(ctx, ds, dg, n, k_in, dx, copies, r, row0, n_out, flag_words=words, epoch=2,
                                           sorted_layout=sorted_layout)
    for r in range(world):
        lib.llvq_wait_ranks(ctx, flags[r], world, r, 2)
    torch.cuda.synchronize()
    assert lib.llvq_last_error(ctx) == (0, 0)
    for r in range(world):
        f = flags[r].cpu().numpy()
        assert all(f[p] == (0 if p == r else 2) for p in range(world))
        y = copies[r].float().cpu().numpy()
        assert np.isnan(y[batch]).all()            # nothing written past the matrix
        assert gemv_error(y[:batch], want) <= TOL_BF16_OUT
        assert torch.equal(copies[r][:batch], copies[0][:batch])


def test_degenerate_bands_still_raise_their_flags(lib, ctx, code):
    o = code
    stream, gain, _ = gen.make_layer(o.N, o.W, 8, 48, 1, seed=2)
    ds, dg, dx = to_dev_u8(stream), to_dev_f16(gain), to_dev_bf16(gen.normal_bf16(48, seed=2))
    copies = [torch.full((16,), 5.0, device="cuda") for _ in range(2)]
    flags = [torch.zeros(2, dtype=torch.int32, device="cuda") for _ in range(2)]
    words = lambda r: [flags[p].data_ptr() + 4 * r for p in range(2)]
    # rank 0 has no rows at all: nothing is written, the peer still hears from it
    lib.llvq_gemv_rowshard(ctx, ds, dg, 0, 48, dx, copies, 0, 0, torch.float32, flag_words=words(0), epoch=3)
    # rank 1 has rows but no columns: its rows are zero everywhere
    lib.llvq_gemv_rowshard(ctx, ds, dg, 8, 0, dx, copies, 1, 8, torch.float32, flag_words=words(1), epoch=3)
    for r in range(2):
        lib.llvq_wait_ranks(ctx, flags[r], 2, r, 3)
    torch.cuda.synchronize()
    assert lib.llvq_last_error(ctx) == (0, 0)
    assert flags[0].tolist() == [0, 3] and flags[1].tolist() == [3, 0]
    for c in copies:
        assert c[:8].tolist() == [5.0] * 8 and c[8:].tolist() == [0.0] * 8


def test_wait_runs_out_on_a_flag_nobody_raises(lib, ctx):
    flags = torch.zeros(4, dtype=torch.int32, device="cuda")
    flags[1] = 7
    lib.llvq_wait_ranks(ctx, flags, 4, 0, 7, max_spins=64)               # words 2 and 3 stay at 0
    torch.cuda.synchronize()
    assert lib.llvq_last_error(ctx) == (0, lib.LLVQ_FLAG_WAIT_TIMEOUT)
    flags[2:] = 9                                                         # beyond the epoch counts as reached
    lib.llvq_wait_ranks(ctx, flags, 4, 0, 7, max_spins=64)
    torch.cuda.synchronize()
    assert lib.llvq_last_error(ctx) == (0, 0)                             # the context is as usable as before


def test_epochs_may_wrap(lib, ctx):
    flags = torch.tensor([3, 3], dtype=torch.int32, device="cuda")       # the writers are already past the wrap
    lib.llvq_wait_ranks(ctx, flags, 2, -1, 0xfffffffe, max_spins=64)
    torch.cuda.synchronize()
    assert lib.llvq_last_error(ctx) == (0, 0)
    flags[:] = -3                                                         # 0xfffffffd: one before the epoch
    lib.llvq_wait_ranks(ctx, flags, 2, -1, 0xfffffffe, max_spins=64)
    torch.cuda.synchronize()
    assert lib.llvq_last_error(ctx) == (0, lib.LLVQ_FLAG_WAIT_TIMEOUT)


def test_argument_checks(lib, ctx, code):
    o = code
    stream, gain, _ = gen.make_layer(o.N, o.W, 16, 48, 1, seed=1)
    ds, dg, dx = to_dev_u8(stream), to_dev_f16(gain), to_dev_bf16(gen.normal_bf16(48, seed=1))
    y = torch.zeros(16, device="cuda")
    for y_all, own in [([y] * 9, 0), ([y], 1), ([y], -1), ([y, 0], 0)]:
        with pytest.raises((lib.LlvqError, AssertionError)):
            lib.llvq_gemv_rowshard(ctx, ds, dg, 16, 48, dx, y_all, own, 0)
    with pytest.raises(lib.LlvqError):
        lib.llvq_gemv_rowshard(ctx, ds, dg, 16, 48, dx, [y], 0, -8)
    with pytest.raises(lib.LlvqError):
        lib.llvq_wait_ranks(ctx, y, 9, 0, 1)
    with pytest.raises(lib.LlvqError):
        lib.llvq_signal_ranks(ctx, [0], 1)
    torch.cuda.synchronize()
    assert lib.llvq_last_error(ctx) == (0, 0)


def _two_process_rank(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import torch.distributed as dist
    import oracle
    import paper_2603_11021_b200 as P
    from paper_2603_11021_b200.rowshard import RowShardedGemv, band_of_stream, row_bands
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    torch.cuda.set_device(0)                                              # both ranks share the one device
    ctx = P.Context(2, 13, device=0)
    o = oracle.Code(2, 13)
    n_out, k_in = 520, 1536
    stream, gain, _ = gen.make_layer(o.N, o.W, n_out, k_in, 1, seed=44)
    row0, n = row_bands(n_out, world)[rank]
    s, g = band_of_stream(stream, gain, k_in, o.W, row0, n)
    ok = True
    for sorted_layout in (False, True):
        dtype = torch.bfloat16 if sorted_layout else torch.float32
        op = RowShardedGemv(ctx, n_out, k_in, to_dev_u8(s), to_dev_f16(g), dtype, sorted_layout=sorted_layout)
        for step in range(3):
            x = gen.normal_bf16(k_in, seed=100 + step)
            op.launch(to_dev_bf16(x))
            torch.cuda.synchronize()
            dist.barrier()                                                # every rank's band and flag are in place:
            y = op.wait()                                                 # the wait kernel never waits on a running kernel
            torch.cuda.synchronize()
            ok = ok and P.llvq_last_error(ctx) == (0, 0)
            ok = ok and gemv_error(y.float().cpu().numpy(), o.gemv(stream, gain, n_out, k_in, x, threads=2)) <= TOL_BF16_OUT
            dist.barrier()
        op.close()
    out[rank] = ok
    dist.barrier()
    dist.destroy_process_group()


def test_two_processes_exchange_through_ipc_buffers():
    mpc = mp.get_context("spawn")
    with mpc.Manager() as m:
        out = m.dict()
        procs = [mpc.Process(target=_two_process_rank, args=(r, 2, 29547, out)) for r in range(2)]
        for p in procs:
            p.start()
        for p in procs:
            p.join(300)
            assert p.exitcode == 0
        assert dict(out) == {0: True, 1: True}


def test_bench_strong_scaling_leg_runs_on_one_rank():
    # the benchmark's strong-scaling leg (one matrix spread over the ranks, rotating band copies, agreement of all ranks' y,
    # comparison with the unsharded product), driven with a single rank: every code path but the peer stores
    import json
    import subprocess
    env = dict(os.environ, MASTER_PORT="29591")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--steps", "3", "--warmup", "3", "--no-extras", "--no-cpu-baseline",
                        "--rowshard-leg"], capture_output=True, text=True, env=env, timeout=900)
    assert r.returncode == 0, r.stderr[-2000:]
    line = json.loads(r.stdout.strip().splitlines()[-1])
    leg = line["rowshard"]
    assert leg["world"] == 1 and leg["errors"] == [0, 0]
    assert set(leg["shapes"]) == {"11008x4096", "6144x4096", "4096x4096", "28672x4096", "4096x14336"}
    for shape in leg["shapes"].values():
        assert shape["all_ranks_same_y"] and shape["max_rel_diff_to_unsharded"] <= 2.0 ** -7
        assert shape["us_per_step"] >= shape["us_band_gemv"] > 0
