"""Host-side logic of the benchmark's multi-rank path, on CPU with gloo (world size 2): the timing
reduction is a max over ranks, the whole-job value scales with the world size, ranks draw different
layers, and the reference arm prints its line on rank 0 only."""
import json
import os
import subprocess
import sys

import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    import torch.distributed as dist
    sys.path.insert(0, ROOT)
    import bench
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    ms = bench.max_over_ranks(10.0 + 5.0 * rank, dist, "cpu")          # rank 1 is the slow one
    dist.barrier()
    out[rank] = (ms, bench.whole_job_value(world, 1_000_000, ms), bench.rank_seed(rank, 3, 2))
    dist.destroy_process_group()


def test_max_over_ranks_and_weak_scaling_value():
    ctx = mp.get_context("spawn")
    with ctx.Manager() as m:
        out = m.dict()
        procs = [ctx.Process(target=_worker, args=(r, 2, 29533, out)) for r in range(2)]
        for p in procs:
            p.start()
        for p in procs:
            p.join(120)
            assert p.exitcode == 0
        res = dict(out)
    assert res[0][0] == res[1][0] == 15.0                              # max over ranks, seen by both
    assert abs(res[0][1] - 2 * 1_000_000 / 15e-3 / 1e9) < 1e-12        # whole job = world x per-rank bytes / max time
    assert res[0][2] != res[1][2]                                      # ranks draw different layers


def _agree_worker(rank, world, port, out):
    import torch
    import torch.distributed as dist
    sys.path.insert(0, ROOT)
    import bench
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    same = torch.arange(64, dtype=torch.float32).to(torch.bfloat16)
    differs = same.clone()
    if rank == 1:
        differs[17] = -1.0                                             # one rank ends up with another value in one row
    plans = [bench.rowshard_plan(11008, 4096, world, r) for r in range(world)]
    out[rank] = (bench.ranks_agree(same, dist), bench.ranks_agree(differs, dist), plans)
    dist.destroy_process_group()


def test_strong_scaling_leg_host_logic():
    # the band plan of the row-sharded leg covers the matrix, and the agreement check fails on every rank as soon as one
    # rank's copy of y differs
    ctx = mp.get_context("spawn")
    with ctx.Manager() as m:
        out = m.dict()
        procs = [ctx.Process(target=_agree_worker, args=(r, 2, 29537, out)) for r in range(2)]
        for p in procs:
            p.start()
        for p in procs:
            p.join(120)
            assert p.exitcode == 0
        res = dict(out)
    for r in range(2):
        agree_same, agree_differs, plans = res[r]
        assert agree_same is True and agree_differs is False
        assert [p["row0"] for p in plans] == [0, 5504] and sum(p["rows"] for p in plans) == 11008
        assert all(p["rows"] % 8 == 0 for p in plans)
        assert plans[0]["band_bytes"] == 5504 * 171 * 8 + 2 * 4096 + 2 * 5504


def test_single_process_path_has_no_collective():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(3.5, None, "cpu") == 3.5
    assert bench.algorithmic_bytes(4096, 4096) == 700416 * 8 + 4096 * 2 + 4096 * 2


def test_reference_arm_prints_on_rank0_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "1", "--warmup", "0"],
                       capture_output=True, text=True, env=env, timeout=300)
    assert r.returncode == 0 and r.stdout.strip() == ""
    env["RANK"] = "0"
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "1", "--warmup", "0", "--gpus", "2"],
                       capture_output=True, text=True, env=env, timeout=300)
    assert r.returncode == 0
    line = json.loads(r.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["cpu_baseline"]["kind"] == "oracle" and line["value"] > 0
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["unit"] == "GB/s"


def test_counter_file_vouches_for_its_sources_only(tmp_path):
    # the benchmark quotes profiler counters only while the sources the captured kernel is compiled from are unchanged
    sys.path.insert(0, ROOT)
    from paper_2603_11021_b200 import ncu_counters as nc
    raw = tmp_path / "raw.csv"
    raw.write_text('"ID","Kernel Name","gpu__time_duration.sum","dram__bytes_read.sum","smsp__inst_executed.sum"\n'
                   '"","","us","Mbyte","inst"\n'
                   '"0","void k<1>(int)","120.5","45.0","1000"\n')
    d = nc.parse_raw_csv(str(raw))
    assert d["kernel"] == "void k<1>" and d["duration_ns"] == 120500.0 and d["dram_bytes_read"] == 45e6 and d["warp_instructions"] == 1000.0
    good = tmp_path / "good.json"
    good.write_text(json.dumps({"duration_ns": 1.0, "sources": ["tables.h"], "source_hash": nc.source_hash(["tables.h"])}))
    assert nc.load(str(good))["duration_ns"] == 1.0
    stale = tmp_path / "stale.json"
    stale.write_text(json.dumps({"duration_ns": 1.0, "sources": ["tables.h"], "source_hash": "0" * 16}))
    assert nc.load(str(stale)) is None and nc.load(str(tmp_path / "missing.json")) is None
    assert nc.source_hash(["tables.h"]) != nc.source_hash(["tables.h", "fast.cuh"])
