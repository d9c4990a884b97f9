"""The multi-rank path of the benchmark is "replicas only": no data-path collective, only a barrier
and a maximum over ranks of the device-timed interval.  The slice-sharded iteration has one real
exchange: the all-reduce of the per-layer moment sums.  These tests run that host logic as two gloo
ranks on the CPU (no GPU, no CUDA library needed)."""
import json
import os
import socket
import subprocess
import sys
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

RANK_SCRIPT = textwrap.dedent("""
    import json, os, sys
    sys.path.insert(0, %r)
    import torch, torch.distributed as dist
    import bench
    rank, world = int(os.environ["RANK"]), int(os.environ["WORLD_SIZE"])
    dist.init_process_group("gloo")
    ms = bench.max_over_ranks(10.0 + 5.0 * rank, world, "cpu")        # rank 1 is the slow replica
    wl = bench.replica_workload(rank, n_users=1)
    g = wl.gradient(0)[:, :4096]                                      # this replica's own draw
    digest = torch.tensor([float(g.double().abs().sum())], dtype=torch.float64)
    all_d = [torch.zeros(1, dtype=torch.float64) for _ in range(world)]
    dist.all_gather(all_d, digest)
    dist.barrier()
    if rank == 0:
        print(json.dumps({"ms": ms, "value": bench.job_throughput_gbs(world, 4.0e9, 10, ms),
                          "digests": [float(x) for x in all_d], "ld": wl.ld, "d": wl.d}))
    dist.destroy_process_group()
""") % ROOT


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def test_two_replicas_report_the_slowest_time_and_the_sum_of_the_work():
    port = _free_port()
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), WORLD_SIZE="2", LOCAL_RANK=str(rank),
                   MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, "-c", RANK_SCRIPT], env=env, cwd=ROOT,
                                      stdout=subprocess.PIPE, stderr=subprocess.PIPE, text=True))
    outs = [p.communicate(timeout=240) for p in procs]
    assert all(p.returncode == 0 for p in procs), [o[1][-2000:] for o in outs]
    assert outs[1][0].strip() == ""                                   # only rank 0 prints
    r = json.loads(outs[0][0].strip().splitlines()[-1])
    assert r["ms"] == 15.0                                            # max over ranks, not rank 0's 10 ms
    assert abs(r["value"] - 2 * 4.0e9 * 10 / 15.0e-3 / 1e9) < 1e-6    # both replicas' bytes over that time
    assert r["digests"][0] != r["digests"][1]                         # replicas draw different gradients
    assert r["ld"] % 4096 == 0 and r["ld"] >= r["d"]


def test_reference_arm_runs_on_rank_0_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    p = subprocess.run([sys.executable, "bench.py", "--impl", "reference", "--gpus", "2", "--steps", "1"],
                       env=env, cwd=ROOT, capture_output=True, text=True, timeout=240)
    assert p.returncode == 0 and p.stdout.strip() == ""


SLICE_SCRIPT = textwrap.dedent("""
    import json, os, sys
    sys.path.insert(0, %r)
    import torch, torch.distributed as dist
    from paper_2203_09044_b200 import sharded
    rank, world = int(os.environ["RANK"]), int(os.environ["WORLD_SIZE"])
    dist.init_process_group("gloo")
    d, off = 20000, [0, 3000, 3000, 9000, 12288, 20000]             # segment 1 is empty, 2 and 3 span the cut
    lay = sharded.SliceLayout(d, off, rank, world)
    # stand-in for the exported sums: every local segment reports its element count and two multiples
    n = torch.tensor([lay.local_offsets[i + 1] - lay.local_offsets[i] for i in range(len(lay.seg_ids))],
                     dtype=torch.float64)
    local = torch.stack([n, 0.5 * n, 0.25 * n * (rank + 1)], dim=1)
    pooled = sharded.all_reduce_sum(lay.to_global(local))
    mine = lay.to_local(pooled)
    print(json.dumps({"rank": rank, "lo": lay.lo, "hi": lay.hi, "seg_ids": lay.seg_ids,
                      "local_offsets": lay.local_offsets, "pooled": pooled.tolist(), "mine": mine.tolist()}))
    dist.destroy_process_group()
""") % ROOT


def test_slices_pool_their_layer_moments_with_one_all_reduce():
    port = _free_port()
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), WORLD_SIZE="2", LOCAL_RANK=str(rank),
                   MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, "-c", SLICE_SCRIPT], env=env, cwd=ROOT,
                                      stdout=subprocess.PIPE, stderr=subprocess.PIPE, text=True))
    outs = [p.communicate(timeout=240) for p in procs]
    assert all(p.returncode == 0 for p in procs), [o[1][-2000:] for o in outs]
    r0, r1 = (json.loads(o[0].strip().splitlines()[-1]) for o in outs)
    # 5 tiles of 4096 for 2 ranks: 3 + 2, cut at 12288
    assert (r0["lo"], r0["hi"], r1["lo"], r1["hi"]) == (0, 12288, 12288, 20000)
    assert r0["seg_ids"] == [0, 2, 3] and r0["local_offsets"] == [0, 3000, 9000, 12288]
    assert r1["seg_ids"] == [4] and r1["local_offsets"] == [0, 20000 - 12288]
    sizes = [3000, 0, 6000, 3288, 7712]
    assert r0["pooled"] == r1["pooled"]                               # every rank ends with the same table
    assert [row[0] for row in r0["pooled"]] == sizes                  # entries of each layer over all slices
    assert [row[1] for row in r0["pooled"]] == [0.5 * n for n in sizes]
    assert r0["pooled"][4][2] == 0.25 * 7712 * 2 and r0["pooled"][0][2] == 0.25 * 3000
    assert r0["mine"] == [r0["pooled"][i] for i in (0, 2, 3)] and r1["mine"] == [r1["pooled"][4]]


def test_slice_bounds_cover_d_in_whole_tiles():
    from paper_2203_09044_b200 import sharded
    import pytest
    for d, world in [(4096, 1), (20000, 2), (11_173_962, 8), (124_439_808, 3), (65536, 16)]:
        b = sharded.slice_bounds(d, world)
        assert b[0][0] == 0 and b[-1][1] == d and len(b) == world
        assert all(b[i][1] == b[i + 1][0] for i in range(world - 1))
        assert all(lo % 4096 == 0 and hi > lo for lo, hi in b)
        tiles = [-(-(hi - lo) // 4096) for lo, hi in b]
        assert max(tiles) - min(tiles) <= 1
    with pytest.raises(ValueError):
        sharded.slice_bounds(8000, 3)
    # a layer cut by the slice boundary appears in both layouts under the same global index
    off = [0, 5000, 30000]
    a, c = sharded.SliceLayout(30000, off, 0, 2), sharded.SliceLayout(30000, off, 1, 2)
    assert a.seg_ids == [0, 1] and c.seg_ids == [1] and a.hi == c.lo == 16384
