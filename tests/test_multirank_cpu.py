"""The multi-rank path of the benchmark is "replicas only": no data-path collective, only a barrier
and a maximum over ranks of the device-timed interval.  These tests run that host logic as two gloo
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
