"""Host-side logic of the multi-rank bench run, on CPU: two gloo ranks, no GPU.

The path shards by batch with no exchange step (replicas only), so the only multi-rank code is the
aggregation of the per-rank timings: whole-job units divided by the slowest rank's time.
"""
import json
import os
import socket
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r"""
import os, sys, json
sys.path.insert(0, os.environ["PSB_ROOT"])
import torch.distributed as dist
import bench
rank = int(os.environ["RANK"])
dist.init_process_group("gloo", init_method="tcp://127.0.0.1:%s" % os.environ["PSB_PORT"],
                        rank=rank, world_size=int(os.environ["WORLD_SIZE"]))
# rank r took (1 + r) seconds for 100 * (r + 1) units
sec, units = bench.aggregate_over_ranks(1.0 + rank, 100.0 * (rank + 1), dist)
dist.barrier()
dist.destroy_process_group()
print(json.dumps({"rank": rank, "sec": sec, "units": units}))
"""


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def test_two_ranks_report_the_sum_of_units_over_the_slowest_time():
    port = _free_port()
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), WORLD_SIZE="2", PSB_PORT=str(port), PSB_ROOT=ROOT,
                   MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, "-c", WORKER], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.PIPE, text=True))
    outs = []
    for p in procs:
        out, err = p.communicate(timeout=240)
        assert p.returncode == 0, err[-2000:]
        outs.append(json.loads(out.strip().splitlines()[-1]))
    for o in outs:
        assert o["sec"] == 2.0          # the slower rank's time
        assert o["units"] == 300.0      # units of both ranks


def test_single_process_aggregation_is_the_identity():
    sys.path.insert(0, ROOT)
    import bench

    assert bench.aggregate_over_ranks(0.5, 7) == (0.5, 7)


def test_reference_arm_runs_on_rank_zero_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "1",
                        "--warmup", "0"], env=env, capture_output=True, text=True, timeout=240)
    assert r.returncode == 0 and r.stdout.strip() == ""
