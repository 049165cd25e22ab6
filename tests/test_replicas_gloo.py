"""The N > 1 path of bench.py is request-sharded replicas: each rank draws its own batch, no collective touches
the data path, and only the timing / token totals are reduced.  Checked here with two gloo ranks on CPU."""
import os
import subprocess
import sys

import numpy as np
import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r"""
import os, sys, json
sys.path.insert(0, os.environ["BS_ROOT"])
import torch, torch.distributed as dist
import bench, bs_inputs
rank, world, local = bench.dist_env()
dist.init_process_group("gloo", rank=rank, world_size=world)
dev = torch.device("cpu")
wl = bs_inputs.workload(2, seed=bench.shard_seed(0, rank))
t = bench.max_over_ranks(1.0 + rank, world, dev)            # slowest rank defines the time
c = bench.sum_over_ranks(float(wl.committed_target()), world, dev)
bench.barrier(world)
print(json.dumps({"rank": rank, "t": t, "c": c, "own": wl.committed_target(),
                  "p": [r.p for r in wl.requests]}), flush=True)
dist.destroy_process_group()
"""


def test_two_gloo_ranks_shard_by_request_and_reduce_only_totals(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    env = dict(os.environ, BS_ROOT=ROOT, MASTER_ADDR="127.0.0.1", MASTER_PORT="29653", WORLD_SIZE="2")
    procs = []
    for rank in range(2):
        e = dict(env, RANK=str(rank), LOCAL_RANK=str(rank))
        procs.append(subprocess.Popen([sys.executable, str(script)], env=e, stdout=subprocess.PIPE,
                                      stderr=subprocess.PIPE, text=True))
    outs = []
    for p in procs:
        out, err = p.communicate(timeout=180)
        assert p.returncode == 0, err[-2000:]
        outs.append(eval(out.strip().splitlines()[-1].replace("true", "True")))
    outs.sort(key=lambda o: o["rank"])
    assert outs[0]["t"] == outs[1]["t"] == 2.0                     # max over ranks
    assert outs[0]["c"] == outs[1]["c"] == outs[0]["own"] + outs[1]["own"]   # whole-job token total
    assert outs[0]["p"] != outs[1]["p"]                            # each replica serves its own batch
    import bs_inputs
    import bench
    again = bs_inputs.workload(2, seed=bench.shard_seed(0, 1))
    assert [r.p for r in again.requests] == outs[1]["p"]           # and the draw is reproducible


def test_reference_arm_runs_on_rank_zero_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "1",
                        "--warmup", "0"], env=env, capture_output=True, text=True, timeout=120)
    assert r.returncode == 0 and r.stdout.strip() == ""


STUB = r"""
import os, sys, json
import torch.distributed as dist
rank, world = int(os.environ["RANK"]), int(os.environ["WORLD_SIZE"])
dist.init_process_group("gloo", rank=rank, world_size=world)
dist.barrier()
if rank == 0:
    print(json.dumps({"n_gpus": world, "argv": sys.argv[1:], "local_rank": os.environ["LOCAL_RANK"]}), flush=True)
dist.destroy_process_group()
"""


def test_plain_start_with_gpus_n_launches_n_ranks(tmp_path):
    """`python bench.py --gpus N` without a launcher must start N ranks itself: here the launcher runs a stub worker
    (gloo, CPU) and both ranks must meet at the rendezvous it set up; rank 0's line names the world size."""
    import json
    sys.path.insert(0, ROOT)
    import bench
    stub = tmp_path / "stub.py"
    stub.write_text(STUB)
    res = bench.launch_ranks(2, ["--gpus", "2", "--steps", "1"], worker=[sys.executable, str(stub)],
                             check_devices=False, timeout_s=120)
    assert [rc for rc, _ in res] == [0, 0]
    line = json.loads(res[0][1].strip().splitlines()[-1])
    assert line["n_gpus"] == 2 and line["argv"] == ["--gpus", "2", "--steps", "1"] and line["local_rank"] == "0"
    assert res[1][1].strip() == ""                       # only rank 0 prints


def test_more_ranks_than_devices_is_refused():
    import torch
    sys.path.insert(0, ROOT)
    import bench
    with pytest.raises(SystemExit):
        bench.launch_ranks(torch.cuda.device_count() + 1, [])
