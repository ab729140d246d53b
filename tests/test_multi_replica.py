"""The N > 1 path of bench.py on CPU: two gloo ranks.

The hot path is single-GPU; with several GPUs bench.py runs independent replicas, lets the ranks
load one at a time and reports the whole-job rate from the slowest rank's time.  These helpers are
exercised here with two processes and the gloo backend (no GPU involved)."""
import os
import subprocess
import sys
import textwrap
from pathlib import Path

ROOT = Path(__file__).resolve().parent.parent

WORKER = textwrap.dedent("""
    import os, sys, time, json
    sys.path.insert(0, %r)
    import torch.distributed as dist
    import bench
    rank, world = int(os.environ["RANK"]), int(os.environ["WORLD_SIZE"])
    dist.init_process_group("gloo")
    log = os.environ["TURN_LOG"]
    def load():
        with open(log, "a") as f: f.write("enter %%d\\n" %% rank)
        time.sleep(0.2)
        with open(log, "a") as f: f.write("leave %%d\\n" %% rank)
        return rank * 10
    got = bench.take_turns(rank, world, dist.barrier, load)
    ms, e2e = bench.max_over_ranks([10.0 + rank, 100.0 - rank], world, "cpu")
    rate = bench.whole_job_rate(world, 1000, 5, ms)
    print(json.dumps({"rank": rank, "got": got, "ms": ms, "e2e": e2e, "rate": rate}), flush=True)
    dist.destroy_process_group()
""") % str(ROOT)


def test_two_gloo_ranks_take_turns_and_agree_on_the_slowest_time(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    log = tmp_path / "turns.log"
    env = dict(os.environ, MASTER_ADDR="127.0.0.1", MASTER_PORT="29653", WORLD_SIZE="2", TURN_LOG=str(log),
               CUDA_VISIBLE_DEVICES="")
    procs = [subprocess.Popen([sys.executable, str(script)], env=dict(env, RANK=str(r)), stdout=subprocess.PIPE,
                              stderr=subprocess.PIPE, text=True) for r in range(2)]
    outs = [p.communicate(timeout=180) for p in procs]
    assert all(p.returncode == 0 for p in procs), outs
    import json
    res = sorted((json.loads(o[0].strip().splitlines()[-1]) for o in outs), key=lambda d: d["rank"])
    assert [d["got"] for d in res] == [0, 10]                      # each rank got its own result
    assert all(d["ms"] == 11.0 and d["e2e"] == 100.0 for d in res)  # maximum over ranks, on every rank
    assert all(d["rate"] == 2 * 1000 * 5 / 11e-3 for d in res)     # whole job: both replicas' units
    assert log.read_text().split() == "enter 0 leave 0 enter 1 leave 1".split()   # loads never overlap


def test_single_rank_helpers_are_identities():
    sys.path.insert(0, str(ROOT))
    import bench
    assert bench.take_turns(0, 1, lambda: None, lambda: 7) == 7
    assert bench.max_over_ranks([1.5, 2.5], 1, "cpu") == [1.5, 2.5]
    assert bench.whole_job_rate(1, 100, 2, 50.0) == 4000.0
