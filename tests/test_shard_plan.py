"""The column-shard plan on CPU with two gloo ranks: each rank buckets its own shard with the library's host
bucketer and checks it, bit for bit, against the oracle's tiles restricted to the shard's columns; together
the shards hold every stored entry exactly once.  No GPU is involved."""
import json
import os
import subprocess
import sys
import textwrap
from pathlib import Path

import numpy as np

ROOT = Path(__file__).resolve().parent.parent

WORKER = textwrap.dedent("""
    import os, sys, json
    sys.path.insert(0, %r)
    import numpy as np
    import torch
    import torch.distributed as dist
    from oracle import dsfacto_oracle as O
    from paper_2004_13940_b200 import dsfacto as D
    from paper_2004_13940_b200 import workloads as W
    rank, world = int(os.environ["RANK"]), int(os.environ["WORLD_SIZE"])
    dist.init_process_group("gloo")
    ok = True
    total = 0
    for name, p in (("C1", 4), ("C3", 64), ("C2", 16), ("C1", 7)):
        wl = W.make(name, p=p)
        tp_o, rows_o, cols_o, vals_o = O.bucket(wl.n, wl.d, p, wl.indptr, wl.indices, wl.values)
        rc, kept, tp, rows, cols, vals = D.dsfacto_bucket_host_shard(wl.n, wl.d, p, rank, world, wl.indptr, wl.indices, wl.values)
        lo = -(-((rank * p) // world) * wl.d // p)
        hi = -(-(((rank + 1) * p) // world) * wl.d // p)
        keep = (cols_o >= lo) & (cols_o < hi)
        ok &= rc == 0 and kept == int(keep.sum())
        ok &= np.array_equal(rows, rows_o[keep]) and np.array_equal(cols, cols_o[keep])
        ok &= np.array_equal(vals.view(np.uint32), vals_o[keep].view(np.uint32))
        # tile sizes: the oracle's tile by tile, counting only this shard's columns
        tile_of = np.repeat(np.arange(p * p), np.diff(tp_o))
        ok &= np.array_equal(np.diff(tp), np.bincount(tile_of[keep], minlength=p * p))
        t = torch.tensor([kept], dtype=torch.int64)
        dist.all_reduce(t)
        ok &= int(t.item()) == wl.nnz          # every stored entry in exactly one shard
        total += int(t.item())
    print(json.dumps({"rank": rank, "ok": bool(ok), "total": total}), flush=True)
    dist.destroy_process_group()
""") % str(ROOT)


def test_two_gloo_ranks_bucket_their_shards_like_the_oracle(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    env = dict(os.environ, MASTER_ADDR="127.0.0.1", MASTER_PORT="29671", WORLD_SIZE="2", CUDA_VISIBLE_DEVICES="")
    procs = [subprocess.Popen([sys.executable, str(script)], env=dict(env, RANK=str(r)), stdout=subprocess.PIPE,
                              stderr=subprocess.PIPE, text=True) for r in range(2)]
    outs = [p.communicate(timeout=300) for p in procs]
    assert all(p.returncode == 0 for p in procs), outs
    res = [json.loads(o[0].strip().splitlines()[-1]) for o in outs]
    assert all(r["ok"] for r in res), res
    assert res[0]["total"] == res[1]["total"] > 0


def test_shard_bucketer_argument_checks():
    sys.path.insert(0, str(ROOT))
    from paper_2004_13940_b200 import dsfacto as D
    indptr = np.array([0, 1, 2], np.int64)
    indices = np.array([0, 1], np.int32)
    values = np.ones(2, np.float32)
    assert D.dsfacto_bucket_host_shard(2, 2, 2, 2, 2, indptr, indices, values)[0] == D.ERR_INVALID_ARG   # shard out of range
    assert D.dsfacto_bucket_host_shard(2, 2, 2, 0, 3, indptr, indices, values)[0] == D.ERR_INVALID_ARG   # more shards than blocks
    rc, kept, tp, rows, cols, vals = D.dsfacto_bucket_host_shard(2, 2, 2, 1, 2, indptr, indices, values)
    assert rc == D.OK and kept == 1 and rows.tolist() == [1] and cols.tolist() == [1]
