"""Column-sharded DS-FACTO epochs: the partition of Section 4.2 (column blocks of w and V spread over the
workers, every worker sees the rows) with one exchange per epoch.

Every shard is a handle made by dsfacto_create_shard; all arithmetic runs inside libdsfacto.so.  This module
only moves the shards' partial auxiliaries [A | lin | q] to where they are added up:

  ShardGroup     all shards live in this process on one GPU; the buffers are added with one torch add per
                 shard.  This is how the sharded path is tested where only one GPU can be had.
  DistributedShard   one shard per rank of an initialised torch.distributed group; the buffers are added with
                 one all_reduce (NCCL on GPUs).  The reduction runs on this rank's own tensor: no peer memory
                 is handed to a library kernel, and nothing here uses multicast loads.

The objective of eq. (fm_obj) needs the squared norms of all columns: each shard returns those of its own
columns and they are added here (a second, four-number reduction in the distributed case)."""
from __future__ import annotations

import numpy as np

from . import dsfacto as D


class _Shard:
    def __init__(self, n, d, K, p, loss, lambda_w, lambda_v, eta, seed, shard, nshards, device):
        import torch

        self.h = D.DSFacto(n, d, K, p, loss, lambda_w, lambda_v, eta, seed, shard=shard, nshards=nshards)
        self.lambda_w, self.lambda_v, self.n = float(lambda_w), float(lambda_v), int(n)
        self.count = self.h.shard_partial_count()
        self.buf = torch.empty(self.count, dtype=torch.float32, device=device)

    def partial(self):
        self.h.shard_partial(self.buf.data_ptr(), self.count)
        return self.buf


class ShardGroup:
    """nshards column shards in one process, on one device."""

    def __init__(self, n, d, K, p, loss, lambda_w, lambda_v, eta, seed, nshards, device="cuda:0"):
        self.shards = [_Shard(n, d, K, p, loss, lambda_w, lambda_v, eta, seed, s, nshards, device) for s in range(nshards)]
        self.n, self.d, self.K = int(n), int(d), int(K)
        self.objective = float("nan")

    def close(self):
        for s in self.shards:
            s.h.close()

    def __enter__(self):
        return self

    def __exit__(self, *exc):
        self.close()

    def _exchange(self) -> float:
        import torch

        total = torch.zeros_like(self.shards[0].buf)
        for s in self.shards:                      # fixed order: the same bits on every run
            total += s.partial()
        torch.cuda.synchronize()
        sums = [s.h.shard_epoch_end(total.data_ptr(), s.count) for s in self.shards]
        lw, lv = self.shards[0].lambda_w, self.shards[0].lambda_v
        self.objective = sums[0][0] / self.n + 0.5 * lw * sum(x[2] for x in sums) + 0.5 * lv * sum(x[3] for x in sums)
        return self.objective

    def load_csr(self, indptr, indices, values, y) -> float:
        for s in self.shards:
            s.h.load_csr(indptr, indices, values, y)
        return self._exchange()

    def epoch(self) -> float:
        for s in self.shards:
            s.h.shard_epoch_begin()
        return self._exchange()

    def get_params(self):
        """w0, w, V assembled from the columns each shard owns."""
        w = np.empty(self.d, np.float32)
        V = np.empty((self.d, self.K), np.float32)
        w0 = 0.0
        for s in self.shards:
            lo, hi = s.h.shard_columns()
            w0, ws, Vs = s.h.get_params()
            w[lo:hi], V[lo:hi] = ws[lo:hi], Vs[lo:hi]
        return w0, w, V

    def get_aux(self):
        return self.shards[0].h.get_aux()


class DistributedShard:
    """This rank's shard of a torch.distributed group (one rank per GPU)."""

    def __init__(self, n, d, K, p, loss, lambda_w, lambda_v, eta, seed, device):
        import torch.distributed as dist

        self.rank, self.world = dist.get_rank(), dist.get_world_size()
        self.s = _Shard(n, d, K, p, loss, lambda_w, lambda_v, eta, seed, self.rank, self.world, device)
        self.objective = float("nan")

    def close(self):
        self.s.h.close()

    def _exchange(self) -> float:
        import torch
        import torch.distributed as dist

        buf = self.s.partial()
        dist.all_reduce(buf)                       # sum of the shards' [A | lin | q]
        sums = self.s.h.shard_epoch_end(buf.data_ptr(), self.s.count)
        norms = torch.tensor(sums[2:], dtype=torch.float64, device=buf.device)
        dist.all_reduce(norms)
        w2, v2 = (float(x) for x in norms.tolist())
        self.objective = sums[0] / self.s.n + 0.5 * self.s.lambda_w * w2 + 0.5 * self.s.lambda_v * v2
        return self.objective

    def load_csr(self, indptr, indices, values, y) -> float:
        self.s.h.load_csr(indptr, indices, values, y)
        return self._exchange()

    def epoch(self) -> float:
        self.s.h.shard_epoch_begin()
        return self._exchange()
