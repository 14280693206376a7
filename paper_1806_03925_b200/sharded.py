"""The step with the tables partitioned by ID across devices (host-side plumbing).

Paper, Section 3: the Slowgear Workers serve the Fastgear Workers' requests "by partition of Image ID"; Section 4
runs N Fastgear and N Slowgear workers.  Here every rank plays both roles on its GPU:

  owner   (Slowgear role) holds the rows of every table whose ID is congruent to its rank modulo the number of ranks
          (ID i lives at row i // world of rank i % world): embeddings, cached DFVs, the gradient store, the timestamps.
          It answers row requests (gear_fetch_rows), applies the embedding gradients that arrive
          (gear_apply_emb_grad), feeds the arriving (Image ID, gradient) pairs to its store
          (gear_accumulate_collect) and scans its own timestamps (gear_collect_expired).
  worker  (Fastgear role) takes its share of the page views, asks the owners for the rows it needs, runs the head
          forward and backward on them (gear_forward_backward over the received rows, addressed 0, 1, 2, ...), and
          sends every gradient row back to the owner of its ID: one embedding-gradient row per view and table
          (columns of dX) and one DFV-gradient row per image occurrence (gear_step_out.dfv_grad, event 5).

Three all-to-all(v) exchanges per table and step: IDs out, rows back, gradient rows out.  Rows land in the
receiver's own memory before any kernel reads them.  At an owner, rows arrive sender by sender, each sender's rows
in its own row order: that is the arrival order of the store (the paper's workers push asynchronously, so any order
is a valid one; this one is reproducible).  The workers do not rescale their gradients by the number of ranks: as
in the paper, every worker's batch is a batch of its own.

Nothing here computes anything of the method: routing by ID (remainder, quotient, a stable partition by owner),
copies and collectives.  `Exchange` has two forms with the same interface: `DistExchange` runs one rank per process
over torch.distributed (NCCL on GPUs, gloo on CPU tensors); `LoopbackExchange` holds all ranks in one process and
moves the pieces by indexing, so that the whole sharded step can be run and checked on a single GPU, rank after rank,
with no kernel of one rank waiting on another's.
"""
from __future__ import annotations

from dataclasses import dataclass, replace
from typing import List, Optional, Sequence

import numpy as np
import torch

from . import binding as gb
from .session import DeviceBatch, GearSession
from .workloads import BF16, Batch, GearPreset


@dataclass
class Route:
    """How one rank's ID list travels: order sorts its entries by owner (stable); send_counts[o] of them go to rank
    o; recv_counts[s] entries arrive from rank s, their owner-local row numbers in recv_local (sender by sender)."""
    order: torch.Tensor
    send_counts: List[int]
    recv_counts: List[int]
    recv_local: torch.Tensor


def partition_by_owner(ids: torch.Tensor, world: int):
    """(order, send_counts, local): stable partition of the entries by owner = id mod world; local = id div world
    (floor: a negative ID stays negative and is refused by its owner)."""
    ids64 = ids.to(torch.int64)
    owner = torch.remainder(ids64, world)
    local = torch.div(ids64, world, rounding_mode="floor").to(torch.int32)
    order = torch.sort(owner, stable=True).indices
    counts = torch.bincount(owner, minlength=world)
    return order, [int(c) for c in counts.tolist()], local


class LoopbackExchange:
    """All ranks in this process: lists passed in and returned hold one entry per rank."""

    def __init__(self, world: int):
        self.world = world
        self.local_ranks = list(range(world))

    def route(self, ids_per_rank: Sequence[torch.Tensor]) -> List[Route]:
        W = self.world
        parts = [partition_by_owner(ids, W) for ids in ids_per_rank]
        routes = []
        for o in range(W):
            pieces, recv_counts = [], []
            for s in range(W):
                order, counts, local = parts[s]
                lo = sum(counts[:o])
                pieces.append(local[order[lo:lo + counts[o]]])
                recv_counts.append(counts[o])
            routes.append(Route(parts[o][0], parts[o][1], recv_counts, torch.cat(pieces)))
        return routes

    def reply(self, routes: Sequence[Route], rows_at_owner: Sequence[torch.Tensor]) -> List[torch.Tensor]:
        """rows_at_owner[o] is aligned with routes[o].recv_local; returns, per rank, the rows of its own request in
        the order of its ID list."""
        W = self.world
        out = []
        for s in range(W):
            pieces = []
            for o in range(W):
                lo = sum(routes[o].recv_counts[:s])
                pieces.append(rows_at_owner[o][lo:lo + routes[o].recv_counts[s]])
            got = torch.cat(pieces)
            rows = torch.empty_like(got)
            rows[routes[s].order] = got
            out.append(rows)
        return out

    def push(self, routes: Sequence[Route], rows_per_rank: Sequence[torch.Tensor]) -> List[torch.Tensor]:
        """rows_per_rank[s] is aligned with rank s's ID list; returns, per owner, the rows aligned with its recv_local."""
        W = self.world
        sorted_rows = [rows[routes[s].order] for s, rows in enumerate(rows_per_rank)]
        out = []
        for o in range(W):
            pieces = []
            for s in range(W):
                lo = sum(routes[s].send_counts[:o])
                pieces.append(sorted_rows[s][lo:lo + routes[s].send_counts[o]])
            out.append(torch.cat(pieces))
        return out

    def mean_over_ranks(self, tensors: Sequence[torch.Tensor]) -> None:
        """In place: every rank's tensor becomes the mean over the ranks (the small head's gradient)."""
        # stands in for the reduction that the collective performs between real ranks (NCCL's AVG)
        reduced = torch.stack(list(tensors)).mean(0)
        for t in tensors:
            t.copy_(reduced)


class DistExchange:
    """One rank per process over torch.distributed; the lists hold this rank's single entry."""

    def __init__(self, rank: int, world: int, group=None):
        self.rank, self.world, self.group = rank, world, group
        self.local_ranks = [rank]

    def _all_to_all(self, send: torch.Tensor, send_counts: List[int], recv_counts: List[int]) -> torch.Tensor:
        recv = torch.empty((sum(recv_counts),) + tuple(send.shape[1:]), dtype=send.dtype, device=send.device)
        if self.world == 1:
            recv.copy_(send)
            return recv
        import torch.distributed as dist
        dist.all_to_all_single(recv, send.contiguous(), output_split_sizes=recv_counts, input_split_sizes=send_counts,
                               group=self.group)
        return recv

    def route(self, ids_per_rank: Sequence[torch.Tensor]) -> List[Route]:
        (ids,) = ids_per_rank
        order, send_counts, local = partition_by_owner(ids, self.world)
        if self.world == 1:
            recv_counts = list(send_counts)
        else:
            import torch.distributed as dist
            sc = torch.tensor(send_counts, dtype=torch.int64, device=ids.device)
            rc = torch.empty_like(sc)
            dist.all_to_all_single(rc, sc, group=self.group)
            recv_counts = [int(c) for c in rc.tolist()]
        recv_local = self._all_to_all(local[order], send_counts, recv_counts)
        return [Route(order, send_counts, recv_counts, recv_local)]

    def reply(self, routes: Sequence[Route], rows_at_owner: Sequence[torch.Tensor]) -> List[torch.Tensor]:
        (r,), (rows,) = routes, rows_at_owner
        got = self._all_to_all(rows, r.recv_counts, r.send_counts)
        out = torch.empty_like(got)
        out[r.order] = got
        return [out]

    def push(self, routes: Sequence[Route], rows_per_rank: Sequence[torch.Tensor]) -> List[torch.Tensor]:
        (r,), (rows,) = routes, rows_per_rank
        return [self._all_to_all(rows[r.order], r.send_counts, r.recv_counts)]

    def mean_over_ranks(self, tensors: Sequence[torch.Tensor]) -> None:
        if self.world == 1:
            return
        import torch.distributed as dist
        (t,) = tensors
        if t.is_cuda:
            dist.all_reduce(t, op=dist.ReduceOp.AVG, group=self.group)       # the reduction runs inside the collective
        else:
            raise NotImplementedError("the mean over ranks is taken by the NCCL collective; CPU tensors have no such path")


def shard_rows(vocab: int, rank: int, world: int) -> int:
    """Rows of a table of `vocab` IDs that live on `rank`."""
    return (vocab - rank + world - 1) // world


class ShardedGear:
    """Owner and worker sessions of the local ranks (one under DistExchange, all under LoopbackExchange)."""

    def __init__(self, p: GearPreset, head_params: np.ndarray, ex, max_batch_local: int, max_nnz_local: int,
                 tables: Optional[dict] = None, seed: int = 0, now: int = 0, device: str = "cuda"):
        """tables (optional): the WHOLE tables as host arrays (user_emb, url_emb, dfv, ts), of which every owner takes
        its rows (rank, rank + world, ...); without them every shard gets its own procedural fill."""
        self.p, self.ex, self.world = p, ex, ex.world
        W = self.world
        self.owners: List[GearSession] = []
        self.workers: List[GearSession] = []
        for r in ex.local_ranks:
            sp = replace(p, user_vocab=shard_rows(p.user_vocab, r, W), url_vocab=shard_rows(p.url_vocab, r, W),
                         img_vocab=shard_rows(p.img_vocab, r, W))
            mine = None
            if tables is not None:
                mine = {k: np.ascontiguousarray(v[r::W]) for k, v in tables.items()}
            self.owners.append(GearSession(sp, head_params, max_batch=max_batch_local * W, max_nnz=max_nnz_local * W,
                                           seed=seed + r, fill=True, now=now, tables=mine, device=device))
            wp = replace(p, user_vocab=max_batch_local, url_vocab=max_batch_local, img_vocab=max_nnz_local)
            dfv_np = np.uint16 if p.dfv_dtype == BF16 else np.float32
            blank = dict(user_emb=np.zeros((max_batch_local, p.emb_dim), np.float32),
                         url_emb=np.zeros((max_batch_local, p.emb_dim), np.float32),
                         dfv=np.zeros((max_nnz_local, p.dfv_dim), dfv_np), ts=np.zeros(max_nnz_local, np.int64))
            wk = GearSession(wp, head_params, max_batch=max_batch_local, max_nnz=max_nnz_local, tables=blank,
                             expired_cap=1, ready_cap=1, device=device)
            wk.dfv_grad = torch.zeros((max_nnz_local, p.dfv_dim), dtype=torch.float32, device=device)
            wk._step_out = None
            self.workers.append(wk)
        self._iota = torch.arange(max(max_batch_local, max_nnz_local), dtype=torch.int32, device=device)

    def step(self, batches: Sequence[Batch], now: int, lr: Optional[float] = None, mean_head_grad: bool = True):
        """One step of every local rank.  batches[i]: the page views of local rank i (host arrays).  Returns per local
        rank (averages handed over by its owner, IDs its owner's scan listed)."""
        p, ex = self.p, self.ex
        lr = p.lr if lr is None else lr
        E = p.emb_dim
        dev = self.workers[0].dev
        ids = {k: [torch.from_numpy(np.ascontiguousarray(getattr(b, k))).to(dev) for b in batches]
               for k in ("user_id", "url_id", "img_id")}
        # events 1-3: IDs to the owners, rows back into the workers' row buffers
        routes = {k: ex.route(ids[k]) for k in ids}
        for k, which, buf in (("user_id", gb.GEAR_TABLE_USER, "user_emb"), ("url_id", gb.GEAR_TABLE_URL, "url_emb"),
                              ("img_id", gb.GEAR_TABLE_DFV, "dfv")):
            rows = []
            for ow, rt in zip(self.owners, routes[k]):
                n = int(rt.recv_local.shape[0])
                out = torch.empty((n,) + tuple(getattr(ow, buf).shape[1:]), dtype=getattr(ow, buf).dtype, device=dev)
                gb.gear_fetch_rows(ow.ctx, which, rt.recv_local, n, out)
                rows.append(out)
            for wk, got in zip(self.workers, ex.reply(routes[k], rows)):
                getattr(wk, buf)[:got.shape[0]].copy_(got)
        # event 4 on the workers: the received rows are rows 0, 1, 2, ... of the worker's tables
        for wk, b in zip(self.workers, batches):
            db = DeviceBatch(self._iota[:b.B], self._iota[:b.B], torch.from_numpy(b.img_off).to(dev), self._iota[:b.nnz],
                             torch.from_numpy(b.label).to(dev), b.B, b.nnz)
            wk.forward_backward(db, lr=0.0)          # the worker's copies of the rows are scratch: nothing to update
        if mean_head_grad:
            ex.mean_over_ranks([wk.head_grad for wk in self.workers])
        # events 4 (push) and 5: gradient rows to the owners of their IDs
        g_user = ex.push(routes["user_id"], [wk.dX[:b.B, :E].contiguous() for wk, b in zip(self.workers, batches)])
        g_url = ex.push(routes["url_id"], [wk.dX[:b.B, E:2 * E].contiguous() for wk, b in zip(self.workers, batches)])
        g_img = ex.push(routes["img_id"], [wk.dfv_grad[:b.nnz] for wk, b in zip(self.workers, batches)])
        out = []
        for i, ow in enumerate(self.owners):
            ru, rh, ri = routes["user_id"][i], routes["url_id"][i], routes["img_id"][i]
            gb.gear_apply_emb_grad(ow.ctx, gb.GEAR_TABLE_USER, ru.recv_local, g_user[i], int(ru.recv_local.shape[0]), lr)
            gb.gear_apply_emb_grad(ow.ctx, gb.GEAR_TABLE_URL, rh.recv_local, g_url[i], int(rh.recv_local.shape[0]), lr)
            # event 6 at the owner, then its own expiry scan
            n_ready = ow.accumulate_collect_rows(ri.recv_local, g_img[i]) if ri.recv_local.shape[0] else ow.collect_ready()
            n_exp = ow.collect_expired(now, restamp=True)
            out.append((n_ready, n_exp))
        return out

    def close(self):
        for s in self.owners + self.workers:
            s.close()
