"""Device-memory plumbing around the C calls: allocates the tables, the
workspace and the per-step outputs as torch tensors and issues the calls of one
step in order.  No arithmetic of the method happens here.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import Dict, Optional

import numpy as np
import torch

from . import binding as gb
from .workloads import BF16, Batch, GearPreset


@dataclass
class DeviceBatch:
    user_id: torch.Tensor
    url_id: torch.Tensor
    img_off: torch.Tensor
    img_id: torch.Tensor
    label: torch.Tensor
    B: int
    nnz: int
    fast: Optional[torch.Tensor] = None       # [B][fast_dim] fp32: the views' own dense input

    @staticmethod
    def from_host(b: Batch, device="cuda") -> "DeviceBatch":
        f = lambda a: torch.from_numpy(np.ascontiguousarray(a)).to(device)
        return DeviceBatch(f(b.user_id), f(b.url_id), f(b.img_off), f(b.img_id), f(b.label), b.B, b.nnz,
                           None if b.fast is None else f(b.fast))


class GearSession:
    """Tables + ctx + output buffers for one configuration on one GPU."""

    GUARD_I = -7
    GUARD_F = 12345.0

    def __init__(self, p: GearPreset, head_params: np.ndarray, max_batch: Optional[int] = None,
                 max_nnz: Optional[int] = None, seed: int = 0, fill: bool = True, now: int = 0,
                 tables: Optional[Dict[str, np.ndarray]] = None, ready_cap: int = 0, device: str = "cuda",
                 want_emb_grad: bool = False, want_debug: bool = False, expired_cap: Optional[int] = None,
                 accum_mode: int = gb.GEAR_ACC_SORT, adam: Optional["gb.gear_adam"] = None):
        gb.load()
        self.p = p
        self.dev = torch.device(device)
        self.max_batch = int(max_batch or p.batch)
        self.max_nnz = int(max_nnz or self.max_batch * p.img_hi)
        self.d_in = p.d_in
        dfv_t = torch.bfloat16 if p.dfv_dtype == BF16 else torch.float32
        self.cfg = gb.make_config(p.user_vocab, p.url_vocab, p.img_vocab, p.emb_dim, p.dfv_dim,
                                  gb.GEAR_BF16 if p.dfv_dtype == BF16 else gb.GEAR_F32,
                                  gb.GEAR_BF16 if p.head_dtype == BF16 else gb.GEAR_F32,
                                  list(p.hidden), p.M, p.expire, self.max_batch, self.max_nnz, ready_cap, accum_mode,
                                  fast_dim=p.fast_dim)
        dev = self.dev
        if tables is None:
            self.user_emb = torch.empty((p.user_vocab, p.emb_dim), dtype=torch.float32, device=dev)
            self.url_emb = torch.empty((p.url_vocab, p.emb_dim), dtype=torch.float32, device=dev)
            self.dfv = torch.empty((p.img_vocab, p.dfv_dim), dtype=dfv_t, device=dev)
            self.dfv_ts = torch.zeros(p.img_vocab, dtype=torch.int64, device=dev)
        else:
            fill = False
            self.user_emb = torch.from_numpy(tables["user_emb"]).to(dev)
            self.url_emb = torch.from_numpy(tables["url_emb"]).to(dev)
            dfv = tables["dfv"]
            if dfv.dtype == np.uint16:
                self.dfv = torch.from_numpy(dfv.view(np.int16)).to(dev).view(torch.bfloat16)
            else:
                self.dfv = torch.from_numpy(dfv).to(dev)
            assert self.dfv.dtype == dfv_t
            self.dfv_ts = torch.from_numpy(tables["ts"]).to(dev)
        self.dfv_gsum = torch.zeros((p.img_vocab, p.dfv_dim), dtype=torch.float32, device=dev)
        self.dfv_gcnt = torch.zeros(p.img_vocab, dtype=torch.int32, device=dev)
        self.head_params = torch.from_numpy(np.ascontiguousarray(head_params, dtype=np.float32)).to(dev)
        assert self.head_params.numel() == p.n_params
        self.workspace = torch.empty(gb.gear_workspace_bytes(self.cfg), dtype=torch.uint8, device=dev)
        self.ctx = gb.gear_init_tables(self.cfg, self.user_emb, self.url_emb, self.dfv, self.dfv_gsum, self.dfv_gcnt,
                                       self.dfv_ts, self.head_params, self.workspace, seed=seed, fill=fill, now=now)
        B, nnz = self.max_batch, self.max_nnz
        # loss and the two counts share one small buffer, so that a caller can read them back with a single copy
        self.scalars = torch.zeros(3, dtype=torch.int64, device=dev)
        self.loss = self.scalars[0:1].view(torch.float32)[0:1]
        self.prob = torch.zeros(B, dtype=torch.float32, device=dev)
        self.head_grad = torch.zeros(p.n_params, dtype=torch.float32, device=dev)
        self.dX = torch.zeros((B, self.d_in), dtype=torch.float32, device=dev)
        self.row_view = torch.zeros(nnz, dtype=torch.int32, device=dev)
        self.inv_n = torch.zeros(B, dtype=torch.float32, device=dev)
        self.x_debug = (torch.zeros((B, self.d_in), dtype=torch.bfloat16 if p.head_dtype == BF16 else torch.float32,
                                    device=dev) if want_debug else None)
        # event 5's rows in materialised form (what a worker would send to the owners of the images); with want_debug
        self.dfv_grad = torch.zeros((nnz, p.dfv_dim), dtype=torch.float32, device=dev) if want_debug else None
        self.user_grad = torch.zeros_like(self.user_emb) if want_emb_grad else None
        self.url_grad = torch.zeros_like(self.url_emb) if want_emb_grad else None
        # Section 4's optimiser for the embedding tables: first and second moments per table row
        self.adam = adam
        self.adam_step = 0
        self.user_m = torch.zeros_like(self.user_emb) if adam is not None else None
        self.user_v = torch.zeros_like(self.user_emb) if adam is not None else None
        self.url_m = torch.zeros_like(self.url_emb) if adam is not None else None
        self.url_v = torch.zeros_like(self.url_emb) if adam is not None else None
        # every output list is followed by one guard entry the library must never write (guards_intact checks them)
        self.ready_cap = int(ready_cap or nnz)
        self._ready_ids_g = torch.full((self.ready_cap + 1,), self.GUARD_I, dtype=torch.int32, device=dev)
        self._ready_seq_g = torch.full((self.ready_cap + 1,), self.GUARD_I, dtype=torch.int32, device=dev)
        self._ready_avg_g = torch.zeros((self.ready_cap + 1, p.dfv_dim), dtype=torch.float32, device=dev)
        self._ready_avg_g[self.ready_cap].fill_(self.GUARD_F)
        self.ready_ids, self.ready_seq = self._ready_ids_g[:self.ready_cap], self._ready_seq_g[:self.ready_cap]
        self.ready_avg = self._ready_avg_g[:self.ready_cap]
        self.expired_cap = int(expired_cap if expired_cap is not None else p.img_vocab)
        self._expired_ids_g = torch.full((self.expired_cap + 1,), self.GUARD_I, dtype=torch.int32, device=dev)
        self.expired_ids = self._expired_ids_g[:self.expired_cap]
        self.d_counts = self.scalars[1:3]
        self._expiry_stream = None
        self._step_out = None

    # ---- the four calls of a step ---------------------------------------------------------------
    def forward_backward(self, b: DeviceBatch, lr: Optional[float] = None):
        # the output struct never changes and a batch's struct only in its counts: both are made once
        if self._step_out is None:
            self._step_out = gb.make_step_out(self.loss, self.head_grad, self.dX, prob=self.prob, row_view=self.row_view,
                                              inv_n=self.inv_n, x_debug=self.x_debug, user_grad=self.user_grad,
                                              url_grad=self.url_grad, dfv_grad=self.dfv_grad, adam=self.adam, user_m=self.user_m,
                                              user_v=self.user_v, url_m=self.url_m, url_v=self.url_v)
        if self.adam is not None:
            self.adam_step += 1
            self._step_out.adam_step = self.adam_step
        bt = b.__dict__.get("_c_batch")
        if bt is None:
            bt = b.__dict__["_c_batch"] = gb.make_batch(b.user_id, b.url_id, b.img_off, b.img_id, b.label, fast=b.fast)
        bt.B, bt.nnz = b.B, b.nnz
        return gb.gear_forward_backward_structs(self.ctx, bt, self.p.lr if lr is None else lr, self._step_out)

    def accumulate_from_step(self, b: DeviceBatch, reuse_sorted_ids: bool = True):
        """Event 5 in its indirect form: row r of the batch is dX[row_view[r], 2E:] * inv_n[row_view[r]].
        With reuse_sorted_ids the image IDs sorted during forward_backward are used (img_id = NULL)."""
        if b.nnz == 0:
            return 0
        ptr = self.dX.data_ptr() + 4 * 2 * self.p.emb_dim
        return gb.gear_accumulate_dfv_grad(self.ctx, None if reuse_sorted_ids else b.img_id, ptr, self.d_in,
                                           self.row_view, self.inv_n, b.nnz)

    def accumulate_rows(self, img_id: torch.Tensor, grads: torch.Tensor):
        assert grads.dtype == torch.float32 and grads.shape[1] == self.p.dfv_dim
        return gb.gear_accumulate_dfv_grad(self.ctx, img_id, grads.data_ptr(), grads.stride(0), None, None,
                                           int(img_id.shape[0]))

    def accumulate_collect_from_step(self, b: DeviceBatch, sync: bool = True, reuse_sorted_ids: bool = True):
        """Events 5 and 6 of a step as one call: the batch's gradient rows (indirect form, as in
        accumulate_from_step) are added and the averages of the completed groups handed over."""
        ptr = self.dX.data_ptr() + 4 * 2 * self.p.emb_dim
        return gb.gear_accumulate_collect(self.ctx, None if (reuse_sorted_ids and b.nnz > 0) else b.img_id, ptr, self.d_in,
                                          self.row_view, self.inv_n, b.nnz, self.ready_ids, self.ready_seq,
                                          self.ready_avg, self.ready_cap, d_n=self.d_counts[0:1], sync=sync)

    def accumulate_collect_rows(self, img_id: torch.Tensor, grads: torch.Tensor, sync: bool = True):
        assert grads.dtype == torch.float32 and grads.shape[1] == self.p.dfv_dim
        return gb.gear_accumulate_collect(self.ctx, img_id, grads.data_ptr(), grads.stride(0) if grads.shape[0] else
                                          self.p.dfv_dim, None, None, int(img_id.shape[0]), self.ready_ids, self.ready_seq,
                                          self.ready_avg, self.ready_cap, d_n=self.d_counts[0:1], sync=sync)

    def collect_ready(self, sync: bool = True):
        return gb.gear_collect_ready(self.ctx, self.ready_ids, self.ready_seq, self.ready_avg, self.ready_cap,
                                     d_n=self.d_counts[0:1], sync=sync)

    def collect_expired(self, now: int, restamp: bool = True, sync: bool = True):
        return gb.gear_collect_expired(self.ctx, now, restamp, self.expired_ids, self.expired_cap,
                                       d_n=self.d_counts[1:2], sync=sync)

    def refresh_dfv(self, ids: torch.Tensor, rows: torch.Tensor, now: int, n: Optional[int] = None, d_n=None):
        """Recomputed DFVs replace cached ones (rows fp32) and restart their clocks."""
        return gb.gear_refresh_dfv(self.ctx, ids, rows, int(ids.shape[0]) if n is None else n, now, d_n=d_n)

    # ---- a linear Dense Part on the same device ---------------------------------------------------
    def dense_forward(self, raw: torch.Tensor, Wd: torch.Tensor, ids: torch.Tensor, rows: torch.Tensor, n=None, d_n=None):
        return gb.gear_dense_forward(self.ctx, raw, Wd, ids, int(ids.shape[0]) if n is None else n, rows, d_n=d_n)

    def dense_backward(self, raw: torch.Tensor, n: int, Wd_grad: torch.Tensor, d_n=None):
        """Back-propagation of the averages just handed over (ready_ids, ready_avg) through the Dense Part."""
        return gb.gear_dense_backward(self.ctx, raw, self.ready_ids, self.ready_avg, n, Wd_grad, d_n=d_n)

    def step(self, b: DeviceBatch, now: int, sync: bool = False, expiry_beside: Optional[bool] = None):
        """One pass of the whole hot path over one batch.  The expiry scan depends on nothing the training calls
        produce: with expiry_beside it goes to a stream of its own, starts when the step starts and is joined
        at the step's end, so that it runs beside the gather and the head.  Default: beside for tables of 4M images
        or more (the fork and join cost the host more than a scan of a small table takes on the device)."""
        if expiry_beside is None:
            expiry_beside = self.p.img_vocab >= (1 << 22)
        if not expiry_beside:
            self.forward_backward(b)
            n_ready = self.accumulate_collect_from_step(b, sync=sync)
            n_exp = self.collect_expired(now, restamp=True, sync=sync)
            return n_ready, n_exp
        main = torch.cuda.current_stream()
        if self._expiry_stream is None:
            self._expiry_stream = torch.cuda.Stream()
            self._ev_fork, self._ev_join = torch.cuda.Event(), torch.cuda.Event()
        self._ev_fork.record(main)
        self._expiry_stream.wait_event(self._ev_fork)      # earlier readers of expired_ids and the count are done
        with torch.cuda.stream(self._expiry_stream):
            n_exp = self.collect_expired(now, restamp=True, sync=sync)
            self._ev_join.record(self._expiry_stream)
        self.forward_backward(b)
        n_ready = self.accumulate_collect_from_step(b, sync=sync)
        main.wait_event(self._ev_join)
        return n_ready, n_exp

    def status(self):
        return gb.gear_status(self.ctx)

    def guards_intact(self) -> bool:
        """The entry after the end of each output list still holds the value it was created with."""
        return bool(int(self._ready_ids_g[-1]) == self.GUARD_I and int(self._ready_seq_g[-1]) == self.GUARD_I and
                    int(self._expired_ids_g[-1]) == self.GUARD_I and
                    bool((self._ready_avg_g[-1] == self.GUARD_F).all()))

    def close(self):
        if self.ctx is not None:
            gb.gear_destroy(self.ctx)
            self.ctx = None
