"""Runs the CUDA library and the CPU oracle side by side on the same seeded inputs.

The oracle never sees anything the GPU produced: both sides get the batches from
the workload generators and the tables either from host-built arrays or, for the
procedural fill, each from its own implementation of the generator.

For vocabularies too large for dense host tables the oracle works on a compact
problem: only the rows the batches touch are generated (row by row, from the
procedural definition) and the IDs are renumbered; GPU results are read back at
those rows.  The timestamp table is always kept in full.
"""
from __future__ import annotations

from typing import Dict, List, Optional

import numpy as np
import torch

import oracle
from oracle import GearOracle
from paper_1806_03925_b200 import workloads
from paper_1806_03925_b200.session import DeviceBatch, GearSession
from paper_1806_03925_b200.workloads import BF16, Batch, GearPreset

TOL_F32 = 1e-5      # relative tolerance for fp32 configurations (normwise: against the largest reference entry)
TOL_BF16 = 1e-2     # for configurations whose DFVs / head operands are bfloat16

# How close to zero a hidden pre-activation a = sum_i in_i * w_ij + b_j has to be for the device's ReLU branch to be
# allowed to differ from the oracle's, relative to max|in| * max|w| of the unit's layer:
#   * both sides add the same K products, the device in fp32 in its own order, the oracle in fp64: the sums differ by
#     about sqrt(K) * 2^-24 * (rms term) * sqrt(K) <= K * 2^-24 * max|in| * max|w|; eight times that is allowed;
#   * bf16 heads: the operand in_i is itself a rounded fp32 value (pooled mean, or the layer below's activation); where
#     the two sides' values straddle a rounding boundary the operands differ by one bf16 unit in the last place, at
#     most 2^-7 |in_i|, which moves a by at most 2^-7 * max|in| * max|w|.
# A unit outside this band must take the oracle's branch.
def relu_margin_rel(p: GearPreset) -> float:
    k_max = max((p.d_in,) + tuple(p.hidden))
    accum = 8.0 * k_max * 2.0 ** -24
    return accum + (2.0 ** -7 if p.head_dtype == BF16 else 0.0)


MAX_FLIPS_PER_VIEW = 3      # branches of one view that may differ from the oracle's (each inside the band above)


def max_views_with_flips(B: int, listed: int = 0) -> int:
    """Views of a batch whose ReLU branches may validly differ from the oracle's before a test calls it a failure:
    a few per 512 views, and one more per 2048 units the oracle lists inside the rounding band (only those can differ;
    a wide layer lists many more units per view than a narrow one)."""
    return 2 + B // 512 + listed // 2048


def tol_of(p: GearPreset) -> float:
    return TOL_BF16 if (p.head_dtype == BF16 or p.dfv_dtype == BF16) else TOL_F32


def assert_close(got, want, tol, what=""):
    got = np.asarray(got, dtype=np.float64)
    want = np.asarray(want, dtype=np.float64)
    assert got.shape == want.shape, (what, got.shape, want.shape)
    if want.size == 0:
        return
    scale = max(np.abs(want).max(), 1e-30)
    err = np.abs(got - want).max()
    assert err <= tol * scale, "%s: max abs error %.3e > %.1e * %.3e" % (what, err, tol, scale)


def count_nonzero(t: torch.Tensor) -> int:
    """Non-zero entries of a (possibly very large) tensor, counted in pieces so that no table-sized temporary is made."""
    flat = t.reshape(-1)
    step, total = 1 << 28, 0
    for i in range(0, flat.numel(), step):
        total += int(torch.count_nonzero(flat[i:i + step]).item())
    return total


def _rows(t: torch.Tensor, rows: np.ndarray) -> np.ndarray:
    return _np(t[torch.from_numpy(rows).to(t.device)])


def _np(t: torch.Tensor) -> np.ndarray:
    if t.dtype == torch.bfloat16:
        return t.float().cpu().numpy()
    return t.cpu().numpy()


class Remap:
    """Renumbering of the IDs that occur (sorted) to 0..n-1; out-of-range IDs map to -1."""

    def __init__(self, ids: np.ndarray, vocab: int, dense: bool):
        self.vocab = vocab
        if dense:
            self.rows = np.arange(vocab, dtype=np.int64)
        else:
            ok = ids[(ids >= 0) & (ids < vocab)]
            self.rows = np.unique(ok).astype(np.int64)
        self.dense = dense

    def __call__(self, ids: np.ndarray) -> np.ndarray:
        ids = np.asarray(ids)
        ok = (ids >= 0) & (ids < self.vocab)
        out = np.full(ids.shape, -1, dtype=np.int32)
        if self.dense:
            out[ok] = ids[ok]
        else:
            out[ok] = np.searchsorted(self.rows, ids[ok]).astype(np.int32)
        return out

    @property
    def n(self) -> int:
        return len(self.rows)


class Pair:
    """A GearSession on the GPU and a GearOracle on the CPU over the same problem."""

    def __init__(self, p: GearPreset, batches: List[Batch], seed: int = 0, dense: Optional[bool] = None,
                 now0: int = 0, ready_cap: int = 0, want_emb_grad: bool = False, extra_img_ids=None,
                 atomic: bool = False, fused: bool = False):
        # atomic: GEAR_ACC_ATOMIC on the device against the oracle's order-free (pooled) store
        # fused: a step's events 5 and 6 go through gear_accumulate_collect instead of the two separate calls
        self.p, self.seed, self.atomic, self.fused = p, seed, atomic, fused
        if dense is None:
            dense = max(p.user_vocab, p.url_vocab, p.img_vocab) <= 200_000
        cat = lambda k: np.concatenate([getattr(b, k) for b in batches]) if batches else np.zeros(0, np.int32)
        img_all = cat("img_id")
        if extra_img_ids is not None:
            img_all = np.concatenate([img_all, extra_img_ids])
        self.ru = Remap(cat("user_id"), p.user_vocab, dense)
        self.rh = Remap(cat("url_id"), p.url_vocab, dense)
        self.ri = Remap(img_all, p.img_vocab, dense)
        self.params = workloads.head_params(p, seed)
        max_b = max([b.B for b in batches] + [1])
        max_nnz = max([b.nnz for b in batches] + [1])
        if extra_img_ids is not None:
            max_nnz = max(max_nnz, len(extra_img_ids))
        self.gpu = GearSession(p, self.params, max_batch=max_b, max_nnz=max_nnz, seed=seed, fill=True, now=now0,
                               ready_cap=ready_cap, want_emb_grad=want_emb_grad, want_debug=True,
                               accum_mode=1 if atomic else 0)
        dfv_np = np.uint16 if p.dfv_dtype == BF16 else np.float32
        self.cpu = GearOracle(
            oracle.fill_rows(seed, oracle.TAG_USER, p.emb_dim, self.ru.rows, self.ru.n, np.float32),
            oracle.fill_rows(seed, oracle.TAG_URL, p.emb_dim, self.rh.rows, self.rh.n, np.float32),
            oracle.fill_rows(seed, oracle.TAG_DFV, p.dfv_dim, self.ri.rows, self.ri.n, dfv_np),
            p.hidden, p.M, p.expire, round_bf16=(p.head_dtype == BF16),
            ts=oracle.fill_ts(seed, p.expire, now0, None, p.img_vocab), fast_dim=p.fast_dim)
        self.tol = tol_of(p)
        self.want_emb_grad = want_emb_grad
        self.updated_user = np.zeros(0, np.int32)
        self.updated_url = np.zeros(0, np.int32)
        self.relu_flips_accepted = 0
        self.relu_views_flipped = 0
        self.last_relu = dict(views=0, units=0, listed=0)
        self.status_bits = 0       # device status bits seen so far (reading the word clears it)
        self.status_rc = 0

    def status(self):
        rc, bits, pending = self.gpu.status()
        self.status_bits |= bits
        if rc != 0 and self.status_rc == 0:
            self.status_rc = rc
        return pending

    # ---- one full step on both sides, compared call by call ------------------------------------
    def step_and_compare(self, b: Batch, now: int, lr: Optional[float] = None, check_tables: bool = True):
        p, gpu, cpu, tol = self.p, self.gpu, self.cpu, self.tol
        lr = p.lr if lr is None else lr
        E, D = p.emb_dim, p.dfv_dim
        db = DeviceBatch.from_host(b)
        gpu.forward_backward(db, lr)
        uid, hid, img = self.ru(b.user_id), self.rh(b.url_id), self.ri(b.img_id)
        params64 = self.params.astype(np.float64)
        r = cpu.forward_backward(params64, uid, hid, b.img_off, img, b.label, relu_margin=0.0,
                                 relu_margin_rel=relu_margin_rel(p), near_cap=max(65536, 64 * b.B), fast=b.fast)

        B = b.B
        X = _np(gpu.x_debug[:B])
        # gathered rows are copies: bit-exact (after the same bf16 rounding for bf16 heads) for every row
        # of a table that no earlier step has updated (an updated row agrees to rounding only)
        fresh_u = ~np.isin(uid, self.updated_user)
        fresh_h = ~np.isin(hid, self.updated_url)
        assert np.array_equal(X[fresh_u, :E].astype(np.float64), r.X[fresh_u, :E]), "user embedding rows"
        assert np.array_equal(X[fresh_h, E:2 * E].astype(np.float64), r.X[fresh_h, E:2 * E]), "url embedding rows"
        n_b = np.diff(b.img_off)
        single = (n_b == 1)
        assert np.array_equal(X[single, 2 * E:].astype(np.float64), r.X[single, 2 * E:]), "single-image pooled rows"
        if p.fast_dim:      # the view's own dense input is a copy (rounded once for bf16 heads)
            assert np.array_equal(X[:, 2 * E + D:].astype(np.float64), r.X[:, 2 * E + D:]), "fast-side dense input"
        assert_close(X, r.X, tol, "head input")
        assert_close(_np(gpu.prob[:B]), r.prob, tol, "prob")
        assert_close(_np(gpu.loss), [r.loss], tol, "loss")
        r = self.resolve_relu_decisions(r, params64, uid, hid, b.img_off, img, b.label, b.fast)
        assert_close(_np(gpu.head_grad), r.head_grad, tol, "head_grad")
        assert_close(_np(gpu.dX[:B]), r.dX, tol, "dX")
        view_of = np.repeat(np.arange(B, dtype=np.int32), n_b)
        assert np.array_equal(_np(gpu.row_view[:b.nnz]), view_of), "row_view"
        inv = np.where(n_b > 0, 1.0 / np.maximum(n_b, 1), 0.0)
        assert_close(_np(gpu.inv_n[:B]), inv, 1e-7, "inv_n")
        # event 5 in its materialised form: one gradient row per image occurrence
        assert_close(_np(gpu.dfv_grad[:b.nnz]), cpu.dfv_grad_rows(b.img_off, r.dX), tol, "DFV gradient rows")

        # embedding gradients / in-place update
        if self.want_emb_grad:
            gu = cpu.emb_grad("user", uid, r.dX)
            gh = cpu.emb_grad("url", hid, r.dX)
            assert_close(_rows(gpu.user_grad, self.ru.rows), gu, tol, "user_grad")
            assert_close(_rows(gpu.url_grad, self.rh.rows), gh, tol, "url_grad")
            gpu.user_grad.zero_()
            gpu.url_grad.zero_()
        else:
            cpu.emb_apply("user", uid, r.dX, -lr)
            cpu.emb_apply("url", hid, r.dX, -lr)
            if lr != 0.0:
                self.updated_user = np.union1d(self.updated_user, uid)
                self.updated_url = np.union1d(self.updated_url, hid)
            if check_tables:
                assert_close(_rows(gpu.user_emb, self.ru.rows), cpu.user_emb, tol, "user_emb after update")
                assert_close(_rows(gpu.url_emb, self.rh.rows), cpu.url_emb, tol, "url_emb after update")

        # event 5 + 6
        if self.fused:
            n_fused = gpu.accumulate_collect_from_step(db)
        else:
            gpu.accumulate_from_step(db)
        cpu.accumulate(img, cpu.dfv_grad_rows(b.img_off, r.dX), pooled=self.atomic)
        self.compare_store(check_tables)
        n_ready = self.collect_and_compare(n_fused if self.fused else None)
        n_exp = self.expire_and_compare(now)
        assert self.status() == 0
        out = dict(loss=r.loss, n_ready=n_ready, n_expired=n_exp, status=self.status_bits, rc=self.status_rc,
                   bad=r.bad_ids, relu=dict(self.last_relu))
        self.status_bits = self.status_rc = 0
        return out

    def resolve_relu_decisions(self, r, params64, uid, hid, img_off, img, label, fast=None):
        """The backward pass depends on the sign of every hidden pre-activation.  Where the oracle's own
        pre-activation lies inside the rounding band of relu_margin_rel (r.near_units) the device may validly have
        taken the other branch; a unit's branch only affects its own view's row of dX (and, through the sums over
        views, the head gradients).

        Views whose dX row fails the strict comparison are looked at one by one: the candidates are that view's
        listed units alone, smallest |pre-activation| first (the oracle's list, not the device's error, picks them);
        the oracle is re-run on that single view with subsets of at most MAX_FLIPS_PER_VIEW of them on the other
        branch until the row matches.  The expected values are then recomputed BY THE ORACLE over the whole batch
        with the accepted units flipped.  The number of views that needed this is bounded by the caller."""
        import itertools
        from oracle import decode_unit
        B = len(uid)
        got_dx, got_hg = _np(self.gpu.dX[:B]), _np(self.gpu.head_grad)
        scale = max(np.abs(r.dX).max(), 1e-30)
        bad_views = np.nonzero(np.abs(got_dx - r.dX).max(1) > self.tol * scale)[0]
        self.last_relu = dict(views=0, units=0, listed=0 if r.near_units is None else len(r.near_units))
        if len(bad_views) == 0 or r.near_units is None or len(r.near_units) == 0:
            return r
        if len(bad_views) > max_views_with_flips(B, len(r.near_units)):
            return r                                        # not a matter of a few branches: the strict asserts report
        order = np.argsort(r.near_abs, kind="stable")
        by_view = {}
        for k in order:
            l, v, j = decode_unit(r.near_units[k], B)
            by_view.setdefault(v, []).append((l, j))
        off = np.asarray(img_off)
        all_flips = []
        for v in bad_views:
            cands = by_view.get(int(v), [])[:6]
            lo, hi = int(off[v]), int(off[v + 1])
            found = None
            for k in range(1, min(MAX_FLIPS_PER_VIEW, len(cands)) + 1):
                for subset in itertools.combinations(cands, k):
                    codes = np.array([(l * 1 + 0) * 1024 + j for (l, j) in subset], dtype=np.int64)
                    one = self.cpu.forward_backward(params64, uid[v:v + 1], hid[v:v + 1], np.array([0, hi - lo], np.int32),
                                                    img[lo:hi], label[v:v + 1], flip_units=codes,
                                                    fast=None if fast is None else fast[v:v + 1])
                    # a batch of one view divides by 1 where the batch divides by B
                    if np.abs(got_dx[v] - one.dX[0] / B).max() <= self.tol * scale:
                        found = subset
                        break
                if found:
                    break
            if not found:
                return r                                    # the strict asserts report the mismatch
            all_flips += [(l * B + int(v)) * 1024 + j for (l, j) in found]
        res = self.cpu.forward_backward(params64, uid, hid, img_off, img, label,
                                        flip_units=np.array(all_flips, dtype=np.int64), fast=fast)
        self.last_relu.update(views=len(bad_views), units=len(all_flips))
        self.relu_flips_accepted += len(all_flips)
        self.relu_views_flipped += len(bad_views)
        print("ReLU branches taken the other way inside the rounding band: %d units in %d of %d views (%d units listed)"
              % (len(all_flips), len(bad_views), B, self.last_relu["listed"]))
        return res

    def compare_store(self, check_tables: bool = True):
        gpu, cpu = self.gpu, self.cpu
        rows = torch.from_numpy(self.ri.rows).to(gpu.dev)
        assert np.array_equal(_np(gpu.dfv_gcnt[rows]), cpu.gcnt), "open-group counts"
        assert int(gpu.dfv_gcnt.sum().item()) == int(cpu.gcnt.sum()), "counts outside the touched rows"
        if check_tables:
            assert_close(_np(gpu.dfv_gsum[rows]), cpu.gsum, self.tol, "open-group sums")
            # nothing may land in the accumulator row of an image the batches never name (a row written too wide
            # would spill into its neighbour): the table's non-zero entries are all inside the touched rows
            assert count_nonzero(gpu.dfv_gsum) == count_nonzero(gpu.dfv_gsum[rows]), "sums outside the touched rows"

    def collect_and_compare(self, n_handed_over: Optional[int] = None) -> int:
        """n_handed_over: the count a gear_accumulate_collect call returned (the hand-over has happened already)."""
        gpu, cpu = self.gpu, self.cpu
        if n_handed_over is None:
            assert self.status() == cpu.pending_ready, "pending ready count"
            n = gpu.collect_ready()
        else:
            assert self.status() == 0, "the queue is empty after a fused call"
            n = n_handed_over
            assert int(gpu.d_counts[0].item()) == n, "device-side count of the fused call"
        eid, eseq, eavg = oracle.sort_emissions(*cpu.collect_ready())
        assert n == len(eid), "number of emissions"
        gid = _np(gpu.ready_ids[:n])
        assert np.array_equal(self.ri(gid), eid), "emitted ids"
        assert np.array_equal(_np(gpu.ready_seq[:n]), eseq), "emission numbers"
        assert_close(_np(gpu.ready_avg[:n]), eavg, self.tol, "averaged gradients")
        assert gpu.guards_intact(), "an output list was written past its end"
        return n

    def expire_and_compare(self, now: int, restamp: bool = True) -> int:
        gpu, cpu = self.gpu, self.cpu
        n = gpu.collect_expired(now, restamp)
        want = cpu.collect_expired(now, restamp)
        assert n == len(want), "number of expired entries"
        assert np.array_equal(_np(gpu.expired_ids[:n]), want), "expired ids"
        assert np.array_equal(_np(gpu.dfv_ts), cpu.ts), "timestamps after the scan"
        assert gpu.guards_intact(), "an output list was written past its end"
        return n

    def close(self):
        self.gpu.close()
