#!/usr/bin/env python
"""Accumulate-only measurements of the gradient store (events 5 and 6 of the paper's Section 3).

    python -m paper_1806_03925_b200.microbench [--config micro|skew|refresh|all] [--steps K] [--rows N]

micro   n gradient rows of dim 128 fp32 (IDs uniform or Zipf 1.1) into a 4M-image sum+count table, followed by
        the count >= M compaction and hand-over, M in {8, 64}: time and bytes-moved rate of
        gear_accumulate_collect (events 5 and 6 as one call) against the measured HBM copy rate.
skew    the skew-stress shapes (32768 views, 4M images, Zipf 1.3, dim 128 fp32), M in {1, 64, 1024}:
        sort + segmented reduction (GEAR_ACC_SORT) against fp32 reductions (GEAR_ACC_ATOMIC) under contention.

refresh gear_refresh_dfv: 2^20 recomputed DFVs (256 x fp32 each) written into a 20M-image table, bf16 and fp32
        storage, distinct random IDs in ascending order (the shape of an expiry list): bytes-moved rate.

One JSON line per case.  Inputs are synthetic and seeded; gradient rows are the procedural fill.  The bytes
counted are the ones the method has to move: every gradient row once, one accumulator row read (if it holds
anything) and written per distinct image, one averaged row per emission; the key sort's traffic is overhead
and not counted.
"""
from __future__ import annotations

import argparse
import json
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def _peak_gbs() -> tuple:
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        return json.load(open(path))["hbm_gbs"], "measured"
    return 6650.0, "fallback"


def _run_case(name, ids_np, V, D, M, mode, steps, warmup=2):
    import torch
    from . import binding as gb
    from .session import GearSession
    from .workloads import PRESETS

    n = len(ids_np)
    uniq = len(np.unique(ids_np))
    p = PRESETS["skew"].scaled(img_vocab=V, dfv_dim=D, M=M, user_vocab=64, url_vocab=64, expire=1 << 40)
    ready_cap = n // M + uniq + 1024 if mode == "sort" else 2 * n
    ready_cap = min(ready_cap, 2 * n)
    sess = GearSession(p, np.zeros(p.n_params, np.float32), max_batch=8, max_nnz=n, ready_cap=ready_cap, fill=True,
                       accum_mode=gb.GEAR_ACC_ATOMIC if mode == "atomic" else gb.GEAR_ACC_SORT, expired_cap=1)
    try:
        ids = torch.from_numpy(ids_np).cuda()
        grads = torch.empty((n, D), dtype=torch.float32, device="cuda")
        gb.gear_fill_uniform(grads, seed=5, tag=gb.GEAR_TAG_GRAD, amp=1.0)
        stream = torch.cuda.current_stream()
        t_acc, t_col, n_ready = [], [], []
        launches0 = gb.gear_launch_count(sess.ctx)
        for s in range(warmup + steps):
            e0, e1, e2 = (torch.cuda.Event(enable_timing=True) for _ in range(3))
            e0.record(stream)
            k = sess.accumulate_collect_rows(ids, grads, sync=True)     # events 5 and 6 as one call
            e1.record(stream)
            e2.record(stream)
            torch.cuda.synchronize()
            if s >= warmup:
                t_acc.append(e0.elapsed_time(e1)); t_col.append(e1.elapsed_time(e2)); n_ready.append(k)
        launches_per_step = (gb.gear_launch_count(sess.ctx) - launches0) / (warmup + steps)
        # one more call with per-kernel events (serialised, so each kernel is timed alone)
        gb.gear_profile_enable(sess.ctx, True)
        sess.accumulate_collect_rows(ids, grads, sync=True)
        prof = gb.gear_profile_read(sess.ctx, 64)
        gb.gear_profile_enable(sess.ctx, False)
        kernels = {k: round(v[0], 4) for k, v in sorted(prof.items(), key=lambda kv: -kv[1][0])}
        rc, status, _ = sess.status()
        acc_ms, col_ms, ready = float(np.median(t_acc)), float(np.median(t_col)), float(np.mean(n_ready))
        bytes_acc = n * D * 4 + n * 4 + uniq * (D * 4 + 4) * 2 + ready * (D * 4 + 4)
        bytes_col = 0.0 if "collect_move" not in prof else ready * (2 * D * 4 + 16)      # a separate hand-over pass, if one ran
        peak, src = _peak_gbs()
        gbs = (bytes_acc + bytes_col) / ((acc_ms + col_ms) * 1e-3) / 1e9
        return {"case": name, "mode": mode, "rows": n, "img_vocab": V, "dim": D, "M": M, "distinct_images": uniq,
                "emissions_per_call": ready, "accumulate_ms": round(acc_ms, 4), "collect_ms": round(col_ms, 4),
                "rows_per_s": round(n / ((acc_ms + col_ms) * 1e-3), 1),
                "algorithmic_GB": round((bytes_acc + bytes_col) / 1e9, 3), "GB/s": round(gbs, 1),
                "frac_of_hbm_peak": round(gbs / peak, 4), "hbm_peak_GB/s": peak, "peak_source": src,
                "frac_of_8TBs": round(gbs / 8000.0, 4), "kernel_ms": kernels, "launches_per_step": launches_per_step,
                "device_status": status, "dtype": "f32", "data": "synthetic"}
    finally:
        sess.close()


def _run_refresh(dfv_dtype: str, n: int, steps: int, V: int = 20_000_000, D: int = 256):
    import torch
    from . import binding as gb
    from .session import GearSession
    from .workloads import PRESETS
    p = PRESETS["tiny"].scaled(img_vocab=V, dfv_dim=D, dfv_dtype=dfv_dtype, user_vocab=64, url_vocab=64, expire=1 << 40)
    sess = GearSession(p, np.zeros(p.n_params, np.float32), max_batch=8, max_nnz=8, fill=True, expired_cap=1)
    try:
        rng = np.random.default_rng(1)
        ids = torch.from_numpy(np.sort(rng.choice(V, n, replace=False)).astype(np.int32)).cuda()
        rows = torch.empty((n, D), dtype=torch.float32, device="cuda")
        gb.gear_fill_uniform(rows, seed=6, tag=gb.GEAR_TAG_GRAD, amp=1.0)
        stream = torch.cuda.current_stream()
        ts = []
        for s in range(2 + steps):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            sess.refresh_dfv(ids, rows, now=s)
            e1.record(stream)
            torch.cuda.synchronize()
            if s >= 2:
                ts.append(e0.elapsed_time(e1))
        ms = float(np.median(ts))
        esz = 2 if dfv_dtype == "bf16" else 4
        nbytes = n * (D * 4 + D * esz + 12)
        peak, src = _peak_gbs()
        gbs = nbytes / (ms * 1e-3) / 1e9
        rc, status, _ = sess.status()
        return {"case": "refresh_%s" % dfv_dtype, "rows": n, "img_vocab": V, "dim": D, "ms": round(ms, 4),
                "rows_per_s": round(n / (ms * 1e-3), 1), "algorithmic_GB": round(nbytes / 1e9, 3), "GB/s": round(gbs, 1),
                "frac_of_hbm_peak": round(gbs / peak, 4), "hbm_peak_GB/s": peak, "peak_source": src,
                "frac_of_8TBs": round(gbs / 8000.0, 4), "device_status": status, "dtype": dfv_dtype, "data": "synthetic"}
    finally:
        sess.close()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--config", default="all", choices=["micro", "skew", "refresh", "all"])
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--rows", type=int, default=None, help="rows of the micro cases (default 2^24)")
    ap.add_argument("--vocab", type=int, default=20_000_000, help="images in the table of the refresh cases")
    args = ap.parse_args()
    import torch
    if not torch.cuda.is_available():
        raise SystemExit("needs a CUDA device: libgear has no CPU path")
    from . import workloads
    from .workloads import MICRO_PRESETS, PRESETS, BatchSource
    if args.config in ("micro", "all"):
        for name, mp in MICRO_PRESETS.items():
            ids = workloads.micro_ids(mp, seed=0, n_rows=args.rows)
            print(json.dumps(_run_case(name, ids, mp.img_vocab, mp.dfv_dim, mp.M, "sort", args.steps)), flush=True)
    if args.config in ("refresh", "all"):
        for dt in ("bf16", "f32"):
            print(json.dumps(_run_refresh(dt, min(1 << 20, args.vocab // 2), args.steps, V=args.vocab)), flush=True)
    if args.config in ("skew", "all"):
        p = PRESETS["skew"]
        ids = BatchSource(p, 0).batch(0).img_id
        for M in (1, 64, 1024):
            for mode in ("sort", "atomic"):
                print(json.dumps(_run_case("skew_M%d" % M, ids, p.img_vocab, p.dfv_dim, M, mode, args.steps)),
                      flush=True)


if __name__ == "__main__":
    main()
