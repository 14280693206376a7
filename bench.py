#!/usr/bin/env python
"""Throughput of the Gear Training sparse-part step on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload large|medium|tiny]

One "step" is one pass of the whole hot path over one batch of synthetic page views:
gear_forward_backward (gather, head forward/backward, embedding scatter), gear_accumulate_dfv_grad,
gear_collect_ready and gear_collect_expired.  Prints ONE JSON line (rank 0).

value      page views/s with the batches already resident in HBM (device-timed, max over ranks)
e2e        the same with the batch arrays in pinned HOST memory, every step's batch copied in inside the timed
           region (one step ahead, on a copy stream) and every step's loss and two counts read back by the host
roofline   the kernel with the largest share of the step, timed per launch with CUDA events inside the
           library (a second pass of K steps with profiling on), against the measured machine peaks
cpu_baseline  the CPU oracle, as it stands, on a bounded sample of the same workload (rank 0, N=1)

With --gpus N > 1 (launched under torchrun) every rank runs an independent replica on its own GPU: the
path has no exchange step on one GPU and the multi-GPU sharding is not built, so scaling is "weak".
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "page views/sec per step (1 B200); gather+accumulate HBM GB/s vs ~8 TB/s peak"
UNIT = "page views/s"
N_BATCHES = 8          # distinct pre-generated batches the timed loop cycles through
MIN_TIMED_MS = 1000.0  # device time measured per arm, whatever --steps is: the K-step region is repeated until then
MAX_REGIONS = 400


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        d = json.load(open(path))
        return dict(hbm_gbs=d["hbm_gbs"], bf16_tflops=d["bf16_tflops"], bf16_sustained=d.get("bf16_tflops_sustained"),
                    source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, bf16_sustained=1400.0, source="fallback")


# fp32 FMA peak of the plain-ALU head: 148 SMs x 128 lanes x 2 flop x max SM clock
ALU_F32_TFLOPS = 148 * 128 * 2 * 1.965e9 / 1e12


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu, self.proc, self.lines = gpu_index, None, []
        self.t_open = self.t_close = None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.gpu), "--query-gpu=" + self.FIELDS,
                                          "--format=csv,noheader,nounits", "-lms", "50"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append((time.monotonic(), line.strip()))

    def open_window(self):
        """Samples count from here (the start of the first timed region) ..."""
        self.t_open = time.monotonic()

    def close_window(self):
        """... to here (the end of the last one)."""
        self.t_close = time.monotonic()

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        t0 = self.t_open if self.t_open is not None else 0.0
        t1 = self.t_close if self.t_close is not None else float("inf")
        inside = [ln for (t, ln) in self.lines if t0 <= t <= t1 + 0.05]
        for line in inside:
            f = [x.strip() for x in line.split(",")]
            if len(f) < 8:
                continue
            try:
                sm.append(float(f[0])); mx.append(float(f[1]))
            except ValueError:
                continue
            for name, v in zip(names, f[4:8]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


def preset_for(name: str):
    from paper_1806_03925_b200.workloads import PRESETS
    return PRESETS[name]


# ---------------------------------------------------------------------------------------------
# algorithmic work per launch of each kernel (bytes the method must move, or flops)
# ---------------------------------------------------------------------------------------------
def kernel_models(p, stats):
    """name -> (bound, work per launch, unit).  stats: per-step means measured on the generated batches."""
    B, nnz = stats["B"], stats["nnz"]
    E, D, Din = p.emb_dim, p.dfv_dim, p.d_in
    dsz = 2 if p.dfv_dtype == "bf16" else 4
    xsz = 2 if p.head_dtype == "bf16" else 4
    m = {}
    m["gather_pool"] = ("hbm", B * 2 * E * 4 + nnz * D * dsz + B * Din * xsz + (3 * B + 1 + 2 * nnz) * 4 + B * 4)
    # gradient rows: the B pooled-gradient rows are read (each once from HBM; repeats hit L2), one accumulator row
    # is read (if open) and written per distinct image, complete groups write one averaged row
    m["acc_reduce"] = ("hbm", B * D * 4 + nnz * 8 + stats["uniq_img"] * (D * 4 + 4) * 2 + stats["n_ready"] * (D * 4 + 4))
    m["expiry_mark"] = ("hbm", p.img_vocab * 8 + p.img_vocab // 8)
    m["emb_reduce"] = ("hbm", 2 * (B * E * 4 + B * 8 + stats["uniq_emb"] * E * 4 * 2))      # both tables, one launch
    m["collect_move"] = ("hbm", stats["n_ready"] * (D * 4 * 2 + 16))
    fan = [Din] + list(p.hidden)
    L = len(p.hidden)
    m["head_out"] = ("hbm", B * fan[L] * xsz * 2 + B * 12)          # top activations in, their gradients out
    # the head's products: (flops, bytes) per launch.  Launches of one name share the step's products of that kind
    # evenly.  Bytes: every operand and the output once, in the dtype it has in memory (the weights' fp32 gradient,
    # dX fp32, everything else in the head dtype); the ReLU mask of a hidden-layer gradient is one more operand.
    def avg(xs):
        return sum(xs) / max(len(xs), 1)
    layers = range(L)
    m["gemm"] = {
        "fwd": (avg([2 * B * fan[l] * fan[l + 1] for l in layers]),
                avg([(B * fan[l] + fan[l] * fan[l + 1] + B * fan[l + 1]) * xsz for l in layers])),
        "dw": (avg([2 * B * fan[l] * fan[l + 1] for l in layers]),
               avg([(B * fan[l] + B * fan[l + 1]) * xsz + fan[l] * fan[l + 1] * 4 for l in layers])),
        "dh": (avg([2 * B * fan[l] * fan[l + 1] for l in layers if l > 0]),
               avg([(B * fan[l + 1] + fan[l] * fan[l + 1] + 2 * B * fan[l]) * xsz for l in layers if l > 0])),
        "dx": (2 * B * fan[0] * fan[1], (B * fan[1] + fan[0] * fan[1]) * xsz + B * fan[0] * 4),
    }
    return m


# DRAM bytes per launch (dram__bytes_read.sum + dram__bytes_write.sum) from the ncu --set full captures summarised under
# profiles/, taken on the large_2m workload (same batch and head, 4.6 GB of tables; a full-set capture of the 48.9 GB
# workload would save and restore tens of GB per pass).  Second entry: what the figure scales with when the bench
# runs another workload -- "work" = the kernel's algorithmic bytes (table-bound kernels: traffic grows with the rows
# touched), "vocab" = image vocabulary, None = same shapes, taken as is.  ncu flushes the L2 before every pass, so
# re-reads that hit the L2 in a real step count as DRAM traffic here.  A kernel that has changed since its capture
# must be taken out of this table (traffic is then reported as null).
NCU_TRAFFIC_LARGE_2M = {
    "gather_pool": (64.1e6, "l2"), "acc_reduce": (238.0e6, "work"), "expiry_mark": (16.0e6, "vocab"),
    "head_out": (34.5e6, None), "emb_reduce": (46.9e6, "work"),
    "tc_gemm_fwd": (69.0e6, None), "tc_gemm_dw": (113.6e6, None), "tc_gemm_dh": (130.4e6, None), "tc_gemm_dx": (110.3e6, None),
}
# algorithmic bytes per launch of the table-bound kernels on large_2m (kernel_models on that workload's batches)
NCU_WORK_LARGE_2M = {"gather_pool": 222.0e6, "acc_reduce": 224.5e6, "emb_reduce": 58.9e6}


def ncu_traffic(name, p, work):
    """(DRAM traffic per launch of kernel `name` on workload p, where the figure comes from); (None, reason) if there
    is no figure that holds for this workload."""
    if name not in NCU_TRAFFIC_LARGE_2M:
        return None, "no ncu capture of this kernel as it stands"
    if not p.name.startswith("large"):
        return None, "ncu captures exist for the large-table shapes only"
    bytes_2m, scales_with = NCU_TRAFFIC_LARGE_2M[name]
    if p.name == "large_2m":
        return round(bytes_2m), "ncu --set full on this workload (large_2m)"
    if scales_with == "vocab":
        return round(bytes_2m * p.img_vocab / 2_000_000), "ncu on large_2m, scaled by the image vocabulary"
    if scales_with == "work":
        if not work or name not in NCU_WORK_LARGE_2M:
            return None, "no algorithmic-bytes figure to scale by"
        return round(bytes_2m * work / NCU_WORK_LARGE_2M[name]), "ncu on large_2m, scaled by algorithmic bytes"
    if scales_with == "l2":
        return None, ("ncu on large_2m only: the L2 serves a share of the rows of a 2M-image table that it cannot "
                      "serve of a 20M-image one, so the figure does not scale")
    return round(bytes_2m), "ncu on large_2m, same shapes"


def roofline_for(name, ms_per_launch, p, stats, peaks):
    """Roofline object of one kernel from its live per-launch time."""
    models = kernel_models(p, stats)
    sec = ms_per_launch * 1e-3
    if name in models and isinstance(models[name], tuple):
        work = models[name][1]
        ach = work / sec / 1e9
        traffic, source = ncu_traffic(name, p, work)
        return {"kernel": name, "bound": "hbm", "achieved": round(ach, 1), "peak": peaks["hbm_gbs"], "unit": "GB/s",
                "frac": round(ach / peaks["hbm_gbs"], 4), "traffic": traffic, "traffic_source": source,
                "peak_source": peaks["source"], "work_per_launch": work}
    if name.startswith("simt_gemm") or name.startswith("tc_gemm"):
        # The head's products are dense contractions: rated by their flops against the tensor peak (bf16 heads; the
        # sustained figure, since they run inside a long step) or the fp32 FMA peak (fp32 heads).  memory_frac is
        # the secondary figure: every operand and the output once, over the measured copy rate.
        flops, nbytes = models["gemm"][name.rsplit("_", 1)[1]]
        if name.startswith("tc_gemm"):
            peak, bound, src = peaks["bf16_sustained"] or peaks["bf16_tflops"], "tensor", peaks["source"] + " (sustained bf16)"
        else:
            peak, bound, src = ALU_F32_TFLOPS, "alu", "148 SMs x 128 FMA lanes x 2 x 1.965 GHz"
        ach = flops / sec / 1e12
        traffic, source = ncu_traffic(name, p, None) if bound == "tensor" else (None, "fp32 head: no capture")
        return {"kernel": name, "bound": bound, "achieved": round(ach, 2), "peak": round(peak, 1), "unit": "TFLOP/s",
                "frac": round(ach / peak, 4), "traffic": traffic, "traffic_source": source,
                "peak_source": src, "work_per_launch": flops, "memory_frac": round(nbytes / sec / 1e9 / peaks["hbm_gbs"], 4)}
    return {"kernel": name, "bound": "latency", "achieved": None, "peak": None, "unit": None, "frac": None,
            "traffic": None, "traffic_source": None}


def step_roofline(p, stats, ms_per_step, peaks):
    """The whole step against both rooflines: the bytes the method has to move per step (gather, embedding scatter,
    accumulate, emit, expiry scan; intermediates of the head not counted) and the head's flops, over the step time."""
    m = kernel_models(p, stats)
    nbytes = sum(m[k][1] for k in ("gather_pool", "acc_reduce", "expiry_mark", "emb_reduce"))
    nbytes += stats.get("n_ready", 0.0) * (p.dfv_dim * 4 + 8) if not stats.get("emit_direct") else 0.0
    fan = [p.d_in] + list(p.hidden)
    flops = 6.0 * stats["B"] * (sum(fan[l] * fan[l + 1] for l in range(len(p.hidden))) + fan[-1])
    sec = ms_per_step * 1e-3
    tensor_peak = (peaks["bf16_sustained"] or peaks["bf16_tflops"]) if p.head_dtype == "bf16" else ALU_F32_TFLOPS
    return {"bytes_per_step": round(nbytes), "flops_per_step": round(flops),
            "hbm_GB/s": round(nbytes / sec / 1e9, 1), "hbm_frac": round(nbytes / sec / 1e9 / peaks["hbm_gbs"], 4),
            "math_TFLOP/s": round(flops / sec / 1e12, 2), "math_frac": round(flops / sec / 1e12 / tensor_peak, 4),
            "math_peak": round(tensor_peak, 1), "math_bound": "tensor" if p.head_dtype == "bf16" else "alu",
            "lower_bound_ms": round(max(nbytes / (peaks["hbm_gbs"] * 1e9), flops / (tensor_peak * 1e12)) * 1e3, 4),
            "peak_source": peaks["source"]}


# ---------------------------------------------------------------------------------------------
# reference arm: the CPU oracle
# ---------------------------------------------------------------------------------------------
def oracle_sample_run(p, src, sample_views: int, step: int = 0, seed: int = 0):
    """One bounded sample of a step on the CPU oracle.  Returns (seconds for the per-view part on the sample,
    seconds for the expiry scan of the whole timestamp table, views in the sample)."""
    import oracle
    from oracle import GearOracle
    b = src.batch(step)
    views = slice(0, min(sample_views, b.B))
    nv = views.stop
    off = b.img_off[:nv + 1].astype(np.int32)
    img = b.img_id[:off[-1]]
    uid, hid = b.user_id[:nv], b.url_id[:nv]
    ru, iu = np.unique(uid, return_inverse=True)
    rh, ih = np.unique(hid, return_inverse=True)
    ri, ii = np.unique(img, return_inverse=True)
    dfv_np = np.uint16 if p.dfv_dtype == "bf16" else np.float32
    orc = GearOracle(oracle.fill_rows(seed, oracle.TAG_USER, p.emb_dim, ru, len(ru), np.float32),
                     oracle.fill_rows(seed, oracle.TAG_URL, p.emb_dim, rh, len(rh), np.float32),
                     oracle.fill_rows(seed, oracle.TAG_DFV, p.dfv_dim, ri, len(ri), dfv_np),
                     p.hidden, p.M, p.expire, round_bf16=(p.head_dtype == "bf16"),
                     ts=oracle.fill_ts(seed, p.expire, 0, None, p.img_vocab))
    from paper_1806_03925_b200 import workloads
    params = workloads.head_params(p, seed).astype(np.float64)
    t0 = time.perf_counter()
    r = orc.forward_backward(params, iu.astype(np.int32), ih.astype(np.int32), off, ii.astype(np.int32), b.label[:nv])
    orc.emb_apply("user", iu.astype(np.int32), r.dX, -p.lr)
    orc.emb_apply("url", ih.astype(np.int32), r.dX, -p.lr)
    orc.accumulate(ii.astype(np.int32), orc.dfv_grad_rows(off, r.dX))
    orc.collect_ready()
    t1 = time.perf_counter()
    orc.collect_expired(step + 1, True)
    t2 = time.perf_counter()
    return t1 - t0, t2 - t1, nv


def cpu_baseline(p, src, sample_views: int):
    t_views, t_exp, nv = oracle_sample_run(p, src, sample_views)
    step_s = t_views * (p.batch / nv) + t_exp
    return {"value": round(p.batch / step_s, 1), "unit": UNIT, "cores": 1, "kind": "oracle",
            "sample": "first %d of the %d views of one %s step (gather, head, embedding apply, accumulate, collect) "
                      "scaled to the full batch, plus one expiry scan of all %d timestamps; %.1f s of CPU time"
                      % (nv, p.batch, p.name, p.img_vocab, t_views + t_exp)}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from paper_1806_03925_b200.workloads import BatchSource
    p = preset_for(args.workload)
    src = BatchSource(p, 0)
    sample = {"large": 1024, "medium": 1024, "tiny": 256}.get(args.workload, 512)
    times = []
    for s in range(args.warmup + args.steps):
        t_views, t_exp, nv = oracle_sample_run(p, src, sample, step=s % 2)
        if s >= args.warmup:
            times.append(t_views * (p.batch / nv) + t_exp)
    step_s = float(np.mean(times))
    value = p.batch / step_s
    line = {"impl": "reference", "metric": METRIC, "value": round(value, 1), "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": round(step_s * 1e3, 3),
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": "%s tables" % p.name if p.name == "large" else p.name, "batch": p.batch,
                       "note": "CPU oracle, one thread; each step is a sample of %d views scaled to the batch" % sample},
            "cpu_baseline": {"value": round(value, 1), "unit": UNIT, "cores": 1, "kind": "oracle",
                             "sample": "%d views per step scaled to %d, plus the full expiry scan" % (sample, p.batch)},
            "e2e": {"value": round(value, 1), "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


# ---------------------------------------------------------------------------------------------
# our arm
# ---------------------------------------------------------------------------------------------
def run_ours(args):
    import torch
    from paper_1806_03925_b200 import binding as gb
    from paper_1806_03925_b200.replicas import Replicas
    from paper_1806_03925_b200 import workloads
    from paper_1806_03925_b200.session import DeviceBatch, GearSession
    from paper_1806_03925_b200.workloads import BatchSource

    reps = Replicas.from_env()
    rank, world, local = reps.rank, reps.world, reps.local_rank
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: libgear has no CPU path")
    torch.cuda.set_device(local)
    reps.init("nccl", torch.device("cuda", local))
    gb.load()
    p = preset_for(args.workload)
    K, W = args.steps, args.warmup
    sampler = ClockSampler(local)          # started early: nvidia-smi needs a moment before its first line
    sampler.start()
    seed = reps.seed                              # every replica draws its own tables and batches
    src = BatchSource(p, seed)
    host_batches = [src.batch(s) for s in range(N_BATCHES)]
    max_nnz = max(b.nnz for b in host_batches)
    sess = GearSession(p, workloads.head_params(p, seed), max_batch=p.batch, max_nnz=max_nnz, seed=seed, fill=True,
                       now=0, expired_cap=p.img_vocab)
    dev_batches = [DeviceBatch.from_host(b) for b in host_batches]
    stats = {"B": p.batch, "nnz": float(np.mean([b.nnz for b in host_batches])),
             "uniq_img": float(np.mean([len(np.unique(b.img_id)) for b in host_batches])),
             "uniq_emb": float(np.mean([(len(np.unique(b.user_id)) + len(np.unique(b.url_id))) / 2 for b in host_batches]))}

    stream = torch.cuda.current_stream()
    now = [0]

    expiry_beside_default = p.img_vocab >= (1 << 22)       # GearSession.step's own rule

    def one_step(db, expiry_beside=None):
        now[0] += 1
        sess.step(db, now[0], sync=False, expiry_beside=expiry_beside)

    def barrier():
        torch.cuda.synchronize()
        reps.barrier()
        torch.cuda.synchronize()

    def timed(fn, steps):
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        ev0.record(stream)
        for s in range(steps):
            fn(s)
        ev1.record(stream)
        barrier()
        return reps.max_over_ranks(ev0.elapsed_time(ev1), device="cuda")

    # ---- device-resident throughput (clock samples count from here to the end of the end-to-end pass:
    #      every region in between runs the same step under load)
    sampler.open_window()
    for s in range(W):
        one_step(dev_batches[s % N_BATCHES])
    def regions_of(region_fn):
        """Repeats the K-step timed region until MIN_TIMED_MS of device time have been measured (at least 3 regions):
        a few steps alone are too short for the clock sampler to see and for the clocks to settle under load.  The
        loop count follows from the max-over-ranks time, so every rank runs the same number of regions."""
        out = []
        while (sum(out) < args.min_timed_ms or len(out) < 3) and len(out) < MAX_REGIONS:
            out.append(region_fn())
        return out

    launches0 = gb.gear_launch_count(sess.ctx)
    ms = timed(lambda s: one_step(dev_batches[s % N_BATCHES]), K)
    launches = gb.gear_launch_count(sess.ctx) - launches0
    region_ms = [ms] + regions_of(lambda: timed(lambda s: one_step(dev_batches[s % N_BATCHES]), K))
    ms = float(np.median(region_ms))
    rc, status, _ = sess.status()
    n_ready_mean = None

    # ---- end to end: host batches in, loss and counts out, every step
    # One pinned host buffer per batch holding its five arrays back to back (16-byte aligned), and two device buffers
    # of the same layout whose slices are the batch a step reads: one host->device copy per step, issued on a copy
    # stream one step ahead, so that batch s+1 travels while step s computes.  The loss and the two counts of a step
    # come back with one device->host copy of the session's 24-byte scalar block; the host reads them one step
    # late (while the next step runs) and the last step's before the timed region ends.
    def packed_layout(nnz_cap):
        sizes = [p.batch * 4, p.batch * 4, (p.batch + 1) * 4, nnz_cap * 4, p.batch * 4]
        offs, o = [], 0
        for sz in sizes:
            offs.append(o)
            o = (o + sz + 15) // 16 * 16
        return offs, o
    offs, total_bytes = packed_layout(max_nnz)
    dev_packs = [torch.empty(total_bytes, dtype=torch.uint8, device="cuda") for _ in range(2)]

    def view(buf, off, n, dt):
        return buf[off:off + n * 4].view(dt)
    stages = [DeviceBatch(view(dp, offs[0], p.batch, torch.int32), view(dp, offs[1], p.batch, torch.int32),
                          view(dp, offs[2], p.batch + 1, torch.int32), view(dp, offs[3], max_nnz, torch.int32),
                          view(dp, offs[4], p.batch, torch.float32), B=p.batch, nnz=0) for dp in dev_packs]
    host_packs = []
    for hb in host_batches:
        hp = torch.zeros(total_bytes, dtype=torch.uint8).pin_memory()
        for off, arr in zip(offs, (hb.user_id, hb.url_id, hb.img_off, hb.img_id, hb.label)):
            raw = torch.from_numpy(np.ascontiguousarray(arr)).view(torch.uint8)
            hp[off:off + raw.numel()].copy_(raw)
        host_packs.append(hp)
    h2d_bytes = total_bytes
    host_scalars = [torch.zeros(3, dtype=torch.int64).pin_memory() for _ in range(2)]
    copy_stream = torch.cuda.Stream()
    ev_arrived = [torch.cuda.Event() for _ in range(2)]      # batch in device buffer i has landed
    ev_consumed = [torch.cuda.Event() for _ in range(2)]     # the step that read device buffer i is done
    ev_result = [torch.cuda.Event() for _ in range(2)]       # the scalars of that step are in host buffer i
    results = []

    def send(s):
        i = s % 2
        with torch.cuda.stream(copy_stream):
            copy_stream.wait_event(ev_consumed[i])            # the buffer's previous batch has been used
            dev_packs[i].copy_(host_packs[s % N_BATCHES], non_blocking=True)
            ev_arrived[i].record(copy_stream)

    def e2e_run(steps):
        for i in range(2):
            ev_consumed[i].record(stream)
        send(0)
        for s in range(steps):
            i = s % 2
            if s + 1 < steps:
                send(s + 1)
            stream.wait_event(ev_arrived[i])
            stages[i].nnz = host_batches[s % N_BATCHES].nnz
            one_step(stages[i])
            ev_consumed[i].record(stream)
            host_scalars[i].copy_(sess.scalars, non_blocking=True)
            ev_result[i].record(stream)
            if s > 0:
                ev_result[1 - i].synchronize()                # the caller reads the loss and the counts of step s-1
                results.append(int(host_scalars[1 - i][1]))
        ev_result[(steps - 1) % 2].synchronize()
        results.append(int(host_scalars[(steps - 1) % 2][1]))

    def timed_run(fn, steps):
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        ev0.record(stream)
        fn(steps)
        ev1.record(stream)
        barrier()
        return reps.max_over_ranks(ev0.elapsed_time(ev1), device="cuda")

    e2e_run(min(W, 3))
    e2e_region_ms = regions_of(lambda: timed_run(e2e_run, K))
    ms_e2e = float(np.median(e2e_region_ms))
    sampler.close_window()
    clocks = sampler.stop()
    d2h_bytes = 24

    # ---- per-kernel timing pass (profiling on; not part of the throughput numbers)
    ready_counts = []
    KP = min(K, 50)
    gb.gear_profile_enable(sess.ctx, True)
    for s in range(KP):
        one_step(dev_batches[s % N_BATCHES], expiry_beside=False)      # every kernel alone, on one stream
        ready_counts.append(int(sess.d_counts[0].item()))
    prof = gb.gear_profile_read(sess.ctx, 64)
    gb.gear_profile_enable(sess.ctx, False)
    stats["n_ready"] = float(np.mean(ready_counts)) if ready_counts else 0.0
    total_ms = sum(v[0] for v in prof.values()) or 1.0
    kernels = sorted(({"name": k, "launches_per_step": v[1] / KP, "ms_per_step": v[0] / KP, "share": v[0] / total_ms,
                       "ms_per_launch": v[0] / v[1]} for k, v in prof.items()), key=lambda d: -d["ms_per_step"])
    peaks = measured_peaks()
    # the dominant kernel of the step's critical path: the ID sort runs on a side stream beside the gather and the
    # head in the throughput passes and has no bandwidth or flop roofline, so it is not a candidate
    roof = None
    for kd in kernels:
        r = roofline_for(kd["name"], kd["ms_per_launch"], p, stats, peaks)
        if r["bound"] in ("hbm", "tensor", "alu"):
            roof = r
            roof["share_of_step"] = round(kd["share"], 4)
            break
    if roof is None:
        roof = roofline_for(kernels[0]["name"], kernels[0]["ms_per_launch"], p, stats, peaks)
    hbm_kernels = []
    for kd in kernels:
        r = roofline_for(kd["name"], kd["ms_per_launch"], p, stats, peaks)
        if r["bound"] == "hbm":
            hbm_kernels.append({"kernel": kd["name"], "GB/s": r["achieved"], "frac_of_measured": r["frac"],
                                "frac_of_8TBs": round(r["achieved"] / 8000.0, 4), "ms": round(kd["ms_per_launch"], 4)})

    stats["emit_direct"] = any(k["name"] == "acc_reduce" for k in kernels) and not any(k["name"] == "collect_move" for k in kernels)
    spread = lambda xs: {"regions": len(xs), "min_ms_per_step": round(min(xs) / K, 4), "median_ms_per_step": round(float(np.median(xs)) / K, 4),
                         "max_ms_per_step": round(max(xs) / K, 4), "timed_ms": round(sum(xs), 1)}
    line = {"metric": METRIC, "value": round(reps.whole_job_rate(p.batch * K, ms), 1), "unit": UNIT, "n_gpus": world, "steps": K,
            "warmup": W, "ms_per_step": round(ms / K, 4), "regions": spread(region_ms),
            "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16" if p.head_dtype == "bf16" else "f32", "data": "synthetic",
            "config": {"workload": "large tables" if p.name == "large" else p.name, "batch": p.batch,
                       "tables_gb": round((p.user_vocab + p.url_vocab) * p.emb_dim * 4 / 1e9 + p.img_vocab * p.dfv_dim *
                                          ((2 if p.dfv_dtype == "bf16" else 4) + 4) / 1e9 + p.img_vocab * 12 / 1e9, 1),
                       "M": p.M, "expire": p.expire, "mean_nnz": round(stats["nnz"], 1),
                       "l2": "tables far exceed the 126 MB L2 and rows are Zipf-random; %d pre-generated batches cycle; "
                             "no explicit flush" % N_BATCHES,
                       "streams": ("training calls on one stream, the expiry scan of the same step on a second one, "
                                   "forked at the step's start and joined at its end (inside the timed region)")
                       if expiry_beside_default else "all calls on one stream",
                       "outputs": "the averaged-gradient list (ids, seq, avg) and the expired-ID list of every step stay in "
                                  "device memory, where a Dense Part on the same GPU would consume them; the end-to-end arm "
                                  "reads back the loss and the two counts (24 bytes)",
                       "parallelism": "replicas only" if world > 1 else "single GPU"},
            "clocks": clocks,
            "e2e": {"value": round(reps.whole_job_rate(p.batch * K, ms_e2e), 1), "unit": UNIT, "h2d_bytes_per_step": h2d_bytes,
                    "d2h_bytes_per_step": d2h_bytes, "ms_per_step": round(ms_e2e / K, 4), "regions": spread(e2e_region_ms)},
            "gpu_launches": int(launches),
            "roofline": roof,
            "roofline_step": step_roofline(p, stats, ms / K, peaks),
            "products": [roofline_for(k["name"], k["ms_per_launch"], p, stats, peaks) for k in kernels
                         if k["name"].startswith(("tc_gemm", "simt_gemm"))],
            "kernels": [{"name": k["name"], "ms_per_step": round(k["ms_per_step"], 4), "share": round(k["share"], 4),
                         "launches_per_step": round(k["launches_per_step"], 2)} for k in kernels],
            "hbm_kernels": hbm_kernels,
            "device_status": status}
    if rank == 0:
        if world == 1 and not args.no_cpu_baseline:
            # sized for roughly 10-30 s of single-thread CPU time
            sample = {"large": 32768, "large_2m": 32768, "medium": 4096, "tiny": 256}.get(args.workload, 8192)
            line["cpu_baseline"] = cpu_baseline(p, BatchSource(p, 0), sample)
        else:
            line["cpu_baseline"] = None
        print(json.dumps(line), flush=True)
    sess.close()
    reps.close()


# ---------------------------------------------------------------------------------------------
# configurations 4 and 5: accumulate-only micro-benchmark, sort against atomics under skew
# ---------------------------------------------------------------------------------------------
def oracle_accumulate_sample(ids, V, D, M, n_sample, seed=5):
    """The CPU oracle's accumulate + collect on the first n_sample rows of the case; returns seconds."""
    import oracle
    from oracle import GearOracle
    n = min(n_sample, len(ids))
    rows = oracle.fill_rows(seed, oracle.TAG_GRAD, D, None, n, np.float32, amp=1.0).astype(np.float64)
    orc = GearOracle(np.zeros((1, 4), np.float32), np.zeros((1, 4), np.float32), np.zeros((V, D), np.uint16), (8,), M, 1 << 40)
    t0 = time.perf_counter()
    orc.accumulate(ids[:n], rows)
    orc.collect_ready()
    return time.perf_counter() - t0, n


def accumulate_line(case, args, sampler_gpu, peaks, with_cpu=True):
    """One JSON line for one accumulate-only case (a dict from microbench._run_case plus the keys of the contract)."""
    acc_ms = case["kernel_ms"].get("acc_reduce")
    total_ms = case["accumulate_ms"] + case["collect_ms"]
    n, D, uniq, ready = case["rows"], case["dim"], case["distinct_images"], case["emissions_per_call"]
    line = {"metric": METRIC, "value": case["rows_per_s"], "unit": "gradient rows/s", "n_gpus": 1, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": round(total_ms, 4), "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {"workload": case["case"], "mode": case["mode"], "rows": n, "img_vocab": case["img_vocab"], "dim": D,
                       "M": case["M"], "distinct_images": uniq, "emissions_per_call": ready,
                       "step": "one gear_accumulate_collect over all rows (accumulate + hand-over of the completed groups)",
                       "l2": "8.6 GB of gradient rows and a 2 GB store per call: far beyond the 126 MB L2"},
            "clocks": sampler_gpu, "gpu_launches": case.get("launches_per_step"),
            "e2e": None, "e2e_note": "the rows are produced on the device by the head's backward pass and never cross "
                                     "PCIe in the method: no host-buffer arm for this kernel-level case",
            "kernel_ms": case["kernel_ms"], "device_status": case["device_status"],
            "roofline_step": {"bytes_per_step": round(case["algorithmic_GB"] * 1e9), "hbm_GB/s": case["GB/s"],
                              "hbm_frac": case["frac_of_hbm_peak"], "frac_of_8TBs": case["frac_of_8TBs"],
                              "peak_source": case["peak_source"]}}
    if acc_ms:
        work = n * D * 4 + n * 8 + uniq * (D * 4 + 4) * 2 + ready * (D * 4 + 4)
        ach = work / (acc_ms * 1e-3) / 1e9
        line["roofline"] = {"kernel": "acc_reduce", "bound": "hbm", "achieved": round(ach, 1), "peak": peaks["hbm_gbs"],
                            "unit": "GB/s", "frac": round(ach / peaks["hbm_gbs"], 4), "traffic": None,
                            "traffic_source": "no ncu capture at this size", "peak_source": peaks["source"],
                            "work_per_launch": work}
    return line


def run_accumulate_cases(args, which):
    import torch
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: libgear has no CPU path")
    from paper_1806_03925_b200 import microbench, workloads
    from paper_1806_03925_b200.workloads import MICRO_PRESETS, PRESETS, BatchSource
    peaks = measured_peaks()
    cases = []
    if which == "micro":
        for name, mp in MICRO_PRESETS.items():
            cases.append((name, workloads.micro_ids(mp, seed=0), mp.img_vocab, mp.dfv_dim, mp.M, "sort"))
    else:
        p = PRESETS["skew"]
        ids = BatchSource(p, 0).batch(0).img_id
        for M in (1, 64, 1024):
            for mode in ("sort", "atomic"):
                cases.append(("skew_M%d" % M, ids, p.img_vocab, p.dfv_dim, M, mode))
    for name, ids, V, D, M, mode in cases:
        sampler = ClockSampler(0)
        sampler.start()
        time.sleep(0.3)
        sampler.open_window()
        case = microbench._run_case(name, ids, V, D, M, mode, steps=max(args.steps, 5), warmup=max(args.warmup, 3))
        sampler.close_window()
        line = accumulate_line(case, args, sampler.stop(), peaks)
        if not args.no_cpu_baseline:
            sec, n_s = oracle_accumulate_sample(ids, V, D, M, 1 << 21)
            line["cpu_baseline"] = {"value": round(n_s / sec, 1), "unit": "gradient rows/s", "cores": 1, "kind": "oracle",
                                    "sample": "the first %d rows of the case through orc_accumulate and the hand-over, "
                                              "%.1f s of CPU time" % (n_s, sec)}
        print(json.dumps(line), flush=True)


# ---------------------------------------------------------------------------------------------
# tables partitioned by ID over the ranks (opt-in; the default multi-GPU arm runs independent replicas)
# ---------------------------------------------------------------------------------------------
def run_sharded(args):
    """Every rank owns the table rows whose ID is congruent to its rank and works on its own batch of the workload's
    size; IDs, rows and gradient rows cross between the ranks by all-to-all (NCCL).  A step includes the host->device
    copy of the batch's ID arrays, so the one figure reported is an end-to-end one."""
    import torch
    from paper_1806_03925_b200 import binding as gb, workloads
    from paper_1806_03925_b200.replicas import Replicas
    from paper_1806_03925_b200.sharded import DistExchange, ShardedGear
    from paper_1806_03925_b200.workloads import BatchSource
    reps = Replicas.from_env()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: libgear has no CPU path")
    torch.cuda.set_device(reps.local_rank)
    reps.init("nccl", torch.device("cuda", reps.local_rank))
    gb.load()
    p = preset_for(args.workload)
    K, W = args.steps, max(args.warmup, 3)
    sampler = ClockSampler(reps.local_rank)
    sampler.start()
    src = BatchSource(p, reps.rank)
    batches = [src.batch(s) for s in range(N_BATCHES)]
    sg = ShardedGear(p, workloads.head_params(p, 0), DistExchange(reps.rank, reps.world), max_batch_local=p.batch,
                     max_nnz_local=max(b.nnz for b in batches), seed=0)
    stream = torch.cuda.current_stream()
    now = [0]

    def one(s):
        now[0] += 1
        sg.step([batches[s % N_BATCHES]], now[0])

    for s in range(W):
        one(s)
    launches0 = sum(gb.gear_launch_count(x.ctx) for x in sg.owners + sg.workers)
    region_ms = []
    sampler.open_window()
    while (sum(region_ms) < args.min_timed_ms or len(region_ms) < 3) and len(region_ms) < MAX_REGIONS:
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize(); reps.barrier(); torch.cuda.synchronize()
        ev0.record(stream)
        for s in range(K):
            one(s)
        ev1.record(stream)
        torch.cuda.synchronize(); reps.barrier(); torch.cuda.synchronize()
        region_ms.append(reps.max_over_ranks(ev0.elapsed_time(ev1), device="cuda"))
    sampler.close_window()
    launches = (sum(gb.gear_launch_count(x.ctx) for x in sg.owners + sg.workers) - launches0) / len(region_ms)
    ms = float(np.median(region_ms))
    h2d = int(np.mean([b.user_id.nbytes + b.url_id.nbytes + b.img_id.nbytes + b.img_off.nbytes + b.label.nbytes for b in batches]))
    value = round(reps.whole_job_rate(p.batch * K, ms), 1)
    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": reps.world, "steps": K, "warmup": W,
            "ms_per_step": round(ms / K, 4), "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "bf16" if p.head_dtype == "bf16" else "f32", "data": "synthetic",
            "config": {"workload": "large tables" if p.name == "large" else p.name, "batch": p.batch,
                       "parallelism": "tables partitioned by ID over %d ranks, a batch per rank, three all-to-all "
                                      "exchanges per table and step" % reps.world,
                       "l2": "tables far exceed the 126 MB L2; %d pre-generated batches cycle" % N_BATCHES},
            "regions": {"regions": len(region_ms), "min_ms_per_step": round(min(region_ms) / K, 4),
                        "max_ms_per_step": round(max(region_ms) / K, 4)},
            "clocks": sampler.stop(), "gpu_launches": int(launches),
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": 16,
                    "note": "the timed step itself copies the batch in and reads the two counts back"},
            "roofline": None, "cpu_baseline": None,
            "device_status": [x.status()[1] for x in sg.owners + sg.workers]}
    if reps.rank == 0:
        print(json.dumps(line), flush=True)
    sg.close()
    reps.close()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=None)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="large", choices=["large", "large_2m", "medium", "tiny", "skew", "micro", "skew_modes"],
                    help="large (default): the configuration the metric is quoted on.  micro: the accumulate-only "
                         "micro-benchmark, one line per case.  skew: the skew-stress step.  skew_modes: its accumulate call, "
                         "sort against atomics, M in {1, 64, 1024}, one line per case")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--min-timed-ms", type=float, default=MIN_TIMED_MS,
                    help="device time to measure per arm: the K-step region is repeated until then (default 1000; a "
                         "profiler capture passes 0 to keep the run to three short regions)")
    ap.add_argument("--sharded", action="store_true",
                    help="tables partitioned by ID over the ranks instead of independent replicas (not the default: this "
                         "arm has only ever run on one GPU)")
    args = ap.parse_args()
    # defaults: a few hundred milliseconds of device time per timed region for the CUDA path (so that the
    # clock sampler sees it), a couple of minutes of host time for the CPU oracle
    if args.steps is None:
        args.steps = 400 if args.impl == "ours" else 20
    if args.warmup is None:
        args.warmup = 20 if args.impl == "ours" else 2
    if args.warmup < 3 and args.impl == "ours":
        args.warmup = 3
    if args.impl == "reference":
        if args.workload in ("micro", "skew_modes"):
            raise SystemExit("the reference arm times the whole step: use --workload large, medium, tiny or skew")
        run_reference(args)
    elif args.sharded:
        if args.steps == 400:
            args.steps = 50
        run_sharded(args)
    elif args.workload in ("micro", "skew_modes"):
        if args.steps == 400:
            args.steps = 7
        run_accumulate_cases(args, "micro" if args.workload == "micro" else "skew")
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
