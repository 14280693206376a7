"""Python access to the CPU oracle (oracle/gear_oracle.c).

TEST INFRASTRUCTURE ONLY: imported by the tests, the smoke check and the
benchmark's CPU-baseline leg.  The CUDA library and its binding never import
this package, and this package never imports them.

The wrapper only marshals numpy arrays into the C functions; every step of the
method is computed in gear_oracle.c.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from dataclasses import dataclass
from typing import Optional, Sequence, Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "gear_oracle.c")
_LIB = os.path.join(_HERE, "libgear_oracle.so")

ORC_F64, ORC_F32, ORC_BF16 = 0, 1, 2

# table tags of the procedural fill (the CUDA library documents the same numbers in its header)
TAG_USER, TAG_URL, TAG_DFV, TAG_TS, TAG_GRAD = 1, 2, 3, 4, 5
FILL_AMP = 0.17320508075688773   # uniform half-width giving standard deviation 0.1


def build(force: bool = False) -> str:
    """Compile the oracle with gcc -O2 into oracle/libgear_oracle.so."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".%d.tmp" % os.getpid()
        subprocess.check_call(["gcc", "-O2", "-std=c99", "-ffp-contract=off", "-shared", "-fPIC",
                               "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


class _Model(C.Structure):
    _fields_ = [("user_vocab", C.c_int64), ("url_vocab", C.c_int64), ("img_vocab", C.c_int64),
                ("emb_dim", C.c_int32), ("dfv_dim", C.c_int32), ("n_hidden", C.c_int32),
                ("hidden", C.c_int32 * 2), ("round_bf16", C.c_int32), ("fast_dim", C.c_int32)]


_lib = None


def lib():
    global _lib
    if _lib is None:
        L = C.CDLL(build())
        vp, i32, i64, u64, dbl = C.c_void_p, C.c_int32, C.c_int64, C.c_uint64, C.c_double
        L.orc_round_bf16.restype = dbl
        L.orc_round_bf16.argtypes = [dbl]
        L.orc_mix64.restype = u64
        L.orc_mix64.argtypes = [u64]
        L.orc_draw.restype = u64
        L.orc_draw.argtypes = [u64, u64, u64]
        L.orc_fill_rows.restype = C.c_int
        L.orc_fill_rows.argtypes = [u64, u64, i32, dbl, vp, i64, C.c_int, vp]
        L.orc_fill_ts.restype = C.c_int
        L.orc_fill_ts.argtypes = [u64, u64, i64, i64, vp, i64, vp]
        L.orc_head_param_count.restype = i64
        L.orc_head_param_count.argtypes = [C.POINTER(_Model)]
        L.orc_forward_backward.restype = i64
        L.orc_forward_backward.argtypes = [C.POINTER(_Model), vp, C.c_int, vp, C.c_int, vp, C.c_int, vp,
                                           i32, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp,
                                           dbl, dbl, vp, vp, i64, vp, vp, i64]
        L.orc_emb_apply.restype = i64
        L.orc_emb_apply.argtypes = [vp, C.c_int, i64, i32, vp, i32, vp, i32, i32, dbl, vp]
        L.orc_dfv_grad_rows.restype = None
        L.orc_dfv_grad_rows.argtypes = [i32, i32, vp, vp, i32, i32, vp]
        L.orc_accumulate.restype = i64
        L.orc_accumulate.argtypes = [vp, vp, vp, i64, i32, i32, vp, vp, i64, vp, vp, vp, i64, vp, vp]
        L.orc_accumulate_pooled.restype = i64
        L.orc_accumulate_pooled.argtypes = [vp, vp, vp, i64, i32, i32, vp, vp, i64, vp, vp, vp, i64, vp]
        L.orc_collect_ready.restype = None
        L.orc_collect_ready.argtypes = [vp, vp, i64]
        L.orc_collect_expired.restype = i64
        L.orc_collect_expired.argtypes = [vp, i64, i64, i64, C.c_int, vp]
        L.orc_refresh_dfv.restype = i64
        L.orc_refresh_dfv.argtypes = [vp, C.c_int, i64, i32, vp, i64, vp, vp, vp, i64, i64, i64]
        L.orc_dense_forward.restype = i64
        L.orc_dense_forward.argtypes = [vp, C.c_int, i64, i32, vp, i32, vp, i64, vp]
        L.orc_dense_backward.restype = i64
        L.orc_dense_backward.argtypes = [vp, C.c_int, i64, i32, i32, vp, vp, i64, vp]
        L.orc_adam_step.restype = None
        L.orc_adam_step.argtypes = [vp, vp, vp, vp, i64, i64, dbl, dbl, dbl, dbl]
        L.orc_emb_adam.restype = i64
        L.orc_emb_adam.argtypes = [vp, C.c_int, vp, vp, i64, i32, vp, i32, vp, i32, i32, i64, dbl, dbl, dbl, dbl]
        _lib = L
    return _lib


def _ptr(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _dtype_tag(a: np.ndarray) -> int:
    if a.dtype == np.float64:
        return ORC_F64
    if a.dtype == np.float32:
        return ORC_F32
    if a.dtype == np.uint16:
        return ORC_BF16
    raise TypeError("table dtype must be float64, float32 or uint16 (bf16 bits), got %s" % a.dtype)


def _c(a: np.ndarray, dtype) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=dtype)


def round_bf16(v: float) -> float:
    return lib().orc_round_bf16(float(v))


def draw(seed: int, tag: int, idx: int) -> int:
    return lib().orc_draw(seed, tag, idx)


def fill_rows(seed: int, tag: int, dim: int, rows: Optional[np.ndarray], n_rows: int,
              dtype=np.float32, amp: float = FILL_AMP) -> np.ndarray:
    """Rows of the procedural table (seed, tag); rows=None means rows 0..n_rows-1."""
    out = np.empty((n_rows, dim), dtype=dtype)
    r = None if rows is None else _c(rows, np.int64)
    lib().orc_fill_rows(seed, tag, dim, amp, _ptr(r), n_rows, _dtype_tag(out), _ptr(out))
    return out


def fill_ts(seed: int, expire: int, now: int, rows: Optional[np.ndarray], n_rows: int) -> np.ndarray:
    out = np.empty(n_rows, dtype=np.int64)
    r = None if rows is None else _c(rows, np.int64)
    lib().orc_fill_ts(seed, TAG_TS, expire, now, _ptr(r), n_rows, _ptr(out))
    return out


@dataclass
class StepResult:
    X: np.ndarray
    prob: Optional[np.ndarray]
    loss: float
    head_grad: Optional[np.ndarray]
    dX: Optional[np.ndarray]
    bad_ids: int
    near_units: Optional[np.ndarray] = None   # coded (layer * B + view) * 1024 + column
    near_abs: Optional[np.ndarray] = None     # |pre-activation| of each listed unit


def decode_unit(code: int, B: int) -> Tuple[int, int, int]:
    """(layer, view, column) of a unit code of forward_backward's near_units list."""
    j = int(code) % 1024
    lb = int(code) // 1024
    return lb // B, lb % B, j


class GearOracle:
    """State (tables, gradient store, timestamps) plus the oracle's calls.

    Tables are used in place in the dtype they are given in: float64 / float32
    arrays, or uint16 arrays holding bfloat16 bit patterns.
    """

    def __init__(self, user_emb: np.ndarray, url_emb: np.ndarray, dfv: np.ndarray,
                 hidden: Sequence[int], M: int, expire: int, round_bf16: bool = False,
                 ts: Optional[np.ndarray] = None, fast_dim: int = 0):
        """ts may be longer than the DFV table: a test that keeps only the touched rows of a huge
        table still scans every timestamp."""
        self.user_emb = np.ascontiguousarray(user_emb)
        self.url_emb = np.ascontiguousarray(url_emb)
        self.dfv = np.ascontiguousarray(dfv)
        self.E = int(self.user_emb.shape[1])
        self.D = int(self.dfv.shape[1])
        self.V = int(self.dfv.shape[0])
        self.hidden = tuple(int(h) for h in hidden)
        self.M = int(M)
        self.expire = int(expire)
        m = _Model()
        m.user_vocab, m.url_vocab, m.img_vocab = self.user_emb.shape[0], self.url_emb.shape[0], self.V
        m.emb_dim, m.dfv_dim = self.E, self.D
        m.n_hidden = len(self.hidden)
        for i, h in enumerate(self.hidden):
            m.hidden[i] = h
        m.round_bf16 = 1 if round_bf16 else 0
        m.fast_dim = self.F = int(fast_dim)
        self.model = m
        self.d_in = 2 * self.E + self.D + self.F
        self.n_params = int(lib().orc_head_param_count(C.byref(m)))
        self.gsum = np.zeros((self.V, self.D), dtype=np.float64)
        self.gcnt = np.zeros(self.V, dtype=np.int32)
        self.seq = np.zeros(self.V, dtype=np.int32)
        self.ts = np.zeros(self.V, dtype=np.int64) if ts is None else _c(ts, np.int64).copy()
        self._emit_id = np.zeros(0, dtype=np.int32)
        self._emit_seq = np.zeros(0, dtype=np.int32)
        self._emit_avg = np.zeros((0, self.D), dtype=np.float64)

    # -- events 1, 3, 4 -----------------------------------------------------
    def forward_backward(self, params: np.ndarray, user_id, url_id, img_off, img_id, label,
                         backward: bool = True, relu_margin: Optional[float] = None,
                         flip_units: Optional[Sequence[int]] = None, relu_margin_rel: float = 0.0,
                         near_cap: int = 65536, fast: Optional[np.ndarray] = None) -> StepResult:
        """relu_margin / relu_margin_rel: list the hidden units whose pre-activation a has
        |a| <= relu_margin + relu_margin_rel * max|input row| * max|layer weights| (None: no list)."""
        B = int(len(user_id))
        params = _c(params, np.float64)
        assert params.shape[0] == self.n_params
        uid, hid = _c(user_id, np.int32), _c(url_id, np.int32)
        off, img = _c(img_off, np.int32), _c(img_id, np.int32)
        y = _c(label, np.float64)
        fast64 = None
        if self.F:
            fast64 = _c(fast, np.float64)
            assert fast64.shape == (B, self.F)
        X = np.zeros((B, self.d_in), dtype=np.float64)
        prob = np.zeros(B, dtype=np.float64)
        loss = C.c_double(0.0)
        hg = np.zeros(self.n_params, dtype=np.float64) if backward else None
        dX = np.zeros((B, self.d_in), dtype=np.float64) if backward else None
        near = np.zeros(near_cap, dtype=np.int64) if relu_margin is not None else None
        near_abs = np.zeros(near_cap, dtype=np.float64) if relu_margin is not None else None
        n_near = C.c_int64(0)
        flips = _c(flip_units, np.int64) if flip_units is not None and len(flip_units) else None
        bad = lib().orc_forward_backward(
            C.byref(self.model), _ptr(self.user_emb), _dtype_tag(self.user_emb),
            _ptr(self.url_emb), _dtype_tag(self.url_emb), _ptr(self.dfv), _dtype_tag(self.dfv),
            _ptr(params), B, _ptr(uid), _ptr(hid), _ptr(off), _ptr(img), _ptr(y), _ptr(fast64),
            _ptr(X), _ptr(prob), C.byref(loss), _ptr(hg), _ptr(dX),
            0.0 if relu_margin is None else float(relu_margin), float(relu_margin_rel), _ptr(near), _ptr(near_abs),
            0 if near is None else len(near), C.byref(n_near), _ptr(flips), 0 if flips is None else len(flips))
        if near is not None:
            assert n_near.value <= len(near), "near-zero unit list overflowed"
            near = near[:n_near.value].copy()
            near_abs = near_abs[:n_near.value].copy()
        return StepResult(X, prob, loss.value, hg, dX, int(bad), near, near_abs)

    def emb_grad(self, which: str, ids, dX: np.ndarray) -> np.ndarray:
        """Dense summed gradient G[vocab, E] of one embedding table."""
        table, col0 = (self.user_emb, 0) if which == "user" else (self.url_emb, self.E)
        G = np.zeros((table.shape[0], self.E), dtype=np.float64)
        ids = _c(ids, np.int32)
        dX = _c(dX, np.float64)
        lib().orc_emb_apply(None, 0, table.shape[0], self.E, _ptr(ids), len(ids), _ptr(dX),
                            dX.shape[1], col0, 0.0, _ptr(G))
        return G

    def emb_apply(self, which: str, ids, dX: np.ndarray, alpha: float) -> int:
        """table[id] += alpha * G[id] in place."""
        table, col0 = (self.user_emb, 0) if which == "user" else (self.url_emb, self.E)
        ids = _c(ids, np.int32)
        dX = _c(dX, np.float64)
        return int(lib().orc_emb_apply(_ptr(table), _dtype_tag(table), table.shape[0], self.E, _ptr(ids),
                                       len(ids), _ptr(dX), dX.shape[1], col0, float(alpha), None))

    # -- event 5 --------------------------------------------------------------
    def dfv_grad_rows(self, img_off, dX: np.ndarray) -> np.ndarray:
        off = _c(img_off, np.int32)
        dX = _c(dX, np.float64)
        B = len(off) - 1
        rows = np.zeros((int(off[-1]), self.D), dtype=np.float64)
        lib().orc_dfv_grad_rows(B, self.D, _ptr(off), _ptr(dX), dX.shape[1], 2 * self.E, _ptr(rows))
        return rows

    # -- event 6 --------------------------------------------------------------
    def accumulate(self, img_id, grads: np.ndarray, want_members: bool = False, pooled: bool = False):
        """pooled: the order-free store (orc_accumulate_pooled): emissions carry the mean of all
        gradients pooled for the image."""
        ids = _c(img_id, np.int32)
        g = _c(grads, np.float64)
        n = len(ids)
        assert g.shape == (n, self.D)
        n0 = len(self._emit_id)
        # room for the emissions this call can add: every emission takes M arrivals, old (still open) or new
        cap = n0 + (n + int(self.gcnt.sum(dtype=np.int64))) // self.M + 1
        eid = np.zeros(cap, dtype=np.int32); eid[:n0] = self._emit_id
        eseq = np.zeros(cap, dtype=np.int32); eseq[:n0] = self._emit_seq
        eavg = np.zeros((cap, self.D), dtype=np.float64); eavg[:n0] = self._emit_avg
        n_emit = C.c_int64(n0)
        members = np.zeros(n, dtype=np.int64) if want_members else None
        if pooled:
            assert not want_members
            bad = lib().orc_accumulate_pooled(_ptr(self.gsum), _ptr(self.gcnt), _ptr(self.seq), self.V, self.D,
                                              self.M, _ptr(ids), _ptr(g), n, _ptr(eid), _ptr(eseq), _ptr(eavg), cap,
                                              C.byref(n_emit))
        else:
            bad = lib().orc_accumulate(_ptr(self.gsum), _ptr(self.gcnt), _ptr(self.seq), self.V, self.D, self.M,
                                       _ptr(ids), _ptr(g), n, _ptr(eid), _ptr(eseq), _ptr(eavg), cap,
                                       C.byref(n_emit), _ptr(members))
        assert bad >= 0
        k = n_emit.value
        self._emit_id, self._emit_seq, self._emit_avg = eid[:k], eseq[:k], eavg[:k]
        return (int(bad), members) if want_members else int(bad)

    @property
    def pending_ready(self) -> int:
        return len(self._emit_id)

    def collect_ready(self) -> Tuple[np.ndarray, np.ndarray, np.ndarray]:
        """(ids, seq, avg) in emission order; clears the list."""
        out = (self._emit_id.copy(), self._emit_seq.copy(), self._emit_avg.copy())
        lib().orc_collect_ready(_ptr(self.seq), _ptr(self._emit_id), len(self._emit_id))
        self._emit_id = np.zeros(0, dtype=np.int32)
        self._emit_seq = np.zeros(0, dtype=np.int32)
        self._emit_avg = np.zeros((0, self.D), dtype=np.float64)
        return out

    # -- expiry -----------------------------------------------------------------
    def collect_expired(self, now: int, restamp: bool = True) -> np.ndarray:
        out = np.zeros(len(self.ts), dtype=np.int32)
        n = lib().orc_collect_expired(_ptr(self.ts), len(self.ts), int(now), self.expire, 1 if restamp else 0,
                                      _ptr(out))
        return out[:n].copy()


    # -- refresh of cached inference results ----------------------------------------
    def refresh_dfv(self, ids, rows: np.ndarray, now: int, ts_ids=None) -> int:
        """Stores rows[k] (fp32) as the cached DFV of image ids[k], rounded to the table's dtype, and stamps the
        image with now.  ts_ids: index into the timestamp array where it differs from the table row (see __init__).
        Returns the number of skipped (out-of-range) IDs."""
        ids = _c(np.asarray(ids), np.int32)
        rows = _c(np.asarray(rows), np.float32)
        assert rows.ndim == 2 and rows.shape[0] == len(ids) and rows.shape[1] == self.D
        tid = None if ts_ids is None else _c(np.asarray(ts_ids), np.int32)
        return int(lib().orc_refresh_dfv(_ptr(self.dfv), _dtype_tag(self.dfv), self.V, self.D, _ptr(self.ts), len(self.ts),
                                         _ptr(ids), _ptr(tid), _ptr(rows), rows.shape[1], len(ids), int(now)))


# -- a linear Dense Part and the optimiser ------------------------------------------
def dense_forward(raw: np.ndarray, Wd: np.ndarray, ids) -> np.ndarray:
    """DFV rows raw[ids] . Wd of a linear Dense Part (raw in its storage type, Wd float64 [R][D])."""
    raw = np.ascontiguousarray(raw)
    Wd = _c(Wd, np.float64)
    ids = _c(np.asarray(ids), np.int32)
    rows = np.zeros((len(ids), Wd.shape[1]), dtype=np.float64)
    lib().orc_dense_forward(_ptr(raw), _dtype_tag(raw), raw.shape[0], raw.shape[1], _ptr(Wd), Wd.shape[1], _ptr(ids),
                            len(ids), _ptr(rows))
    return rows


def dense_backward(raw: np.ndarray, ids, avg: np.ndarray) -> np.ndarray:
    """dLoss/dWd [R][D] of a linear Dense Part from the emitted (id, averaged gradient) pairs."""
    raw = np.ascontiguousarray(raw)
    ids = _c(np.asarray(ids), np.int32)
    avg = _c(avg, np.float64)
    G = np.zeros((raw.shape[1], avg.shape[1] if avg.ndim == 2 else 0), dtype=np.float64)
    lib().orc_dense_backward(_ptr(raw), _dtype_tag(raw), raw.shape[0], raw.shape[1], G.shape[1], _ptr(ids), _ptr(avg),
                             len(ids), _ptr(G))
    return G


@dataclass
class AdamConfig:
    lr: float = 1e-4          # the paper's learning rate
    beta1: float = 0.9
    beta2: float = 0.999
    eps: float = 1e-8


def adam_step(p: np.ndarray, g: np.ndarray, m: np.ndarray, v: np.ndarray, t: int, cfg: AdamConfig) -> None:
    """In place on float64 arrays of equal size."""
    for a in (p, g, m, v):
        assert a.dtype == np.float64 and a.flags.c_contiguous and a.size == p.size
    lib().orc_adam_step(_ptr(p), _ptr(g), _ptr(m), _ptr(v), p.size, int(t), cfg.lr, cfg.beta1, cfg.beta2, cfg.eps)


def emb_adam(table: np.ndarray, m: np.ndarray, v: np.ndarray, ids, dX: np.ndarray, col0: int, t: int,
             cfg: AdamConfig) -> int:
    """Adam on the rows of an embedding table that received a gradient (in place; m, v float64 [vocab][E])."""
    ids = _c(np.asarray(ids), np.int32)
    dX = _c(dX, np.float64)
    assert table.flags.c_contiguous and m.dtype == np.float64 and v.dtype == np.float64
    return int(lib().orc_emb_adam(_ptr(table), _dtype_tag(table), _ptr(m), _ptr(v), table.shape[0], table.shape[1],
                                  _ptr(ids), len(ids), _ptr(dX), dX.shape[1], col0, int(t), cfg.lr, cfg.beta1,
                                  cfg.beta2, cfg.eps))


def sort_emissions(ids: np.ndarray, seq: np.ndarray, avg: np.ndarray):
    """Emission order is arrival order, which the paper leaves arbitrary;
    comparisons are made after sorting by (id, seq)."""
    order = np.lexsort((seq, ids))
    return ids[order], seq[order], avg[order]
