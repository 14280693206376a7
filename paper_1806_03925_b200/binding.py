"""ctypes binding of libgear.so (C ABI in include/gear.h).

Argument marshalling only: every step of the method runs in the CUDA kernels
behind the C calls.  PyTorch is used for device memory and streams.  There is
no CPU fallback: loading fails loudly when the library has not been built, and
every call raises on a non-zero return code.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Sequence

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libgear.so")

GEAR_OK, GEAR_ERR_ARG, GEAR_ERR_CAPACITY, GEAR_ERR_BAD_ID, GEAR_ERR_CUDA, GEAR_ERR_STATE = 0, -1, -2, -3, -4, -5
GEAR_F32, GEAR_BF16 = 0, 1
GEAR_ACC_SORT, GEAR_ACC_ATOMIC = 0, 1
GEAR_DEV_BAD_ID, GEAR_DEV_READY_OVERFLOW, GEAR_DEV_OUT_CAPACITY, GEAR_DEV_BAD_CSR = 1, 2, 4, 8
GEAR_TAG_USER, GEAR_TAG_URL, GEAR_TAG_DFV, GEAR_TAG_TS, GEAR_TAG_GRAD = 1, 2, 3, 4, 5
GEAR_TABLE_USER, GEAR_TABLE_URL, GEAR_TABLE_DFV = 0, 1, 2

EXPORTS = ("gear_workspace_bytes", "gear_init_tables", "gear_forward_backward", "gear_accumulate_dfv_grad",
           "gear_collect_ready", "gear_collect_expired", "gear_status", "gear_destroy", "gear_fill_uniform",
           "gear_last_error", "gear_profile_enable", "gear_profile_read", "gear_launch_count",
           "gear_collect_expired_static", "gear_refresh_dfv", "gear_accumulate_collect", "gear_dense_forward",
           "gear_dense_backward", "gear_adam_dense", "gear_fetch_rows", "gear_apply_emb_grad", "gear_profile_timeline")
GEAR_STATIC_EXPIRY_MAX_VOCAB = 16777216


class GearError(RuntimeError):
    def __init__(self, code: int, where: str, detail: str = ""):
        super().__init__("%s failed with code %d%s" % (where, code, (": " + detail) if detail else ""))
        self.code = code


class gear_config(C.Structure):
    _fields_ = [("user_vocab", C.c_int64), ("url_vocab", C.c_int64), ("img_vocab", C.c_int64),
                ("emb_dim", C.c_int32), ("dfv_dim", C.c_int32), ("dfv_dtype", C.c_int32), ("head_dtype", C.c_int32),
                ("n_hidden", C.c_int32), ("hidden", C.c_int32 * 2), ("M", C.c_int32), ("expire", C.c_int64),
                ("max_batch", C.c_int32), ("max_nnz", C.c_int64), ("ready_cap", C.c_int64), ("accum_mode", C.c_int32),
                ("fast_dim", C.c_int32)]


class gear_buffers(C.Structure):
    _fields_ = [("user_emb", C.c_void_p), ("url_emb", C.c_void_p), ("dfv", C.c_void_p), ("dfv_gsum", C.c_void_p),
                ("dfv_gcnt", C.c_void_p), ("dfv_ts", C.c_void_p), ("head_params", C.c_void_p),
                ("workspace", C.c_void_p), ("workspace_bytes", C.c_size_t)]


class gear_batch(C.Structure):
    _fields_ = [("B", C.c_int32), ("nnz", C.c_int64), ("user_id", C.c_void_p), ("url_id", C.c_void_p),
                ("img_off", C.c_void_p), ("img_id", C.c_void_p), ("label", C.c_void_p), ("fast", C.c_void_p)]


class gear_adam(C.Structure):
    _fields_ = [("lr", C.c_float), ("beta1", C.c_float), ("beta2", C.c_float), ("eps", C.c_float)]


class gear_step_out(C.Structure):
    _fields_ = [("loss", C.c_void_p), ("prob", C.c_void_p), ("head_grad", C.c_void_p), ("dX", C.c_void_p),
                ("row_view", C.c_void_p), ("inv_n", C.c_void_p), ("x_debug", C.c_void_p), ("dfv_grad", C.c_void_p),
                ("user_grad", C.c_void_p), ("url_grad", C.c_void_p),
                ("adam", C.POINTER(gear_adam)), ("adam_step", C.c_int64),
                ("user_m", C.c_void_p), ("user_v", C.c_void_p), ("url_m", C.c_void_p), ("url_v", C.c_void_p)]


_lib = None


def load() -> C.CDLL:
    """Load libgear.so (built by paper_1806_03925_b200.build).  Raises if it is missing."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise ImportError("libgear.so is not built: run `python -m paper_1806_03925_b200.build` "
                          "(needs nvcc); there is no CPU fallback")
    L = C.CDLL(LIB_PATH)
    vp, i32, i64, u64 = C.c_void_p, C.c_int32, C.c_int64, C.c_uint64
    L.gear_workspace_bytes.restype = C.c_int
    L.gear_workspace_bytes.argtypes = [C.POINTER(gear_config), C.POINTER(C.c_size_t)]
    L.gear_init_tables.restype = C.c_int
    L.gear_init_tables.argtypes = [C.POINTER(vp), C.POINTER(gear_config), C.POINTER(gear_buffers), u64, C.c_int,
                                   i64, vp]
    L.gear_forward_backward.restype = C.c_int
    L.gear_forward_backward.argtypes = [vp, C.POINTER(gear_batch), C.c_float, C.POINTER(gear_step_out), vp]
    L.gear_accumulate_dfv_grad.restype = C.c_int
    L.gear_accumulate_dfv_grad.argtypes = [vp, vp, vp, i64, vp, vp, i64, vp]
    L.gear_collect_ready.restype = C.c_int
    L.gear_collect_ready.argtypes = [vp, vp, vp, vp, i64, vp, C.POINTER(i64), vp]
    L.gear_accumulate_collect.restype = C.c_int
    L.gear_accumulate_collect.argtypes = [vp, vp, vp, i64, vp, vp, i64, vp, vp, vp, i64, vp, C.POINTER(i64), vp]
    L.gear_fetch_rows.restype = C.c_int
    L.gear_fetch_rows.argtypes = [vp, i32, vp, i64, vp, vp]
    L.gear_apply_emb_grad.restype = C.c_int
    L.gear_apply_emb_grad.argtypes = [vp, i32, vp, vp, i64, i64, C.c_float, vp]
    L.gear_dense_forward.restype = C.c_int
    L.gear_dense_forward.argtypes = [vp, vp, i32, vp, vp, i64, vp, vp, i64, vp]
    L.gear_dense_backward.restype = C.c_int
    L.gear_dense_backward.argtypes = [vp, vp, i32, vp, vp, i64, vp, vp, vp]
    L.gear_adam_dense.restype = C.c_int
    L.gear_adam_dense.argtypes = [vp, vp, vp, vp, i64, i64, C.POINTER(gear_adam), vp]
    L.gear_collect_expired.restype = C.c_int
    L.gear_collect_expired.argtypes = [vp, i64, C.c_int, vp, i64, vp, C.POINTER(i64), vp]
    L.gear_status.restype = C.c_int
    L.gear_refresh_dfv.restype = C.c_int
    L.gear_refresh_dfv.argtypes = [vp, vp, vp, i64, i64, vp, i64, vp]
    L.gear_status.argtypes = [vp, C.POINTER(i32), C.POINTER(i64)]
    L.gear_destroy.restype = C.c_int
    L.gear_destroy.argtypes = [vp]
    L.gear_fill_uniform.restype = C.c_int
    L.gear_fill_uniform.argtypes = [vp, i32, i64, i32, u64, u64, C.c_double, vp]
    L.gear_profile_enable.restype = C.c_int
    L.gear_profile_enable.argtypes = [vp, C.c_int]
    L.gear_profile_read.restype = C.c_int
    L.gear_profile_read.argtypes = [vp, C.c_char_p, C.POINTER(C.c_float), C.POINTER(i32), i32, C.POINTER(i32)]
    L.gear_profile_timeline.restype = C.c_int
    L.gear_profile_timeline.argtypes = [vp, C.c_char_p, C.POINTER(C.c_float), C.POINTER(C.c_float), i32, C.POINTER(i32)]
    L.gear_launch_count.restype = C.c_int
    L.gear_launch_count.argtypes = [vp, C.POINTER(i64)]
    L.gear_collect_expired_static.restype = C.c_int
    L.gear_collect_expired_static.argtypes = [vp, i64, i64, i64, C.c_int, vp, i64, vp, C.POINTER(i64), vp]
    L.gear_last_error.restype = C.c_char_p
    L.gear_last_error.argtypes = []
    _lib = L
    return L


def _check(rc: int, where: str, allow: Sequence[int] = ()):
    if rc != GEAR_OK and rc not in allow:
        raise GearError(rc, where, load().gear_last_error().decode())
    return rc


def _p(t: Optional[torch.Tensor]):
    """Device pointer of a CUDA tensor (None -> NULL)."""
    if t is None:
        return None
    if not t.is_cuda:
        raise TypeError("libgear takes device memory; got a %s tensor" % t.device)
    if not t.is_contiguous():
        raise TypeError("libgear takes contiguous tensors")
    return C.c_void_p(t.data_ptr())


def _stream(stream: Optional[torch.cuda.Stream]):
    s = torch.cuda.current_stream() if stream is None else stream
    return C.c_void_p(s.cuda_stream)


def make_config(user_vocab, url_vocab, img_vocab, emb_dim, dfv_dim, dfv_dtype, head_dtype, hidden, M, expire,
                max_batch, max_nnz, ready_cap=0, accum_mode=GEAR_ACC_SORT, fast_dim=0) -> gear_config:
    c = gear_config()
    c.user_vocab, c.url_vocab, c.img_vocab = user_vocab, url_vocab, img_vocab
    c.emb_dim, c.dfv_dim, c.dfv_dtype, c.head_dtype = emb_dim, dfv_dim, dfv_dtype, head_dtype
    c.n_hidden = len(hidden)
    for i, h in enumerate(hidden):
        c.hidden[i] = h
    c.M, c.expire, c.max_batch, c.max_nnz, c.ready_cap, c.accum_mode = M, expire, max_batch, max_nnz, ready_cap, accum_mode
    c.fast_dim = fast_dim
    return c


# ---------------------------------------------------------------------------
# the C calls, same names, tensors in place of raw pointers
# ---------------------------------------------------------------------------
def gear_workspace_bytes(cfg: gear_config) -> int:
    n = C.c_size_t(0)
    _check(load().gear_workspace_bytes(C.byref(cfg), C.byref(n)), "gear_workspace_bytes")
    return n.value


def gear_fill_uniform(dst: torch.Tensor, seed: int, tag: int, amp: float = 0.17320508075688773, stream=None):
    assert dst.dim() == 2 and dst.dtype in (torch.float32, torch.bfloat16)
    dt = GEAR_BF16 if dst.dtype == torch.bfloat16 else GEAR_F32
    _check(load().gear_fill_uniform(_p(dst), dt, dst.shape[0], dst.shape[1], seed, tag, amp, _stream(stream)),
           "gear_fill_uniform")


def gear_init_tables(cfg: gear_config, user_emb, url_emb, dfv, dfv_gsum, dfv_gcnt, dfv_ts, head_params, workspace,
                     seed: int = 0, fill: bool = True, now: int = 0, stream=None) -> C.c_void_p:
    b = gear_buffers()
    b.user_emb, b.url_emb, b.dfv = user_emb.data_ptr(), url_emb.data_ptr(), dfv.data_ptr()
    b.dfv_gsum, b.dfv_gcnt, b.dfv_ts = dfv_gsum.data_ptr(), dfv_gcnt.data_ptr(), dfv_ts.data_ptr()
    b.head_params, b.workspace = head_params.data_ptr(), workspace.data_ptr()
    b.workspace_bytes = workspace.numel() * workspace.element_size()
    for t in (user_emb, url_emb, dfv, dfv_gsum, dfv_gcnt, dfv_ts, head_params, workspace):
        _p(t)
    ctx = C.c_void_p()
    _check(load().gear_init_tables(C.byref(ctx), C.byref(cfg), C.byref(b), seed, 1 if fill else 0, now,
                                   _stream(stream)), "gear_init_tables")
    return ctx


def make_batch(user_id, url_id, img_off, img_id, label, B: Optional[int] = None, nnz: Optional[int] = None,
               fast=None) -> gear_batch:
    """The C struct of a batch whose arrays are device tensors (a caller that reuses the tensors may keep it)."""
    bt = gear_batch()
    bt.B = int(user_id.shape[0]) if B is None else B
    bt.nnz = int(img_id.shape[0]) if nnz is None else nnz
    bt.user_id, bt.url_id, bt.img_off = _p(user_id).value, _p(url_id).value, _p(img_off).value
    bt.img_id, bt.label = _p(img_id).value, _p(label).value
    bt.fast = None if fast is None else _p(fast).value
    return bt


def make_adam(lr: float = 1e-4, beta1: float = 0.9, beta2: float = 0.999, eps: float = 1e-8) -> gear_adam:
    """The optimiser's constants (defaults: the paper's learning rate, Kingma and Ba's other constants)."""
    return gear_adam(lr, beta1, beta2, eps)


def make_step_out(loss, head_grad, dX, prob=None, row_view=None, inv_n=None, x_debug=None, user_grad=None,
                  url_grad=None, adam: Optional[gear_adam] = None, adam_step: int = 0, user_m=None, user_v=None,
                  url_m=None, url_v=None, dfv_grad=None) -> gear_step_out:
    o = gear_step_out()
    for name, t in (("loss", loss), ("prob", prob), ("head_grad", head_grad), ("dX", dX), ("row_view", row_view),
                    ("inv_n", inv_n), ("x_debug", x_debug), ("user_grad", user_grad), ("url_grad", url_grad),
                    ("dfv_grad", dfv_grad),
                    ("user_m", user_m), ("user_v", user_v), ("url_m", url_m), ("url_v", url_v)):
        setattr(o, name, None if t is None else _p(t).value)
    if adam is not None:
        o.adam = C.pointer(adam)
        o._adam_keepalive = adam
    o.adam_step = adam_step
    return o


def gear_forward_backward_structs(ctx, bt: gear_batch, lr: float, o: gear_step_out, stream=None):
    """gear_forward_backward on structs made by make_batch / make_step_out."""
    return _check(load().gear_forward_backward(ctx, C.byref(bt), lr, C.byref(o), _stream(stream)),
                  "gear_forward_backward")


def gear_forward_backward(ctx, user_id, url_id, img_off, img_id, label, lr: float, loss, head_grad, dX, prob=None,
                          row_view=None, inv_n=None, x_debug=None, user_grad=None, url_grad=None, stream=None,
                          B: Optional[int] = None, nnz: Optional[int] = None):
    bt = make_batch(user_id, url_id, img_off, img_id, label, B, nnz)
    o = make_step_out(loss, head_grad, dX, prob, row_view, inv_n, x_debug, user_grad, url_grad)
    return gear_forward_backward_structs(ctx, bt, lr, o, stream)


def gear_accumulate_dfv_grad(ctx, img_id, grads_ptr: int, ld: int, src_row, scale, n: int, stream=None):
    """grads_ptr is a raw device address so that a column offset into dX can be passed."""
    return _check(load().gear_accumulate_dfv_grad(ctx, _p(img_id), C.c_void_p(grads_ptr), ld, _p(src_row), _p(scale),
                                                  n, _stream(stream)), "gear_accumulate_dfv_grad")


def gear_collect_ready(ctx, ids, seq, avg, cap: int, d_n=None, sync: bool = True, stream=None) -> Optional[int]:
    """Returns the number of entries (raises GearError(GEAR_ERR_CAPACITY) if cap was too small)
    when sync is True, else None."""
    h = C.c_int64(-1)
    _check(load().gear_collect_ready(ctx, _p(ids), _p(seq), _p(avg), cap, _p(d_n), C.byref(h) if sync else None,
                                     _stream(stream)), "gear_collect_ready")
    return h.value if sync else None


def gear_accumulate_collect(ctx, img_id, grads_ptr: int, ld: int, src_row, scale, n: int, ids, seq, avg, cap: int,
                            d_n=None, sync: bool = True, stream=None) -> Optional[int]:
    """gear_accumulate_dfv_grad and gear_collect_ready as one call; returns the number of entries when sync."""
    h = C.c_int64(-1)
    _check(load().gear_accumulate_collect(ctx, _p(img_id), C.c_void_p(grads_ptr), ld, _p(src_row), _p(scale), n,
                                          _p(ids), _p(seq), _p(avg), cap, _p(d_n), C.byref(h) if sync else None,
                                          _stream(stream)), "gear_accumulate_collect")
    return h.value if sync else None


def gear_collect_expired(ctx, now: int, restamp: bool, ids, cap: int, d_n=None, sync: bool = True,
                         stream=None) -> Optional[int]:
    h = C.c_int64(-1)
    _check(load().gear_collect_expired(ctx, now, 1 if restamp else 0, _p(ids), cap, _p(d_n),
                                       C.byref(h) if sync else None, _stream(stream)), "gear_collect_expired")
    return h.value if sync else None


def gear_refresh_dfv(ctx, ids, rows, n: int, now: int, d_n=None, stream=None):
    """rows: fp32 [>= n][ld] device tensor (stride(0) = ld); processes min(n, *d_n) entries when d_n is given."""
    assert rows.is_cuda and rows.dtype == torch.float32 and rows.dim() == 2 and rows.stride(1) == 1
    _check(load().gear_refresh_dfv(ctx, _p(ids), C.c_void_p(rows.data_ptr()), rows.stride(0), n, _p(d_n), now, _stream(stream)),
           "gear_refresh_dfv")


def gear_fetch_rows(ctx, which: int, ids, n: int, out, stream=None):
    """out[k] = row ids[k] of table `which` (bit-exact copies, the table's storage type), k < n."""
    _check(load().gear_fetch_rows(ctx, which, _p(ids), n, _p(out), _stream(stream)), "gear_fetch_rows")


def gear_apply_emb_grad(ctx, which: int, ids, rows, n: int, lr: float, stream=None):
    """table[id] -= lr * sum of the rows that carry id (rows fp32 [>= n][ld])."""
    assert rows.dtype == torch.float32 and rows.stride(1) == 1
    _check(load().gear_apply_emb_grad(ctx, which, _p(ids), C.c_void_p(rows.data_ptr()), rows.stride(0), n, lr,
                                      _stream(stream)), "gear_apply_emb_grad")


def gear_dense_forward(ctx, raw, Wd, ids, n: int, rows, d_n=None, stream=None):
    """rows[k] = raw[ids[k]] . Wd for k < n (and k < *d_n); rows fp32 [>= n][ld]."""
    assert raw.dtype == torch.float32 and Wd.dtype == torch.float32 and rows.dtype == torch.float32 and rows.stride(1) == 1
    _check(load().gear_dense_forward(ctx, _p(raw), raw.shape[1], _p(Wd), _p(ids), n, _p(d_n), C.c_void_p(rows.data_ptr()),
                                     rows.stride(0), _stream(stream)), "gear_dense_forward")


def gear_dense_backward(ctx, raw, ids, avg, n: int, Wd_grad, d_n=None, stream=None):
    """Wd_grad[r][c] += sum_e raw[ids[e]][r] * avg[e][c] over the emissions e < n (and e < *d_n)."""
    assert raw.dtype == torch.float32 and avg.dtype == torch.float32 and Wd_grad.dtype == torch.float32
    _check(load().gear_dense_backward(ctx, _p(raw), raw.shape[1], _p(ids), _p(avg), n, _p(d_n), _p(Wd_grad),
                                      _stream(stream)), "gear_dense_backward")


def gear_adam_dense(param, grad, m, v, t: int, cfg: gear_adam, stream=None):
    n = param.numel()
    assert grad.numel() == n and m.numel() == n and v.numel() == n
    _check(load().gear_adam_dense(_p(param), _p(grad), _p(m), _p(v), n, t, C.byref(cfg), _stream(stream)),
           "gear_adam_dense")


def gear_status(ctx, raise_on_error: bool = False):
    """(return code, device status bits, pending ready count); synchronises."""
    st, pend = C.c_int32(0), C.c_int64(0)
    rc = load().gear_status(ctx, C.byref(st), C.byref(pend))
    if raise_on_error:
        _check(rc, "gear_status")
    return rc, st.value, pend.value


def gear_destroy(ctx):
    return _check(load().gear_destroy(ctx), "gear_destroy")


def gear_profile_enable(ctx, on):
    """on: False / True (every kernel alone on the caller's stream) / 2 (timeline mode: the side stream stays)."""
    return _check(load().gear_profile_enable(ctx, int(on)), "gear_profile_enable")


def gear_profile_timeline(ctx, cap: int = 256):
    """[(kernel name, start ms, stop ms)] of every launch since timeline mode was switched on; synchronises."""
    names = C.create_string_buffer(64 * cap)
    t0, t1 = (C.c_float * cap)(), (C.c_float * cap)()
    n = C.c_int32(0)
    _check(load().gear_profile_timeline(ctx, names, t0, t1, cap, C.byref(n)), "gear_profile_timeline")
    return [(names.raw[64 * k:64 * (k + 1)].split(b"\0", 1)[0].decode(), float(t0[k]), float(t1[k])) for k in range(n.value)]


def gear_profile_read(ctx, cap: int = 64):
    """{kernel name: (total ms, launches)} since the last read; synchronises."""
    names = C.create_string_buffer(64 * cap)
    ms = (C.c_float * cap)()
    cnt = (C.c_int32 * cap)()
    n = C.c_int32(0)
    _check(load().gear_profile_read(ctx, names, ms, cnt, cap, C.byref(n)), "gear_profile_read")
    out = {}
    for k in range(n.value):
        name = names.raw[64 * k:64 * (k + 1)].split(b"\0", 1)[0].decode()
        out[name] = (float(ms[k]), int(cnt[k]))
    return out


def gear_launch_count(ctx) -> int:
    n = C.c_int64(0)
    _check(load().gear_launch_count(ctx, C.byref(n)), "gear_launch_count")
    return n.value


def gear_collect_expired_static(dfv_ts, expire: int, now: int, restamp: bool, ids, cap: int, d_n=None,
                                sync: bool = True, stream=None, img_vocab: Optional[int] = None) -> Optional[int]:
    """The expiry scan without a ctx or workspace, for callers that may not allocate device memory: the
    scratch lives in a fixed array inside libgear (tables of at most GEAR_STATIC_EXPIRY_MAX_VOCAB entries).
    Returns the count when sync is True.  Raises GearError(GEAR_ERR_CAPACITY) for a table beyond that bound
    or a cap that is too small."""
    h = C.c_int64(-1)
    n = int(dfv_ts.shape[0]) if img_vocab is None else img_vocab
    rc = load().gear_collect_expired_static(_p(dfv_ts), n, expire, now, 1 if restamp else 0, _p(ids), cap, _p(d_n),
                                            C.byref(h) if sync else None, _stream(stream))
    if rc != GEAR_OK:
        raise GearError(rc, "gear_collect_expired_static")
    return h.value if sync else None
