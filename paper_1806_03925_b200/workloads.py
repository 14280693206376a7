"""Seeded synthetic page-view workloads for the Gear Training sparse-part step.

This module only *draws inputs*: page-view records (User ID, URL-hash ID and a
ragged list of Image IDs per view, as in the paper's Table 1), labels, head
parameters and timestamps.  It contains none of the method's arithmetic and is
the one module that both the CPU oracle's tests and the CUDA path's tests and
benchmark may import.  It depends on numpy only.

The paper's production page views are not public, so the presets below stand
in for them shape-wise: few IDs per view, far fewer images than views (paper,
Conclusion), hence heavy ID reuse, modelled as Zipf-distributed IDs.

All random draws come from numpy's counter-based Philox generator keyed by
(seed, stream, step), so that any batch can be regenerated on its own.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field, replace
from typing import Dict, Optional, Tuple

import numpy as np

F32 = "f32"
BF16 = "bf16"

# Philox stream tags (one independent stream per kind of draw).
_STREAM_BATCH = 1
_STREAM_PARAMS = 2
_STREAM_TS = 3
_STREAM_MICRO = 4


@dataclass(frozen=True)
class GearPreset:
    """Shapes and distributions of one workload configuration."""
    name: str
    batch: int
    steps: int
    user_vocab: int
    url_vocab: int
    img_vocab: int
    emb_dim: int
    dfv_dim: int
    dfv_dtype: str            # storage type of the DFV table
    head_dtype: str           # arithmetic type of the head GEMM operands
    hidden: Tuple[int, ...]   # hidden layer widths; output layer is always 1 logistic unit
    M: int                    # gradients per image before one averaged emission
    expire: int               # inference-expired time, in steps
    zipf_user: float
    zipf_url: float
    zipf_img: float
    img_dist: str             # "uniform" or "poisson"
    img_lo: int
    img_hi: int
    img_lambda: float = 0.0
    label_rate: float = 0.05
    lr: float = 0.05
    fast_dim: int = 0         # dense input columns a view brings itself (the Fastgear side's share of the image)

    @property
    def d_in(self) -> int:
        return 2 * self.emb_dim + self.dfv_dim + self.fast_dim

    @property
    def n_params(self) -> int:
        n, fan_in = 0, self.d_in
        for h in self.hidden:
            n += fan_in * h + h
            fan_in = h
        return n + fan_in + 1

    def scaled(self, **kw) -> "GearPreset":
        return replace(self, **kw)


PRESETS: Dict[str, GearPreset] = {
    "tiny": GearPreset(
        name="tiny", batch=256, steps=16, user_vocab=10_000, url_vocab=10_000, img_vocab=5_000,
        emb_dim=16, dfv_dim=64, dfv_dtype=F32, head_dtype=F32, hidden=(64,), M=4, expire=1000,
        zipf_user=1.1, zipf_url=1.1, zipf_img=1.1, img_dist="uniform", img_lo=1, img_hi=4),
    "medium": GearPreset(
        name="medium", batch=4096, steps=200, user_vocab=1_000_000, url_vocab=1_000_000,
        img_vocab=1_000_000, emb_dim=32, dfv_dim=128, dfv_dtype=BF16, head_dtype=BF16,
        hidden=(256, 128), M=16, expire=100,
        zipf_user=1.05, zipf_url=1.05, zipf_img=1.05, img_dist="poisson", img_lo=1, img_hi=8,
        img_lambda=3.0),
    "large": GearPreset(
        name="large", batch=65536, steps=30, user_vocab=50_000_000, url_vocab=20_000_000,
        img_vocab=20_000_000, emb_dim=64, dfv_dim=256, dfv_dtype=BF16, head_dtype=BF16,
        hidden=(512, 256), M=32, expire=100,
        zipf_user=1.05, zipf_url=1.05, zipf_img=1.05, img_dist="poisson", img_lo=1, img_hi=16,
        img_lambda=4.0),
    # the large-table shapes on tables of a few GB: the case profiler captures run on
    "large_2m": GearPreset(
        name="large_2m", batch=65536, steps=30, user_vocab=4_000_000, url_vocab=2_000_000,
        img_vocab=2_000_000, emb_dim=64, dfv_dim=256, dfv_dtype=BF16, head_dtype=BF16,
        hidden=(512, 256), M=32, expire=100,
        zipf_user=1.05, zipf_url=1.05, zipf_img=1.05, img_dist="poisson", img_lo=1, img_hi=16,
        img_lambda=4.0),
    # the shape of the paper's CIFAR100 experiment (Section 4): every 32x32x3 image is cut in two, the top half
    # (16x32x3 = 1536 values) goes to the Fastgear side as a dense input of its own, the bottom half is the Slowgear
    # side's image (one image per view, its DFV cached).  Values are synthetic.
    "split_image": GearPreset(
        name="split_image", batch=1024, steps=8, user_vocab=10_000, url_vocab=10_000, img_vocab=50_000,
        emb_dim=16, dfv_dim=64, dfv_dtype=F32, head_dtype=F32, hidden=(256, 64), M=4, expire=20,
        zipf_user=1.1, zipf_url=1.1, zipf_img=1.05, img_dist="uniform", img_lo=1, img_hi=1, fast_dim=1536),
    "skew": GearPreset(
        name="skew", batch=32768, steps=30, user_vocab=1_000_000, url_vocab=1_000_000,
        img_vocab=4_000_000, emb_dim=32, dfv_dim=128, dfv_dtype=F32, head_dtype=F32,
        hidden=(256, 128), M=64, expire=10,
        zipf_user=1.05, zipf_url=1.05, zipf_img=1.3, img_dist="poisson", img_lo=1, img_hi=8,
        img_lambda=3.0),
}


@dataclass(frozen=True)
class MicroPreset:
    """Accumulate-only micro-benchmark: n gradient rows into a sum+count table."""
    name: str
    n_rows: int
    img_vocab: int
    dfv_dim: int
    M: int
    zipf_s: float             # 0.0 = uniform IDs


MICRO_PRESETS: Dict[str, MicroPreset] = {
    "micro_uniform_m8": MicroPreset("micro_uniform_m8", 1 << 24, 1 << 22, 128, 8, 0.0),
    "micro_uniform_m64": MicroPreset("micro_uniform_m64", 1 << 24, 1 << 22, 128, 64, 0.0),
    "micro_zipf_m8": MicroPreset("micro_zipf_m8", 1 << 24, 1 << 22, 128, 8, 1.1),
    "micro_zipf_m64": MicroPreset("micro_zipf_m64", 1 << 24, 1 << 22, 128, 64, 1.1),
}


def _rng(seed: int, stream: int, step: int = 0) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(key=[seed & (2**64 - 1), stream], counter=[step, 0, 0, 0]))


def _coprime_multiplier(vocab: int) -> int:
    """An odd multiplier near vocab/golden-ratio that is coprime to vocab."""
    a = int(vocab * 0.6180339887498949) | 1
    while math.gcd(a, vocab) != 1:
        a += 2
    return a


class ZipfIds:
    """Zipf(s) over ranks 1..V by inverse CDF; rank r is mapped to the ID
    (r * a + c) mod V with a coprime to V, so that hot rows are scattered over
    the table rather than packed at its start.  s == 0 gives uniform IDs."""

    def __init__(self, vocab: int, s: float, scatter: bool = True):
        self.vocab = int(vocab)
        self.s = float(s)
        self.a = _coprime_multiplier(self.vocab) if scatter else 1
        self.c = (self.vocab // 3) if scatter else 0
        self._cdf: Optional[np.ndarray] = None

    def _table(self) -> np.ndarray:
        if self._cdf is None:
            w = np.arange(1, self.vocab + 1, dtype=np.float64)
            np.power(w, -self.s, out=w)
            np.cumsum(w, out=w)
            w /= w[-1]
            self._cdf = w
        return self._cdf

    def rank_to_id(self, rank0: np.ndarray) -> np.ndarray:
        return ((rank0.astype(np.int64) * self.a + self.c) % self.vocab).astype(np.int32)

    def sample(self, rng: np.random.Generator, n: int) -> np.ndarray:
        if self.s == 0.0:
            return rng.integers(0, self.vocab, size=n, dtype=np.int64).astype(np.int32)
        u = rng.random(n)
        rank0 = np.searchsorted(self._table(), u, side="left")
        np.minimum(rank0, self.vocab - 1, out=rank0)
        return self.rank_to_id(rank0)


@dataclass
class Batch:
    """One batch of page views in CSR form."""
    user_id: np.ndarray   # int32 [B]
    url_id: np.ndarray    # int32 [B]
    img_off: np.ndarray   # int32 [B+1], img_off[0] == 0, non-decreasing
    img_id: np.ndarray    # int32 [nnz]
    label: np.ndarray     # float32 [B], 0.0 or 1.0
    fast: Optional[np.ndarray] = None   # float32 [B, fast_dim]: the views' own dense input (presets with fast_dim > 0)

    @property
    def B(self) -> int:
        return int(self.user_id.shape[0])

    @property
    def nnz(self) -> int:
        return int(self.img_id.shape[0])


class BatchSource:
    """Draws the batches of one preset; batch k depends on (seed, k) only."""

    def __init__(self, preset: GearPreset, seed: int = 0, scatter: bool = True):
        self.p = preset
        self.seed = seed
        self.users = ZipfIds(preset.user_vocab, preset.zipf_user, scatter)
        self.urls = ZipfIds(preset.url_vocab, preset.zipf_url, scatter)
        self.imgs = ZipfIds(preset.img_vocab, preset.zipf_img, scatter)

    def images_per_view(self, rng: np.random.Generator, B: int) -> np.ndarray:
        p = self.p
        if p.img_dist == "uniform":
            n = rng.integers(p.img_lo, p.img_hi + 1, size=B)
        elif p.img_dist == "poisson":
            n = np.clip(rng.poisson(p.img_lambda, size=B), p.img_lo, p.img_hi)
        else:
            raise ValueError(p.img_dist)
        return n.astype(np.int64)

    def batch(self, step: int, B: Optional[int] = None) -> Batch:
        p = self.p
        B = p.batch if B is None else B
        rng = _rng(self.seed, _STREAM_BATCH, step)
        n = self.images_per_view(rng, B)
        off = np.zeros(B + 1, dtype=np.int64)
        np.cumsum(n, out=off[1:])
        nnz = int(off[-1])
        return Batch(
            user_id=self.users.sample(rng, B),
            url_id=self.urls.sample(rng, B),
            img_off=off.astype(np.int32),
            img_id=self.imgs.sample(rng, nnz),
            label=(rng.random(B) < p.label_rate).astype(np.float32),
            fast=(rng.random((B, p.fast_dim), dtype=np.float32) - 0.5) if p.fast_dim > 0 else None,   # "pixels" in [-0.5, 0.5)
        )


def head_params(preset: GearPreset, seed: int = 0) -> np.ndarray:
    """Packed fp32 head parameters: for each hidden layer W[in, out] row-major
    then b[out]; then the output weights w[in] and the output bias.  Weights
    are uniform with standard deviation 1/sqrt(fan_in) (the paper's 0.1 for
    all variables would saturate the wide layers); biases start at zero."""
    rng = _rng(seed, _STREAM_PARAMS)
    parts, fan_in = [], preset.d_in
    for h in tuple(preset.hidden) + (1,):
        a = math.sqrt(3.0 / fan_in)
        parts.append(rng.uniform(-a, a, size=fan_in * h).astype(np.float32))
        parts.append(np.zeros(h, dtype=np.float32))
        fan_in = h
    return np.concatenate(parts)


def timestamps(img_vocab: int, expire: int, seed: int = 0, now: int = 0) -> np.ndarray:
    """Uniform integer timestamps in {now-expire+1 .. now}: with restamping,
    about 1/expire of the images expire at every step."""
    rng = _rng(seed, _STREAM_TS)
    span = max(int(expire), 1)
    return (now - rng.integers(0, span, size=img_vocab, dtype=np.int64)).astype(np.int64)


def random_table(rows: int, dim: int, seed: int, stream: int, std: float = 0.1) -> np.ndarray:
    """A small dense fp32 table, uniform with the given standard deviation
    (the paper initialises all variables with standard deviation 0.1)."""
    rng = _rng(seed, 100 + stream)
    a = std * math.sqrt(3.0)
    return rng.uniform(-a, a, size=(rows, dim)).astype(np.float32)


def micro_ids(preset: MicroPreset, seed: int = 0, n_rows: Optional[int] = None,
              img_vocab: Optional[int] = None) -> np.ndarray:
    """Image IDs of the accumulate-only micro-benchmark (uniform or Zipf)."""
    n = preset.n_rows if n_rows is None else n_rows
    v = preset.img_vocab if img_vocab is None else img_vocab
    rng = _rng(seed, _STREAM_MICRO)
    return ZipfIds(v, preset.zipf_s).sample(rng, n)


def float_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round-to-nearest-even fp32 -> bf16, returned as uint16 bit patterns
    (a storage conversion for host-built input tables, not model arithmetic)."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    bias = ((u >> 16) & 1) + np.uint32(0x7FFF)
    return ((u + bias) >> 16).astype(np.uint16)


def bf16_bits_to_float(b: np.ndarray) -> np.ndarray:
    return (b.astype(np.uint32) << 16).view(np.float32)
