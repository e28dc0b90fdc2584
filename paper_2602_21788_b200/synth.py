"""Seeded synthetic packed batches shaped like the heterogeneous-length workloads of the paper.

This module only draws numbers: sequence lengths, per-sequence context-parallel (CP) degrees and
N(0,1) tensors rounded to bf16.  It contains none of the method's arithmetic, so both the CPU
oracle's tests and the CUDA path's tests may feed on it.  The paper's datasets (Sec. 5.1,
Appendix A.1) are only characterised qualitatively there ("mostly short, a few several times
longer"); the five workloads below are synthetic stand-ins with that shape.

Everything is a pure function of (workload name, seed) through numpy's PCG64.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field

import numpy as np

__all__ = [
    "Workload", "make_workload", "WORKLOADS", "bf16_round", "bf16_bits_to_f32", "bf16_bits_to_f64",
    "normal_bf16", "reduced",
]


# --------------------------------------------------------------------------------------------
# bf16 helpers (storage conversions only)
# --------------------------------------------------------------------------------------------
def bf16_round(x32: np.ndarray) -> np.ndarray:
    """float32 array -> uint16 bf16 bit patterns, round-to-nearest-even (finite inputs)."""
    x32 = np.ascontiguousarray(x32, dtype=np.float32)
    u = x32.view(np.uint32)
    lsb = (u >> np.uint32(16)) & np.uint32(1)
    r = (u + np.uint32(0x7FFF) + lsb) >> np.uint32(16)
    return r.astype(np.uint16)


def bf16_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    return (bits.astype(np.uint32) << np.uint32(16)).view(np.float32)


def bf16_bits_to_f64(bits: np.ndarray) -> np.ndarray:
    return bf16_bits_to_f32(bits).astype(np.float64)


def normal_bf16(rng: np.random.Generator, shape, block_rows: int = 1 << 14) -> np.ndarray:
    """N(0,1) samples rounded to bf16, returned as uint16 bit patterns of the given shape.

    Drawn in row blocks so that very large tensors never need a float64 temporary.
    """
    shape = tuple(int(s) for s in shape)
    out = np.empty(shape, dtype=np.uint16)
    flat = out.reshape(shape[0], -1) if len(shape) > 1 else out.reshape(-1, 1)
    for r0 in range(0, flat.shape[0], block_rows):
        r1 = min(flat.shape[0], r0 + block_rows)
        blk = rng.standard_normal((r1 - r0, flat.shape[1]), dtype=np.float32)
        flat[r0:r1] = bf16_round(blk)
    return out


# --------------------------------------------------------------------------------------------
# workloads
# --------------------------------------------------------------------------------------------
@dataclass
class Workload:
    name: str
    seed: int
    seqlens: np.ndarray            # int32 [B]
    cp_degrees: np.ndarray         # int32 [B]
    hq: int
    hkv: int
    head_dim: int
    note: str = ""
    extra: dict = field(default_factory=dict)
    spans: list | None = None      # per sequence a list of (begin, end) bidirectional spans, or None (causal)

    @property
    def total_tokens(self) -> int:
        return int(self.seqlens.sum())

    @property
    def cu_seqlens(self) -> np.ndarray:
        cu = np.zeros(len(self.seqlens) + 1, dtype=np.int64)
        np.cumsum(self.seqlens, out=cu[1:])
        return cu

    @property
    def sum_sq(self) -> int:
        return int((self.seqlens.astype(np.int64) ** 2).sum())

    def flops_fwd(self) -> float:
        """Forward FLOPs by the headline accounting: 2 * sum L^2 * hq * D for a causal batch (4 * D per
        (query, key) pair over L^2 / 2 pairs); a span of m tokens adds its m(m-1)/2 pairs above the diagonal."""
        extra = sum((e - a) * (e - a - 1) // 2 for sp in (self.spans or []) for a, e in sp)
        return (2.0 * self.sum_sq + 4.0 * extra) * self.hq * self.head_dim

    @property
    def visible_pairs(self) -> int:
        """(query, key) pairs the mask keeps: L(L+1)/2 per sequence plus m(m-1)/2 per span of m tokens."""
        n = int((self.seqlens.astype(np.int64) * (self.seqlens.astype(np.int64) + 1) // 2).sum())
        for sp in self.spans or []:
            n += sum((e - a) * (e - a - 1) // 2 for a, e in sp)
        return n

    def flops_fwd_bwd(self) -> float:
        return 3.5 * self.flops_fwd()

    def device_tensors(self, with_do: bool = True):
        """The same distributions drawn on the current CUDA device by torch's seeded generator, as bf16
        tensors: for workloads whose host draw would take minutes (billions of values).  A pure
        function of (seed, shape) like `tensors`, but a different stream of numbers."""
        import torch
        g = torch.Generator(device="cuda")
        g.manual_seed(0xFC9 + 7919 * int(self.seed))
        T, D = self.total_tokens, self.head_dim
        mk = lambda h: torch.randn((T, h, D), dtype=torch.bfloat16, device="cuda", generator=g)
        out = (mk(self.hq), mk(self.hkv), mk(self.hkv))
        return out + (mk(self.hq),) if with_do else out

    def tensors(self, with_do: bool = True):
        """q[T,hq,D], k[T,hkv,D], v[T,hkv,D] (and dO[T,hq,D]) as bf16 bit patterns (uint16)."""
        rng = np.random.Generator(np.random.PCG64([self.seed, 0xFC9]))
        T = self.total_tokens
        q = normal_bf16(rng, (T, self.hq, self.head_dim))
        k = normal_bf16(rng, (T, self.hkv, self.head_dim))
        v = normal_bf16(rng, (T, self.hkv, self.head_dim))
        if not with_do:
            return q, k, v
        do = normal_bf16(rng, (T, self.hq, self.head_dim))
        return q, k, v, do


def _fill_to_total(draw, total: int, min_len: int, first=()):
    """Draw lengths until the remainder is below ``min_len``; the last draw absorbs it."""
    lens = [int(x) for x in first]
    remaining = total - sum(lens)
    assert remaining >= 0
    i = 0
    while remaining >= min_len:
        L = int(draw(i))
        i += 1
        L = min(L, remaining)
        lens.append(L)
        remaining -= L
    if remaining > 0:
        lens[-1] += remaining
    return np.asarray(lens, dtype=np.int32)


def _tiny(rng):
    lens = rng.integers(64, 1025, size=8).astype(np.int32)
    deg = rng.integers(1, 4, size=8).astype(np.int32)
    return lens, deg, dict(hq=4, hkv=4, head_dim=64)


def _llama8b_64k(rng):
    mu, sigma = math.log(2048.0), 1.0

    def draw(_i):
        return int(np.clip(round(float(rng.lognormal(mu, sigma))), 128, 32768))

    lens = _fill_to_total(draw, 65536, 128)
    deg = np.minimum(8, -(-lens // 4096)).astype(np.int32)
    deg[deg == 7] = 8          # the degree set {1,2,3,4,5,6,8} has no 7
    return lens, deg, dict(hq=32, hkv=8, head_dim=128)


def _longtail_256k(rng):
    lens = _fill_to_total(lambda _i: rng.integers(256, 4097), 262144, 256, first=(131072,))
    deg = np.ones(len(lens), dtype=np.int32)
    deg[0] = 7
    return lens, deg, dict(hq=40, hkv=8, head_dim=128)


def _bimodal_128k(rng):
    def draw(i):
        return rng.integers(512, 2049) if i % 2 == 0 else rng.integers(16384, 65537)

    lens = _fill_to_total(draw, 131072, 512)
    deg = np.where(lens < 8192, 1, np.where(lens <= 24576, 3, np.where(lens <= 40960, 5, 6)))
    return lens, deg.astype(np.int32), dict(hq=32, hkv=32, head_dim=128)


def _extreme_512k(rng, d_long=7):
    support = np.arange(128, 8193, dtype=np.float64)
    w = support ** (-1.2)
    cdf = np.cumsum(w / w.sum())

    def draw(_i):
        return int(support[min(int(np.searchsorted(cdf, rng.random())), len(support) - 1)])

    lens = _fill_to_total(draw, 524288, 128, first=(393216,))
    deg = np.ones(len(lens), dtype=np.int32)
    deg[0] = d_long
    return lens, deg, dict(hq=64, hkv=8, head_dim=128)


def _bimodal_128k_spans(rng):
    """The bimodal batch with image spans: every long (image/video-token-heavy) sequence alternates text
    runs of U{64..512} tokens with bidirectional spans of U{256..2048} tokens; short sequences stay causal."""
    lens, deg, shape = _bimodal_128k(rng)
    spans = []
    for L in lens:
        sp, pos = [], 0
        if L >= 16384:
            while True:
                pos += int(rng.integers(64, 513))
                m = int(rng.integers(256, 2049))
                if pos + m > L:
                    break
                sp.append((pos, pos + m))
                pos += m
        spans.append(sp)
    return lens, deg, dict(shape, spans=spans)


WORKLOADS = {
    "tiny": _tiny,
    "llama8b_64k": _llama8b_64k,
    "longtail_256k": _longtail_256k,
    "bimodal_128k": _bimodal_128k,
    "extreme_512k": _extreme_512k,
    "bimodal_128k_spans": _bimodal_128k_spans,
}


def make_workload(name: str, seed: int = 0, **kw) -> Workload:
    rng = np.random.Generator(np.random.PCG64([seed, 0x5EED]))
    lens, deg, shape = WORKLOADS[name](rng, **kw)
    return Workload(name=name, seed=seed, seqlens=lens.astype(np.int32), cp_degrees=deg.astype(np.int32), **shape)


def reduced(w: Workload, len_div: int = 16, max_heads: int = 8) -> Workload:
    """Same generator and degrees, lengths divided by ``len_div`` (at least 1), at most 8 query heads
    with the query:KV head ratio kept.  Small enough for the fp64 oracle to finish in seconds."""
    g = w.hq // w.hkv
    hq = min(w.hq, max_heads)
    hq = max(g, (hq // g) * g) if g <= max_heads else g
    hkv = max(1, hq // g)
    lens = np.maximum(1, w.seqlens // len_div).astype(np.int32)
    spans = None
    if w.spans is not None:      # span bounds scale with the lengths; spans that collapse are dropped
        spans = [[(a // len_div, min(e // len_div, int(L))) for a, e in sp if min(e // len_div, int(L)) > a // len_div]
                 for sp, L in zip(w.spans, lens)]
    return Workload(name=w.name + "_reduced", seed=w.seed, seqlens=lens, cp_degrees=w.cp_degrees.copy(),
                    hq=hq, hkv=hkv, head_dim=w.head_dim, note=f"lengths/{len_div}", spans=spans)
