"""Seeded synthetic inputs shaped like Qwen3-VL workloads.

This module only *draws inputs*: importance scores, position ids and opaque
bf16 payloads.  It contains none of the method's arithmetic (no ordering, no
selection, no gather) and is the one module both the CPU oracle's tests and the
CUDA path's tests/bench may import.

The paper evaluates on benchmark images and videos that are not available
offline; the five workloads below stand in for them.  Their token grids,
budgets K = floor(n * keep ratio), hidden sizes and K/V row shapes follow the
Qwen3-VL configurations the paper's Section 4.1 setup names (14x14 .. 56x56
merged-token grids, 2048/4096-wide hidden rows, 8 KV heads of 128).

Scores come from a counter-based generator (SplitMix64) evaluated with numpy
integer arithmetic, so they do not depend on the torch version or the device.
Bulk payload values never influence control flow on either side; they are
drawn with torch's seeded generator on whichever device is asked for.
"""

from __future__ import annotations

import dataclasses
import math
from typing import Optional, Tuple

import numpy as np

SEED_BASE = 260528115

_U64 = np.uint64
_MASK = (1 << 64) - 1


def _splitmix64(x: np.ndarray) -> np.ndarray:
    """SplitMix64 output function applied element-wise to uint64 counters."""
    with np.errstate(over="ignore"):
        z = (x + _U64(0x9E3779B97F4A7C15)).astype(np.uint64)
        z = (z ^ (z >> _U64(30))) * _U64(0xBF58476D1CE4E5B9)
        z = (z ^ (z >> _U64(27))) * _U64(0x94D049BB133111EB)
        z = z ^ (z >> _U64(31))
    return z


def raw_u64(seed: int, stream: int, count: int) -> np.ndarray:
    """`count` 64-bit words of stream `stream` under `seed` (pure function)."""
    base = _splitmix64(np.array([(seed * 0x100000001B3 + stream) & _MASK], dtype=np.uint64))[0]
    with np.errstate(over="ignore"):
        ctr = base + np.arange(count, dtype=np.uint64) * _U64(0x9E3779B97F4A7C15)
    return _splitmix64(ctr)


def uniform24(seed: int, stream: int, count: int) -> np.ndarray:
    """U[0,1) on a 2^-24 lattice: every value is exact in fp32. Returns fp64."""
    return (raw_u64(seed, stream, count) >> _U64(40)).astype(np.float64) / float(1 << 24)


def uniform53(seed: int, stream: int, count: int) -> np.ndarray:
    """U(0,1) with 53 random bits, never exactly 0 (safe under log)."""
    return ((raw_u64(seed, stream, count) >> _U64(11)).astype(np.float64) + 0.5) / float(1 << 53)


def normal(seed: int, stream: int, count: int) -> np.ndarray:
    """N(0,1) by Box-Muller in fp64 from two independent streams."""
    u1 = uniform53(seed, 2 * stream, count)
    u2 = uniform53(seed, 2 * stream + 1, count)
    return np.sqrt(-2.0 * np.log(u1)) * np.cos(2.0 * np.pi * u2)


@dataclasses.dataclass(frozen=True)
class Workload:
    """One synthetic workload: a batch of equally shaped segments.

    A segment is one image or one video: a (t, h, w) grid of merged visual
    tokens, n = t*h*w, linearised row-major.  The retention floor tiles every
    temporal slice into region_h x region_w token tiles and keeps at least
    `floor_m` tokens of each tile.  `k` tokens survive per segment.
    """

    name: str
    config_id: int
    n_seg: int
    t: int
    h: int
    w: int
    region_h: int
    region_w: int
    floor_m: int
    k: int
    score_kind: str  # uniform | lognormal | blobs | quant256
    hidden_dim: int = 0  # bf16 elements per hidden row; 0 = no hidden payload
    n_layers: int = 0  # 0 = no K/V payload
    kv_heads: int = 8
    head_dim: int = 128
    text_before: int = 0  # text tokens in front of the visual span
    text_after: int = 0  # text tokens behind it
    pos_t_from_grid: bool = True  # False: t coordinate written as 0

    @property
    def n(self) -> int:
        return self.t * self.h * self.w

    @property
    def n_regions(self) -> int:
        return self.t * math.ceil(self.h / self.region_h) * math.ceil(self.w / self.region_w)

    @property
    def seq_len(self) -> int:
        return self.text_before + self.n + self.text_after

    @property
    def s_out(self) -> int:
        return self.text_before + self.k + self.text_after

    @property
    def hidden_row_bytes(self) -> int:
        return 2 * self.hidden_dim

    @property
    def kv_row_bytes(self) -> int:
        return 2 * self.kv_heads * self.head_dim

    @property
    def seed(self) -> int:
        return SEED_BASE + 1000 * self.config_id

    def replace(self, **kw) -> "Workload":
        return dataclasses.replace(self, **kw)


# The five configurations of the benchmark definition (1-based ids).  c3 carries
# the hidden/pos payload of c2's per-image shape as well, so that one pass over
# it exercises every step of the path; c5 exists once per keep ratio.
C1 = Workload("c1_single_448", 1, 1, 1, 14, 14, 2, 2, 1, 65, "uniform", hidden_dim=2048,
              pos_t_from_grid=False)
C2 = Workload("c2_batch8_896", 2, 8, 1, 32, 32, 4, 4, 1, 341, "lognormal", hidden_dim=4096)
C3 = Workload("c3_kv_qwen3vl8b", 3, 16, 1, 32, 32, 4, 4, 1, 341, "lognormal", hidden_dim=4096,
              n_layers=36, text_before=16, text_after=48)
C4 = Workload("c4_video_32f", 4, 1, 16, 14, 14, 2, 2, 1, 1045, "blobs", hidden_dim=4096)
C5_HALF = Workload("c5_hires_keep_1_2", 5, 4, 1, 56, 56, 4, 4, 1, 1568, "quant256",
                   hidden_dim=4096, n_layers=36)
C5_THIRD = C5_HALF.replace(name="c5_hires_keep_1_3", k=1045)
C5_QUARTER = C5_HALF.replace(name="c5_hires_keep_1_4", k=784)

ALL = (C1, C2, C3, C4, C5_HALF, C5_THIRD, C5_QUARTER)
BY_NAME = {wl.name: wl for wl in ALL}

# Selection alone on segments beyond one thread block (long videos, Section 5 of the paper):
# no payload, K = n / 3.  A 128-frame clip at 56 x 56 tokens per two frames, a batch of eight
# 32-frame clips, and a batch of four 8-frame clips.
LONG_VIDEO = Workload("longsel_video_128f", 6, 1, 64, 56, 56, 4, 4, 1, 64 * 56 * 56 // 3, "quant256")
LONG_BATCH8 = Workload("longsel_batch8_32f", 7, 8, 16, 56, 56, 4, 4, 1, 16 * 56 * 56 // 3, "lognormal")
LONG_BATCH4 = Workload("longsel_batch4_8f", 8, 4, 4, 56, 56, 4, 4, 1, 4 * 56 * 56 // 3, "uniform")
LONG_BY_NAME = {wl.name: wl for wl in (LONG_VIDEO, LONG_BATCH8, LONG_BATCH4)}


def scores(wl: Workload, seg: Optional[int] = None) -> np.ndarray:
    """Importance scores, fp32.  [n_seg, n], or [n] for one segment."""
    if seg is None:
        return np.stack([scores(wl, s) for s in range(wl.n_seg)])
    seed = wl.seed + seg
    n = wl.n
    if wl.score_kind == "uniform":
        out = uniform24(seed, 0, n)
    elif wl.score_kind == "lognormal":
        out = np.exp(normal(seed, 0, n))
    elif wl.score_kind == "quant256":
        out = np.floor(uniform24(seed, 0, n) * 256.0) / 256.0
    elif wl.score_kind == "blobs":
        out = _blob_scores(wl, seed)
    else:
        raise ValueError(wl.score_kind)
    return out.astype(np.float32)


def _blob_scores(wl: Workload, seed: int, blobs_per_group: int = 8) -> np.ndarray:
    """Per temporal group: a sum of 2-D Gaussian bumps plus 0.05*U[0,1) noise.

    Centres ~ U(0,h) x U(0,w), widths ~ U(1,3) tokens, amplitudes ~ U(0.5,1);
    evaluated in fp64 (rounded to fp32 by the caller).
    """
    hh, ww = np.meshgrid(np.arange(wl.h, dtype=np.float64), np.arange(wl.w, dtype=np.float64),
                         indexing="ij")
    out = np.empty((wl.t, wl.h, wl.w), dtype=np.float64)
    for g in range(wl.t):
        u = uniform53(seed, 16 + g, 4 * blobs_per_group).reshape(blobs_per_group, 4)
        acc = np.zeros((wl.h, wl.w), dtype=np.float64)
        for cy, cx, sg, am in u:
            cy, cx = cy * wl.h, cx * wl.w
            sigma = 1.0 + 2.0 * sg
            amp = 0.5 + 0.5 * am
            acc += amp * np.exp(-((hh - cy) ** 2 + (ww - cx) ** 2) / (2.0 * sigma * sigma))
        out[g] = acc
    noise = uniform24(seed, 1, wl.n).reshape(wl.t, wl.h, wl.w)
    return (out + 0.05 * noise).reshape(-1)


def pos_ids(wl: Workload) -> np.ndarray:
    """3-D position ids int32 [n_seg, n, 3] = (t, h, w) of every token."""
    t, h, w = np.meshgrid(np.arange(wl.t), np.arange(wl.h), np.arange(wl.w), indexing="ij")
    if not wl.pos_t_from_grid:
        t = np.zeros_like(t)
    one = np.stack([t.reshape(-1), h.reshape(-1), w.reshape(-1)], axis=1).astype(np.int32)
    return np.repeat(one[None], wl.n_seg, axis=0).copy()


def payload_bf16(shape: Tuple[int, ...], seed: int, device="cpu"):
    """bf16 N(0,1) tensor from torch's seeded generator on `device`."""
    import torch

    g = torch.Generator(device=device)
    g.manual_seed(seed)
    numel = 1
    for s in shape:
        numel *= s
    # draw in slabs to bound the fp32 temporary
    out = torch.empty(numel, dtype=torch.bfloat16, device=device)
    slab = 1 << 26
    for lo in range(0, numel, slab):
        hi = min(numel, lo + slab)
        out[lo:hi] = torch.randn(hi - lo, generator=g, device=device, dtype=torch.float32).to(torch.bfloat16)
    return out.view(*shape)


def hidden(wl: Workload, device="cpu"):
    """Hidden states at the projector boundary, bf16 [n_seg, n, hidden_dim]."""
    return payload_bf16((wl.n_seg, wl.n, wl.hidden_dim), wl.seed + 500, device)


def kv_layer(wl: Workload, layer: int, which: int, device="cpu"):
    """One layer's K (which=0) or V (which=1), bf16 [n_seg, seq_len, heads, head_dim]."""
    return payload_bf16((wl.n_seg, wl.seq_len, wl.kv_heads, wl.head_dim),
                        wl.seed + 600 + 2 * layer + which, device)


def stamp_rows(x, row_elems: int) -> None:
    """Overwrite the first 8 bytes of every row (`row_elems` bf16 elements) of a
    contiguous tensor with the row's linear id, so that any misplaced row is
    distinguishable."""
    import torch

    assert x.is_contiguous() and x.dtype == torch.bfloat16 and row_elems >= 4
    as_i16 = x.view(torch.int16).view(-1, row_elems)
    rows = as_i16
    ids = torch.arange(rows.shape[0], device=x.device, dtype=torch.int64)
    for b in range(4):
        as_i16[:, b] = ((ids >> (16 * b)) & 0xFFFF).to(torch.int16)


def kv_algorithmic_bytes(wl: Workload) -> int:
    """Bytes the K/V compaction must move: every kept row read once and written once."""
    return 2 * (wl.n_layers * 2 * wl.n_seg * wl.s_out * wl.kv_row_bytes)


def hidden_algorithmic_bytes(wl: Workload) -> int:
    return 2 * wl.n_seg * wl.k * (wl.hidden_row_bytes + 12)


# ---------------------------------------------------------------- compact visual aggregation (Eq. 8)

@dataclasses.dataclass(frozen=True)
class AggWorkload:
    """Dense patch embeddings of a batch of images and a shared set of compact anchors."""

    name: str
    n_img: int
    t_e: int  # dense patch tokens per image (before the 2x2 merge)
    m_e: int  # compact anchors
    d_v: int  # vision width
    tau: float
    seed: int = SEED_BASE + 9000

    @property
    def flops(self) -> int:
        """Both contractions: Q_A K_0^T and W_A X_0, 2 flops per multiply-add."""
        return 2 * 2 * self.n_img * self.m_e * self.t_e * self.d_v


# 8 images of 896x896: 64x64 = 4096 patches of 14x14 pixels each (they become the 32x32 merged
# tokens of the batch-8 selection workload), vision width 1152, 1024 anchors (256 compact tokens
# after the 2x2 merger), temperature 0.07.
AGG_896 = AggWorkload("agg_batch8_896", 8, 4096, 1024, 1152, 0.07)
AGG_896_X2 = AggWorkload("agg_batch2_896", 2, 4096, 1024, 1152, 0.07)  # a quarter of it, for profiler captures
AGG_448 = AggWorkload("agg_single_448", 1, 1024, 256, 1152, 0.07)
AGG_BY_NAME = {w.name: w for w in (AGG_896, AGG_896_X2, AGG_448)}


def agg_inputs(w: AggWorkload, device="cpu"):
    """(x0 bf16 [n_img, t_e, d_v] ~ 1.5 N(0,1) + 0.7, anchors fp32 [m_e, d_v] ~ N(0,1)), seeded."""
    import torch

    x0 = payload_bf16_affine((w.n_img, w.t_e, w.d_v), w.seed, device, 1.5, 0.7)
    g = torch.Generator(device=device)
    g.manual_seed(w.seed + 1)
    anchors = torch.randn((w.m_e, w.d_v), generator=g, device=device, dtype=torch.float32)
    return x0, anchors


def payload_bf16_affine(shape, seed: int, device, scale: float, offset: float):
    """bf16 scale * N(0,1) + offset from torch's seeded generator on `device`."""
    import torch

    g = torch.Generator(device=device)
    g.manual_seed(seed)
    numel = 1
    for s in shape:
        numel *= s
    out = torch.empty(numel, dtype=torch.bfloat16, device=device)
    slab = 1 << 26
    for lo in range(0, numel, slab):
        hi = min(numel, lo + slab)
        out[lo:hi] = (torch.randn(hi - lo, generator=g, device=device, dtype=torch.float32) * scale
                      + offset).to(torch.bfloat16)
    return out.view(*shape)


# ---------------------------------------------------------------- KV-compressed attention (Eq. 9)

@dataclasses.dataclass(frozen=True)
class KvAttnWorkload:
    """Projected Q, K, V of one compact vision layer for a batch of images, and a shared assignment."""

    name: str
    n_img: int
    m_e: int      # compact tokens
    n_heads: int
    head_dim: int
    s: int        # memory anchors
    seed: int = SEED_BASE + 9500

    @property
    def dim(self) -> int:
        return self.n_heads * self.head_dim

    @property
    def flops(self) -> int:
        """Compression of K and V (2 GEMMs) and the two contractions of the attention."""
        return 2 * 2 * self.n_img * self.s * self.m_e * self.dim * 2


# 8 images, 1024 compact tokens, 16 heads of 64 (vision width 1024), 256 memory anchors
KVATTN_896 = KvAttnWorkload("kvattn_batch8_896", 8, 1024, 16, 64, 256)
# the same layer on a 1152-wide tower (16 heads of 72), and with Table 2's 512 memory anchors
KVATTN_896_W1152 = KvAttnWorkload("kvattn_batch8_896_w1152", 8, 1024, 16, 72, 256)
KVATTN_896_S512 = KvAttnWorkload("kvattn_batch8_896_s512", 8, 1024, 16, 64, 512)
KVATTN_BY_NAME = {w.name: w for w in (KVATTN_896, KVATTN_896_W1152, KVATTN_896_S512)}


def kvattn_inputs(w: KvAttnWorkload, device="cpu"):
    """(q, k, v bf16 [n_img, m_e, dim] ~ 1.2 N(0,1); r fp32 [m_e, s]: row-wise softmax of 3 N(0,1)), seeded."""
    import torch

    q, k, v = (payload_bf16_affine((w.n_img, w.m_e, w.dim), w.seed + i, device, 1.2, 0.0) for i in range(3))
    g = torch.Generator(device=device)
    g.manual_seed(w.seed + 3)
    r = torch.softmax(torch.randn((w.m_e, w.s), generator=g, device=device, dtype=torch.float32) * 3.0, dim=1)
    return q, k, v, r
