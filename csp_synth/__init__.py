"""Seeded synthetic multimodal KV caches shaped like multi-image VLM prompts.

This module only *makes inputs*: token layouts (which positions are text, which are visual),
sequence lengths, integer budgets and random Q/K/V tensors.  It contains none of the pruning
method's arithmetic and is the one module that both the CPU oracle's tests and the CUDA
library's tests and bench draw their inputs from.

Values: Q, K, V ~ N(0,1) i.i.d. per channel; rows of K at visual positions get a constant
added to every channel (+0.5, or a per-image draw from U(0.2, 0.8)); two "sink" keys
(position 0 and the first visual token) have their K row multiplied by 4; everything is
rounded to the storage type (bf16 or fp32) before anyone reads it.  The random stream of a
tensor depends on (seed, layer, tensor) and on the device it is drawn on; a comparison always
feeds both sides the same bytes.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from fractions import Fraction
from typing import List, Optional, Sequence, Tuple

import numpy as np
import torch

TEXT, VISUAL = 0, 1
Span = Tuple[int, int]  # (modality label, length)


def round_half_even(x: Fraction) -> int:
    """Nearest integer, ties to the even one."""
    fl = x.numerator // x.denominator
    rem = x - fl
    if rem > Fraction(1, 2) or (rem == Fraction(1, 2) and fl % 2 == 1):
        return fl + 1
    return fl


@dataclass
class CacheConfig:
    """One synthetic workload: shapes, token layouts and budgets of every sequence."""
    name: str
    n_layers: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    dtype: torch.dtype
    window: int
    recent: int
    layouts: List[List[Span]]                 # per sequence: ordered (label, length) spans
    budgets: np.ndarray                       # int32 [B, 4]: k_self_text, k_self_vis, k_cross_text, k_cross_vis
    total_budget: Optional[np.ndarray] = None  # int32 [B] = T of the pruning procedure, if used
    seed: int = 0
    visual_shift: float = 0.5                 # constant added to visual K rows
    per_image_shift: bool = False             # draw the shift per image from U(0.2, 0.8) instead
    sink_scale: float = 4.0
    max_len: int = field(init=False)

    def __post_init__(self):
        lens = self.seq_lens
        self.max_len = int(max(lens)) if len(lens) else 0

    @property
    def batch(self) -> int:
        return len(self.layouts)

    @property
    def seq_lens(self) -> np.ndarray:
        return np.array([sum(n for _, n in lay) for lay in self.layouts], np.int32)

    @property
    def group(self) -> int:
        return self.n_q_heads // self.n_kv_heads

    def modality(self) -> np.ndarray:
        """uint8 [B, max_len]; padding positions are labelled text."""
        m = np.zeros((self.batch, self.max_len), np.uint8)
        for b, lay in enumerate(self.layouts):
            pos = 0
            for label, n in lay:
                m[b, pos:pos + n] = label
                pos += n
        return m

    def out_capacity(self) -> int:
        """Rows per head that the compacted cache needs: kept keys plus the recent block."""
        kept = self.budgets.astype(np.int64).sum(axis=1) + self.recent
        return int(max(int(kept.max()), 1))


def candidate_counts(layout: Sequence[Span], recent: int) -> Tuple[int, int]:
    """(text, visual) keys among the candidates, i.e. all but the last `recent` positions."""
    labels = np.concatenate([np.full(n, lab, np.uint8) for lab, n in layout])
    cand = labels[:len(labels) - recent]
    n_vis = int((cand != 0).sum())
    return len(cand) - n_vis, n_vis


def budgets_from_percent(layout: Sequence[Span], recent: int, visual_pct: int, text_pct: int) -> List[int]:
    """Per-modality budgets for a prompt that ends in text: the visual share is spent on the
    inter-modality score of visual keys, the text share on the intra-modality score of text keys."""
    n_text, n_vis = candidate_counts(layout, recent)
    return [round_half_even(Fraction(text_pct * n_text, 100)), 0, 0,
            round_half_even(Fraction(visual_pct * n_vis, 100))]


def budgets_from_total(total: int, recent: int, rho: Fraction = Fraction(1, 2)) -> List[int]:
    """Split a total cache budget T: K_cross = round(rho (T - R)), K_self = the rest."""
    k_cross = round_half_even(rho * (total - recent))
    return [total - recent - k_cross, 0, 0, k_cross]


def interleaved_layout(text_spans: Sequence[int], image_len: int) -> List[Span]:
    """text, image, text, image, ..., text"""
    lay: List[Span] = []
    for i, n in enumerate(text_spans):
        if n:
            lay.append((TEXT, int(n)))
        if i + 1 < len(text_spans):
            lay.append((VISUAL, int(image_len)))
    return lay


def _even_text_spans(total_text: int, n_spans: int) -> List[int]:
    base = total_text // n_spans
    spans = [base] * n_spans
    spans[-1] += total_text - base * n_spans
    return spans


def config(index: int, budget_pct: int = 20) -> CacheConfig:
    """The five benchmark shapes.  `budget_pct` only matters for shape 4 (its budget sweep)."""
    bf16, f32 = torch.bfloat16, torch.float32
    if index == 0:
        lay = [(TEXT, 64), (VISUAL, 384), (TEXT, 128), (VISUAL, 384), (TEXT, 64)]
        return CacheConfig("tiny-fp32", 1, 4, 4, 64, f32, 16, 16, [lay],
                           np.array([budgets_from_percent(lay, 16, 50, 50)], np.int32), seed=0)
    if index == 1:
        lay = interleaved_layout([64] * 6 + [256], 576)
        return CacheConfig("llava-7b-4k", 32, 32, 32, 128, bf16, 32, 32, [lay],
                           np.array([budgets_from_percent(lay, 32, 20, 50)], np.int32), seed=1)
    if index == 2:
        lay = interleaved_layout([64] * 24 + [1024], 576)
        total = round_half_even(Fraction(10 * 16384, 100))
        return CacheConfig("multi-image-16k", 32, 32, 32, 128, bf16, 32, 32, [lay],
                           np.array([budgets_from_total(total, 32)], np.int32),
                           total_budget=np.array([total], np.int32), seed=2, per_image_shift=True)
    if index == 3:
        lays, buds = [], []
        for L in (8192, 16384, 24576, 32768):
            n_img = -((-85 * L) // (100 * 1024))   # ceil(0.85 L / 1024): 7, 14, 21, 28 images
            lay = interleaved_layout(_even_text_spans(L - n_img * 1024, n_img + 1), 1024)
            lays.append(lay)
            buds.append(budgets_from_percent(lay, 32, 15, 40))
        return CacheConfig("gqa-qwen2vl-7b", 28, 28, 4, 128, bf16, 32, 32, lays,
                           np.array(buds, np.int32), seed=3)
    if index == 4:
        rng = np.random.RandomState(4)
        lays, buds, totals = [], [], []
        for _ in range(32):
            L = int(rng.randint(2048, 8193))
            n_img = int(rng.randint(2, min(8, (L - 512) // 576) + 1))
            text = L - n_img * 576
            free = text - 64                      # the final span keeps at least 64 tokens
            cuts = np.sort(rng.randint(0, free + 1, size=n_img))
            spans = np.diff(np.concatenate([[0], cuts, [free]])).tolist()
            spans[-1] += 64
            lay = interleaved_layout(spans, 576)
            total = round_half_even(Fraction(budget_pct * L, 100))
            lays.append(lay)
            buds.append(budgets_from_total(total, 32))
            totals.append(total)
        return CacheConfig(f"serving-b32-{budget_pct}pct", 32, 32, 32, 128, bf16, 32, 32, lays,
                           np.array(buds, np.int32), total_budget=np.array(totals, np.int32), seed=4)
    raise ValueError(f"no such config: {index}")


def _generator(cfg: CacheConfig, layer: int, tensor_id: int, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed((cfg.seed * 1_000_003 + layer) * 16 + tensor_id)
    return g


def make_layer(cfg: CacheConfig, layer: int, device="cpu"):
    """Q window, K and V of one layer.

    Returns (q [B,Hq,W,d], k [B,Hkv,max_len,d], v [B,Hkv,max_len,d]) in cfg.dtype on `device`.
    Rows of k/v at positions >= the sequence's length are padding (random, to be ignored).
    """
    dev = torch.device(device)
    B, W, d, Lm = cfg.batch, cfg.window, cfg.head_dim, cfg.max_len
    q = torch.randn((B, cfg.n_q_heads, W, d), generator=_generator(cfg, layer, 0, dev),
                    device=dev, dtype=torch.float32)
    k = torch.randn((B, cfg.n_kv_heads, Lm, d), generator=_generator(cfg, layer, 1, dev),
                    device=dev, dtype=torch.float32)
    v = torch.randn((B, cfg.n_kv_heads, Lm, d), generator=_generator(cfg, layer, 2, dev),
                    device=dev, dtype=torch.float32)
    shift_rng = np.random.RandomState(cfg.seed * 7919 + 17)
    shift = np.zeros((B, Lm), np.float32)
    gain = np.ones((B, Lm), np.float32)
    for b, lay in enumerate(cfg.layouts):
        pos, first_visual = 0, None
        for label, n in lay:
            if label != TEXT:
                if first_visual is None:
                    first_visual = pos
                shift[b, pos:pos + n] = (shift_rng.uniform(0.2, 0.8) if cfg.per_image_shift
                                         else cfg.visual_shift)
            pos += n
        if pos > 0:
            gain[b, 0] = cfg.sink_scale
        if first_visual is not None:
            gain[b, first_visual] = cfg.sink_scale
    shift_t = torch.from_numpy(shift).to(dev)[:, None, :, None]
    gain_t = torch.from_numpy(gain).to(dev)[:, None, :, None]
    k.add_(shift_t).mul_(gain_t)
    return q.to(cfg.dtype), k.to(cfg.dtype), v.to(cfg.dtype)


def small_config(name: str, layouts: List[List[Span]], n_q_heads: int, n_kv_heads: int, head_dim: int,
                 window: int, recent: int, dtype=torch.bfloat16, visual_pct: int = 30,
                 text_pct: int = 50, seed: int = 0, **kw) -> CacheConfig:
    """A one-layer workload with percent budgets, for tests."""
    buds = np.array([budgets_from_percent(l, recent, visual_pct, text_pct) for l in layouts], np.int32)
    return CacheConfig(name, 1, n_q_heads, n_kv_heads, head_dim, dtype, window, recent, layouts, buds,
                       seed=seed, **kw)
