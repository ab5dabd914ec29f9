"""Seeded synthetic inputs shaped like FiCoCo's workloads.

This module only draws random numbers and arranges them (fields on a patch grid,
softmax-normalised attention logits, ragged packing).  It contains none of the
token-reduction arithmetic, so both the CUDA path and the CPU checker can be fed
from it without sharing any of the method's code.

Shapes follow the models the paper evaluates (Sec. "Implementation Details",
backbone list): a CLIP-ViT-L/14-336 encoder (1 CLS + 24x24 patches, width 1024),
multi-crop high-resolution inputs (5 crops of 576 patches), dynamic-resolution
ragged batches (width 1280, no CLS) and an LLM decoder layer (576 vision + 64 text
tokens, width 4096).

bf16 tensors are carried as ``uint16`` bit patterns in numpy (numpy has no bf16).
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import List, Optional, Sequence, Tuple

import numpy as np

# ----------------------------------------------------------------------------
# bf16 <-> fp32 bit helpers (storage format only)
# ----------------------------------------------------------------------------

def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round fp32 to bf16 (round-to-nearest-even), returned as uint16 bit patterns."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    lsb = (u >> np.uint32(16)) & np.uint32(1)
    r = u + np.uint32(0x7FFF) + lsb
    return (r >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    """Exact widening of bf16 bit patterns to fp32."""
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def rng_for(seed: int, *stream: int) -> np.random.Generator:
    """Counter-based generator (Philox) keyed by a seed and a stream id tuple."""
    key = np.random.SeedSequence([int(seed) & 0xFFFFFFFF, *[int(s) & 0xFFFFFFFF for s in stream]])
    return np.random.Generator(np.random.Philox(key))


# ----------------------------------------------------------------------------
# Token fields
# ----------------------------------------------------------------------------

def _blur_matrix(n: int, corr_len: float) -> np.ndarray:
    """Row-normalised Gaussian smoothing matrix on a 1-D grid of n cells."""
    idx = np.arange(n, dtype=np.float64)
    d = idx[:, None] - idx[None, :]
    g = np.exp(-0.5 * (d / float(corr_len)) ** 2)
    return g / g.sum(axis=1, keepdims=True)


def smooth_field(rng: np.random.Generator, gh: int, gw: int, dim: int, corr_len: float,
                 noise_std: float = 0.1) -> np.ndarray:
    """[gh*gw, dim] fp32: per channel a spatially smooth Gaussian random field with the
    given correlation length (in patches), rescaled to unit variance, plus white noise."""
    white = rng.standard_normal((gh, gw, dim), dtype=np.float32).astype(np.float64)
    bh = _blur_matrix(gh, corr_len)
    bw = _blur_matrix(gw, corr_len)
    f = np.einsum("ij,jkd->ikd", bh, white)
    f = np.einsum("kl,ild->ikd", bw, f)
    f -= f.mean(axis=(0, 1), keepdims=True)
    f /= f.std(axis=(0, 1), keepdims=True) + 1e-12
    f = f.reshape(gh * gw, dim)
    f += noise_std * rng.standard_normal((gh * gw, dim), dtype=np.float32)
    return f.astype(np.float32)


def softmax_attention(rng: np.random.Generator, heads: int, n: int, logit_std: float) -> np.ndarray:
    """[heads, n] fp32: each head is a softmax over N(0, logit_std) logits."""
    z = logit_std * rng.standard_normal((heads, n), dtype=np.float32).astype(np.float64)
    z -= z.max(axis=1, keepdims=True)
    e = np.exp(z)
    return (e / e.sum(axis=1, keepdims=True)).astype(np.float32)


def relation_map(rng: np.random.Generator, patches: np.ndarray, sharpness: float = 8.0,
                 logit_std: float = 1.0) -> np.ndarray:
    """[Np, Np] fp32 stand-in for a head-averaged self-attention map over the patch tokens:
    row i is a softmax over sharpness * cos(x_i, x_j) + N(0, logit_std) logits, so rows sum to 1,
    the map is not symmetric and similar tokens attend to each other."""
    x = patches.astype(np.float64)
    xh = x / np.sqrt((x * x).sum(axis=1, keepdims=True))
    z = sharpness * (xh @ xh.T) + logit_std * rng.standard_normal((x.shape[0], x.shape[0]))
    z -= z.max(axis=1, keepdims=True)
    e = np.exp(z)
    return (e / e.sum(axis=1, keepdims=True)).astype(np.float32)


def causal_text_to_vision_attention(rng: np.random.Generator, heads: int, n_vision: int,
                                    n_text: int, logit_std: float = 1.0) -> np.ndarray:
    """[heads, n_text, n_vision] fp32: the vision block of a causal softmax.  Text row k
    attends to all vision tokens and to text tokens 0..k; only the vision columns are
    returned (they therefore sum to less than one)."""
    out = np.empty((heads, n_text, n_vision), dtype=np.float32)
    for k in range(n_text):
        z = logit_std * rng.standard_normal((heads, n_vision + k + 1), dtype=np.float32).astype(np.float64)
        z -= z.max(axis=1, keepdims=True)
        e = np.exp(z)
        p = e / e.sum(axis=1, keepdims=True)
        out[:, k, :] = p[:, :n_vision].astype(np.float32)
    return out


# ----------------------------------------------------------------------------
# Batches
# ----------------------------------------------------------------------------

@dataclass
class VBatch:
    """One FiCoCo-V reduce-step input.

    tokens : list (per image) of [c + Np, D] arrays; fp32, or uint16 bf16 bit patterns
    attn   : list of [H, Np] fp32 (CLS->patch weights per head, over alive patches)
    pos    : list of [Np] int32 (linear index of each alive patch on the original grid)
    grid   : list of (gh, gw)
    keep   : list of int, number of patch tokens preserved (N^T)
    """
    dtype: str
    has_cls: bool
    dim: int
    heads: int
    tokens: List[np.ndarray]
    attn: List[np.ndarray]
    pos: List[np.ndarray]
    grid: List[Tuple[int, int]]
    keep: List[int]
    name: str = ""

    @property
    def batch(self) -> int:
        return len(self.tokens)

    def uniform(self) -> bool:
        n0 = self.tokens[0].shape[0]
        return (all(t.shape[0] == n0 for t in self.tokens)
                and all(k == self.keep[0] for k in self.keep)
                and all(g == self.grid[0] for g in self.grid))


@dataclass
class LBatch:
    """One FiCoCo-L reduce-step input.

    tokens   : list of [N + M, D] arrays (vision rows first, then text rows)
    attn_t2v : list of [H, M, N] fp32 text->vision attention weights
    keep     : list of int, number of vision tokens preserved
    """
    dtype: str
    dim: int
    heads: int
    n_vision: int
    n_text: int
    tokens: List[np.ndarray]
    attn_t2v: List[np.ndarray]
    keep: List[int]
    name: str = ""

    @property
    def batch(self) -> int:
        return len(self.tokens)


def _store(x: np.ndarray, dtype: str) -> np.ndarray:
    if dtype == "bf16":
        return f32_to_bf16_bits(x)
    if dtype == "fp32":
        return np.ascontiguousarray(x, dtype=np.float32)
    raise ValueError(dtype)


def vit_image(seed: int, image: int, gh: int, gw: int, dim: int, dtype: str, has_cls: bool,
              corr_len: Sequence[float] | float = 3.0, crop_rows: Optional[int] = None,
              noise_std: float = 0.1) -> np.ndarray:
    """Token matrix of one image: optional CLS row N(0,1), then gh*gw patch rows.

    ``crop_rows``: when given, the grid is a vertical stack of crops of that many rows,
    each an independent field with its own correlation length (``corr_len`` sequence)."""
    rng = rng_for(seed, image, 1)
    if crop_rows is None:
        patches = smooth_field(rng, gh, gw, dim, float(corr_len), noise_std)
    else:
        assert gh % crop_rows == 0
        ncrop = gh // crop_rows
        cl = list(corr_len) if not np.isscalar(corr_len) else [float(corr_len)] * ncrop
        patches = np.concatenate(
            [smooth_field(rng, crop_rows, gw, dim, cl[c], noise_std) for c in range(ncrop)], axis=0)
    rows = [patches]
    if has_cls:
        rows.insert(0, rng.standard_normal((1, dim), dtype=np.float32))
    return _store(np.concatenate(rows, axis=0), dtype)


def make_v_batch(seed: int, batch: int, gh: int, gw: int, dim: int, heads: int, keep: int,
                 dtype: str = "bf16", has_cls: bool = True, logit_std: float = 1.0,
                 corr_len: float = 3.0, name: str = "") -> VBatch:
    """Uniform batch: every image has the same grid and keep count, all patches alive."""
    npatch = gh * gw
    toks, attn, pos = [], [], []
    for b in range(batch):
        toks.append(vit_image(seed, b, gh, gw, dim, dtype, has_cls, corr_len))
        attn.append(softmax_attention(rng_for(seed, b, 2), heads, npatch, logit_std))
        pos.append(np.arange(npatch, dtype=np.int32))
    return VBatch(dtype, has_cls, dim, heads, toks, attn, pos, [(gh, gw)] * batch, [keep] * batch, name)


def make_multicrop_batch(seed: int, batch: int, crops: int, crop_hw: int, dim: int, heads: int,
                         keep: int, dtype: str = "bf16", logit_std: float = 1.0,
                         name: str = "") -> VBatch:
    """High-resolution multi-crop images: crops stacked vertically on one grid
    (crops*crop_hw rows x crop_hw columns), per-crop correlation length ~ U[2, 6]."""
    gh, gw = crops * crop_hw, crop_hw
    toks, attn, pos = [], [], []
    for b in range(batch):
        cl = rng_for(seed, b, 3).uniform(2.0, 6.0, size=crops)
        toks.append(vit_image(seed, b, gh, gw, dim, dtype, True, cl, crop_rows=crop_hw))
        attn.append(softmax_attention(rng_for(seed, b, 2), heads, gh * gw, logit_std))
        pos.append(np.arange(gh * gw, dtype=np.int32))
    return VBatch(dtype, True, dim, heads, toks, attn, pos, [(gh, gw)] * batch, [keep] * batch, name)


def make_ragged_batch(seed: int, batch: int, lo: int, hi: int, dim: int, heads: int,
                      keep_div: int = 9, dtype: str = "bf16", logit_std: float = 1.0,
                      name: str = "") -> VBatch:
    """Dynamic-resolution batch without CLS: grid sides drawn uniformly from [lo, hi];
    each image keeps ceil(N / keep_div) tokens."""
    r = rng_for(seed, 0, 4)
    toks, attn, pos, grid, keep = [], [], [], [], []
    for b in range(batch):
        gh = int(r.integers(lo, hi + 1))
        gw = int(r.integers(lo, hi + 1))
        n = gh * gw
        toks.append(vit_image(seed, b, gh, gw, dim, dtype, False, 3.0))
        attn.append(softmax_attention(rng_for(seed, b, 2), heads, n, logit_std))
        pos.append(np.arange(n, dtype=np.int32))
        grid.append((gh, gw))
        keep.append(-(-n // keep_div))
    return VBatch(dtype, False, dim, heads, toks, attn, pos, grid, keep, name)


def make_l_batch(seed: int, batch: int, n_vision: int, n_text: int, dim: int, heads: int,
                 keep: int, dtype: str = "bf16", scale: float = 1.0 / 64.0,
                 name: str = "") -> LBatch:
    """Decoder-layer hidden states N(0,1)*scale, with causal text->vision attention."""
    toks, attn = [], []
    for b in range(batch):
        x = rng_for(seed, b, 1).standard_normal((n_vision + n_text, dim), dtype=np.float32) * np.float32(scale)
        toks.append(_store(x, dtype))
        attn.append(causal_text_to_vision_attention(rng_for(seed, b, 2), heads, n_vision, n_text))
    return LBatch(dtype, dim, heads, n_vision, n_text, toks, attn, [keep] * batch, name)


def make_keys(seed: int, n_tokens: List[int], heads: int, head_dim: int, dtype: str = "bf16",
              common: float = 0.5) -> List[np.ndarray]:
    """Key states for the no-CLS equivalent token, one [T, H, d] array per image (token-major,
    as a key projection writes them).  Every entry is N(0, 1) plus a per-image direction shared
    by all tokens and heads (scale `common`), so that the cosines with the mean key spread over
    a range instead of hovering around zero."""
    out = []
    for b, t in enumerate(n_tokens):
        r = rng_for(seed, b, 7)
        k = r.standard_normal((t, heads, head_dim))
        shared = r.standard_normal(head_dim)
        gain = r.uniform(0.0, 2.0, size=(t, 1, 1))          # how much of it each token carries
        out.append(_store(k + common * gain * shared[None, None, :], dtype))
    return out


def regenerate_attention(batch: VBatch, seed: int, step: int, logit_std: float) -> None:
    """Replace the attention of every image by fresh per-head softmax weights over its
    currently alive patches (used between the steps of a progressive schedule)."""
    for b in range(batch.batch):
        n = batch.pos[b].shape[0]
        batch.attn[b] = softmax_attention(rng_for(seed, b, 100 + step), batch.heads, n, logit_std)


# ----------------------------------------------------------------------------
# The five workload shapes (full size and a scaled-down variant of each)
# ----------------------------------------------------------------------------

def workload(idx: int, small: bool = False, seed: Optional[int] = None):
    """Return the first-step input of workload ``idx`` (1..5).

    1: single ViT-L/14-336 image, fp32, discard 64 of 576
    2: batch 32, bf16, first step of the 576->288->144->64 schedule (logit std 1.5)
    3: batch 8 multi-crop (5x576 patches), bf16, first step of 2880->1440->720->320
    4: ragged batch 16, grids 16..64 per side, width 1280, no CLS, keep ceil(N/9)
    5: FiCoCo-L, batch 16, 576 vision + 64 text, width 4096, keep 64
    ``small`` shrinks batch / grid / width so a CPU check finishes in seconds while still
    spanning several tiles and a ragged tail.
    """
    s = 1000 * idx if seed is None else seed
    if idx == 1:
        if small:
            return make_v_batch(s, 1, 10, 10, 256, 4, 100 - 12, "fp32", True, 1.0, name="c1-small")
        return make_v_batch(s, 1, 24, 24, 1024, 16, 576 - 64, "fp32", True, 1.0, name="c1")
    if idx == 2:
        if small:
            return make_v_batch(s, 3, 12, 12, 256, 4, 72, "bf16", True, 1.5, name="c2-small")
        return make_v_batch(s, 32, 24, 24, 1024, 16, 288, "bf16", True, 1.5, name="c2")
    if idx == 3:
        if small:
            return make_multicrop_batch(s, 2, 3, 12, 256, 4, 216, "bf16", name="c3-small")
        return make_multicrop_batch(s, 8, 5, 24, 1024, 16, 1440, "bf16", name="c3")
    if idx == 4:
        if small:
            return make_ragged_batch(s, 4, 8, 20, 320, 4, 9, "bf16", name="c4-small")
        return make_ragged_batch(s, 16, 16, 64, 1280, 16, 9, "bf16", name="c4")
    if idx == 5:
        if small:
            return make_l_batch(s, 2, 144, 16, 512, 4, 16, "bf16", name="c5-small")
        return make_l_batch(s, 16, 576, 64, 4096, 32, 64, "bf16", name="c5")
    raise ValueError(idx)


SCHEDULES = {2: [288, 144, 64], 3: [1440, 720, 320]}
SCHEDULES_SMALL = {2: [72, 36, 16], 3: [216, 108, 48]}
