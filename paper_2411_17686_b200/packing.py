"""Pack synthetic batches (lists of per-image numpy arrays) into the flat layouts of the
C ABI, as torch tensors on a device or in pinned host memory.  Marshalling only."""
from __future__ import annotations

from dataclasses import dataclass
from typing import List, Optional

import numpy as np

from .binding import to_torch


@dataclass
class PackedV:
    tokens: object
    attn: object
    pos: object
    seqlens: Optional[List[int]]
    n_tokens: int
    keep: List[int]
    grid_h: List[int]
    grid_w: List[int]
    heads: int
    has_cls: bool

    def call_kwargs(self):
        return dict(n_tokens=self.n_tokens, seqlens=self.seqlens, pos=self.pos)


@dataclass
class PackedL:
    tokens: object
    attn_t2v: object
    keep: List[int]
    n_vision: int
    n_text: int
    heads: int


def pack_v(batch, device=None, pin: bool = False, with_pos: bool = True) -> PackedV:
    tokens = np.concatenate(batch.tokens, axis=0)
    attn = np.concatenate([a.reshape(-1) for a in batch.attn]).astype(np.float32)
    pos = np.concatenate(batch.pos).astype(np.int32)
    uniform = batch.uniform()
    return PackedV(
        tokens=to_torch(tokens, device, pin), attn=to_torch(attn, device, pin),
        pos=to_torch(pos, device, pin) if with_pos else None,
        seqlens=None if uniform else [int(t.shape[0]) for t in batch.tokens],
        n_tokens=int(batch.tokens[0].shape[0]) if uniform else 0,
        keep=[int(k) for k in batch.keep], grid_h=[int(g[0]) for g in batch.grid],
        grid_w=[int(g[1]) for g in batch.grid], heads=batch.heads, has_cls=batch.has_cls)


def pack_l(batch, device=None, pin: bool = False) -> PackedL:
    tokens = np.concatenate(batch.tokens, axis=0)
    attn = np.stack(batch.attn_t2v, axis=0).astype(np.float32)
    return PackedL(to_torch(tokens, device, pin), to_torch(attn, device, pin),
                   [int(k) for k in batch.keep], batch.n_vision, batch.n_text, batch.heads)
