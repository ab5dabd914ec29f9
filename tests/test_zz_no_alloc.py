"""The allocation-free entry point, for callers that must not allocate device memory (a
serving engine's step callback, say, whose engine owns every byte of it): its result has to
equal what the ordinary, context-based entry point computes.

ficoco_v_reduce with lambda = 1 and the local penalty off returns exactly the vision-aware
redundancy as its scores, so that is the reference.  Two calls in a row, the second on a
different and smaller batch, show that the fixed scratch array carries nothing over from one
call to the next.  This file sorts last on purpose: a run that stops at the first failure has
then already run every other test.
"""
import numpy as np
import pytest
import torch

from oracle import ficoco_oracle as fo
from paper_2411_17686_b200 import binding, packing, synth

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _reference(ctx, pk, n_tokens):
    prm = binding.make_params(lam=1.0, local_penalty=False)
    res = ctx.ficoco_v_reduce(pk.tokens, pk.attn, pk.keep, pk.grid_h, pk.grid_w, pk.heads, params=prm,
                              want_scores=True, n_tokens=n_tokens, pos=pk.pos)
    return binding.to_numpy(res.scores).astype(np.float64)


def test_noalloc_matches_context_entry_point_twice():
    ctx = binding.Context(max_tokens=8192, max_dim=1024, max_batch=8, device=0)
    cases = [synth.make_v_batch(901, 5, 14, 13, 384, 3, 90, "bf16", True, 1.0),
             synth.make_v_batch(902, 2, 7, 9, 96, 2, 30, "fp32", True, 1.0)]
    for batch in cases:
        n_tokens = batch.tokens[0].shape[0]
        pk = packing.pack_v(batch, DEV)
        want = _reference(ctx, pk, n_tokens)
        v_out = torch.full((batch.batch * (n_tokens - 1),), float("nan"), dtype=torch.float32, device=DEV)
        got = binding.ficoco_vision_redundancy_noalloc(pk.tokens, n_tokens, True, v_out=v_out)
        torch.cuda.synchronize()
        got = got.cpu().numpy().astype(np.float64)
        scale = float(np.mean(np.abs(want)))
        assert np.all(np.abs(got - want) <= 1e-5 * np.maximum(np.abs(want), scale))
        # and against the float64 checker: the first term of Eq. 1 from the literal N x N relation
        np_ = n_tokens - 1
        for b in range(batch.batch):
            P = fo.widen(batch.tokens[b])[1:]
            exact = fo.vision_redundancy(fo.cosine_relation(P))
            assert np.all(np.abs(got[b * np_:(b + 1) * np_] - exact) <= 1e-5 * np.abs(exact) + 1e-7)
    ctx.close()


def test_noalloc_rejects_what_does_not_fit():
    lib = binding.load_library()
    t = torch.zeros((16, 4096), dtype=torch.bfloat16, device=DEV)
    v = torch.zeros((16,), dtype=torch.float32, device=DEV)
    args = lambda batch, n, dim: lib.ficoco_vision_redundancy_noalloc(  # noqa: E731
        t.data_ptr(), binding.FICOCO_BF16, batch, n, dim, 0, v.data_ptr(), None)
    assert args(1, 16, 4096) == -9          # hidden size beyond the fixed scratch
    assert args(65, 4, 64) == -9            # too many images
    assert args(64, 1024, 64) == -9         # too many token rows in total
    assert args(1, 16, 12) == -2            # rows not 16-byte aligned
    assert b"allocation-free" in lib.ficoco_strerror(-9)
