"""GPU parity of the equivalent token (no-CLS variant) against the float64 checker."""
import numpy as np
import pytest
import torch

from oracle import ficoco_oracle as fo
from paper_2411_17686_b200 import binding, synth

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
# fp32 sums of at most a few thousand terms of order one, then a quotient of magnitude <= 1:
# a few 1e-7 in practice; 5e-6 absolute leaves room for the longest images.
ATOL = 5e-6


def run(n_tokens, heads, dk, dtype, has_cls, seed, ragged):
    keys = synth.make_keys(seed, n_tokens, heads, dk, dtype)
    packed = np.concatenate([k.reshape(k.shape[0], heads * dk) for k in keys], axis=0)
    kt = binding.to_torch(packed, DEV)
    if ragged:
        got = binding.ficoco_equivalent_token(kt, heads, dk, seqlens=n_tokens, has_cls=has_cls)
    else:
        got = binding.ficoco_equivalent_token(kt, heads, dk, n_tokens=n_tokens[0], has_cls=has_cls)
    torch.cuda.synchronize()
    got = got.cpu().numpy()
    exp = np.concatenate([fo.equivalent_token(k, 1 if has_cls else 0) for k in keys])
    assert got.shape == exp.shape
    assert np.isfinite(got).all()
    np.testing.assert_allclose(got, exp, atol=ATOL, rtol=0)
    return kt, got


def test_uniform_batch_like_clip_large():
    # 32 images x (1 CLS + 576 patches), 16 heads of 64: the shape of the headline workload
    kt, a = run([577] * 32, 16, 64, "bf16", True, 301, ragged=False)
    # bit-reproducible: fixed summation order everywhere
    b = binding.ficoco_equivalent_token(kt, 16, 64, n_tokens=577, has_cls=True)
    assert np.array_equal(a, b.cpu().numpy())


def test_ragged_batch_without_cls_head_dim_80():
    r = np.random.default_rng(5)
    n = [int(h * w) for h, w in zip(r.integers(16, 65, 12), r.integers(16, 65, 12))]
    run(n, 16, 80, "bf16", False, 302, ragged=True)


@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
def test_small_and_degenerate_sizes(dtype):
    run([2, 3, 9, 17, 130], 4, 32, dtype, True, 303, ragged=True)      # fewer patches than CTAs in a cluster
    run([1, 1, 5], 2, 8, dtype, False, 304, ragged=True)               # one patch: a = -1
    run([40] * 3, 1, 256, dtype, False, 305, ragged=False)             # one head, widest head


def test_feeds_the_reduce_step_and_limits():
    keys = synth.make_keys(306, [100] * 2, 4, 16, "bf16")
    kt = binding.to_torch(np.concatenate([k.reshape(100, 64) for k in keys]), DEV)
    a = binding.ficoco_equivalent_token(kt, 4, 16, n_tokens=100, has_cls=False)
    batch = synth.make_v_batch(306, 2, 10, 10, 64, 1, 40, "bf16", False, 1.0)
    from paper_2411_17686_b200 import packing
    pk = packing.pack_v(batch, DEV)
    ctx = binding.Context(max_tokens=1000, max_dim=64, max_batch=2, max_text=0, device=0)
    try:
        prm = binding.make_params(has_cls=False)
        res = ctx.ficoco_v_reduce(pk.tokens, a, 40, 10, 10, 1, params=prm, **pk.call_kwargs())
        torch.cuda.synchronize()
        assert ctx.ficoco_status() == 0
        assert res.out_rows == [40, 40]
    finally:
        ctx.close()
    # an image too long for a cluster's shared memory, a misaligned row, a bad dtype
    big = torch.zeros((70000, 64), dtype=torch.bfloat16, device=DEV)
    with pytest.raises(binding.FicocoError):
        binding.ficoco_equivalent_token(big, 1, 64, n_tokens=70000, has_cls=False)
    odd = torch.zeros((8, 4), dtype=torch.bfloat16, device=DEV)
    with pytest.raises(binding.FicocoError):
        binding.ficoco_equivalent_token(odd, 1, 4, n_tokens=8, has_cls=False)
