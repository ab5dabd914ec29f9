"""The input-repair harness: after it ran, every discontinuous decision of the reduce step
has a margin above its floor, the repair is deterministic, and it only touches inputs."""
import copy

import numpy as np
import pytest

from oracle import ficoco_oracle as fo, gaps
from paper_2411_17686_b200 import synth


@pytest.mark.parametrize("idx", [1, 2, 3, 4])
def test_repair_v_clears_margins(idx):
    batch = synth.workload(idx, small=True)
    before = copy.deepcopy(batch)
    log = gaps.repair_v(batch)
    p = fo.Params()
    for b in range(batch.batch):
        r = fo.ficoco_v_reduce(batch.tokens[b], batch.attn[b], batch.pos[b], batch.grid[b],
                               batch.keep[b], batch.has_cls, p)
        m = gaps.margins(r, batch.pos[b].astype(np.int64), batch.grid[b], p, True)
        assert gaps.ok(m), m
        assert batch.tokens[b].shape == before.tokens[b].shape
        assert batch.tokens[b].dtype == before.tokens[b].dtype
    again = copy.deepcopy(before)
    assert gaps.repair_v(again) == log
    for b in range(batch.batch):
        assert np.array_equal(again.tokens[b], batch.tokens[b])
        assert np.array_equal(again.attn[b], batch.attn[b])


def test_repair_l_clears_margins():
    batch = synth.workload(5, small=True)
    gaps.repair_l(batch)
    p = fo.Params()
    for b in range(batch.batch):
        r = fo.ficoco_l_reduce(batch.tokens[b], batch.attn_t2v[b], batch.n_vision, batch.keep[b], p)
        assert gaps.ok(gaps.margins(r, None, None, p, False))


def test_margins_flag_a_planted_near_tie():
    batch = synth.make_v_batch(3, 1, 6, 6, 32, 2, 20, "fp32")
    gaps.repair_v(batch)
    p = fo.Params()
    r = fo.ficoco_v_reduce(batch.tokens[0], batch.attn[0], None, (6, 6), 20, True, p)
    m = gaps.margins(r, batch.pos[0].astype(np.int64), (6, 6), p, True)
    # move the first preserved token's score to within 1e-5 of the last discarded one
    hi, lo = m.sel_pair
    shift = (m.sel_gap - 1e-5) / (1.0 - p.lam)
    scale = 2.0 if r.score[lo] != r.score_raw[lo] else 1.0
    batch.attn[0][:, lo] -= np.float32(shift / scale)
    r2 = fo.ficoco_v_reduce(batch.tokens[0], batch.attn[0], None, (6, 6), 20, True, p)
    m2 = gaps.margins(r2, batch.pos[0].astype(np.int64), (6, 6), p, True)
    assert not gaps.ok(m2)
