"""Pins for the float64 checker: everything here is fixed by the paper's equations or by
mathematics, not by the checker itself (hand-worked values, an independent scalar-loop
transcription, closed forms, invariants, library routines for special cases)."""
import json
import os

import numpy as np
import pytest
import torch

from oracle import ficoco_oracle as fo
from paper_2411_17686_b200 import synth
from tests import brute_force as bf

HERE = os.path.dirname(os.path.abspath(__file__))


def tiny_v(seed, n_side=4, dim=8, heads=3, keep=10, dtype="fp32"):
    return synth.make_v_batch(seed, 1, n_side, n_side, dim, heads, keep, dtype, True, 1.0, corr_len=1.5)


# ---------------------------------------------------------------------------
# hand-worked example (Eq. 1, Eq. 2)
# ---------------------------------------------------------------------------

def test_hand_worked_example():
    g = json.load(open(os.path.join(HERE, "golden", "hand_example.json")))
    P = np.array(g["patches"], dtype=np.float32)
    attn = np.array(g["cls_attention"], dtype=np.float32)
    for case in g["cases"]:
        p = fo.Params(lam=g["lambda"], eps=case["eps"], local_penalty=False)
        r = fo.ficoco_v_reduce(P, attn, None, (2, 2), g["keep"], has_cls=False, p=p)
        # float32 storage of 0.1 / 0.4 attention limits the agreement to ~1e-8
        np.testing.assert_allclose(r.v, g["vision_redundancy"], atol=1e-12)
        np.testing.assert_allclose(r.score, g["score"], atol=1e-8)
        assert sorted(r.S.tolist()) == g["S"] and r.T.tolist() == g["T"]
        order = np.argsort(r.S)
        C = r.C[order]
        np.testing.assert_allclose(C, g["C"], atol=1e-12)
        for k, si in enumerate(order):
            assert r.J[si].tolist() == case["J"][k]
            np.testing.assert_allclose(r.alpha[si], case["alpha"][k], atol=1e-12)
        np.testing.assert_allclose(r.out.astype(np.float64), case["merged"], rtol=1e-6)
        assert r.kept_idx.tolist() == g["T"]


def _golden():
    return json.load(open(os.path.join(HERE, "golden", "hand_example.json")))


def check_fixed_k_hand_cases():
    """Fixed K on the hand-worked example: K = 1 is its eps = 1 case, K = 2 = N^T its eps = 0 case,
    and tau_i is the smallest correlation still taken."""
    g = _golden()
    P = np.array(g["patches"], dtype=np.float32)
    attn = np.array(g["cls_attention"], dtype=np.float32)
    for case in g["fixed_k_cases"]:
        p = fo.Params(lam=g["lambda"], local_penalty=False, max_targets=case["max_targets"])
        r = fo.ficoco_v_reduce(P, attn, None, (2, 2), g["keep"], has_cls=False, p=p)
        order = np.argsort(r.S)
        for k, si in enumerate(order):
            assert r.J[si].tolist() == case["J"][k]
            np.testing.assert_allclose(r.alpha[si], case["alpha"][k], atol=1e-12)
            np.testing.assert_allclose(r.tau[si], case["tau"][k], atol=1e-12)
        np.testing.assert_allclose(r.out.astype(np.float64), case["merged"], rtol=1e-6)


def check_tie_hand_cases():
    """Equal scores: across the selection boundary the lower token index is discarded; inside a
    local-penalty window the lower token index is the one multiplied."""
    t = _golden()["tie_cases"]
    P = np.array(t["patches"], dtype=np.float32)
    attn = np.array(t["cls_attention"], dtype=np.float32)
    for c in t["selection"]:
        r = fo.ficoco_v_reduce(P, attn, None, (2, 2), c["keep"], False, fo.Params(lam=t["lambda"], local_penalty=False))
        np.testing.assert_allclose(r.score, t["score"], atol=1e-8)
        assert r.score[0] == r.score[1] and r.score[2] == r.score[3]
        assert sorted(r.S.tolist()) == c["S"] and r.T.tolist() == c["T"]
        assert r.kept_idx.tolist() == c["T"]
    w = t["window"]
    r = fo.ficoco_v_reduce(P, attn, None, tuple(w["grid"]), w["keep"], False,
                           fo.Params(lam=t["lambda"], window=w["window"], penalty_coef=w["coef"]))
    np.testing.assert_allclose(r.score, w["score_after_penalty"], atol=1e-8)
    assert sorted(r.S.tolist()) == w["S"] and r.T.tolist() == w["T"]
    wo = t["window_only"]
    out = fo.local_penalty(np.array(wo["scores"]), np.array(wo["pos"]), tuple(wo["grid"]), wo["window"], wo["coef"])
    assert out.tolist() == wo["expected"]
    # the selection helper on its own, ties inside and across the boundary
    S, T = fo.filter_topk(np.array([0.3, 0.5, 0.5, 0.1, 0.5]), 2)
    assert S.tolist() == [1, 2] and T.tolist() == [0, 3, 4]
    S, T = fo.filter_topk(np.array([0.5, 0.5, 0.5]), 1)
    assert S.tolist() == [0] and T.tolist() == [1, 2]


def test_fixed_k_and_tie_hand_cases():
    check_fixed_k_hand_cases()
    check_tie_hand_cases()


# ---------------------------------------------------------------------------
# independent scalar-loop transcription on tiny inputs
# ---------------------------------------------------------------------------

def _compare_with_brute(r, b, P64):
    np.testing.assert_allclose(r.score_raw, b["s_raw"], rtol=0, atol=1e-12)
    np.testing.assert_allclose(r.score, b["s"], rtol=0, atol=1e-12)
    assert r.S.tolist() == b["S"]
    assert r.T.tolist() == b["T"]
    Tl = r.T.tolist()
    for k, i in enumerate(r.S.tolist()):
        assert [Tl[j] for j in r.J[k].tolist()] == b["J"][i]
        for jj, a in zip(r.J[k].tolist(), r.alpha[k].tolist()):
            assert abs(a - b["alpha"][(i, Tl[jj])]) < 1e-12
        for jj, j in enumerate(Tl):
            assert abs(r.C[k, jj] - b["C"][(i, j)]) < 1e-12
        if i in b["tau"]:
            assert abs(r.tau[k] - b["tau"][i]) < 1e-12
    return Tl


@pytest.mark.parametrize("seed", [1, 2, 3, 4])
@pytest.mark.parametrize("penalty", [True, False])
@pytest.mark.parametrize("eps", [0.998, 0.7])
def test_v_matches_brute_force(seed, penalty, eps):
    batch = tiny_v(seed)
    # knock out some grid cells so that padding of discarded positions is exercised
    alive = np.sort(synth.rng_for(seed, 9).permutation(16)[:13]).astype(np.int32)
    tok = np.concatenate([batch.tokens[0][:1], batch.tokens[0][1:][alive]])
    attn = batch.attn[0][:, alive]
    p = fo.Params(eps=eps, local_penalty=penalty)
    r = fo.ficoco_v_reduce(tok, attn, alive, (4, 4), 8, True, p)
    P = tok[1:].astype(np.float64)
    b = bf.reduce_v(P.tolist(), attn.astype(np.float64).tolist(), alive.tolist(), 4, 4, 8,
                    eps=eps, penalty=penalty)
    Tl = _compare_with_brute(r, b, P)
    for jj, j in enumerate(Tl):
        np.testing.assert_allclose(r.out[1 + jj].astype(np.float64), b["merged"][j], rtol=2e-7, atol=1e-7)
    assert r.kept_idx.tolist() == [0] + [1 + j for j in Tl]
    assert r.pos_out.tolist() == [int(alive[j]) for j in Tl]


@pytest.mark.parametrize("seed", [11, 12, 13])
@pytest.mark.parametrize("eps", [0.998, 0.6])
def test_l_matches_brute_force(seed, eps):
    lb = synth.make_l_batch(seed, 1, 14, 5, 8, 3, 6, "fp32", scale=1.0)
    p = fo.Params(eps=eps)
    r = fo.ficoco_l_reduce(lb.tokens[0], lb.attn_t2v[0], 14, 6, p)
    P = lb.tokens[0][:14].astype(np.float64)
    b = bf.reduce_l(P.tolist(), lb.attn_t2v[0].astype(np.float64).tolist(), 6, eps=eps)
    Tl = _compare_with_brute(r, b, P)
    for jj, j in enumerate(Tl):
        np.testing.assert_allclose(r.out[jj].astype(np.float64), b["merged"][j], rtol=2e-7, atol=1e-7)
    # text rows pass through untouched after the preserved vision rows
    assert np.array_equal(r.out[len(Tl):], lb.tokens[0][14:])
    assert r.kept_idx.tolist() == Tl + list(range(14, 19))


@pytest.mark.parametrize("seed", [1, 2, 3])
@pytest.mark.parametrize("kfix", [0, 1, 2, 3, 8, 11])
def test_fixed_k_matches_brute_force_v(seed, kfix):
    """Fixed-K ablation (every discarded token to its K most correlated targets) against the
    scalar transcription, K from 0 (pruning) to beyond N^T = 8."""
    batch = tiny_v(seed)
    tok, attn = batch.tokens[0], batch.attn[0]
    r = fo.ficoco_v_reduce(tok, attn, None, (4, 4), 8, True, fo.Params(max_targets=kfix))
    P = tok[1:].astype(np.float64)
    b = bf.reduce_v(P.tolist(), attn.astype(np.float64).tolist(), list(range(16)), 4, 4, 8, max_targets=kfix)
    Tl = _compare_with_brute(r, b, P)
    assert all(len(j) == min(kfix, 8) for j in r.J) or kfix == 0
    for jj, j in enumerate(Tl):
        np.testing.assert_allclose(r.out[1 + jj].astype(np.float64), b["merged"][j], rtol=2e-7, atol=1e-7)


@pytest.mark.parametrize("kfix", [1, 2, 3, 9])
def test_fixed_k_matches_brute_force_l(kfix):
    lb = synth.make_l_batch(14, 1, 14, 5, 8, 3, 6, "fp32", scale=1.0)
    r = fo.ficoco_l_reduce(lb.tokens[0], lb.attn_t2v[0], 14, 6, fo.Params(max_targets=kfix))
    P = lb.tokens[0][:14].astype(np.float64)
    b = bf.reduce_l(P.tolist(), lb.attn_t2v[0].astype(np.float64).tolist(), 6, max_targets=kfix)
    Tl = _compare_with_brute(r, b, P)
    for jj, j in enumerate(Tl):
        np.testing.assert_allclose(r.out[jj].astype(np.float64), b["merged"][j], rtol=2e-7, atol=1e-7)


def test_fixed_k_ties_go_to_the_lower_column():
    C = np.array([[0.5, 0.9, 0.9, 0.1], [0.2, 0.2, 0.2, 0.2]])
    J, A, tau = fo.targets_and_weights(C, fo.Params(max_targets=1))
    assert J[0].tolist() == [1] and J[1].tolist() == [0] and tau.tolist() == [0.9, 0.2]
    J, A, tau = fo.targets_and_weights(C, fo.Params(max_targets=3))
    assert J[0].tolist() == [0, 1, 2] and J[1].tolist() == [0, 1, 2] and tau.tolist() == [0.5, 0.2]
    np.testing.assert_allclose(A[0], np.array([0.5, 0.9, 0.9]) / 2.3, atol=1e-15)


def test_planted_mistakes_in_fixed_k_and_tie_rules_are_caught(monkeypatch):
    """The fixed-K branch and the two tie rules, each flipped in the checker, must break a pin."""
    real_tw, real_topk, real_pen = fo.targets_and_weights, fo.filter_topk, fo.local_penalty

    def fails(check):
        try:
            check()
        except AssertionError:
            return True
        return False

    def brute_k():
        batch = tiny_v(2)
        tok, attn = batch.tokens[0], batch.attn[0]
        P = tok[1:].astype(np.float64)
        for kfix in (1, 2, 3):
            r = fo.ficoco_v_reduce(tok, attn, None, (4, 4), 8, True, fo.Params(max_targets=kfix))
            b = bf.reduce_v(P.tolist(), attn.astype(np.float64).tolist(), list(range(16)), 4, 4, 8, max_targets=kfix)
            Tl = _compare_with_brute(r, b, P)
            for jj, j in enumerate(Tl):
                np.testing.assert_allclose(r.out[1 + jj].astype(np.float64), b["merged"][j], rtol=2e-7, atol=1e-7)

    assert not fails(brute_k) and not fails(check_fixed_k_hand_cases) and not fails(check_tie_hand_cases)

    def tw_variant(kind):
        def wrong(C, p):
            if p.max_targets is None or p.max_targets == 0:
                return real_tw(C, p)
            J, A, tau = [], [], np.full(C.shape[0], np.nan)
            for i in range(C.shape[0]):
                row = C[i]
                k = min(p.max_targets, C.shape[1])
                if kind == "one_more":
                    order = np.argsort(-row, kind="stable")[:k + 1]
                elif kind == "ascending":
                    order = np.argsort(row, kind="stable")[:k]
                else:
                    order = np.argsort(-row, kind="stable")[:k]
                tau[i] = row[order[0]] if kind == "tau_first" else row[order[-1]]
                j = np.sort(order)
                cpos = np.maximum(row[j], 0.0)
                J.append(j.astype(np.int64)); A.append(cpos / max(cpos.sum(), 1e-300))
            return J, A, tau
        return wrong

    for kind in ("one_more", "ascending", "tau_first"):
        with monkeypatch.context() as m:
            m.setattr(fo, "targets_and_weights", tw_variant(kind))
            assert fails(brute_k), f"fixed-K mistake '{kind}' passes the scalar transcription"
            assert fails(check_fixed_k_hand_cases), f"fixed-K mistake '{kind}' passes the hand example"

    def topk_high(s, n_src):     # ties to the higher index
        order = np.argsort(-s[::-1], kind="stable")
        S = (s.shape[0] - 1 - order)[:n_src]
        mask = np.ones(s.shape[0], dtype=bool)
        mask[S] = False
        return S.astype(np.int64), np.nonzero(mask)[0].astype(np.int64)

    def penalty_high(s, pos, grid, window, coef):   # ties inside a window to the higher index
        n = s.shape[0]
        return real_pen(s[::-1].copy(), np.asarray(pos)[::-1].copy(), grid, window, coef)[::-1].copy()

    with monkeypatch.context() as m:
        m.setattr(fo, "filter_topk", topk_high)
        assert fails(check_tie_hand_cases), "selection tie rule flipped, no pin noticed"
    with monkeypatch.context() as m:
        m.setattr(fo, "local_penalty", penalty_high)
        assert fails(check_tie_hand_cases), "window tie rule flipped, no pin noticed"


def test_planted_mistakes_are_caught(monkeypatch):
    """Each plausible slip in the checker must break agreement with the scalar transcription."""
    batch = tiny_v(5)
    tok, attn = batch.tokens[0], batch.attn[0]
    P = tok[1:].astype(np.float64)
    b = bf.reduce_v(P.tolist(), attn.astype(np.float64).tolist(), list(range(16)), 4, 4, 10, eps=0.6)

    def disagree():
        r = fo.ficoco_v_reduce(tok, attn, None, (4, 4), 10, True, fo.Params(eps=0.6))
        try:
            Tl = _compare_with_brute(r, b, P)
            for jj, j in enumerate(Tl):
                np.testing.assert_allclose(r.out[1 + jj].astype(np.float64), b["merged"][j],
                                           rtol=2e-7, atol=1e-7)
        except AssertionError:
            return True
        return False

    assert not disagree()
    mistakes = {
        "score_v": lambda v, a, lam: lam * v + (1 - lam) * a,                       # wrong sign
        "vision_redundancy": lambda R: (R.sum(axis=1) - 1.0) / R.shape[0],          # dropped j = i
        "correlation_v": lambda R, S, T: R[np.ix_(T, S)].T[::-1],                   # wrong index
        "head_mean": lambda attn: attn.astype(np.float64).sum(axis=0),              # no 1/H
        "quantile_threshold": lambda row, eps: float(np.sort(row)[int(eps * (len(row) - 1))]),  # no interpolation
    }
    for name, wrong in mistakes.items():
        with monkeypatch.context() as m:
            m.setattr(fo, name, wrong)
            assert disagree(), f"planted mistake in {name} went unnoticed"


# ---------------------------------------------------------------------------
# closed forms and invariants
# ---------------------------------------------------------------------------

def test_relation_properties_and_closed_form_row_mean():
    batch = synth.make_v_batch(21, 1, 6, 6, 32, 2, 20, "fp32")
    P = batch.tokens[0][1:].astype(np.float64)
    R = fo.cosine_relation(P)
    assert np.allclose(np.diag(R), 1.0, atol=1e-14)
    assert np.allclose(R, R.T, atol=1e-15)
    assert np.abs(R).max() <= 1.0 + 1e-14
    Ph = P / np.linalg.norm(P, axis=1, keepdims=True)
    closed = Ph @ Ph.mean(axis=0)           # (1/N) sum_j R_ij = x_hat_i . mean_j x_hat_j
    np.testing.assert_allclose(fo.vision_redundancy(R), closed, atol=1e-14)
    # against torch's cosine similarity routine
    tP = torch.from_numpy(P)
    Rt = torch.nn.functional.cosine_similarity(tP[:, None, :], tP[None, :, :], dim=-1).numpy()
    np.testing.assert_allclose(R, Rt, atol=1e-12)


def test_lambda_extremes():
    batch = synth.make_v_batch(22, 1, 6, 6, 32, 2, 20, "fp32")
    tok, attn = batch.tokens[0], batch.attn[0]
    r1 = fo.ficoco_v_reduce(tok, attn, None, (6, 6), 20, True, fo.Params(lam=1.0, local_penalty=False))
    assert set(r1.S.tolist()) == set(np.argsort(-r1.v, kind="stable")[:16].tolist())
    r0 = fo.ficoco_v_reduce(tok, attn, None, (6, 6), 20, True, fo.Params(lam=0.0, local_penalty=False))
    a = attn.astype(np.float64).mean(axis=0)
    assert set(r0.S.tolist()) == set(np.argsort(a, kind="stable")[:16].tolist())  # lowest CLS attention


def test_local_penalty_special_cases():
    batch = synth.make_v_batch(23, 1, 6, 6, 32, 2, 20, "fp32")
    tok, attn = batch.tokens[0], batch.attn[0]
    off = fo.ficoco_v_reduce(tok, attn, None, (6, 6), 20, True, fo.Params(local_penalty=False))
    one = fo.ficoco_v_reduce(tok, attn, None, (6, 6), 20, True, fo.Params(penalty_coef=1.0))
    assert np.array_equal(off.score, one.score) and np.array_equal(off.out, one.out)
    w1 = fo.ficoco_v_reduce(tok, attn, None, (6, 6), 20, True, fo.Params(window=1))
    np.testing.assert_allclose(w1.score, 2.0 * w1.score_raw, rtol=0, atol=0)
    # default: exactly one token per 2x2 window is doubled, and it is the window maximum
    d = fo.ficoco_v_reduce(tok, attn, None, (6, 6), 20, True)
    changed = np.nonzero(d.score != d.score_raw)[0]
    assert changed.shape[0] == 9
    grid = d.score_raw.reshape(3, 2, 3, 2).transpose(0, 2, 1, 3).reshape(9, 4)
    np.testing.assert_allclose(np.sort(d.score[changed]), np.sort(2.0 * grid.max(axis=1)))
    # odd grid: edge windows are smaller, discarded cells are padding
    s = np.array([0.3, -0.2, 0.1, 0.5, -0.4, -0.1], dtype=np.float64)
    pos = np.array([0, 1, 2, 3, 5, 8])
    out = fo.local_penalty(s, pos, (3, 3), 2, 2.0)
    # windows: {0,1,3,(4 dead)} -> max 0.5 at pos 3 ; {2,5} -> 0.1 ; {(6,7 dead)} none ; {8} -> -0.1
    np.testing.assert_allclose(out, [0.3, -0.2, 0.2, 1.0, -0.4, -0.2])


def test_selection_invariants_and_permutation_equivariance():
    batch = synth.make_v_batch(24, 1, 6, 6, 32, 2, 20, "fp32")
    tok, attn = batch.tokens[0], batch.attn[0]
    p = fo.Params(local_penalty=False)
    r = fo.ficoco_v_reduce(tok, attn, None, (6, 6), 20, True, p)
    assert r.out.shape[0] == 1 + 20 and r.kept_idx[0] == 0
    assert np.array_equal(r.out[0], tok[0])
    S, T = set(r.S.tolist()), set(r.T.tolist())
    assert not (S & T) and (S | T) == set(range(36)) and len(S) == 16
    assert np.all(np.diff(r.T) > 0)
    perm = synth.rng_for(24, 5).permutation(36)
    tok2 = np.concatenate([tok[:1], tok[1:][perm]])
    r2 = fo.ficoco_v_reduce(tok2, attn[:, perm], None, (6, 6), 20, True, p)
    assert set(perm[r2.S].tolist()) == S
    # same merged rows, in the permuted order
    inv = {int(perm[j]): k for k, j in enumerate(r2.T.tolist())}
    for k, j in enumerate(r.T.tolist()):
        np.testing.assert_allclose(r.out[1 + k], r2.out[1 + inv[j]], rtol=1e-6)


def test_quantile_matches_library_and_eps_one():
    rng = synth.rng_for(25)
    for n in (2, 3, 17, 288, 512, 1440):
        row = rng.standard_normal(n)
        for eps in (0.998, 0.5, 0.0, 1.0, 0.9731):
            assert abs(fo.quantile_threshold(row, eps) - float(np.quantile(row, eps))) < 1e-12
            tq = float(torch.quantile(torch.from_numpy(row), eps))
            assert abs(fo.quantile_threshold(row, eps) - tq) < 1e-12
    C = rng.standard_normal((5, 40))
    J, A, tau = fo.targets_and_weights(C, fo.Params(eps=1.0))
    for i in range(5):
        assert J[i].tolist() == [int(np.argmax(C[i]))] or C[i].max() <= 0
        if J[i].size:
            assert A[i].tolist() == [1.0]


def test_number_of_targets_follows_the_quantile_level():
    rng = synth.rng_for(26)
    for n, k in ((288, 1), (144, 1), (64, 1), (512, 2), (720, 2), (1440, 3)):
        C = np.abs(rng.standard_normal((3, n))) + 0.01
        J, A, _ = fo.targets_and_weights(C, fo.Params())
        for i in range(3):
            assert J[i].shape[0] == k == n - 1 - int(np.floor(0.998 * (n - 1)))
            assert abs(A[i].sum() - 1.0) < 1e-14
            assert set(J[i].tolist()) == set(np.argsort(-C[i])[:k].tolist())


def test_merge_invariants():
    batch = synth.make_v_batch(27, 1, 8, 8, 16, 2, 24, "fp32")
    tok, attn = batch.tokens[0], batch.attn[0]
    p = fo.Params(eps=0.9)
    r = fo.ficoco_v_reduce(tok, attn, None, (8, 8), 24, True, p)
    P = tok[1:].astype(np.float64)
    # total-mass identity: sum_j (1 + w_j) out_j = sum_{j in T} x_j + sum_{i in S, J_i != {}} x_i
    merged, wsum = fo.compress(P, r.S, r.T, r.J, r.alpha)
    lhs = ((1.0 + wsum)[:, None] * merged).sum(axis=0)
    used = [int(i) for k, i in enumerate(r.S) if r.J[k].size]
    rhs = P[r.T].sum(axis=0) + P[used].sum(axis=0)
    np.testing.assert_allclose(lhs, rhs, atol=1e-10)
    # a target with a single source keeps at least half of itself
    for jj in range(len(r.T)):
        srcs = [k for k in range(len(r.S)) if jj in r.J[k].tolist()]
        if len(srcs) == 1:
            assert 1.0 / (1.0 + wsum[jj]) >= 0.5
    # K = 0 is plain pruning: the output is a gather of the input rows
    r0 = fo.ficoco_v_reduce(tok, attn, None, (8, 8), 24, True, fo.Params(max_targets=0))
    assert np.array_equal(r0.out, tok[r0.kept_idx])
    assert np.array_equal(r0.T, r.T)
    # identical tokens merge to themselves
    same = np.repeat(tok[1:2], 65, axis=0)
    rs = fo.ficoco_v_reduce(same, attn, None, (8, 8), 24, True, p)
    np.testing.assert_allclose(rs.out, same[:25], rtol=1e-6)


def test_average_compression_is_the_group_mean():
    """Ablation 'average compression' (features averaged directly): same S, T, J_i as the default,
    every weight 1, merged rows equal to the plain mean of each group (scalar-loop routine that
    does not go through Eq. 2), rows of size-1 groups untouched, and the count-weighted mass
    identity sum_j |group_j| out_j = sum_{j in T} x_j + sum_i |J_i| x_i."""
    for seed, eps, kfix in ((6, 0.7, None), (7, 0.998, None), (8, 0.998, 2)):
        batch = tiny_v(seed)
        tok, attn = batch.tokens[0], batch.attn[0]
        P = tok[1:].astype(np.float64)
        base = fo.ficoco_v_reduce(tok, attn, None, (4, 4), 9, True, fo.Params(eps=eps, max_targets=kfix))
        r = fo.ficoco_v_reduce(tok, attn, None, (4, 4), 9, True,
                               fo.Params(eps=eps, max_targets=kfix, average_compression=True))
        assert r.S.tolist() == base.S.tolist() and r.T.tolist() == base.T.tolist()
        Tl, Sl = r.T.tolist(), r.S.tolist()
        J = {}
        for k, i in enumerate(Sl):
            assert r.J[k].tolist() == base.J[k].tolist()
            assert r.alpha[k].tolist() == [1.0] * len(r.J[k])
            J[i] = [Tl[jj] for jj in r.J[k].tolist()]
        means = bf.group_means(P.tolist(), Sl, Tl, J)
        sizes = {j: 1 + sum(1 for i in Sl if j in J[i]) for j in Tl}
        assert max(sizes.values()) > 1
        for jj, j in enumerate(Tl):
            np.testing.assert_allclose(r.out[1 + jj].astype(np.float64), means[j], rtol=2e-7, atol=1e-7)
            if sizes[j] == 1:
                assert np.array_equal(r.out[1 + jj], tok[1 + j])
        merged, wsum = fo.compress(P, r.S, r.T, r.J, r.alpha)
        assert wsum.tolist() == [float(sizes[j] - 1) for j in Tl]
        lhs = ((1.0 + wsum)[:, None] * merged).sum(axis=0)
        rhs = P[Tl].sum(axis=0) + sum(len(J[i]) * P[i] for i in Sl)
        np.testing.assert_allclose(lhs, rhs, atol=1e-10)
        # the default weights differ from 1 somewhere, so the two variants really differ
        if kfix is None and eps < 0.9:
            assert not np.array_equal(r.out, base.out)


def test_convergent_correlation_is_one_mean_token():
    """Ablation 'convergent correlation' (all discarded tokens merge into one additional token):
    same S and T as the default method, preserved rows untouched bit for bit, one appended row
    equal to the plain mean of the discarded rows (scalar loops), kept index -1 for it, the mass
    identity N^S * extra = sum_{i in S} x_i, a single discarded token reproduced exactly, nothing
    appended when nothing is discarded, and for FiCoCo-L the row sits before the text rows."""
    import math
    batch = tiny_v(41)
    tok, attn = batch.tokens[0], batch.attn[0]
    P = tok[1:].astype(np.float64)
    base = fo.ficoco_v_reduce(tok, attn, None, (4, 4), 9, True, fo.Params())
    r = fo.ficoco_v_reduce(tok, attn, None, (4, 4), 9, True, fo.Params(convergent=True))
    assert r.S.tolist() == base.S.tolist() and r.T.tolist() == base.T.tolist()
    assert r.out.shape[0] == 1 + 9 + 1 and r.kept_idx.tolist() == base.kept_idx.tolist() + [-1]
    assert np.array_equal(r.out[:10], tok[base.kept_idx])
    Sl = r.S.tolist()
    mean = [math.fsum(P[i][d] for i in Sl) / len(Sl) for d in range(P.shape[1])]
    np.testing.assert_allclose(r.out[10].astype(np.float64), mean, rtol=2e-7, atol=1e-7)
    np.testing.assert_allclose(len(Sl) * fo.convergent_token(P, r.S), P[Sl].sum(axis=0), atol=1e-12)
    assert r.pos_out.tolist() == base.pos_out.tolist()
    one = fo.ficoco_v_reduce(tok, attn, None, (4, 4), 15, True, fo.Params(convergent=True))
    assert one.out.shape[0] == 17 and np.array_equal(one.out[16], tok[1 + int(one.S[0])])
    none = fo.ficoco_v_reduce(tok, attn, None, (4, 4), 16, True, fo.Params(convergent=True))
    assert np.array_equal(none.out, tok) and none.kept_idx.tolist() == list(range(17))
    # bf16 storage: the mean is rounded once
    bb = synth.make_v_batch(42, 1, 4, 4, 8, 2, 6, "bf16", True, 1.0)
    rb = fo.ficoco_v_reduce(bb.tokens[0], bb.attn[0], None, (4, 4), 6, True, fo.Params(convergent=True))
    Pb = fo.widen(bb.tokens[0])[1:]
    exact = Pb[rb.S].sum(axis=0) / 10
    got = fo.widen(rb.out[-1])
    assert np.all(np.abs(got - exact) <= np.abs(exact) * 2.0 ** -8 + 1e-30)
    # FiCoCo-L: preserved vision rows, the additional token, then the text rows
    lb = synth.make_l_batch(43, 1, 14, 5, 8, 3, 6, "fp32", scale=1.0)
    ld = fo.ficoco_l_reduce(lb.tokens[0], lb.attn_t2v[0], 14, 6, fo.Params())
    lc = fo.ficoco_l_reduce(lb.tokens[0], lb.attn_t2v[0], 14, 6, fo.Params(convergent=True))
    assert lc.T.tolist() == ld.T.tolist() and lc.out.shape[0] == 6 + 1 + 5
    assert lc.kept_idx.tolist() == ld.T.tolist() + [-1] + list(range(14, 19))
    assert np.array_equal(lc.out[:6], lb.tokens[0][ld.T]) and np.array_equal(lc.out[7:], lb.tokens[0][14:])
    Pl = lb.tokens[0][:14].astype(np.float64)
    np.testing.assert_allclose(lc.out[6].astype(np.float64), Pl[lc.S].mean(axis=0), rtol=2e-7, atol=1e-7)


def test_relation_argument():
    """The relation argument replaces A^v everywhere and nothing else: (i) given the cosine
    similarity computed by torch it reproduces the default step; (ii) for a symmetric map the two
    directions of the mean agree; (iii) a row-stochastic map makes the printed first term of Eq. 1
    the constant 1/N, so the ranking is that of the attention term alone (lambda = 0); (iv) scores
    and C against scalar loops over the map."""
    batch = synth.make_v_batch(31, 1, 6, 6, 16, 3, 20, "fp32", True, 1.0)
    tok, attn = batch.tokens[0], batch.attn[0]
    P = torch.from_numpy(tok[1:].astype(np.float64))
    R = torch.nn.functional.cosine_similarity(P[:, None, :], P[None, :, :], dim=-1).numpy()
    p = fo.Params(eps=0.9)
    r_def = fo.ficoco_v_reduce(tok, attn, None, (6, 6), 20, True, p)
    for by_col in (False, True):
        r = fo.ficoco_v_reduce(tok, attn, None, (6, 6), 20, True, p, relation=R, by_column=by_col)
        np.testing.assert_allclose(r.score, r_def.score, atol=1e-13)
        assert r.S.tolist() == r_def.S.tolist() and r.kept_idx.tolist() == r_def.kept_idx.tolist()
        assert all(a.tolist() == b.tolist() for a, b in zip(r.J, r_def.J))
        np.testing.assert_allclose(r.out, r_def.out, rtol=1e-6, atol=1e-7)
    A = synth.relation_map(synth.rng_for(31, 5), tok[1:]).astype(np.float64)
    np.testing.assert_allclose(A.sum(axis=1), 1.0, atol=1e-6)
    pn = fo.Params(local_penalty=False)
    r_row = fo.ficoco_v_reduce(tok, attn, None, (6, 6), 20, True, pn, relation=A)
    r_att = fo.ficoco_v_reduce(tok, attn, None, (6, 6), 20, True, fo.Params(lam=0.0, local_penalty=False))
    np.testing.assert_allclose(r_row.v, 1.0 / 36, atol=1e-8)
    assert sorted(r_row.S.tolist()) == sorted(r_att.S.tolist())
    r_col = fo.ficoco_v_reduce(tok, attn, None, (6, 6), 20, True, pn, relation=A, by_column=True)
    a_mean = attn.astype(np.float64).mean(axis=0)
    for i in range(36):
        received = sum(A[j, i] for j in range(36)) / 36
        assert abs(r_col.score_raw[i] - (0.35 * received - 0.65 * a_mean[i])) < 1e-12
    for k, i in enumerate(r_col.S.tolist()):
        for jj, j in enumerate(r_col.T.tolist()):
            assert r_col.C[k, jj] == A[i, j]
    assert not np.array_equal(r_col.S, r_row.S) or not np.allclose(r_col.score_raw, r_row.score_raw)


def test_untouched_rows_keep_their_bits_and_bf16_rounding():
    batch = synth.make_v_batch(28, 2, 8, 8, 64, 2, 40, "bf16")
    for b in range(2):
        r = fo.ficoco_v_reduce(batch.tokens[b], batch.attn[b], None, (8, 8), 40, True)
        untouched = np.nonzero(r.wsum == 0)[0]
        assert untouched.size > 0
        assert np.array_equal(r.out[1 + untouched], batch.tokens[b][1 + r.T[untouched]])
    # the float64 -> bf16 rounding against torch's own conversion, incl. exact halfway cases
    rng = synth.rng_for(28, 1)
    x = rng.standard_normal(20000) * np.exp(rng.uniform(-20, 20, 20000))
    half = (np.arange(1, 200, dtype=np.float64) * 2 + 1) / 512.0   # 9 significant bits: ties
    x = np.concatenate([x, half, -half, [0.0, 1.0, -1.0, 3.0 + 2.0 ** -8, 3.0 + 2.0 ** -7]])
    mine = fo.round_to_bf16_bits(x)
    ref = torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(mine, ref)
    assert np.array_equal(fo.widen(mine), synth.bf16_bits_to_f32(mine).astype(np.float64))
    # widening against torch's own reinterpretation of the bits as bfloat16, all finite patterns
    bits = np.arange(65536, dtype=np.uint32).astype(np.uint16)
    finite = (bits & 0x7F80) != 0x7F80
    tw = torch.from_numpy(bits.view(np.int16).copy()).view(torch.bfloat16).to(torch.float64).numpy()
    assert np.array_equal(fo.widen(bits[finite]), tw[finite])
    assert np.array_equal(np.signbit(fo.widen(bits[finite])), np.signbit(tw[finite]))


def test_ficoco_l_special_cases():
    lb = synth.make_l_batch(29, 1, 40, 6, 32, 3, 12, "fp32", scale=1.0)
    tok, att = lb.tokens[0], lb.attn_t2v[0]
    t = fo.head_mean(att)
    P = tok[:40].astype(np.float64)
    R = fo.cosine_relation(P)
    r = fo.ficoco_l_reduce(tok, att, 40, 12, fo.Params(gamma=1.0))
    np.testing.assert_allclose(r.C, R[np.ix_(r.S, r.T)], atol=0)
    rb = fo.ficoco_l_reduce(tok, att, 40, 12, fo.Params(beta=1.0))
    np.testing.assert_allclose(rb.score, fo.vision_redundancy(R), atol=0)
    G = t.T @ t / t.shape[0]
    assert np.allclose(G, G.T) and np.linalg.eigvalsh(G).min() > -1e-12
    full = fo.ficoco_l_reduce(tok, att, 40, 12)
    expect = 0.6 * R[np.ix_(full.S, full.T)] + 0.4 * G[np.ix_(full.S, full.T)]
    np.testing.assert_allclose(full.C, expect, atol=1e-15)
    assert full.out.shape[0] == 12 + 6


def test_edge_counts():
    batch = synth.make_v_batch(30, 1, 4, 4, 8, 2, 16, "fp32")
    tok, attn = batch.tokens[0], batch.attn[0]
    r = fo.ficoco_v_reduce(tok, attn, None, (4, 4), 16, True)      # discard nothing
    assert np.array_equal(r.out, tok) and r.S.size == 0
    r = fo.ficoco_v_reduce(tok, attn, None, (4, 4), 0, True)       # discard everything
    assert r.out.shape[0] == 1 and np.array_equal(r.out[0], tok[0])
    r = fo.ficoco_v_reduce(tok, attn, None, (4, 4), 1, True)       # one target takes it all
    assert r.out.shape[0] == 2 and all(j.tolist() == [0] for j in r.J if j.size)


# ---------------------------------------------------------------------------
# equivalent token (appendix "Implementation of the Equivalent Token")
# ---------------------------------------------------------------------------

def _eq_token_loops(keys, n_cls):
    """Scalar-loop transcription of the appendix equations (independent of the checker)."""
    T, H, d = keys.shape
    M = [[sum(float(keys[t, h, o]) for h in range(H)) / H for o in range(d)] for t in range(T)]
    P = M[n_cls:]
    mu = [sum(P[i][o] for i in range(len(P))) / len(P) for o in range(d)]
    n_mu = sum(x * x for x in mu) ** 0.5
    out = []
    for row in P:
        n_r = sum(x * x for x in row) ** 0.5
        out.append(-sum(a * b for a, b in zip(mu, row)) / (n_mu * n_r))
    return np.array(out)


def test_equivalent_token_closed_forms():
    # identical patch keys: every cosine with their mean is 1, so a = -1
    k = np.tile(np.array([[[0.3, -1.2, 2.0]]], dtype=np.float32), (5, 2, 1))
    np.testing.assert_allclose(fo.equivalent_token(k, 0), -1.0, atol=1e-12)
    # two orthogonal patch keys of equal length: cos(mean, each) = 1/sqrt(2)
    k = np.zeros((2, 1, 2), dtype=np.float32)
    k[0, 0] = [2, 0]
    k[1, 0] = [0, 2]
    np.testing.assert_allclose(fo.equivalent_token(k, 0), -1.0 / np.sqrt(2.0), atol=1e-12)
    # P = [3u, -u]: the mean is u, so the first token is aligned (a = -1), the second opposed (a = +1)
    u = np.array([0.6, -0.8, 0.0], dtype=np.float32)
    k = np.stack([3 * u, -u])[:, None, :]
    np.testing.assert_allclose(fo.equivalent_token(k.astype(np.float32), 0), [-1.0, 1.0], atol=1e-7)
    # a zero patch key (reading: a = 0) next to ordinary ones
    k = np.array([[[0.0, 0.0]], [[1.0, 0.0]], [[1.0, 1.0]]], dtype=np.float32)
    a = fo.equivalent_token(k, 0)
    assert a[0] == 0.0 and a[1] < 0.0 and a[2] < 0.0


def test_equivalent_token_invariants_and_loops():
    keys = synth.make_keys(11, [9], 3, 5, "fp32")[0]
    a = fo.equivalent_token(keys, 1)
    assert a.shape == (8,) and np.all(np.abs(a) <= 1.0 + 1e-12)
    np.testing.assert_allclose(a, _eq_token_loops(keys, 1), atol=1e-12)
    # the CLS row takes no part; a common positive scale changes nothing
    k2 = keys.copy()
    k2[0] = 123.0
    np.testing.assert_allclose(fo.equivalent_token(k2, 1), a, atol=1e-12)
    np.testing.assert_allclose(fo.equivalent_token((4.0 * keys).astype(np.float32), 1), a, atol=1e-6)
    # heads enter only through their mean: one head holding that mean gives the same result
    m = keys.astype(np.float64).mean(axis=1, keepdims=True)
    np.testing.assert_allclose(fo.equivalent_token(m.astype(np.float32), 1), a, atol=1e-6)
    # without the CLS exclusion the first row would be scored too
    assert fo.equivalent_token(keys, 0).shape == (9,)
    # a planted mistake (mean taken over all rows, CLS included) must not survive the loops pin
    M = keys.astype(np.float64).mean(axis=1)
    mu_wrong = M.mean(axis=0)
    wrong = -(M[1:] @ mu_wrong) / (np.linalg.norm(M[1:], axis=1) * np.linalg.norm(mu_wrong))
    assert np.max(np.abs(wrong - _eq_token_loops(keys, 1))) > 1e-3
    # bf16 storage is widened exactly
    kb = synth.make_keys(12, [6], 2, 4, "bf16")[0]
    kf = synth.bf16_bits_to_f32(kb)
    np.testing.assert_allclose(fo.equivalent_token(kb, 0), fo.equivalent_token(kf, 0), atol=0)
