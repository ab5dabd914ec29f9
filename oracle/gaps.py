"""Decision margins of a reduce step, and deterministic input repair.

TEST INFRASTRUCTURE ONLY (uses the float64 checker; never imported by the product).

The reduce step takes three kinds of discontinuous decisions: which score wins a
local-penalty window, where the top-N^S selection boundary falls, and which preserved
tokens pass the quantile threshold tau_i of a discarded token.  An fp32 GPU path and a
float64 checker can only agree bit-exactly on those decisions when the competing values
are further apart than fp32 rounding noise.  ``margins`` measures the distances;
``repair_v`` / ``repair_l`` perturb the *inputs* (never the expected outputs) until
every distance exceeds its floor, so that both implementations are then given the same,
unambiguous problem.

Repairs applied (each is a change of the synthetic input, recorded in the returned log):
  * selection boundary / window winner too close: the attention column of the lower of
    the two competing tokens is raised (its score falls by (1-lam) * delta);
  * quantile decision too close in row i: a small fresh Gaussian perturbation is added to
    discarded token i's features and the row is re-rounded to the storage dtype.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import List, Optional, Tuple

import numpy as np

from . import ficoco_oracle as fo

SEL_GAP = 2e-4     # floor on the score gap at the top-N^S boundary
WIN_GAP = 1e-5     # floor on the top-1 / top-2 raw-score gap inside a penalty window
ROW_GAP = 1e-5     # floor on the distances around tau_i in a correlation row


@dataclass
class Margins:
    sel_gap: float
    sel_pair: Tuple[int, int]          # (last discarded, first preserved) patch indices
    win_gap: float
    win_pairs: List[Tuple[int, int]]   # (winner, runner-up) pairs closer than WIN_GAP
    row_gap: float
    bad_rows: List[int]                # positions in S whose tau decision is too close


def margins(res: fo.StepResult, pos: Optional[np.ndarray], grid: Optional[Tuple[int, int]],
            p: fo.Params, penalty: bool) -> Margins:
    s = res.score
    ns = res.S.shape[0]
    order = np.argsort(-s, kind="stable")
    if 0 < ns < s.shape[0]:
        sel_gap = float(s[order[ns - 1]] - s[order[ns]])
        sel_pair = (int(order[ns - 1]), int(order[ns]))
    else:
        sel_gap, sel_pair = np.inf, (-1, -1)

    win_gap, win_pairs = np.inf, []
    if penalty and pos is not None:
        gw = grid[1]
        nwc = -(-gw // p.window)
        wid = (pos // gw // p.window) * nwc + (pos % gw) // p.window
        raw = res.score_raw
        by_win = {}
        for i in range(raw.shape[0]):
            by_win.setdefault(int(wid[i]), []).append(i)
        for w, members in by_win.items():
            if len(members) < 2:
                continue
            vals = raw[members]
            o = np.argsort(-vals, kind="stable")
            g = float(vals[o[0]] - vals[o[1]])
            win_gap = min(win_gap, g)
            if g < WIN_GAP:
                win_pairs.append((members[o[0]], members[o[1]]))

    row_gap, bad_rows = np.inf, []
    C = res.C
    nt = C.shape[1] if C.ndim == 2 else 0
    if nt >= 2 and p.max_targets != 0:
        for i in range(C.shape[0]):
            v = np.sort(C[i])
            if p.max_targets is None:
                tau = res.tau[i]
                q = p.eps * (nt - 1)
                lo = int(np.floor(q)); hi = min(lo + 1, nt - 1)
                if q == lo:
                    # tau is the order statistic v[lo] itself (it passes by equality on both
                    # sides); what must be unambiguous is which element holds that rank
                    g = float(v[lo] - v[lo - 1]) if lo >= 1 else np.inf
                else:
                    g = float(np.abs(v - tau).min())
                    # the two order statistics the interpolation uses must be distinct
                    g = min(g, float(v[hi] - v[lo]))
            else:
                k = min(p.max_targets, nt)
                g = float(v[nt - k] - v[nt - k - 1]) if k < nt else np.inf
            row_gap = min(row_gap, g)
            if g < ROW_GAP:
                bad_rows.append(i)
    return Margins(sel_gap, sel_pair, win_gap, win_pairs, row_gap, bad_rows)


def ok(m: Margins) -> bool:
    return m.sel_gap >= SEL_GAP and m.win_gap >= WIN_GAP and m.row_gap >= ROW_GAP


def _band(res: fo.StepResult, m: Margins, rng: np.random.Generator, coeff: float):
    """Preserved tokens whose score lies within 1.5 * SEL_GAP of the last discarded one,
    with the attention increase that takes each of them below that band."""
    if coeff < 1e-3:
        raise ValueError("the attention term has (almost) no weight in the score: it cannot move the boundary")
    s_hi = res.score[m.sel_pair[0]]
    out = []
    for j in res.T.tolist():
        short = 1.5 * SEL_GAP - (s_hi - res.score[j])
        if short > 0.0:
            out.append((int(j), (short + 1e-5 * rng.random()) / coeff))
    return out


def _perturb_row(tokens: np.ndarray, row: int, rng: np.random.Generator, rel: float = 0.02) -> None:
    x = fo.widen(tokens[row:row + 1])[0]
    scale = rel * float(np.sqrt(np.mean(x * x)) + 1e-30)
    x = x + scale * rng.standard_normal(x.shape[0])
    tokens[row] = fo.round_like(x[None, :], tokens)[0]


def repair_v(batch, p: Optional[fo.Params] = None, max_iter: int = 40, seed: int = 7) -> List[str]:
    """Perturb a synthetic VBatch in place until every image's margins clear the floors.
    Returns a log of the changes made."""
    p = p or fo.Params()
    log: List[str] = []
    c = 1 if batch.has_cls else 0
    for b in range(batch.batch):
        for it in range(max_iter):
            res = fo.ficoco_v_reduce(batch.tokens[b], batch.attn[b], batch.pos[b], batch.grid[b],
                                     batch.keep[b], batch.has_cls, p)
            m = margins(res, batch.pos[b].astype(np.int64), batch.grid[b], p, p.local_penalty)
            if ok(m):
                break
            rng = np.random.Generator(np.random.Philox(key=[seed, (b << 16) | it]))
            if m.win_gap < WIN_GAP:
                for (_win, second) in m.win_pairs:
                    d = (2.0 * WIN_GAP + 1e-6 * rng.random()) / (1.0 - p.lam)
                    batch.attn[b][:, second] += np.float32(d)
                    log.append(f"img {b} it {it}: window runner-up {second} attn += {d:.3e}")
            elif m.sel_gap < SEL_GAP:
                # every preserved token inside the band below the last discarded score moves
                # further down (a penalty winner moves by coef times as much, which only helps)
                for lower, d in _band(res, m, rng, 1.0 - p.lam):
                    batch.attn[b][:, lower] += np.float32(d)
                    log.append(f"img {b} it {it}: boundary token {lower} attn += {d:.3e}")
            else:
                for i in m.bad_rows:
                    _perturb_row(batch.tokens[b], c + int(res.S[i]), rng)
                    log.append(f"img {b} it {it}: perturbed discarded token {int(res.S[i])}")
        else:
            raise RuntimeError(f"image {b}: margins not repaired after {max_iter} iterations: {m}")
    return log


def repair_v_relation(batch, rels: List[np.ndarray], by_column: bool, p: Optional[fo.Params] = None,
                      max_iter: int = 60, seed: int = 11) -> List[str]:
    """repair_v for the relation mode (rels[b]: fp32 [Np, Np] map of image b, changed in place).
    Window and boundary margins are repaired through the attention columns as in repair_v; a
    correlation row that is too close to its threshold gets that discarded token's row of the map
    rescaled entry by entry by a few per cent."""
    p = p or fo.Params()
    log: List[str] = []
    for b in range(batch.batch):
        for it in range(max_iter):
            res = fo.ficoco_v_reduce(batch.tokens[b], batch.attn[b], batch.pos[b], batch.grid[b],
                                     batch.keep[b], batch.has_cls, p, relation=rels[b], by_column=by_column)
            m = margins(res, batch.pos[b].astype(np.int64), batch.grid[b], p, p.local_penalty)
            if ok(m):
                break
            rng = np.random.Generator(np.random.Philox(key=[seed, (b << 16) | it]))
            if m.win_gap < WIN_GAP:
                for (_win, second) in m.win_pairs:
                    d = (2.0 * WIN_GAP + 1e-6 * rng.random()) / (1.0 - p.lam)
                    batch.attn[b][:, second] += np.float32(d)
                    log.append(f"img {b} it {it}: window runner-up {second} attn += {d:.3e}")
            elif m.sel_gap < SEL_GAP:
                for lower, d in _band(res, m, rng, 1.0 - p.lam):
                    batch.attn[b][:, lower] += np.float32(d)
                    log.append(f"img {b} it {it}: boundary token {lower} attn += {d:.3e}")
            else:
                for i in m.bad_rows:
                    row = int(res.S[i])
                    f = 1.0 + 0.05 * rng.standard_normal(rels[b].shape[1])
                    rels[b][row] = (rels[b][row].astype(np.float64) * np.abs(f)).astype(np.float32)
                    log.append(f"img {b} it {it}: rescaled relation row {row}")
        else:
            raise RuntimeError(f"image {b}: margins not repaired after {max_iter} iterations: {m}")
    return log


def repair_l(batch, p: Optional[fo.Params] = None, max_iter: int = 40, seed: int = 7) -> List[str]:
    """Same for a synthetic LBatch (no windows; the score's attention term is the text->vision
    column mean, moved by raising that column for every head and text row)."""
    p = p or fo.Params()
    log: List[str] = []
    for b in range(batch.batch):
        for it in range(max_iter):
            res = fo.ficoco_l_reduce(batch.tokens[b], batch.attn_t2v[b], batch.n_vision, batch.keep[b], p)
            m = margins(res, None, None, p, False)
            if ok(m):
                break
            rng = np.random.Generator(np.random.Philox(key=[seed, (b << 16) | it]))
            if m.sel_gap < SEL_GAP:
                for lower, d in _band(res, m, rng, 1.0 - p.beta):
                    batch.attn_t2v[b][:, :, lower] += np.float32(d)
                    log.append(f"seq {b} it {it}: boundary token {lower} attn += {d:.3e}")
            else:
                for i in m.bad_rows:
                    _perturb_row(batch.tokens[b], int(res.S[i]), rng)
                    log.append(f"seq {b} it {it}: perturbed discarded token {int(res.S[i])}")
        else:
            raise RuntimeError(f"sequence {b}: margins not repaired after {max_iter} iterations: {m}")
    return log
