"""CPU checker for the FiCoCo reduce step (filter -> correlate -> compress -> compact).

TEST INFRASTRUCTURE ONLY.  This is a plain, slow, float64 restatement of what the
paper defines, used to judge the CUDA library.  It shares no code with the CUDA path,
is never imported by the product package, and must not be tuned for speed.

Each function names the passage of the paper it follows:
  * Eq. 1 (Sec. "Redundancy-based Token Discard"): redundancy score s^v
  * local penalty paragraph of the same section, window 2x2, coefficient 2
    (Sec. "Implementation Details")
  * Sec. "Correlation-based Information Recycling": correlation matrix C, token-wise
    quantile threshold tau_i, sets J_i / I_j
  * Eq. 2: self-preserving compression and the weights alpha_ij
  * Sec. "Task-Aware Improvements for FiCoCo-L": s^l and C^l
  * Algorithm 1 / Algorithm 2: order of the steps, output = X without the rows of S
  * Appendix "Implementation of the Equivalent Token": a^Eq from the key states

Readings taken where the paper is silent:
  * the token-token relation A_{i,j} between two vision tokens is the cosine similarity
    R = X_hat X_hat^T of the layer's hidden states (the paper itself uses cosine
    similarity in place of attention for encoders without CLS, Appendix
    "Implementation of the Equivalent Token");
  * the CLS token is never scored, discarded or merged into; "N" in the 1/N of Eq. 1 is
    the number of alive patch tokens and the j = i term is included;
  * multi-head attention is averaged over heads;
  * the quantile is the linearly interpolated order statistic at eps*(n-1);
  * weights use max(C, 0) (cosine can be negative, attention cannot); a discarded token
    whose positive mass is zero is pruned;
  * all preserved tokens are updated at once from the pre-update X;
  * "average compression" (ablation tables; "directly averaging the features") keeps J_i as
    it is and sets every alpha_ij to 1, whatever the sign of C_ij;
  * "convergent correlation" (ablation tables; Sec. "Correlation-based Information Recycling":
    all discarded tokens merge into one additional token) says nothing about weights: the
    additional token is the plain mean of the discarded tokens, it is appended after the
    preserved vision tokens (before the text rows of FiCoCo-L), preserved tokens stay as they
    are, and its kept index is -1; with nothing discarded there is no additional token;
  * for FiCoCo-L the supplied text->vision block t (head mean, M x N) is used for both
    the task term (1/M) sum_k t[k,i] and the text-bridged term (1/M) sum_k t[k,i] t[k,j]
    (main-text equations, which carry the 1/M that Algorithm 2 omits).

bf16 tensors are uint16 bit patterns; they are widened exactly to float64.  Merged rows
are computed in float64 and rounded once (round-to-nearest-even) to the I/O dtype;
rows that receive nothing are copied bit for bit.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Dict, List, Optional, Tuple

import numpy as np


# ----------------------------------------------------------------------------
# Hyper-parameters (Sec. "Implementation Details")
# ----------------------------------------------------------------------------

@dataclass
class Params:
    lam: float = 0.35          # lambda, Eq. 1
    beta: float = 0.6          # beta, s^l
    gamma: float = 0.6         # gamma, C^l
    eps: float = 0.998         # quantile level for tau_i
    penalty_coef: float = 2.0  # local-penalty scaling coefficient
    window: int = 2            # local-penalty window side
    local_penalty: bool = True
    max_targets: Optional[int] = None  # None: token-adaptive K (paper); 0: pruning; k>0: fixed K
    average_compression: bool = False  # ablation "average compression": every alpha_ij = 1
    convergent: bool = False           # ablation "convergent correlation": one additional token


# ----------------------------------------------------------------------------
# Storage format helpers
# ----------------------------------------------------------------------------

def widen(tokens: np.ndarray) -> np.ndarray:
    """fp32 array or uint16 bf16 bit patterns -> float64, exactly."""
    if tokens.dtype == np.uint16:
        return (tokens.astype(np.uint32) << np.uint32(16)).view(np.float32).astype(np.float64)
    if tokens.dtype == np.float32:
        return tokens.astype(np.float64)
    raise TypeError(f"tokens must be float32 or uint16 (bf16 bits), got {tokens.dtype}")


def round_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """float64 -> bf16 bit patterns with a single round-to-nearest-even.

    bf16 keeps 8 significand bits (7 stored); a float64 stores 52, so the low 45 stored
    bits are rounded away on the integer representation.  Valid for finite values in the
    normal range of bf16 (|x| >= 2^-126 or x == 0), which is all this checker produces."""
    b = np.ascontiguousarray(x, dtype=np.float64).view(np.int64)
    drop = np.int64(45)
    lsb = (b >> drop) & np.int64(1)
    b = b + ((np.int64(1) << (drop - 1)) - np.int64(1)) + lsb
    b = b & ~((np.int64(1) << drop) - np.int64(1))
    as32 = b.view(np.float64).astype(np.float32)  # exact: value has <= 8 significant bits
    return (as32.view(np.uint32) >> np.uint32(16)).astype(np.uint16)


def round_like(x64: np.ndarray, like: np.ndarray) -> np.ndarray:
    if like.dtype == np.uint16:
        return round_to_bf16_bits(x64)
    return x64.astype(np.float32)


# ----------------------------------------------------------------------------
# Stage 1: Filter
# ----------------------------------------------------------------------------

def cosine_relation(P: np.ndarray) -> np.ndarray:
    """R_ij = x_hat_i . x_hat_j for all alive patch tokens (the stand-in for A^v_{i,j})."""
    norms = np.sqrt(np.sum(P * P, axis=1))
    Ph = P / norms[:, None]
    return Ph @ Ph.T


def vision_redundancy(R: np.ndarray) -> np.ndarray:
    """First term of Eq. 1: (1/N) sum_j A_{i,j}, j = i included."""
    n = R.shape[0]
    return R.sum(axis=1) / n


def head_mean(attn: np.ndarray) -> np.ndarray:
    """Average a per-head quantity over heads (axis 0)."""
    return attn.astype(np.float64).sum(axis=0) / attn.shape[0]


def equivalent_token(keys: np.ndarray, n_cls: int) -> np.ndarray:
    """Appendix "Implementation of the Equivalent Token": the stand-in for the CLS attention
    when the encoder has no CLS token.  keys: [T, H, d] key states of one image, token-major
    (bf16 bit patterns or floats).  M = mean over the H heads; P = the patch rows of M (the
    first n_cls rows are left out); mu = mean of P; a_i = -cos(mu, P_i).
    Reading (the paper does not say): a zero mu or a zero P_i gives a_i = 0."""
    K = widen(keys)
    M = K.mean(axis=1)                       # [T, d]
    P = M[n_cls:]
    mu = P.mean(axis=0)
    out = np.zeros(P.shape[0], dtype=np.float64)
    n_mu = np.sqrt(np.dot(mu, mu))
    for i in range(P.shape[0]):
        n_i = np.sqrt(np.dot(P[i], P[i]))
        if n_mu > 0.0 and n_i > 0.0:
            out[i] = -np.dot(mu, P[i]) / (n_mu * n_i)
    return out


def score_v(v: np.ndarray, a_cls: np.ndarray, lam: float) -> np.ndarray:
    """Eq. 1: s^v_i = lam * v_i - (1 - lam) * a^CLS_i."""
    return lam * v - (1.0 - lam) * a_cls


def score_l(v: np.ndarray, t: np.ndarray, beta: float) -> np.ndarray:
    """s^l_i = beta * v_i - (1 - beta) * (1/M) sum_k t[k, i]  (FiCoCo-L, main text)."""
    m = t.shape[0]
    return beta * v - (1.0 - beta) * (t.sum(axis=0) / m)


def local_penalty(s: np.ndarray, pos: np.ndarray, grid: Tuple[int, int], window: int,
                  coef: float) -> np.ndarray:
    """Local penalty: lay the scores back on the 2-D grid, split it into non-overlapping
    window x window cells (previously discarded positions are padding and never win), and
    multiply the highest alive score of each window by ``coef`` whatever its sign.
    Ties inside a window go to the lower token index."""
    gh, gw = grid
    out = s.copy()
    rows = pos // gw
    cols = pos % gw
    wr = rows // window
    wc = cols // window
    nwc = -(-gw // window)
    wid = wr * nwc + wc
    best: Dict[int, int] = {}
    for i in range(s.shape[0]):
        w = int(wid[i])
        if w not in best or s[i] > s[best[w]]:
            best[w] = i
    for w, i in best.items():
        out[i] = coef * s[i]
    return out


def filter_topk(s: np.ndarray, n_src: int) -> Tuple[np.ndarray, np.ndarray]:
    """Source set S = the n_src highest scores (ties: lower index first), in descending
    score order; target set T = the remaining indices in ascending order."""
    order = np.argsort(-s, kind="stable")
    S = order[:n_src]
    mask = np.ones(s.shape[0], dtype=bool)
    mask[S] = False
    T = np.nonzero(mask)[0]
    return S.astype(np.int64), T.astype(np.int64)


# ----------------------------------------------------------------------------
# Stage 2: Correlate
# ----------------------------------------------------------------------------

def correlation_v(R: np.ndarray, S: np.ndarray, T: np.ndarray) -> np.ndarray:
    """C^v_{i,j} = A^v_{i,j} for i in S, j in T."""
    return R[np.ix_(S, T)]


def correlation_l(R: np.ndarray, t: np.ndarray, S: np.ndarray, T: np.ndarray,
                  gamma: float) -> np.ndarray:
    """C^l_{i,j} = gamma A_{i,j} + (1-gamma) (1/M) sum_k A_{i,k} A_{k,j}, the text-bridged
    term built from the text->vision block t[k, .]."""
    m = t.shape[0]
    indirect = (t[:, S].T @ t[:, T]) / m
    return gamma * R[np.ix_(S, T)] + (1.0 - gamma) * indirect


def quantile_threshold(row: np.ndarray, eps: float) -> float:
    """tau_i = the eps-quantile of one row of C (linear interpolation between the order
    statistics around eps*(n-1))."""
    v = np.sort(row)
    n = v.shape[0]
    q = eps * (n - 1)
    lo = int(np.floor(q))
    hi = min(lo + 1, n - 1)
    return float(v[lo] + (q - lo) * (v[hi] - v[lo]))


def targets_and_weights(C: np.ndarray, p: Params) -> Tuple[List[np.ndarray], List[np.ndarray], np.ndarray]:
    """Per discarded token i: J_i = {j : C_ij >= tau_i} (as column positions in T) and
    alpha_ij = C+_ij / sum_{j in J_i} C+_ij (Eq. 2).  Returns (J, alpha, tau).

    With p.average_compression (the "average compression" row of the ablation tables, which
    Sec. "Ablation Study" describes as directly averaging the features) every alpha_ij is 1,
    so Eq. 2 turns into the plain mean of a preserved token and the tokens sent to it."""
    ns, nt = C.shape
    J: List[np.ndarray] = []
    A: List[np.ndarray] = []
    tau = np.full(ns, np.nan)
    for i in range(ns):
        if nt == 0 or p.max_targets == 0:
            J.append(np.zeros(0, dtype=np.int64)); A.append(np.zeros(0)); continue
        row = C[i]
        if p.max_targets is None:
            tau[i] = quantile_threshold(row, p.eps)
            j = np.nonzero(row >= tau[i])[0]
        else:
            k = min(p.max_targets, nt)
            order = np.argsort(-row, kind="stable")[:k]
            tau[i] = row[order[-1]]
            j = np.sort(order)
        if p.average_compression:
            J.append(j.astype(np.int64)); A.append(np.ones(j.shape[0])); continue
        cpos = np.maximum(row[j], 0.0)
        den = cpos.sum()
        if den <= 1e-12:
            J.append(np.zeros(0, dtype=np.int64)); A.append(np.zeros(0)); continue
        J.append(j.astype(np.int64))
        A.append(cpos / den)
    return J, A, tau


# ----------------------------------------------------------------------------
# Stage 3: Compress, then compact
# ----------------------------------------------------------------------------

def compress(P: np.ndarray, S: np.ndarray, T: np.ndarray, J: List[np.ndarray],
             A: List[np.ndarray]) -> Tuple[np.ndarray, np.ndarray]:
    """Eq. 2: X_j <- (X_j + sum_{i in I_j} alpha_ij X_i) / (1 + sum_{i in I_j} alpha_ij)
    for every preserved token j, all from the pre-update X.  Returns the updated target
    rows (float64) and the per-target total weight sum_{i in I_j} alpha_ij."""
    nt = T.shape[0]
    num = P[T].copy()
    wsum = np.zeros(nt)
    order = np.argsort(S, kind="stable")  # accumulate sources in ascending token index
    for si in order:
        for jj, a in zip(J[si], A[si]):
            num[jj] += a * P[S[si]]
            wsum[jj] += a
    return num / (1.0 + wsum)[:, None], wsum


@dataclass
class StepResult:
    out: np.ndarray            # [c + N^T (+ M), D] in the I/O storage format
    kept_idx: np.ndarray       # int32 row indices into the input (CLS, then T ascending)
    pos_out: Optional[np.ndarray]  # int32 grid positions of the preserved patches (V only)
    score_raw: np.ndarray      # Eq. 1 / s^l before the penalty
    score: np.ndarray          # after the local penalty
    S: np.ndarray              # discarded patch indices, descending score
    T: np.ndarray              # preserved patch indices, ascending
    C: np.ndarray              # correlation matrix [N^S, N^T]
    tau: np.ndarray
    J: List[np.ndarray]        # per discarded token: positions in T
    alpha: List[np.ndarray]
    wsum: np.ndarray           # per preserved token: total received weight
    rn: np.ndarray             # 1 / ||x_i||
    v: np.ndarray              # vision-aware redundancy
    a: np.ndarray              # attention term


def ficoco_v_reduce(tokens: np.ndarray, attn: np.ndarray, pos: Optional[np.ndarray],
                    grid: Tuple[int, int], keep: int, has_cls: bool = True,
                    p: Optional[Params] = None, relation: Optional[np.ndarray] = None,
                    by_column: bool = False) -> StepResult:
    """One FiCoCo-V reduce step on one image (Algorithm 1).

    tokens [c+Np, D]; attn [H, Np]; pos [Np] grid positions (None = identity);
    keep = N^T preserved patch tokens.

    relation: optional [Np, Np] map A^v over the patch tokens (row = query).  When given it is
    used wherever the paper writes A^v: the first term of Eq. 1 is (1/N) sum_j A_{i,j} as
    printed, or with by_column (1/N) sum_j A_{j,i}, the attention token i receives (the prose
    of the same paragraph; for a row-stochastic softmax map the printed sum is the constant
    1/N), and C_ij = A_{S_i, T_j} (Sec. "Correlation-based Information Recycling").  The
    tokens then only feed Eq. 2."""
    p = p or Params()
    c = 1 if has_cls else 0
    X = widen(tokens)
    P = X[c:]
    npatch = P.shape[0]
    if pos is None:
        pos = np.arange(npatch, dtype=np.int64)
    pos = np.asarray(pos, dtype=np.int64)
    assert attn.shape[1] == npatch and 0 <= keep <= npatch
    n_src = npatch - keep

    # Stage 1: Filter
    if relation is None:
        R = cosine_relation(P)
        v = vision_redundancy(R)
    else:
        R = np.asarray(relation, dtype=np.float64)
        assert R.shape == (npatch, npatch)
        v = vision_redundancy(R.T if by_column else R)
    a = head_mean(attn)
    s_raw = score_v(v, a, p.lam)
    s = local_penalty(s_raw, pos, grid, p.window, p.penalty_coef) if p.local_penalty else s_raw.copy()
    S, T = filter_topk(s, n_src)
    # Stage 2: Correlate
    C = correlation_v(R, S, T)
    rn = 1.0 / np.sqrt(np.sum(P * P, axis=1))
    if p.convergent:
        extra = convergent_token(P, S) if n_src > 0 else None
        out = _assemble_convergent(tokens, c, T, extra, 0)
        kept = np.concatenate([np.arange(c), T + c, [-1] if n_src > 0 else []]).astype(np.int32)
        none = [np.zeros(0, dtype=np.int64) for _ in range(n_src)]
        return StepResult(out, kept, pos[T].astype(np.int32), s_raw, s, S, T, C, np.full(n_src, np.nan), none,
                          [np.zeros(0) for _ in range(n_src)], np.zeros(T.shape[0]), rn, v, a)
    # Stage 3: Compress
    J, A, tau = targets_and_weights(C, p)
    merged, wsum = compress(P, S, T, J, A)
    out = _assemble(tokens, c, T, merged, wsum, tail_rows=0)
    kept = np.concatenate([np.arange(c), T + c]).astype(np.int32)
    return StepResult(out, kept, pos[T].astype(np.int32), s_raw, s, S, T, C, tau, J, A, wsum, rn, v, a)


def ficoco_l_reduce(tokens: np.ndarray, attn_t2v: np.ndarray, n_vision: int, keep: int,
                    p: Optional[Params] = None) -> StepResult:
    """One FiCoCo-L reduce step on one sequence (Algorithm 2, with the main-text 1/M).

    tokens [N+M, D], vision rows first; attn_t2v [H, M, N]; keep = preserved vision tokens.
    Text rows pass through unchanged after the preserved vision rows."""
    p = p or Params()
    X = widen(tokens)
    n = n_vision
    m = X.shape[0] - n
    P = X[:n]
    assert attn_t2v.shape[1] == m and attn_t2v.shape[2] == n and 0 <= keep <= n
    n_src = n - keep
    t = head_mean(attn_t2v)            # [M, N]
    R = cosine_relation(P)
    v = vision_redundancy(R)
    s_raw = score_l(v, t, p.beta)      # no local penalty in FiCoCo-L
    S, T = filter_topk(s_raw, n_src)
    C = correlation_l(R, t, S, T, p.gamma)
    rn = 1.0 / np.sqrt(np.sum(P * P, axis=1))
    if p.convergent:
        extra = convergent_token(P, S) if n_src > 0 else None
        out = _assemble_convergent(tokens, 0, T, extra, m)
        kept = np.concatenate([T, [-1] if n_src > 0 else [], np.arange(n, n + m)]).astype(np.int32)
        none = [np.zeros(0, dtype=np.int64) for _ in range(n_src)]
        return StepResult(out, kept, None, s_raw, s_raw.copy(), S, T, C, np.full(n_src, np.nan), none,
                          [np.zeros(0) for _ in range(n_src)], np.zeros(T.shape[0]), rn, v, t.sum(axis=0) / m)
    J, A, tau = targets_and_weights(C, p)
    merged, wsum = compress(P, S, T, J, A)
    out = _assemble(tokens, 0, T, merged, wsum, tail_rows=m)
    kept = np.concatenate([T, np.arange(n, n + m)]).astype(np.int32)
    return StepResult(out, kept, None, s_raw, s_raw.copy(), S, T, C, tau, J, A, wsum, rn, v,
                      t.sum(axis=0) / m)


def convergent_token(P: np.ndarray, S: np.ndarray) -> np.ndarray:
    """Ablation "convergent correlation": the one additional token all discarded tokens merge
    into, taken as their plain mean (float64; the paper gives no weights)."""
    return P[np.sort(S)].sum(axis=0) / S.shape[0]


def _assemble_convergent(tokens: np.ndarray, c: int, T: np.ndarray, extra: Optional[np.ndarray],
                         tail_rows: int) -> np.ndarray:
    """Output of the convergent variant: CLS rows, preserved rows bit for bit, the additional
    token (rounded once to the storage format) when there is one, trailing rows."""
    n_in = tokens.shape[0]
    parts = [tokens[:c], tokens[c + T]]
    if extra is not None:
        parts.append(round_like(extra[None, :], tokens))
    if tail_rows:
        parts.append(tokens[n_in - tail_rows:])
    return np.concatenate(parts, axis=0)


def _assemble(tokens: np.ndarray, c: int, T: np.ndarray, merged: np.ndarray, wsum: np.ndarray,
              tail_rows: int) -> np.ndarray:
    """Compaction (last step of Algorithm 1/2): leading CLS rows, preserved rows in
    ascending order, trailing rows (text) unchanged.  Rows that received no weight keep
    their stored bits."""
    n_in = tokens.shape[0]
    nt = T.shape[0]
    out = np.empty((c + nt + tail_rows, tokens.shape[1]), dtype=tokens.dtype)
    out[:c] = tokens[:c]
    body = tokens[c + T].copy() if nt else tokens[:0].copy()
    touched = wsum > 0.0
    if touched.any():
        body[touched] = round_like(merged[touched], tokens)
    out[c:c + nt] = body
    if tail_rows:
        out[c + nt:] = tokens[n_in - tail_rows:]
    return out


# ----------------------------------------------------------------------------
# Batch helpers
# ----------------------------------------------------------------------------

def v_reduce_batch(batch, p: Optional[Params] = None) -> List[StepResult]:
    """Apply ficoco_v_reduce to every image of a synthetic VBatch (images are independent)."""
    return [ficoco_v_reduce(batch.tokens[b], batch.attn[b], batch.pos[b], batch.grid[b],
                            batch.keep[b], batch.has_cls, p) for b in range(batch.batch)]


def l_reduce_batch(batch, p: Optional[Params] = None) -> List[StepResult]:
    return [ficoco_l_reduce(batch.tokens[b], batch.attn_t2v[b], batch.n_vision, batch.keep[b], p)
            for b in range(batch.batch)]
