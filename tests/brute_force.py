"""Independent pure-Python transcription of the FiCoCo reduce step for tiny inputs.

Written with scalar loops, sets and dicts straight from the paper's element-wise
definitions (Eq. 1, the local-penalty paragraph, the quantile threshold, Eq. 2 and the
FiCoCo-L score / correlation).  It deliberately avoids every helper of ``oracle/`` and
every numpy matrix routine so that a mistake in the checker's vectorised code (a dropped
term, a transposed operand, a wrong index set) shows up as a disagreement.
"""
import math


def _dot(a, b):
    return math.fsum(x * y for x, y in zip(a, b))


def reduce_v(P, cls_attn_heads, pos, gh, gw, keep, lam=0.35, eps=0.998, coef=2.0, window=2,
             penalty=True, max_targets=None):
    """P: list of patch rows (lists of floats); cls_attn_heads: list over heads of lists.
    Returns dict with scores, S (set), T (sorted list), J, alpha, merged rows (floats)."""
    n = len(P)
    H = len(cls_attn_heads)
    norm = [math.sqrt(_dot(x, x)) for x in P]
    A = [[_dot(P[i], P[j]) / (norm[i] * norm[j]) for j in range(n)] for i in range(n)]
    s = []
    for i in range(n):
        vis = math.fsum(A[i][j] for j in range(n)) / n
        a_cls = math.fsum(cls_attn_heads[h][i] for h in range(H)) / H
        s.append(lam * vis - (1.0 - lam) * a_cls)
    s_raw = list(s)
    if penalty:
        windows = {}
        for i in range(n):
            r, c = divmod(pos[i], gw)
            windows.setdefault((r // window, c // window), []).append(i)
        for members in windows.values():
            top = members[0]
            for i in members[1:]:
                if s_raw[i] > s_raw[top]:
                    top = i
            s[top] = coef * s_raw[top]
    n_src = n - keep
    ranked = sorted(range(n), key=lambda i: (-s[i], i))
    S = ranked[:n_src]
    T = sorted(set(range(n)) - set(S))
    return _correlate_compress(P, S, T, lambda i, j: A[i][j], eps, s_raw, s, max_targets)


def reduce_l(P, t2v_heads, keep, beta=0.6, gamma=0.6, eps=0.998, max_targets=None):
    """P: vision rows; t2v_heads[h][k][i]: attention of text token k to vision token i."""
    n = len(P)
    H = len(t2v_heads)
    M = len(t2v_heads[0])
    t = [[math.fsum(t2v_heads[h][k][i] for h in range(H)) / H for i in range(n)] for k in range(M)]
    norm = [math.sqrt(_dot(x, x)) for x in P]
    A = [[_dot(P[i], P[j]) / (norm[i] * norm[j]) for j in range(n)] for i in range(n)]
    s = []
    for i in range(n):
        vis = math.fsum(A[i][j] for j in range(n)) / n
        task = math.fsum(t[k][i] for k in range(M)) / M
        s.append(beta * vis - (1.0 - beta) * task)
    n_src = n - keep
    ranked = sorted(range(n), key=lambda i: (-s[i], i))
    S = ranked[:n_src]
    T = sorted(set(range(n)) - set(S))

    def corr(i, j):
        bridge = math.fsum(t[k][i] * t[k][j] for k in range(M)) / M
        return gamma * A[i][j] + (1.0 - gamma) * bridge

    return _correlate_compress(P, S, T, corr, eps, list(s), s, max_targets)


def _correlate_compress(P, S, T, corr, eps, s_raw, s, max_targets=None):
    """max_targets None: the token-wise quantile threshold; k >= 0: the fixed-K ablation, every
    discarded token goes to its k most correlated preserved tokens (ties: lower token first)."""
    D = len(P[0])
    C = {(i, j): corr(i, j) for i in S for j in T}
    J = {}
    alpha = {}
    taus = {}
    for i in S:
        if not T or max_targets == 0:
            J[i] = []
            continue
        if max_targets is None:
            row = sorted(C[(i, j)] for j in T)
            q = eps * (len(row) - 1)
            lo = int(math.floor(q))
            hi = min(lo + 1, len(row) - 1)
            tau = row[lo] + (q - lo) * (row[hi] - row[lo])
            Ji = [j for j in T if C[(i, j)] >= tau]
        else:
            best = sorted(T, key=lambda j: (-C[(i, j)], j))[:min(max_targets, len(T))]
            tau = C[(i, best[-1])]              # the smallest correlation that is still taken
            Ji = sorted(best)
        taus[i] = tau
        den = math.fsum(max(C[(i, j)], 0.0) for j in Ji)
        if den <= 1e-12:
            J[i] = []
            continue
        J[i] = Ji
        for j in Ji:
            alpha[(i, j)] = max(C[(i, j)], 0.0) / den
    merged = {}
    wsum = {}
    for j in T:
        I_j = [i for i in S if j in J[i]]
        w = math.fsum(alpha[(i, j)] for i in I_j)
        row = []
        for d in range(D):
            num = P[j][d] + math.fsum(alpha[(i, j)] * P[i][d] for i in I_j)
            row.append(num / (1.0 + w))
        merged[j] = row
        wsum[j] = w
    return {"s_raw": s_raw, "s": s, "S": S, "T": T, "J": J, "alpha": alpha, "merged": merged,
            "wsum": wsum, "C": C, "tau": taus}


def group_means(P, S, T, J):
    """'Average compression' written as what it means, not through Eq. 2: every preserved token j
    becomes the arithmetic mean of the group made of itself and the discarded tokens that chose it.
    P: rows (lists of floats); S, T: token indices; J: dict discarded token -> list of targets."""
    out = {}
    for j in T:
        members = [j] + [i for i in S if j in J[i]]
        out[j] = [math.fsum(P[m][d] for m in members) / len(members) for d in range(len(P[0]))]
    return out
