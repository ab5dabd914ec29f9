"""Shared comparison logic for the GPU parity tests: run one reduce step through the C ABI
and compare every stage with the float64 checker on the same (margin-repaired) inputs."""
from __future__ import annotations

from typing import List

import numpy as np

from oracle import ficoco_oracle as fo
from paper_2411_17686_b200 import binding, packing

# Tolerances.  Scores: 1e-5 relative in fp32, measured against the image's score scale for
# entries that nearly cancel.  Merged rows: 2e-2 absolute + 1e-2 relative for bf16 storage
# (one bf16 ulp is 2^-8 relative); fp32 storage is held to 1e-5.
SCORE_RTOL = 1e-5
BF16_ATOL, BF16_RTOL = 2e-2, 1e-2
FP32_ATOL, FP32_RTOL = 1e-5, 1e-5
ALPHA_ATOL = 1e-4
# Largest plain relative score error |got - exp| / |exp| seen by compare_stages (the tolerance is
# measured against max(|s_i|, mean |s|) of the image because lambda v - (1 - lambda) a cancels for
# some tokens); the full-size tests print it.
WORST_PLAIN_REL = {}


def params_to_abi(p: fo.Params, has_cls: bool):
    return binding.make_params(lam=p.lam, beta=p.beta, gamma=p.gamma, eps=p.eps,
                               penalty_coef=p.penalty_coef, window=p.window,
                               max_targets=-1 if p.max_targets is None else p.max_targets,
                               has_cls=has_cls, local_penalty=p.local_penalty,
                               average_compression=p.average_compression, convergent=p.convergent)


def _widen(a: np.ndarray) -> np.ndarray:
    return fo.widen(a)


def compare_tokens(got: np.ndarray, exp: np.ndarray, wsum: np.ndarray, c: int, tail: int, what: str,
                   computed_rows=()):
    """got/exp: output rows of one image in storage format.  computed_rows: rows other than the
    merged preserved tokens that hold computed values (the additional token of the convergent
    variant) and are therefore compared within the tolerance, not bit for bit."""
    assert got.shape == exp.shape, what
    nt = wsum.shape[0]
    untouched = np.ones(got.shape[0], dtype=bool)
    untouched[c:c + nt] = wsum == 0.0
    for r in computed_rows:
        untouched[r] = False
    assert np.array_equal(got[untouched], exp[untouched]), f"{what}: pass-through rows differ"
    g, e = _widen(got[~untouched]), _widen(exp[~untouched])
    if got.dtype == np.uint16:
        tol = BF16_ATOL + BF16_RTOL * np.abs(e)
    else:
        tol = FP32_ATOL + FP32_RTOL * np.abs(e)
    bad = np.abs(g - e) > tol
    assert not bad.any(), f"{what}: {bad.sum()} merged elements off, max err {np.abs(g - e).max():.3e}"
    # much tighter in practice: at most one storage ulp
    if got.dtype == np.uint16 and g.size:
        assert np.abs(g - e).max() <= 2.0 ** -7 * max(1.0, np.abs(e).max()), what


def compare_stages(ctx: binding.Context, results: List[fo.StepResult], n_cls: int, what: str,
                   check_rn: bool = True):
    """Intermediate arrays of the last call vs the checker, image by image."""
    rn = ctx.ficoco_inspect("rnorm")
    s_raw = ctx.ficoco_inspect("score_raw")
    s_pen = ctx.ficoco_inspect("score")
    S = ctx.ficoco_inspect("src_idx")
    T = ctx.ficoco_inspect("tgt_idx")
    cnt = ctx.ficoco_inspect("corr_cnt")
    ctgt = ctx.ficoco_inspect("corr_tgt")
    cw = ctx.ficoco_inspect("corr_w")
    cc = ctx.ficoco_inspect("corr_c")
    tau = ctx.ficoco_inspect("tau")
    p0 = s0 = t0 = 0
    for b, r in enumerate(results):
        npatch, ns, nt = r.score.shape[0], r.S.shape[0], r.T.shape[0]
        tag = f"{what} image {b}"
        if check_rn:
            np.testing.assert_allclose(rn[p0:p0 + npatch], r.rn, rtol=1e-6, err_msg=tag + " rnorm")
        scale = float(np.mean(np.abs(r.score_raw)))
        for got, exp, nm in ((s_raw[p0:p0 + npatch], r.score_raw, "score_raw"),
                             (s_pen[p0:p0 + npatch], r.score, "score")):
            err = np.abs(got.astype(np.float64) - exp)
            tol = SCORE_RTOL * np.maximum(np.abs(exp), scale)
            plain = float(np.max(err / np.maximum(np.abs(exp), 1e-300)))      # plain relative error, no scale floor
            WORST_PLAIN_REL[nm] = max(WORST_PLAIN_REL.get(nm, 0.0), plain)
            assert (err <= tol).all(), (f"{tag} {nm}: max rel err {np.max(err / np.maximum(np.abs(exp), scale)):.3e} "
                                        f"(plain relative, where the two terms of the score cancel: {plain:.3e})")
        # index work: bit exact
        assert np.array_equal(S[s0:s0 + ns], np.sort(r.S)), tag + " S"
        assert np.array_equal(T[t0:t0 + nt], r.T), tag + " T"
        # correlate: same target sets, weights and top correlation values
        order = np.argsort(r.S)
        for k, si in enumerate(order):
            exp_j = r.J[si]
            n = int(cnt[s0 + k])
            assert n == exp_j.shape[0], f"{tag} source {int(r.S[si])}: |J| {n} vs {exp_j.shape[0]}"
            got_j = ctgt[s0 + k, :n]
            o = np.argsort(got_j)
            assert np.array_equal(got_j[o], exp_j), f"{tag} source {int(r.S[si])}: targets differ"
            np.testing.assert_allclose(cw[s0 + k, :n][o], r.alpha[si], atol=ALPHA_ATOL, err_msg=tag + " alpha")
            if n:
                cexp = r.C[si][exp_j]
                cgot = cc[s0 + k, :n][o]
                np.testing.assert_allclose(cgot, cexp, rtol=1e-5, atol=2e-6, err_msg=tag + " C")
                if not np.isnan(r.tau[si]):
                    np.testing.assert_allclose(tau[s0 + k], r.tau[si], rtol=1e-5, atol=2e-6, err_msg=tag + " tau")
        p0 += npatch; s0 += ns; t0 += nt


def run_and_compare_v(ctx: binding.Context, batch, p: fo.Params, device, stages: bool = True,
                      results: List[fo.StepResult] = None, what: str = ""):
    pk = packing.pack_v(batch, device)
    prm = params_to_abi(p, batch.has_cls)
    res = ctx.ficoco_v_reduce(pk.tokens, pk.attn, pk.keep, pk.grid_h, pk.grid_w, pk.heads,
                              params=prm, want_scores=True, **pk.call_kwargs())
    assert ctx.ficoco_status() == 0
    if results is None:
        results = fo.v_reduce_batch(batch, p)
    out = binding.to_numpy(res.out_tokens)
    kidx = binding.to_numpy(res.kept_idx)
    pout = binding.to_numpy(res.pos_out)
    c = 1 if batch.has_cls else 0
    r0 = k0 = 0
    for b, r in enumerate(results):
        nrow = res.out_rows[b]
        assert nrow == r.out.shape[0]
        assert np.array_equal(kidx[r0:r0 + nrow], r.kept_idx), f"{what} image {b}: kept_idx"
        nt = r.T.shape[0]
        assert np.array_equal(pout[k0:k0 + nt], r.pos_out), f"{what} image {b}: pos_out"
        compare_tokens(out[r0:r0 + nrow], r.out, r.wsum, c, 0, f"{what} image {b}",
                       computed_rows=np.nonzero(r.kept_idx < 0)[0])
        r0 += nrow; k0 += nt
    if stages:
        compare_stages(ctx, results, c, what)
        sc = binding.to_numpy(res.scores)
        assert np.array_equal(sc, ctx.ficoco_inspect("score"))
    return res, results


def run_and_compare_v_relation(ctx: binding.Context, batch, rels, by_column: bool, p: fo.Params, device,
                               what: str = ""):
    """ficoco_v_reduce_relation against the checker given the same relation blocks."""
    import torch
    pk = packing.pack_v(batch, device)
    prm = params_to_abi(p, batch.has_cls)
    rel_d = torch.from_numpy(np.concatenate([r.reshape(-1) for r in rels])).to(device)
    res = ctx.ficoco_v_reduce(pk.tokens, pk.attn, pk.keep, pk.grid_h, pk.grid_w, pk.heads, params=prm,
                              want_scores=True, relation=rel_d, by_column=by_column, **pk.call_kwargs())
    assert ctx.ficoco_status() == 0
    results = [fo.ficoco_v_reduce(batch.tokens[b], batch.attn[b], batch.pos[b], batch.grid[b], batch.keep[b],
                                  batch.has_cls, p, relation=rels[b], by_column=by_column)
               for b in range(batch.batch)]
    out = binding.to_numpy(res.out_tokens)
    kidx = binding.to_numpy(res.kept_idx)
    pout = binding.to_numpy(res.pos_out)
    c = 1 if batch.has_cls else 0
    r0 = k0 = 0
    for b, r in enumerate(results):
        nrow = res.out_rows[b]
        assert nrow == r.out.shape[0]
        assert np.array_equal(kidx[r0:r0 + nrow], r.kept_idx), f"{what} image {b}: kept_idx"
        nt = r.T.shape[0]
        assert np.array_equal(pout[k0:k0 + nt], r.pos_out), f"{what} image {b}: pos_out"
        compare_tokens(out[r0:r0 + nrow], r.out, r.wsum, c, 0, f"{what} image {b}")
        r0 += nrow; k0 += nt
    compare_stages(ctx, results, c, what, check_rn=False)
    return res, results


def run_and_compare_l(ctx: binding.Context, batch, p: fo.Params, device, stages: bool = True, what: str = ""):
    pk = packing.pack_l(batch, device)
    prm = params_to_abi(p, False)
    res = ctx.ficoco_l_reduce(pk.tokens, pk.attn_t2v, pk.keep, pk.n_vision, pk.n_text, pk.heads,
                              params=prm, want_scores=True)
    assert ctx.ficoco_status() == 0
    results = fo.l_reduce_batch(batch, p)
    out = binding.to_numpy(res.out_tokens)
    kidx = binding.to_numpy(res.kept_idx)
    r0 = 0
    for b, r in enumerate(results):
        nrow = res.out_rows[b]
        assert np.array_equal(kidx[r0:r0 + nrow], r.kept_idx), f"{what} seq {b}: kept_idx"
        compare_tokens(out[r0:r0 + nrow], r.out, r.wsum, 0, batch.n_text, f"{what} seq {b}",
                       computed_rows=np.nonzero(r.kept_idx < 0)[0])
        r0 += nrow
    if stages:
        compare_stages(ctx, results, 0, what)
    return res, results
