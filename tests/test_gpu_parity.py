"""GPU parity: the CUDA library (through its C ABI) against the float64 checker, element by
element, on seeded inputs whose discrete decisions were made unambiguous beforehand."""
import collections
import copy
import json
import os

import numpy as np
import pytest
import torch

from oracle import ficoco_oracle as fo, gaps
from paper_2411_17686_b200 import binding, packing, synth
from tests import parity

pytestmark = pytest.mark.gpu
VResultLike = collections.namedtuple("VResultLike", "out_tokens kept_idx pos_out")
DEV = "cuda:0"


@pytest.fixture(scope="module")
def ctx():
    c = binding.Context(max_tokens=70000, max_dim=4096, max_batch=32, max_text=64, device=0)
    yield c
    c.close()


# ---------------------------------------------------------------------------------------
# scaled-down versions of the five workloads: several tiles, ragged tails, every stage
# ---------------------------------------------------------------------------------------
@pytest.mark.parametrize("idx", [1, 2, 3, 4])
def test_small_workloads_v(ctx, idx):
    batch = synth.workload(idx, small=True)
    gaps.repair_v(batch)
    parity.run_and_compare_v(ctx, batch, fo.Params(), DEV, what=batch.name)


def test_small_workload_l(ctx):
    batch = synth.workload(5, small=True)
    gaps.repair_l(batch)
    parity.run_and_compare_l(ctx, batch, fo.Params(), DEV, what=batch.name)


@pytest.mark.parametrize("idx", [2, 3])
def test_small_progressive_schedule(ctx, idx):
    """Every step of the schedule is checked on the checker's previous output (so both
    sides always see identical inputs), with attention regenerated and pos chained."""
    batch = synth.workload(idx, small=True)
    sched = synth.SCHEDULES_SMALL[idx]
    p = fo.Params()
    for step, keep in enumerate(sched):
        batch.keep = [keep] * batch.batch
        gaps.repair_v(batch)
        _, results = parity.run_and_compare_v(ctx, batch, p, DEV, what=f"{batch.name} step {step}")
        batch.tokens = [r.out for r in results]
        batch.pos = [r.pos_out for r in results]
        if step + 1 < len(sched):
            synth.regenerate_attention(batch, 1000 * idx, step + 1, 1.5 if idx == 2 else 1.0)


# ---------------------------------------------------------------------------------------
# variants and edge cases
# ---------------------------------------------------------------------------------------
@pytest.mark.parametrize("p", [
    fo.Params(local_penalty=False),
    fo.Params(eps=0.97),                       # longer top lists (several targets per token)
    fo.Params(eps=1.0),                        # tau = row maximum
    fo.Params(max_targets=0),                  # pruning only
    fo.Params(max_targets=2),                  # fixed K
    fo.Params(window=3, penalty_coef=1.5),
    fo.Params(window=1),
    fo.Params(lam=0.8),
    fo.Params(average_compression=True),            # ablation: features averaged directly
    fo.Params(eps=0.97, average_compression=True),
    fo.Params(max_targets=1, average_compression=True),
], ids=["nopenalty", "eps097", "eps1", "prune", "fixedK2", "win3", "win1", "lam08", "avg", "avg-eps097", "avg-K1"])
def test_variants(ctx, p):
    batch = synth.make_v_batch(77, 3, 13, 11, 192, 5, 80, "bf16", True, 1.2)
    gaps.repair_v(batch, p)
    parity.run_and_compare_v(ctx, batch, p, DEV, what="variant")


@pytest.mark.parametrize("dtype", ["bf16", "fp32"])
@pytest.mark.parametrize("keep", [0, 1, 2, 99, 100])
def test_edge_keep_counts(ctx, dtype, keep):
    batch = synth.make_v_batch(78, 2, 10, 10, 64, 3, keep, dtype, True, 1.0)
    gaps.repair_v(batch)
    parity.run_and_compare_v(ctx, batch, fo.Params(), DEV, what=f"keep{keep}")


def test_no_cls_and_holes_in_pos(ctx):
    batch = synth.make_v_batch(79, 2, 12, 12, 128, 4, 50, "bf16", False, 1.0)
    # drop a third of the grid cells so windows are partially or completely empty
    for b in range(2):
        alive = np.sort(synth.rng_for(79, b, 8).permutation(144)[:96]).astype(np.int32)
        batch.tokens[b] = batch.tokens[b][alive]
        batch.attn[b] = batch.attn[b][:, alive].copy()
        batch.pos[b] = alive
    gaps.repair_v(batch)
    parity.run_and_compare_v(ctx, batch, fo.Params(), DEV, what="holes")


@pytest.mark.parametrize("dim", [8, 72, 1280, 2048, 4096])
def test_hidden_sizes(ctx, dim):
    batch = synth.make_v_batch(80, 2, 6, 7, dim, 2, 20, "bf16", True, 1.0)
    gaps.repair_v(batch)
    parity.run_and_compare_v(ctx, batch, fo.Params(), DEV, what=f"dim{dim}")


def test_fp32_wide_rows(ctx):
    batch = synth.make_v_batch(81, 1, 6, 6, 2052, 2, 20, "fp32", True, 1.0)
    gaps.repair_v(batch)
    parity.run_and_compare_v(ctx, batch, fo.Params(), DEV, what="fp32-wide")


@pytest.mark.parametrize("keep", [130, 30])
def test_fp32_tensor_core_correlate_tiles(ctx, keep):
    """fp32 tokens whose hidden size is a multiple of 64 take the tensor-core correlate that splits
    every value into three bf16 terms: several tiles of discarded tokens, column splits with a ragged
    last one, ragged images, fixed K and pruning, all at the fp32 tolerances."""
    batch = synth.make_v_batch(85, 3, 20, 20, 128, 4, keep, "fp32", True, 1.2)
    # ragged: the second image loses a fifth of its cells
    alive = np.sort(synth.rng_for(85, 1, 8).permutation(400)[:320]).astype(np.int32)
    batch.tokens[1] = np.concatenate([batch.tokens[1][:1], batch.tokens[1][1:][alive]], axis=0)
    batch.attn[1] = batch.attn[1][:, alive].copy()
    batch.pos[1] = alive
    for p in (fo.Params(), fo.Params(eps=0.9), fo.Params(max_targets=2), fo.Params(max_targets=0)):
        gaps.repair_v(batch, p)
        parity.run_and_compare_v(ctx, batch, p, DEV, what=f"fp32-umma-keep{keep}")


def _relations(batch, seed, stochastic=True, times_n=False):
    c = 1 if batch.has_cls else 0
    rels = []
    for b in range(batch.batch):
        r = synth.relation_map(synth.rng_for(seed, b, 21), fo.widen(batch.tokens[b])[c:])
        if not stochastic:   # rows of different mass, so that the by-row mean is not a constant
            r = (r * synth.rng_for(seed, b, 22).uniform(0.5, 1.5, size=(r.shape[0], 1))).astype(np.float32)
        if times_n:          # entries of order one whatever the image size
            r = (r * np.float32(r.shape[0])).astype(np.float32)
        rels.append(r)
    return rels


@pytest.mark.parametrize("by_column", [False, True], ids=["by-row", "by-column"])
@pytest.mark.parametrize("dtype", ["bf16", "fp32"])
def test_relation_mode(ctx, by_column, dtype):
    """Caller-supplied relation map in place of the cosine similarity: scores, S / T, target
    sets, weights and merged rows against the checker given the same map."""
    batch = synth.make_v_batch(90, 3, 13, 11, 192, 5, 60, dtype, True, 1.2)
    rels = _relations(batch, 90, stochastic=by_column)
    for p in (fo.Params(), fo.Params(eps=0.97, local_penalty=False)):
        gaps.repair_v_relation(batch, rels, by_column, p)
        parity.run_and_compare_v_relation(ctx, batch, rels, by_column, p, DEV, what="relation")


@pytest.mark.parametrize("by_column", [False, True], ids=["by-row", "by-column"])
def test_relation_mode_rows_on_16_byte_boundaries(ctx, by_column):
    """Np a multiple of four: the score kernel reads the map with 16-byte loads."""
    batch = synth.make_v_batch(93, 2, 12, 12, 128, 3, 50, "bf16", True, 1.0)
    rels = _relations(batch, 93, stochastic=by_column)
    gaps.repair_v_relation(batch, rels, by_column)
    parity.run_and_compare_v_relation(ctx, batch, rels, by_column, fo.Params(), DEV, what="relation-vec")


def test_relation_mode_ragged_no_cls(ctx):
    batch = synth.workload(4, small=True)
    rels = _relations(batch, 91, times_n=True)
    gaps.repair_v_relation(batch, rels, True)
    parity.run_and_compare_v_relation(ctx, batch, rels, True, fo.Params(), DEV, what="relation-ragged")
    # keep everything / keep nothing
    for keep_all in (True, False):
        b2 = synth.make_v_batch(92, 2, 6, 6, 64, 2, 36 if keep_all else 0, "bf16", True, 1.0)
        r2 = _relations(b2, 92)
        gaps.repair_v_relation(b2, r2, True)
        parity.run_and_compare_v_relation(ctx, b2, r2, True, fo.Params(), DEV, what="relation-edge")


def test_l_variants(ctx):
    for p in (fo.Params(gamma=1.0), fo.Params(beta=0.9), fo.Params(eps=0.9), fo.Params(max_targets=0),
              fo.Params(eps=0.9, average_compression=True)):
        batch = synth.make_l_batch(82, 2, 100, 9, 256, 3, 30, "bf16", scale=1.0 / 16)
        gaps.repair_l(batch, p)
        parity.run_and_compare_l(ctx, batch, p, DEV, what="l-variant")
    batch = synth.make_l_batch(83, 1, 70, 5, 128, 2, 20, "fp32", scale=1.0)
    gaps.repair_l(batch)
    parity.run_and_compare_l(ctx, batch, fo.Params(), DEV, what="l-fp32")


def test_run_to_run_determinism_and_host_entry_point(ctx):
    batch = synth.workload(2, small=True)
    gaps.repair_v(batch)
    pk = packing.pack_v(batch, DEV)
    a = ctx.ficoco_v_reduce(pk.tokens, pk.attn, pk.keep, pk.grid_h, pk.grid_w, pk.heads, **pk.call_kwargs())
    a_out, a_idx = binding.to_numpy(a.out_tokens), binding.to_numpy(a.kept_idx)
    b = ctx.ficoco_v_reduce(pk.tokens, pk.attn, pk.keep, pk.grid_h, pk.grid_w, pk.heads, **pk.call_kwargs())
    assert np.array_equal(a_out, binding.to_numpy(b.out_tokens))
    assert np.array_equal(a_idx, binding.to_numpy(b.kept_idx))
    ph = packing.pack_v(batch, None, pin=True)
    h = ctx.ficoco_v_reduce_host(ph.tokens, ph.attn, ph.keep, ph.grid_h, ph.grid_w, ph.heads, **ph.call_kwargs())
    assert np.array_equal(a_out, binding.to_numpy(h.out_tokens))
    assert np.array_equal(a_idx, binding.to_numpy(h.kept_idx))
    lb = synth.workload(5, small=True)
    gaps.repair_l(lb)
    pl = packing.pack_l(lb, DEV)
    d = ctx.ficoco_l_reduce(pl.tokens, pl.attn_t2v, pl.keep, pl.n_vision, pl.n_text, pl.heads)
    plh = packing.pack_l(lb, None, pin=True)
    hh = ctx.ficoco_l_reduce_host(plh.tokens, plh.attn_t2v, plh.keep, plh.n_vision, plh.n_text, plh.heads)
    assert np.array_equal(binding.to_numpy(d.out_tokens), binding.to_numpy(hh.out_tokens))
    assert np.array_equal(binding.to_numpy(d.kept_idx), binding.to_numpy(hh.kept_idx))


def test_l_host_entry_point_in_sequence_groups(ctx):
    """FiCoCo-L host-buffer call on the full-size workload (cut into groups of sequences whose uploads,
    kernels and downloads overlap), with per-sequence keep counts: every output equals the
    device-buffer call on the same bytes."""
    lb = synth.workload(5)
    pl = packing.pack_l(lb, DEV)
    nseq = len(lb.tokens)
    keep = np.array([64 + 3 * (b % 5) for b in range(nseq)], dtype=np.int32)
    scores_d = torch.empty((nseq * pl.n_vision,), dtype=torch.float32, device=DEV)
    d = ctx.ficoco_l_reduce(pl.tokens, pl.attn_t2v, keep, pl.n_vision, pl.n_text, pl.heads, scores_out=scores_d)
    torch.cuda.synchronize()
    plh = packing.pack_l(lb, None, pin=True)
    scores_h = torch.empty((nseq * pl.n_vision,), dtype=torch.float32).pin_memory()
    hh = ctx.ficoco_l_reduce_host(plh.tokens, plh.attn_t2v, keep, plh.n_vision, plh.n_text, plh.heads,
                                  scores_out=scores_h)
    assert np.array_equal(binding.to_numpy(d.out_tokens), binding.to_numpy(hh.out_tokens))
    assert np.array_equal(binding.to_numpy(d.kept_idx), binding.to_numpy(hh.kept_idx))
    assert np.array_equal(scores_d.cpu().numpy(), scores_h.numpy())
    assert ctx.ficoco_status() == 0


def test_back_to_back_steps_without_sync(ctx):
    """Steps queued on one stream with no host synchronisation between them: a step fed
    straight from the outputs of the step before it, and an independent step right behind
    (whose first grid may start under the tail of the step before).  Every result must be
    bit-identical to the same chain run with a device synchronisation after every call."""
    nb, g, heads = 16, 24, 4
    batch = synth.make_v_batch(91, nb, g, g, 512, heads, g * g // 2, "bf16", True, 1.5)
    pk = packing.pack_v(batch, DEV)
    prm = parity.params_to_abi(fo.Params(), True)
    prm.flags |= binding.FICOCO_BACK_TO_BACK       # nothing but reduce steps goes onto the stream below
    gen = torch.Generator().manual_seed(5)
    k1, k2 = g * g // 2, g * g // 4
    attn2 = torch.softmax(1.5 * torch.randn(nb, heads, k1, generator=gen), -1).reshape(-1).to(DEV)

    def chain(sync):
        r1 = ctx.ficoco_v_reduce(pk.tokens, pk.attn, k1, g, g, heads, params=prm, **pk.call_kwargs())
        if sync:
            torch.cuda.synchronize()
        r2 = ctx.ficoco_v_reduce(r1.out_tokens, attn2, k2, g, g, heads, n_tokens=1 + k1, pos=r1.pos_out,
                                 params=prm)
        if sync:
            torch.cuda.synchronize()
        r3 = ctx.ficoco_v_reduce(pk.tokens, pk.attn, k1, g, g, heads, params=prm, **pk.call_kwargs())
        torch.cuda.synchronize()
        assert ctx.ficoco_status() == 0
        return [binding.to_numpy(t) for r in (r1, r2, r3) for t in (r.out_tokens, r.kept_idx, r.pos_out)]

    ref = chain(True)
    assert np.array_equal(ref[0], ref[6]) and np.array_equal(ref[1], ref[7])
    for rep in range(12):
        got = chain(False)
        for i, (a, b) in enumerate(zip(ref, got)):
            assert np.array_equal(a, b), f"repetition {rep}: array {i} differs from the synchronised chain"


@pytest.mark.parametrize("idx", [2, 4])
def test_host_entry_point_in_image_groups(ctx, idx):
    """Host-buffer call on a batch large enough to be cut into image groups (uploads, kernels
    and downloads overlapped): every output equals the device-buffer call on the same bytes.
    Workload 4 is ragged with per-image keep / grid arrays, workload 2 uniform."""
    batch = synth.workload(idx)
    pk = packing.pack_v(batch, DEV)
    prm = parity.params_to_abi(fo.Params(), batch.has_cls)
    keep = pk.keep if idx == 4 else pk.keep[0]
    gh, gw = (pk.grid_h, pk.grid_w) if idx == 4 else (pk.grid_h[0], pk.grid_w[0])
    d = ctx.ficoco_v_reduce(pk.tokens, pk.attn, keep, gh, gw, pk.heads, params=prm, want_scores=True,
                            **pk.call_kwargs())
    torch.cuda.synchronize()
    ph = packing.pack_v(batch, None, pin=True)
    pos_out = torch.empty(d.pos_out.shape, dtype=torch.int32).pin_memory()
    scores = torch.empty(d.scores.shape, dtype=torch.float32).pin_memory()
    h = ctx.ficoco_v_reduce_host(ph.tokens, ph.attn, keep, gh, gw, ph.heads, params=prm, pos_out=pos_out,
                                 scores_out=scores, **ph.call_kwargs())
    assert np.array_equal(binding.to_numpy(d.out_tokens), binding.to_numpy(h.out_tokens))
    assert np.array_equal(binding.to_numpy(d.kept_idx), binding.to_numpy(h.kept_idx))
    assert np.array_equal(binding.to_numpy(d.pos_out), pos_out.numpy())
    # a group is planned on its own, so the column sums fold in another order: scores agree
    # to rounding, the decisions taken from them are the same
    np.testing.assert_allclose(scores.numpy(), binding.to_numpy(d.scores), rtol=1e-4, atol=1e-7)
    assert ctx.ficoco_status() == 0


def test_pairwise_correlation_gap_from_inspection(ctx):
    """The paper's diagnostic for choosing K (Sec. "Correlation-based Information Recycling"):
    top-1 minus top-2 correlation of every discarded token.  With the adaptive threshold the
    library keeps each row's two (or more) largest correlations, so the gap can be read from
    the inspection arrays; it must match the checker's full correlation rows."""
    batch = synth.workload(2, small=True)
    gaps.repair_v(batch)
    p = fo.Params()
    _, results = parity.run_and_compare_v(ctx, batch, p, DEV, what="gap")
    cc = ctx.ficoco_inspect("corr_c")
    s0 = 0
    for r in results:
        order = np.argsort(r.S)
        for k, si in enumerate(order):
            row = np.sort(r.C[si])[::-1]
            np.testing.assert_allclose(cc[s0 + k, 0] - cc[s0 + k, 1], row[0] - row[1], rtol=0, atol=3e-5)
        s0 += r.S.shape[0]


def test_canaries_around_outputs(ctx):
    """Nothing is written outside the documented output extents."""
    batch = synth.workload(4, small=True)
    gaps.repair_v(batch)
    pk = packing.pack_v(batch, DEV)
    rows = sum(pk.keep)
    pad = 64
    out = torch.full((rows + 2 * pad, batch.dim), 7.0, dtype=torch.bfloat16, device=DEV)
    kidx = torch.full((rows + 2 * pad,), -7, dtype=torch.int32, device=DEV)
    pout = torch.full((rows + 2 * pad,), -7, dtype=torch.int32, device=DEV)
    ctx.ficoco_v_reduce(pk.tokens, pk.attn, pk.keep, pk.grid_h, pk.grid_w, pk.heads,
                        params=binding.make_params(has_cls=False),
                        out_tokens=out[pad:pad + rows], kept_idx=kidx[pad:pad + rows],
                        pos_out=pout[pad:pad + rows], **pk.call_kwargs())
    torch.cuda.synchronize()
    for t, v in ((out, 7.0), (kidx, -7), (pout, -7)):
        assert bool((t[:pad] == v).all()) and bool((t[pad + rows:] == v).all())
    assert bool((kidx[pad:pad + rows] >= 0).all())


@pytest.mark.parametrize("dtype", ["bf16", "fp32"])
def test_convergent_correlation_variant(ctx, dtype):
    """Ablation 'convergent correlation': preserved rows bit for bit, one additional row per image
    (the mean of the discarded rows) with kept index -1, against the checker; uniform and ragged
    batches, nothing appended where nothing is discarded, and the FiCoCo-L layout."""
    p = fo.Params(convergent=True)
    batch = synth.make_v_batch(98, 3, 13, 11, 192, 5, 80, dtype, True, 1.2)
    gaps.repair_v(batch, p)
    res, results = parity.run_and_compare_v(ctx, batch, p, DEV, what="convergent")
    assert res.out_rows == [1 + 80 + 1] * 3
    kidx = binding.to_numpy(res.kept_idx).reshape(3, -1)
    assert (kidx[:, -1] == -1).all() and (kidx[:, :-1] >= 0).all()
    ragged = synth.workload(4, small=True)
    ragged.keep[0] = ragged.tokens[0].shape[0]          # this image discards nothing: no additional row
    gaps.repair_v(ragged, p)
    res, results = parity.run_and_compare_v(ctx, ragged, p, DEV, what="convergent-ragged")
    assert res.out_rows[0] == ragged.keep[0] and res.out_rows[1] == ragged.keep[1] + 1
    if dtype == "bf16":
        lb = synth.make_l_batch(99, 2, 100, 9, 256, 3, 30, "bf16", scale=1.0 / 16)
        gaps.repair_l(lb, p)
        res, results = parity.run_and_compare_l(ctx, lb, p, DEV, what="convergent-l")
        kidx = binding.to_numpy(res.kept_idx).reshape(2, -1)
        assert (kidx[:, 30] == -1).all() and kidx[0, 31:].tolist() == list(range(100, 109))


def test_hand_built_ties_follow_the_lower_index(ctx):
    """The two hand-built tie inputs of tests/golden (bit-identical scores across the selection
    boundary, and inside one local-penalty window), with no margin repair: the library takes the
    same decisions as the checker, which the golden file pins by hand."""
    g = json.load(open(os.path.join(os.path.dirname(__file__), "golden", "hand_example.json")))["tie_cases"]
    P = np.array(g["patches"], dtype=np.float32)
    attn = np.array(g["cls_attention"], dtype=np.float32)
    # the same tokens in a wider batch: copies of the image, plus a bf16 variant with more columns
    for dtype in ("fp32", "bf16"):
        tok = P if dtype == "fp32" else synth.f32_to_bf16_bits(np.pad(P, ((0, 0), (0, 4))))
        for case in g["selection"] + [g["window"]]:
            penalty = "window" in case
            batch = synth.VBatch(dtype, False, tok.shape[1], 1, [tok.copy() for _ in range(3)],
                                 [attn.copy() for _ in range(3)], [np.arange(4, dtype=np.int32)] * 3,
                                 [(2, 2)] * 3, [case["keep"]] * 3, "ties")
            p = fo.Params(lam=g["lambda"], local_penalty=penalty)
            res, results = parity.run_and_compare_v(ctx, batch, p, DEV, what="ties")
            kidx = binding.to_numpy(res.kept_idx).reshape(3, -1)
            assert all(kidx[b].tolist() == case["T"] for b in range(3))
            assert all(sorted(r.S.tolist()) == case["S"] for r in results)
    # a larger image with many equal scores: identical tokens and attention in groups of four
    rng = synth.rng_for(95)
    base = rng.standard_normal((40, 64)).astype(np.float32)
    tok = np.repeat(base, 4, axis=0)                      # 160 tokens, every score appears four times
    a = np.repeat(rng.random((2, 40)).astype(np.float32), 4, axis=1)
    a /= a.sum(axis=1, keepdims=True)
    for keep, penalty in ((77, False), (82, False), (61, True)):
        batch = synth.VBatch("fp32", False, 64, 2, [tok], [a], [np.arange(160, dtype=np.int32)], [(10, 16)],
                             [keep], "ties-wide")
        res, results = parity.run_and_compare_v(ctx, batch, fo.Params(local_penalty=penalty, max_targets=0), DEV,
                                                what="ties-wide")
        # groups straddling the boundary exist (160 - keep is not a multiple of four), and the
        # checker's scores really tie bit for bit inside a group
        sraw = results[0].score_raw.reshape(40, 4)
        assert np.all(sraw == sraw[:, :1]) and (160 - keep) % 4 != 0


def test_bounded_wait_runs_out_and_the_context_recovers():
    """A wait between thread blocks that can never be satisfied (the testing hook makes the fused
    filter expect one arrival more than there are pieces) must end by itself: the kernels return,
    bit 2 of the status word is raised, later steps stay off until the status has been read, and
    after that an ordinary call gives exactly the bytes of a clean run."""
    c = binding.Context(max_tokens=8192, max_dim=512, max_batch=8, device=0)
    batch = synth.make_v_batch(96, 6, 16, 16, 256, 4, 128, "bf16", True, 1.2)
    pk = packing.pack_v(batch, DEV)

    def run():
        r = c.ficoco_v_reduce(pk.tokens, pk.attn, pk.keep, pk.grid_h, pk.grid_w, pk.heads, **pk.call_kwargs())
        torch.cuda.synchronize()
        return r

    clean = run()
    assert c.ficoco_status() == 0
    ref = [binding.to_numpy(t) for t in (clean.out_tokens, clean.kept_idx, clean.pos_out)]
    c.ficoco_debug_waits(wait_ns=200_000, extra_arrivals=1)
    run()
    c.ficoco_debug_waits(0, 0)
    sentinel = torch.full_like(clean.out_tokens, 3.0)
    r2 = c.ficoco_v_reduce(pk.tokens, pk.attn, pk.keep, pk.grid_h, pk.grid_w, pk.heads, out_tokens=sentinel,
                           **pk.call_kwargs())
    torch.cuda.synchronize()
    assert bool((sentinel == 3.0).all()), "a step enqueued after the timeout wrote outputs before the status was read"
    assert c.ficoco_status() & 4
    assert c.ficoco_status() == 0
    for rep in range(2):
        again = run()
        assert c.ficoco_status() == 0
        for a, b in zip(ref, (again.out_tokens, again.kept_idx, again.pos_out)):
            assert np.array_equal(a, binding.to_numpy(b))
    c.close()


def test_step_behind_a_foreign_producer_kernel(ctx):
    """Tokens and attention written by other kernels of the same stream right before the step
    (here: device copies) are read in stream order: by default no kernel of the step starts
    early.  With FICOCO_BACK_TO_BACK set on steps that do follow each other directly the results
    are the same bytes."""
    batch = synth.make_v_batch(97, 16, 24, 24, 512, 4, 288, "bf16", True, 1.5)
    pk = packing.pack_v(batch, DEV)
    prm = parity.params_to_abi(fo.Params(), True)
    ref = ctx.ficoco_v_reduce(pk.tokens, pk.attn, pk.keep, pk.grid_h, pk.grid_w, pk.heads, params=prm, **pk.call_kwargs())
    torch.cuda.synchronize()
    want = [binding.to_numpy(t) for t in (ref.out_tokens, ref.kept_idx, ref.pos_out)]
    tok2, attn2 = torch.zeros_like(pk.tokens), torch.zeros_like(pk.attn)
    for rep in range(6):
        tok2.zero_(); attn2.zero_()
        ctx.ficoco_v_reduce(pk.tokens, pk.attn, pk.keep, pk.grid_h, pk.grid_w, pk.heads, params=prm, **pk.call_kwargs())
        tok2.copy_(pk.tokens); attn2.copy_(pk.attn)          # the producers
        got = ctx.ficoco_v_reduce(tok2, attn2, pk.keep, pk.grid_h, pk.grid_w, pk.heads, params=prm,
                                  n_tokens=pk.n_tokens, pos=pk.pos)
        torch.cuda.synchronize()
        for a, b in zip(want, (got.out_tokens, got.kept_idx, got.pos_out)):
            assert np.array_equal(a, binding.to_numpy(b)), f"repetition {rep}"
    b2b = parity.params_to_abi(fo.Params(), True)
    b2b.flags |= binding.FICOCO_BACK_TO_BACK
    outs = [ctx.ficoco_v_reduce(pk.tokens, pk.attn, pk.keep, pk.grid_h, pk.grid_w, pk.heads, params=b2b, **pk.call_kwargs())
            for _ in range(4)]
    torch.cuda.synchronize()
    assert ctx.ficoco_status() == 0
    for o in outs:
        for a, b in zip(want, (o.out_tokens, o.kept_idx, o.pos_out)):
            assert np.array_equal(a, binding.to_numpy(b))


def test_planned_ragged_shape_is_captured_into_a_graph():
    """A ragged shape the context has never seen: ficoco_v_plan builds its plan ahead of time, after
    which the reduce step is captured into a CUDA graph (no synchronisation, no allocation inside
    the call) and the replay gives the bytes of an ordinary call; out_cu_seqlens holds the prefix of
    the output rows.  Without the plan the captured call is refused with FICOCO_ERR_CAPTURE."""
    c = binding.Context(max_tokens=8192, max_dim=256, max_batch=8, device=0)
    batch = synth.make_v_batch(85, 5, 9, 7, 256, 4, 20, "bf16", False, 1.0)
    for b, cut in enumerate((0, 5, 11, 2, 30)):          # five different lengths
        if cut:
            batch.tokens[b] = batch.tokens[b][:-cut]; batch.attn[b] = batch.attn[b][:, :-cut].copy()
            batch.pos[b] = batch.pos[b][:-cut]
    batch.keep = [20, 25, 17, 30, 9]
    pk = packing.pack_v(batch, DEV)
    prm = binding.make_params(has_cls=False)
    rows = sum(batch.keep)
    out = torch.zeros((rows, 256), dtype=torch.bfloat16, device=DEV)
    kidx = torch.zeros((rows,), dtype=torch.int32, device=DEV)
    pout = torch.zeros((rows,), dtype=torch.int32, device=DEV)
    ocu = torch.zeros((6,), dtype=torch.int32, device=DEV)
    st = torch.cuda.Stream()
    kw = dict(params=prm, out_tokens=out, kept_idx=kidx, pos_out=pout, out_cu_seqlens=ocu, stream=st.cuda_stream,
              **pk.call_kwargs())
    g = torch.cuda.CUDAGraph()
    with pytest.raises(binding.FicocoError) as e:
        with torch.cuda.graph(g, stream=st):
            c.ficoco_v_reduce(pk.tokens, pk.attn, pk.keep, pk.grid_h, pk.grid_w, pk.heads, **kw)
    assert e.value.code == -7
    torch.cuda.synchronize()
    c.ficoco_v_reduce(pk.tokens, pk.attn, pk.keep, pk.grid_h, pk.grid_w, pk.heads, plan_only=True, **kw)
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g, stream=st):
        c.ficoco_v_reduce(pk.tokens, pk.attn, pk.keep, pk.grid_h, pk.grid_w, pk.heads, **kw)
    g.replay()
    torch.cuda.synchronize()
    got = [binding.to_numpy(t) for t in (out, kidx, pout)]
    assert ocu.cpu().tolist() == [0, 20, 45, 62, 92, 101]
    ref = c.ficoco_v_reduce(pk.tokens, pk.attn, pk.keep, pk.grid_h, pk.grid_w, pk.heads, params=prm, **pk.call_kwargs())
    torch.cuda.synchronize()
    for a, b in zip(got, (ref.out_tokens, ref.kept_idx, ref.pos_out)):
        assert np.array_equal(a, binding.to_numpy(b))
    assert c.ficoco_status() == 0
    c.close()


def test_graph_of_an_odd_number_of_steps_replayed():
    """Three back-to-back steps captured into one graph and replayed several times, then followed by
    ordinary calls: launches replayed from a graph do not alternate between the fused filter's two
    sets of per-image counters the way consecutive calls do, and every launch must still find its
    set clean.  Every replay reproduces the bytes of an ordinary call."""
    c = binding.Context(max_tokens=8 * 145, max_dim=256, max_batch=8, device=0)
    prm = binding.make_params(has_cls=True, back_to_back=True)
    sets = []
    for i in range(3):
        batch = synth.make_v_batch(120 + i, 8, 12, 12, 256, 4, 64, "bf16", True, 1.0)
        pk = packing.pack_v(batch, DEV)
        ref = c.ficoco_v_reduce(pk.tokens, pk.attn, pk.keep, pk.grid_h, pk.grid_w, pk.heads,
                                params=binding.make_params(has_cls=True), **pk.call_kwargs())
        torch.cuda.synchronize()
        res = VResultLike(torch.zeros_like(ref.out_tokens), torch.zeros_like(ref.kept_idx), torch.zeros_like(ref.pos_out))
        sets.append((pk, ref, res))
    st = torch.cuda.Stream()

    def step(i):
        pk, _, res = sets[i]
        c.ficoco_v_reduce(pk.tokens, pk.attn, pk.keep, pk.grid_h, pk.grid_w, pk.heads, params=prm,
                          out_tokens=res.out_tokens, kept_idx=res.kept_idx, pos_out=res.pos_out,
                          stream=st.cuda_stream, **pk.call_kwargs())

    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g, stream=st):
        for i in range(3):
            step(i)
    for rep in range(5):
        for _, _, res in sets:
            res.out_tokens.zero_(); res.kept_idx.zero_(); res.pos_out.zero_()
        torch.cuda.synchronize()
        with torch.cuda.stream(st):
            g.replay()
            if rep == 2:
                g.replay()            # two replays with nothing in between
        torch.cuda.synchronize()
        for _, ref, res in sets:
            assert np.array_equal(binding.to_numpy(ref.out_tokens), binding.to_numpy(res.out_tokens)), rep
            assert np.array_equal(binding.to_numpy(ref.kept_idx), binding.to_numpy(res.kept_idx)), rep
            assert np.array_equal(binding.to_numpy(ref.pos_out), binding.to_numpy(res.pos_out)), rep
    with torch.cuda.stream(st):           # an ordinary call right behind a replay
        g.replay()
        step(0)
    torch.cuda.synchronize()
    assert np.array_equal(binding.to_numpy(sets[0][1].out_tokens), binding.to_numpy(sets[0][2].out_tokens))
    assert c.ficoco_status(st.cuda_stream) == 0
    c.close()


def test_error_codes_and_status(ctx):
    batch = synth.make_v_batch(84, 2, 6, 6, 64, 2, 20, "bf16", True, 1.0)
    pk = packing.pack_v(batch, DEV)
    kw = pk.call_kwargs()

    def call(**over):
        args = dict(tokens=pk.tokens, attn=pk.attn, keep=pk.keep, grid_h=pk.grid_h, grid_w=pk.grid_w,
                    heads=pk.heads)
        args.update(kw)
        args.update(over)
        return ctx.ficoco_v_reduce(**args)

    with pytest.raises(binding.FicocoError) as e:
        call(keep=[37, 20])
    assert e.value.code == -3
    with pytest.raises(binding.FicocoError) as e:
        call(grid_h=[5, 5])
    assert e.value.code == -8
    with pytest.raises(binding.FicocoError) as e:
        call(params=binding.make_params(eps=0.5))      # top list of 11 of 20 fits; eps=0.1 does not
        call(params=binding.make_params(eps=0.1))
    assert e.value.code == -2
    with pytest.raises(binding.FicocoError) as e:
        call(params=binding.make_params(eps=1.5))
    assert e.value.code == -1
    small = binding.Context(max_tokens=50, max_dim=64, max_batch=2)
    with pytest.raises(binding.FicocoError) as e:
        small.ficoco_v_reduce(pk.tokens, pk.attn, pk.keep, pk.grid_h, pk.grid_w, pk.heads, **kw)
    assert e.value.code == -4
    small.close()
    odd = torch.zeros((74, 12), dtype=torch.bfloat16, device=DEV)
    with pytest.raises(binding.FicocoError) as e:
        ctx.ficoco_v_reduce(odd, pk.attn, pk.keep, pk.grid_h, pk.grid_w, pk.heads, n_tokens=37)
    assert e.value.code == -2
    # outputs may not overlap inputs (Eq. 2 reads the pre-update tokens)
    with pytest.raises(binding.FicocoError) as e:
        call(out_tokens=pk.tokens)
    assert e.value.code == -1
    with pytest.raises(binding.FicocoError) as e:
        call(pos_out=pk.pos)
    assert e.value.code == -1
    # a position outside the grid is reported through the status word, not a fault
    bad = pk.pos.clone()
    bad[5] = 36 + 1000
    call(pos=bad)
    assert ctx.ficoco_status() == 1
    call()
    assert ctx.ficoco_status() == 0


# ---------------------------------------------------------------------------------------
# full-size workloads, in the launch configuration the benchmark times
# ---------------------------------------------------------------------------------------
def _report_plain_score_error(what):
    print(f"\n[{what}] worst plain relative score error so far: "
          + ", ".join(f"{k} {v:.2e}" for k, v in sorted(parity.WORST_PLAIN_REL.items())))


def test_full_c1(ctx):
    batch = synth.workload(1)
    gaps.repair_v(batch)
    parity.run_and_compare_v(ctx, batch, fo.Params(), DEV, what="c1")
    _report_plain_score_error("c1")


def test_full_c2_schedule(ctx):
    batch = synth.workload(2)
    p = fo.Params()
    for step, keep in enumerate(synth.SCHEDULES[2]):
        batch.keep = [keep] * batch.batch
        gaps.repair_v(batch)
        _, results = parity.run_and_compare_v(ctx, batch, p, DEV, what=f"c2 step {step}")
        batch.tokens = [r.out for r in results]
        batch.pos = [r.pos_out for r in results]
        if step + 1 < 3:
            synth.regenerate_attention(batch, 2000, step + 1, 1.5)
    _report_plain_score_error("c2 schedule")


@pytest.mark.parametrize("by_column", [True, False], ids=["by-column", "by-row"])
def test_full_c2_shape_relation_mode(ctx, by_column):
    """The shape bench.py times for the relation mode: 32 images, 576 x 576 maps."""
    batch = synth.workload(2)
    rels = _relations(batch, 94, stochastic=by_column, times_n=True)
    gaps.repair_v_relation(batch, rels, by_column)
    parity.run_and_compare_v_relation(ctx, batch, rels, by_column, fo.Params(), DEV, what="c2-relation")


def test_full_c3_schedule(ctx):
    """2880 -> 1440 -> 720 -> 320 at full size (8 images x 2881 tokens), every step on the checker's
    previous output; the later steps reach top lists of three and two entries."""
    batch = synth.workload(3)
    p = fo.Params()
    for step, keep in enumerate(synth.SCHEDULES[3]):
        batch.keep = [keep] * batch.batch
        gaps.repair_v(batch)
        _, results = parity.run_and_compare_v(ctx, batch, p, DEV, what=f"c3 step {step}")
        batch.tokens = [r.out for r in results]
        batch.pos = [r.pos_out for r in results]
        if step + 1 < 3:
            synth.regenerate_attention(batch, 3000, step + 1, 1.0)
    _report_plain_score_error("c3 schedule")


def _checker_chain(batch, sched, seed, sigma):
    """The checker's chained run of a schedule: per step the (margin-repaired) attention it used,
    and at the end the tokens, the composed kept indices and the positions."""
    p = fo.Params()
    attns, chain = [], None
    for step, keep in enumerate(sched):
        batch.keep = [keep] * batch.batch
        gaps.repair_v(batch)
        attns.append(np.stack(batch.attn, axis=0).astype(np.float32))
        results = fo.v_reduce_batch(batch, p)
        chain = [r.kept_idx if chain is None else c[r.kept_idx] for r, c in zip(results, chain or results)]
        batch.tokens = [r.out for r in results]
        batch.pos = [r.pos_out for r in results]
        if step + 1 < len(sched):
            synth.regenerate_attention(batch, seed, step + 1, sigma)
    return attns, results, chain


@pytest.mark.parametrize("idx,small", [(2, True), (3, True), (2, False)], ids=["c2-small", "c3-small", "c2-full"])
def test_schedule_entry_point_chains_its_own_outputs(ctx, idx, small):
    """ficoco_v_reduce_schedule runs all steps on the GPU's own intermediate outputs; the result is
    compared with the checker's chained run of the same schedule: the composed kept indices and
    the final positions exactly, the final tokens within the bf16 tolerance once per step (a
    merged row may be rounded differently by one ulp in one step and feed the next).  The margins
    that make a step's decisions unambiguous were established on the checker's intermediates; on
    intermediates that differ by an ulp here and there a discarded token whose two best targets are
    nearly tied can go to the other one, which moves two output rows: at most 1 % of the rows may
    be off for that reason (what is kept, and where, must still agree exactly)."""
    batch = synth.workload(idx, small=small)
    sched = (synth.SCHEDULES_SMALL if small else synth.SCHEDULES)[idx]
    pk = packing.pack_v(batch, DEV)
    gh, gw = batch.grid[0]
    attns, results, chain = _checker_chain(batch, sched, 1000 * idx, 1.5 if idx == 2 else 1.0)
    attn_d = [torch.from_numpy(a.reshape(-1)).to(DEV) for a in attns]
    pk.attn = attn_d[0]
    prm = parity.params_to_abi(fo.Params(), True)
    for rep in range(2):                                   # the second call allocates nothing
        res = ctx.ficoco_v_reduce_schedule(pk.tokens, attn_d, sched, gh, gw, pk.heads, n_tokens=pk.n_tokens,
                                           pos=pk.pos, params=prm)
        torch.cuda.synchronize()
        assert ctx.ficoco_status() == 0
        out = binding.to_numpy(res.out_tokens).reshape(batch.batch, 1 + sched[-1], -1)
        kidx = binding.to_numpy(res.kept_idx).reshape(batch.batch, -1)
        pout = binding.to_numpy(res.pos_out).reshape(batch.batch, -1)
        n_steps = len(sched)
        rows_off = rows_all = 0
        for b, r in enumerate(results):
            assert np.array_equal(kidx[b], chain[b]), f"image {b}: composed kept indices"
            assert np.array_equal(pout[b], r.pos_out), f"image {b}: positions"
            g, e = fo.widen(out[b]), fo.widen(r.out)
            tol = n_steps * (parity.BF16_ATOL + parity.BF16_RTOL * np.abs(e))
            rows_off += int(np.any(np.abs(g - e) > tol, axis=1).sum())
            rows_all += g.shape[0]
            assert np.array_equal(out[b][0], r.out[0])   # CLS passes through every step untouched
        assert rows_off <= 0.01 * rows_all, f"{rows_off} of {rows_all} final rows off"
    # the same chain as separate calls gives the same bytes
    cur_tok, cur_pos, n_tok = pk.tokens, pk.pos, pk.n_tokens
    for s, keep in enumerate(sched):
        r1 = ctx.ficoco_v_reduce(cur_tok, attn_d[s], keep, gh, gw, pk.heads, n_tokens=n_tok, pos=cur_pos, params=prm)
        cur_tok, cur_pos, n_tok = r1.out_tokens, r1.pos_out, 1 + keep
    torch.cuda.synchronize()
    assert np.array_equal(binding.to_numpy(cur_tok), binding.to_numpy(res.out_tokens))
    assert np.array_equal(binding.to_numpy(cur_pos), binding.to_numpy(res.pos_out))


def test_full_c4(ctx):
    batch = synth.workload(4)
    gaps.repair_v(batch)
    parity.run_and_compare_v(ctx, batch, fo.Params(), DEV, what="c4")


def test_full_c5(ctx):
    batch = synth.workload(5)
    gaps.repair_l(batch)
    parity.run_and_compare_l(ctx, batch, fo.Params(), DEV, what="c5")
