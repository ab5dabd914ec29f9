#!/usr/bin/env python
"""Benchmark of the FiCoCo-V reduce step.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

A step is one pass of the whole reduce step (filter, correlate, compress, compact) over one
batch of 32 synthetic images of 577 x 1024 bf16 tokens, reducing 576 -> 288 patch tokens.
Rank 0 prints one JSON line.  With N > 1 every rank reduces its own batch (images are
independent, there is no collective on the data path) and the value is the aggregate.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "images/sec of FiCoCo-V reduce step, B=32x577x1024 bf16"
UNIT = "images/s"
B, GH, GW, D, H, KEEP = 32, 24, 24, 1024, 16, 288
WORKLOAD = "c2 step 1: 32 images x (1 CLS + 24x24 patches) x 1024 bf16, 576 -> 288 patch tokens"
N_INSTANCES = 8       # distinct input/output buffer sets cycled through: 8 x 58 MB > 3 x L2
MIN_TIMED_MS = 50.0   # device time the timed repetitions add up to, at least
NOMINAL = {"hbm_gbs": 8000.0, "bf16_tflops": 2250.0}   # vendor figures, reported beside the measured peaks
# dram__bytes_read.sum + dram__bytes_write.sum per launch from the ncu capture summarised under
# profiles/ (bytes); an entry is removed when its kernel changes after the capture.
NCU_TRAFFIC = {"filter_fused": 39088384 + 12800, "correlate_umma": 37963264 + 7680, "merge_compact": 37894912 + 30720}


def algorithmic_bytes() -> dict:
    """Per-step algorithmic HBM traffic: read X once, read attention, write the output, plus
    the index arrays (pos in, kept_idx and pos_out out)."""
    n, npatch = 1 + GH * GW, GH * GW
    x_in = B * n * D * 2
    attn = B * H * npatch * 4
    out = B * (1 + KEEP) * D * 2
    idx = B * 4 * (npatch + 2 * KEEP)
    return {"tokens_in": x_in, "attn": attn, "tokens_out": out, "index": idx,
            "total": x_in + attn + out + idx}


def peaks() -> dict:
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return {"hbm_gbs": float(p["hbm_gbs"]), "bf16_tflops": float(p["bf16_tflops"]), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "source": "fallback"}


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.proc, self.lines = index, None, []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits", "-i", str(self.index),
                 "-lms", "100"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.th = threading.Thread(target=self._read, daemon=True)
            self.th.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=2)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], None, set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in self.lines:
            f = [x.strip() for x in ln.split(",")]
            if len(f) < 7:
                continue
            try:
                sm.append(float(f[0])); mx = float(f[1])
            except ValueError:
                continue
            for nm, v in zip(names, f[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(nm)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": mx,
                "reasons": sorted(reasons), "samples": len(sm)}


def shard_seed(rank: int) -> int:
    """Every rank reduces its own batch of B images (weak scaling): the generator seed differs
    per rank, nothing is exchanged between ranks on the data path."""
    return 2000 + rank


def max_over_ranks(ms: float, world: int, device=None) -> float:
    """Elapsed device time of the slowest rank (all_reduce MAX over the process group)."""
    if world <= 1:
        return ms
    import torch
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    torch.distributed.all_reduce(t, op=torch.distributed.ReduceOp.MAX)
    return float(t.item())


def aggregate_images_per_s(ms_per_step: float, world: int) -> float:
    """Whole-job throughput: all ranks' images per step over the slowest rank's step time."""
    return world * B / (ms_per_step * 1e-3)


def make_instances(rank: int):
    """One generated batch, laid out N_INSTANCES times with the image order rotated, so every
    step reads and writes memory that is not in L2 from the step before."""
    from paper_2411_17686_b200 import synth
    batch = synth.make_v_batch(shard_seed(rank), B, GH, GW, D, H, KEEP, "bf16", True, 1.5, name="c2")
    return batch


def other_workloads(binding, packing, ctx, insts, prm, stream, dev) -> dict:
    """Device times of the other configurations (not the headline metric): the whole progressive
    schedule of the headline batch (576 -> 288 -> 144 -> 64, every step fed from the one before,
    one CUDA graph over the 8 buffer sets) and one reduce step of the other four workloads
    (their inputs are reused every step, so the smaller ones are L2-warm)."""
    import torch
    from paper_2411_17686_b200 import synth
    out = {}
    n = 1 + GH * GW
    k2, k3 = KEEP // 2, 64
    g = torch.Generator().manual_seed(7)
    attn2 = torch.softmax(1.5 * torch.randn(B, H, KEEP, generator=g), -1).reshape(-1).to(dev)
    attn3 = torch.softmax(1.5 * torch.randn(B, H, k2, generator=g), -1).reshape(-1).to(dev)
    o2 = torch.empty((B * (1 + k2), D), dtype=torch.bfloat16, device=dev)
    o3 = torch.empty((B * (1 + k3), D), dtype=torch.bfloat16, device=dev)
    i2 = torch.empty((B * (1 + k2),), dtype=torch.int32, device=dev)
    i3 = torch.empty((B * (1 + k3),), dtype=torch.int32, device=dev)
    p2 = torch.empty((B * k2,), dtype=torch.int32, device=dev)
    p3 = torch.empty((B * k3,), dtype=torch.int32, device=dev)

    def chain(i):
        it = insts[i % N_INSTANCES]
        s = stream.cuda_stream
        ctx.ficoco_v_reduce(it["tokens"], it["attn"], KEEP, GH, GW, H, n_tokens=n, pos=it["pos"], params=prm,
                            out_tokens=it["out"], kept_idx=it["kidx"], pos_out=it["pout"], stream=s)
        ctx.ficoco_v_reduce(it["out"], attn2, k2, GH, GW, H, n_tokens=1 + KEEP, pos=it["pout"], params=prm,
                            out_tokens=o2, kept_idx=i2, pos_out=p2, stream=s)
        ctx.ficoco_v_reduce(o2, attn3, k3, GH, GW, H, n_tokens=1 + k2, pos=p2, params=prm,
                            out_tokens=o3, kept_idx=i3, pos_out=p3, stream=s)

    def schedule(i):
        it = insts[i % N_INSTANCES]
        ctx.ficoco_v_reduce_schedule(it["tokens"], [it["attn"], attn2, attn3], [KEEP, k2, k3], GH, GW, H, n_tokens=n,
                                     pos=it["pos"], params=prm, out_tokens=o3, kept_idx=i3, pos_out=p3,
                                     stream=stream.cuda_stream)

    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    for label, fn in (("c2 schedule 576->288->144->64", chain),
                      ("c2 schedule 576->288->144->64, one ficoco_v_reduce_schedule call", schedule)):
        with torch.cuda.stream(stream):
            fn(0)
        torch.cuda.synchronize()
        gr = torch.cuda.CUDAGraph()
        with torch.cuda.graph(gr, stream=stream):
            for i in range(N_INSTANCES):
                fn(i)
        with torch.cuda.stream(stream):
            gr.replay()
            e0.record(stream)
            for _ in range(5):
                gr.replay()
            e1.record(stream)
        torch.cuda.synchronize()
        us = e0.elapsed_time(e1) * 1e3 / (5 * N_INSTANCES)
        out[label] = {"us_per_schedule": us, "images_per_s": B / (us * 1e-6)}

    # the same step driven by a caller-supplied relation map (fp32 [B, 576, 576], attention each
    # token receives): the map is read once for the scores and its discarded rows once more for C;
    # three maps and the 8 token sets are cycled so that every step starts from HBM
    npatch = GH * GW
    rels = [torch.softmax(4.0 * torch.randn((B, npatch, npatch), generator=g), -1).reshape(-1).to(dev)
            for _ in range(3)]

    def rel_step(i):
        it = insts[i % N_INSTANCES]
        ctx.ficoco_v_reduce(it["tokens"], it["attn"], KEEP, GH, GW, H, n_tokens=n, pos=it["pos"], params=prm,
                            out_tokens=it["out"], kept_idx=it["kidx"], pos_out=it["pout"],
                            stream=stream.cuda_stream, relation=rels[i % 3], by_column=True)

    with torch.cuda.stream(stream):
        for i in range(3):
            rel_step(i)
    torch.cuda.synchronize()
    rel_graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(rel_graph, stream=stream):
        for i in range(24):
            rel_step(i)
    with torch.cuda.stream(stream):
        rel_graph.replay()
        e0.record(stream)
        for _ in range(5):
            rel_graph.replay()
        e1.record(stream)
    torch.cuda.synchronize()
    assert ctx.ficoco_status(stream.cuda_stream) == 0
    rel_us = e0.elapsed_time(e1) * 1e3 / (5 * 24)
    rel_bytes = B * npatch * npatch * 4 + algorithmic_bytes()["total"]
    out["c2 step 1 on a supplied relation map (by column)"] = {
        "us_per_step": rel_us, "images_per_s": B / (rel_us * 1e-6), "algorithmic_bytes": rel_bytes,
        "achieved_gbs": rel_bytes / rel_us / 1e3, "frac_of_hbm_peak": rel_bytes / rel_us / 1e3 / peaks()["hbm_gbs"]}
    del rels

    for idx, label in ((1, "c1: 1 x 577 x 1024 fp32, discard 64"), (3, "c3 step 1: 8 x 2881 x 1024 bf16, 2880 -> 1440"),
                       (4, "c4: 16 ragged images x 1280 bf16, keep 1/9"), (5, "c5: FiCoCo-L 16 x (576+64) x 4096 bf16, 576 -> 64")):
        wl = synth.workload(idx)
        rows = sum(int(t.shape[0]) for t in wl.tokens)
        c2 = binding.Context(max_tokens=rows, max_dim=wl.dim, max_batch=len(wl.tokens),
                             max_text=getattr(wl, "n_text", 0), device=torch.device(dev).index)
        try:
            if idx == 5:
                pk = packing.pack_l(wl, dev)
                pp = binding.make_params(has_cls=False)
                res = c2.ficoco_l_reduce(pk.tokens, pk.attn_t2v, pk.keep, pk.n_vision, pk.n_text, pk.heads, params=pp,
                                         stream=stream.cuda_stream)
                step = lambda: c2.ficoco_l_reduce(pk.tokens, pk.attn_t2v, pk.keep, pk.n_vision, pk.n_text, pk.heads,
                                                  params=pp, out_tokens=res.out_tokens, kept_idx=res.kept_idx,
                                                  stream=stream.cuda_stream)
            else:
                pk = packing.pack_v(wl, dev)
                pp = binding.make_params(has_cls=wl.has_cls)
                res = c2.ficoco_v_reduce(pk.tokens, pk.attn, pk.keep, pk.grid_h, pk.grid_w, pk.heads, params=pp,
                                         stream=stream.cuda_stream, **pk.call_kwargs())
                step = lambda: c2.ficoco_v_reduce(pk.tokens, pk.attn, pk.keep, pk.grid_h, pk.grid_w, pk.heads,
                                                  params=pp, out_tokens=res.out_tokens, kept_idx=res.kept_idx,
                                                  pos_out=res.pos_out, stream=stream.cuda_stream, **pk.call_kwargs())
            with torch.cuda.stream(stream):
                for _ in range(3):
                    step()
                e0.record(stream)
                for _ in range(20):
                    step()
                e1.record(stream)
            torch.cuda.synchronize()
            assert c2.ficoco_status(stream.cuda_stream) == 0
            out[label] = {"us_per_step": e0.elapsed_time(e1) * 1e3 / 20, "images": len(wl.tokens), "token_rows": rows}
            # the library's own events between its launches (serialises them: shares, not a sum to compare)
            c2.ficoco_profile(True)
            with torch.cuda.stream(stream):
                for _ in range(5):
                    step()
            torch.cuda.synchronize()
            out[label]["kernels_us"] = {nm: round(1e3 * t / max(cnt, 1), 2) for nm, t, cnt in c2.ficoco_profile_read()}
            c2.ficoco_profile(False)
        finally:
            c2.close()
    return out


def run_ours(args, rank: int, world: int, local_rank: int):
    import torch
    from paper_2411_17686_b200 import binding, build, packing
    build.build()
    torch.cuda.set_device(local_rank)
    dev = f"cuda:{local_rank}"
    batch = make_instances(rank)
    n = 1 + GH * GW
    base = packing.pack_v(batch, None)
    tok_h = base.tokens.view(B, n, D)
    attn_h = base.attn.view(B, H, GH * GW)
    insts = []
    for k in range(N_INSTANCES):
        perm = [(b + k) % B for b in range(B)]
        insts.append(dict(
            tokens=tok_h[perm].reshape(B * n, D).contiguous().to(dev),
            attn=attn_h[perm].reshape(-1).contiguous().to(dev),
            pos=base.pos.to(dev),
            out=torch.empty((B * (1 + KEEP), D), dtype=torch.bfloat16, device=dev),
            kidx=torch.empty((B * (1 + KEEP),), dtype=torch.int32, device=dev),
            pout=torch.empty((B * KEEP,), dtype=torch.int32, device=dev)))
    ctx = binding.Context(max_tokens=B * n, max_dim=D, max_batch=B, device=local_rank)
    prm = binding.ficoco_default_params()
    prm.flags |= binding.FICOCO_BACK_TO_BACK     # the timed stream carries nothing but reduce steps
    stream = torch.cuda.Stream(device=dev)

    def step(i: int):
        it = insts[i % N_INSTANCES]
        ctx.ficoco_v_reduce(it["tokens"], it["attn"], KEEP, GH, GW, H, n_tokens=n, pos=it["pos"], params=prm,
                            out_tokens=it["out"], kept_idx=it["kidx"], pos_out=it["pout"],
                            stream=stream.cuda_stream)

    def barrier():
        if world > 1:
            torch.distributed.barrier()
        torch.cuda.synchronize()

    with torch.cuda.stream(stream):
        for i in range(max(args.warmup, 3)):
            step(i)
    torch.cuda.synchronize()
    launches_per_step = ctx.ficoco_last_launch_count()

    # The timed steps are always replayed from CUDA graphs (the host's launch cost stays off the GPU
    # timeline whatever --steps is): one graph of a full cycle over the buffer sets, one of the
    # steps % N_INSTANCES remaining steps, together exactly `steps` steps per repetition.
    def capture(n_steps: int):
        if n_steps == 0:
            return None
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=stream):
            for i in range(n_steps):
                step(i)
        return g

    graph = rem_graph = None
    if args.graph:
        graph = capture(N_INSTANCES) if args.steps >= N_INSTANCES else None
        rem_graph = capture(args.steps % N_INSTANCES)
        with torch.cuda.stream(stream):
            for g in (graph, rem_graph):
                if g is not None:
                    g.replay()
        torch.cuda.synchronize()

    def run_steps():
        if not args.graph:
            for i in range(args.steps):
                step(i)
            return
        for _ in range(args.steps // N_INSTANCES):
            graph.replay()
        if rem_graph is not None:
            rem_graph.replay()

    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
        time.sleep(0.3)
    # The `steps`-step region is repeated until at least MIN_TIMED_MS of device time has been timed
    # (at least 3, at most 400 repetitions); every repetition is bracketed by its own pair of events
    # and the reported time per step is the median over the repetitions.
    reps = []
    barrier()
    with torch.cuda.stream(stream):
        probe0, probe1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        probe0.record(stream)
        run_steps()
        probe1.record(stream)
    torch.cuda.synchronize()
    est_ms = max(probe0.elapsed_time(probe1), 1e-3)
    n_rep = int(min(400, max(3, np.ceil(MIN_TIMED_MS / est_ms))))
    if world > 1:                       # every rank runs the same number of repetitions
        t = torch.tensor([n_rep], dtype=torch.int64, device=dev)
        torch.distributed.all_reduce(t, op=torch.distributed.ReduceOp.MAX)
        n_rep = int(t.item())
    evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(n_rep)]
    barrier()
    with torch.cuda.stream(stream):
        for a, b in evs:
            a.record(stream)
            run_steps()
            b.record(stream)
    barrier()
    reps = [a.elapsed_time(b) for a, b in evs]
    clocks = sampler.stop() if rank == 0 else None
    ms = max_over_ranks(float(np.median(reps)), world, dev)
    ms_min = max_over_ranks(float(np.min(reps)), world, dev)
    ms_max = max_over_ranks(float(np.max(reps)), world, dev)
    ms_per_step = ms / args.steps
    value = aggregate_images_per_s(ms_per_step, world)

    if rank != 0:
        return None

    # per-kernel durations, measured live with events between the launches of the same steps
    ctx.ficoco_profile(True)
    with torch.cuda.stream(stream):
        for i in range(args.steps):
            step(i)
    torch.cuda.synchronize()
    prof = ctx.ficoco_profile_read()
    ctx.ficoco_profile(False)
    kern = {nm: {"avg_us": 1e3 * t / max(cnt, 1), "launches_per_step": cnt / args.steps} for nm, t, cnt in prof}
    tot_us = sum(v["avg_us"] * v["launches_per_step"] for v in kern.values())
    for v in kern.values():
        v["share"] = v["avg_us"] * v["launches_per_step"] / tot_us if tot_us else 0.0
    dom = max(kern, key=lambda k: kern[k]["share"])

    pk = peaks()
    ab = algorithmic_bytes()
    roof = kernel_roofline(dom, kern[dom]["avg_us"], pk, ab)
    t_roof_us = max(ab["total"] / (pk["hbm_gbs"] * 1e3), 2.0 * B * (GH * GW - KEEP) * KEEP * D / (pk["bf16_tflops"] * 1e6))

    # the equivalent token of the no-CLS variant on key states of the same shape (B x 577 tokens,
    # 16 heads of 64, bf16): an HBM stream, timed on rotating buffers larger than L2
    eq_keys = [torch.randn((B * n, H * 64), device=dev, dtype=torch.float32).to(torch.bfloat16) for _ in range(4)]
    eq_out = torch.empty((B * (n - 1),), dtype=torch.float32, device=dev)
    with torch.cuda.stream(stream):
        for i in range(4):
            binding.ficoco_equivalent_token(eq_keys[i], H, 64, n_tokens=n, has_cls=True, a_eq=eq_out,
                                            stream=stream.cuda_stream)
    torch.cuda.synchronize()
    eq_graph = torch.cuda.CUDAGraph()          # replayed, so that the host's launch cost is off the timeline
    with torch.cuda.graph(eq_graph, stream=stream):
        for i in range(4):
            binding.ficoco_equivalent_token(eq_keys[i], H, 64, n_tokens=n, has_cls=True, a_eq=eq_out,
                                            stream=stream.cuda_stream)
    with torch.cuda.stream(stream):
        eq_graph.replay()
        q0, q1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        q0.record(stream)
        for _ in range(10):
            eq_graph.replay()
        q1.record(stream)
    torch.cuda.synchronize()
    eq_us = q0.elapsed_time(q1) * 1e3 / 40
    eq_bytes = B * n * H * 64 * 2 + B * (n - 1) * 4
    eq_info = {"us_per_launch": eq_us, "algorithmic_bytes": eq_bytes, "achieved_gbs": eq_bytes / eq_us / 1e3,
               "frac_of_hbm_peak": eq_bytes / eq_us / 1e3 / pk["hbm_gbs"], "launches": 40,
               "workload": "32 x 577 tokens x 16 heads x 64 bf16 keys, 4 buffers cycled"}
    del eq_keys

    extras = other_workloads(binding, packing, ctx, insts, prm, stream, dev) if args.extras else None

    # end to end through the host-buffer entry point (pinned host tensors, copies inside)
    hp = packing.pack_v(batch, None, pin=True)
    out_h = torch.empty((B * (1 + KEEP), D), dtype=torch.bfloat16).pin_memory()
    kidx_h = torch.empty((B * (1 + KEEP),), dtype=torch.int32).pin_memory()
    e2e_steps = max(5, min(args.steps, 50))
    for _ in range(3):
        ctx.ficoco_v_reduce_host(hp.tokens, hp.attn, KEEP, GH, GW, H, n_tokens=n, pos=hp.pos, params=prm,
                                 out_tokens=out_h, kept_idx=kidx_h)
    t0 = time.perf_counter()
    for _ in range(e2e_steps):
        ctx.ficoco_v_reduce_host(hp.tokens, hp.attn, KEEP, GH, GW, H, n_tokens=n, pos=hp.pos, params=prm,
                                 out_tokens=out_h, kept_idx=kidx_h)
    e2e_s = (time.perf_counter() - t0) / e2e_steps
    h2d = hp.tokens.numel() * 2 + hp.attn.numel() * 4 + hp.pos.numel() * 4
    d2h = out_h.numel() * 2 + kidx_h.numel() * 4

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": WORKLOAD, "batch_per_gpu": B, "tokens_per_image": n, "dim": D, "heads": H,
                   "keep": KEEP, "l2": f"inputs larger than L2: {N_INSTANCES} buffer sets cycled",
                   "cuda_graph": bool(args.graph), "repetitions": n_rep,
                   "ms_per_step_min": ms_min / args.steps, "ms_per_step_max": ms_max / args.steps,
                   "timed_ms": float(np.sum(reps)),
                   "stream": "reduce steps only, FICOCO_BACK_TO_BACK set"},
        "tokens_per_s": value * n,
        "clocks": clocks,
        "equivalent_token": eq_info,
        "other_workloads": extras,
        "e2e": {"value": world * B / e2e_s, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "steps": e2e_steps},
        "gpu_launches": launches_per_step * args.steps,
        "roofline": roof,
        "step_roofline": {"bound": "hbm" if ab["total"] / (pk["hbm_gbs"] * 1e3) >= t_roof_us - 1e-9 else "tensor",
                          "t_roof_us": t_roof_us, "t_measured_us": ms_per_step * 1e3,
                          "frac": t_roof_us / (ms_per_step * 1e3),
                          "frac_of_nominal": max(ab["total"] / (NOMINAL["hbm_gbs"] * 1e3),
                                                 2.0 * B * (GH * GW - KEEP) * KEEP * D / (NOMINAL["bf16_tflops"] * 1e6))
                          / (ms_per_step * 1e3),
                          "algorithmic_bytes": ab["total"],
                          "peak": f"{pk['source']} {pk['hbm_gbs']} GB/s, {pk['bf16_tflops']} TFLOP/s bf16"},
        "kernels": kern,
    }
    line["cpu_baseline"] = cpu_baseline(batch, budget_s=args.cpu_budget)
    ctx.close()
    return line


def kernel_roofline(name: str, avg_us: float, pk: dict, ab: dict) -> dict:
    """Roofline entry of the dominant kernel: its own algorithmic bytes (or flops) per launch
    over its measured average duration.  Algorithmic figures per launch (one batch of B images):
      filter_fused / colsum : X read once from HBM (+ attention)          -> hbm
      correlate_*           : 2 * N^S * N^T * D flops per image            -> tensor
      merge_compact         : preserved rows in (L2-resident) + rows out   -> hbm
    """
    npatch, ns = GH * GW, GH * GW - KEEP
    src = pk["source"]
    if name.startswith("correlate"):
        flops = 2.0 * B * ns * KEEP * D
        ach = flops / (avg_us * 1e-6) / 1e12
        return {"kernel": name, "bound": "tensor", "achieved": ach, "peak": pk["bf16_tflops"], "unit": "TFLOP/s",
                "frac": ach / pk["bf16_tflops"], "traffic": NCU_TRAFFIC.get(name), "of": src,
                "algorithmic_flops_per_launch": flops}
    per = {
        "filter_fused": ab["tokens_in"] + ab["attn"] + B * npatch * 4,   # X once, attention, pos
        "colsum": ab["tokens_in"],
        "score": ab["tokens_in"] + ab["attn"],
        "merge_compact": ab["tokens_out"] * 2,
        "select": B * npatch * 4 * 3, "finalize": B * ns * 16, "rownorm": ab["tokens_in"],
    }.get(name, ab["total"])
    ach = per / (avg_us * 1e-6) / 1e9
    return {"kernel": name, "bound": "hbm", "achieved": ach, "peak": pk["hbm_gbs"], "unit": "GB/s",
            "frac": ach / pk["hbm_gbs"], "traffic": NCU_TRAFFIC.get(name), "of": src,
            "algorithmic_bytes_per_launch": per}


def cpu_baseline(batch, budget_s: float = 12.0) -> dict:
    """The float64 checker as it stands, on the host cores, over whole batches of the same
    workload until the time budget is used."""
    from oracle import ficoco_oracle as fo
    cores = os.cpu_count() or 1
    try:
        from threadpoolctl import threadpool_info
        cores = max([p.get("num_threads", 1) for p in threadpool_info()] + [1])
    except Exception:
        pass
    done, t0 = 0, time.perf_counter()
    while True:
        for b in range(batch.batch):
            fo.ficoco_v_reduce(batch.tokens[b], batch.attn[b], batch.pos[b], batch.grid[b], batch.keep[b], True)
            done += 1
            if time.perf_counter() - t0 > budget_s:
                break
        if time.perf_counter() - t0 > budget_s:
            break
    dt = time.perf_counter() - t0
    return {"value": done / dt, "unit": UNIT, "cores": cores, "kind": "oracle",
            "sample": f"{done} images of the same workload in {dt:.1f} s (numpy float64)"}


def run_reference(args, rank: int):
    """Reference arm: the float64 checker on the host cores, each step one whole batch of the
    workload (all 32 images, about a quarter of a second)."""
    if rank != 0:
        return None
    from oracle import ficoco_oracle as fo
    batch = make_instances(0)
    sample = B
    cores = os.cpu_count() or 1
    try:
        from threadpoolctl import threadpool_info
        cores = max([p.get("num_threads", 1) for p in threadpool_info()] + [1])
    except Exception:
        pass

    def step(i):
        for b in range(sample):
            k = (i * sample + b) % batch.batch
            fo.ficoco_v_reduce(batch.tokens[k], batch.attn[k], batch.pos[k], batch.grid[k], batch.keep[k], True)

    for i in range(max(1, min(args.warmup, 3))):
        step(i)
    t0 = time.perf_counter()
    for i in range(args.steps):
        step(i)
    dt = time.perf_counter() - t0
    value = sample * args.steps / dt
    return {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * dt / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": WORKLOAD, "batch_per_gpu": B, "tokens_per_image": 1 + GH * GW, "dim": D, "heads": H,
                   "keep": KEEP, "sample_per_step": f"all {B} images of a batch"},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle",
                         "sample": f"{sample} images per step, {args.steps} steps"},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }


def spawn_ranks(n: int, argv) -> int:
    """`bench.py --gpus N` started as a plain process: start N ranks of this file, one per GPU,
    the way the multi-GPU launch line does (torch.distributed.run on 127.0.0.1), and pass their
    output through."""
    port = 29500 + os.getpid() % 2000
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + list(argv)
    return subprocess.call(cmd)


def run_dry(args, rank: int, world: int):
    """The N > 1 plumbing without a GPU: a gloo group, one shard seed per rank, a made-up step time
    per rank (rank r: 10 + 5 r ms for `steps` steps), the max over ranks and the aggregate."""
    import torch.distributed as dist
    if world > 1:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("gloo")
    ms = max_over_ranks(10.0 + 5.0 * rank, world)
    seeds = [shard_seed(r) for r in range(world)]
    line = None
    if rank == 0:
        line = {"metric": METRIC, "dry_run": True, "n_gpus": world, "steps": args.steps, "unit": UNIT,
                "ms_per_step": ms / args.steps, "value": aggregate_images_per_s(ms / args.steps, world),
                "scaling": "weak", "shard_seeds": seeds}
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()
    return line


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=None)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-graph", dest="graph", action="store_false")
    ap.add_argument("--cpu-budget", type=float, default=12.0)
    ap.add_argument("--no-extras", dest="extras", action="store_false",
                    help="skip the schedule / other-workload timings that follow the headline measurement")
    ap.add_argument("--dry-run", action="store_true",
                    help="exercise the multi-rank plumbing on CPU (gloo, no kernels): ranks, shards, max-over-ranks")
    args = ap.parse_args()
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ and args.impl == "ours":
        sys.exit(spawn_ranks(args.gpus, sys.argv[1:]))
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if args.impl == "reference":
        args.steps = args.steps if args.steps is not None else 20
        args.warmup = args.warmup if args.warmup is not None else 2
        line = run_reference(args, rank)
        if line is not None:
            print(json.dumps(line), flush=True)
        return
    args.steps = args.steps if args.steps is not None else 2000
    args.warmup = args.warmup if args.warmup is not None else 10
    if args.dry_run:
        line = run_dry(args, rank, world)
        if line is not None:
            print(json.dumps(line), flush=True)
        return
    if world > 1:
        import torch
        import torch.distributed as dist
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        torch.cuda.set_device(local_rank)
        dist.init_process_group("nccl", device_id=torch.device(f"cuda:{local_rank}"))
    line = run_ours(args, rank, world, local_rank)
    if line is not None:
        print(json.dumps(line), flush=True)
    if world > 1:
        import torch.distributed as dist
        dist.barrier()
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
