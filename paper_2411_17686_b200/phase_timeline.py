"""In-kernel phase time line of the reduce step in steady state.

Builds the library a second time with -DFICOCO_PHASE_TIMERS (libficoco_phase.so, beside the normal
one), replays N back-to-back steps of the 32 x 577 x 1024 bf16 workload from one CUDA graph and prints,
per launch, when the CTAs of each kernel start and end and how long their phases take.  Thread 0 of
every CTA notes the SM clock at the marks compiled into the kernels, in a record drawn from a
per-kernel counter; consecutive launches of a kernel are told apart by the order of their records.

    python -m paper_2411_17686_b200.phase_timeline [--steps 4] [--workload 2]

The timers cost about 1 % of the step; numbers printed here are for reading the structure of the
step, the bench reports the step time.
"""
from __future__ import annotations

import argparse
import ctypes as C
import os
import subprocess

import numpy as np

from . import binding, build, packing, synth

PHASE_LIB = os.path.join(build.PKG, "libficoco_phase.so")
PH_KERNELS, PH_CTAS, PH_SLOTS = 4, 4096, 16
SM_MHZ = 1965.0
NAMES = {
    0: ("k_filter_fused", ["start", "setup", "pass 1 done", "partials seen", "mean vector ready", "pass 2 done",
                           "merge grid before complete", "scores seen", "end"]),
    1: ("k_correlate_umma", ["start", "setup", "filter grid complete", "lists loaded", "k-loop done", "accumulator ready",
                             "top lists written", "synced", "end"]),
    2: ("k_merge_scan", ["start", "correlate grid complete", "entries filed", "copies done", "light rows done", "end"]),
    3: ("k_correlate_umma_f32", ["start", "setup", "filter grid complete", "lists loaded", "k-loop done",
                                 "accumulator ready", "top lists written", "end"]),
}


def build_phase_library() -> str:
    src = [os.path.join(build.CSRC, s) for s in build.SOURCES]
    newest = max(os.path.getmtime(os.path.join(build.CSRC, f)) for f in os.listdir(build.CSRC))
    if os.path.exists(PHASE_LIB) and os.path.getmtime(PHASE_LIB) > newest:
        return PHASE_LIB
    cmd = [build._nvcc(), "-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-lineinfo", "-std=c++17", "-shared",
           "-Xcompiler", "-fPIC", "-DFICOCO_PHASE_TIMERS", "-o", PHASE_LIB] + src
    r = subprocess.run(cmd, capture_output=True, text=True)
    if r.returncode != 0:
        raise RuntimeError("nvcc failed:\n" + r.stdout + r.stderr)
    return PHASE_LIB


def read_records(lib) -> np.ndarray:
    buf = np.zeros((PH_KERNELS, PH_CTAS, PH_SLOTS), dtype=np.uint64)
    rc = lib.ficoco_phase_read(buf.ctypes.data, buf.nbytes)     # also clears the records on the device
    if rc != 0:
        raise RuntimeError(f"ficoco_phase_read failed: {rc}")
    return buf


def report(buf: np.ndarray, n_steps: int, detail_step: int) -> None:
    t0 = None
    for s in range(n_steps):
        for k in range(PH_KERNELS):
            a = buf[k]
            a = a[a[:, PH_SLOTS - 1] > 0].astype(np.float64)
            if len(a) == 0 or len(a) % n_steps:
                continue
            a = a[np.argsort(a[:, PH_SLOTS - 1], kind="stable")]
            per = len(a) // n_steps
            a = a[s * per:(s + 1) * per]
            if t0 is None:
                t0 = a[:, PH_SLOTS - 1].min()
            name, marks = NAMES[k]
            n = len(marks)
            start = (a[:, PH_SLOTS - 1] - t0) / 1e3                       # us on the global timer
            last = np.nanmax(np.where(a[:, 1:n] > 0, a[:, 1:n], np.nan), axis=1)
            dur = (last - a[:, 0]) / SM_MHZ
            print(f"step {s} {name}: {len(a)} CTAs, start {start.min():7.2f} / {np.median(start):7.2f} / {start.max():7.2f}"
                  f"  end {np.min(start + dur):7.2f} / {np.median(start + dur):7.2f} / {np.max(start + dur):7.2f}"
                  f"  (min / median / max, us)   median CTA {np.median(dur):6.2f} us")
            if s != detail_step:
                continue
            for p in range(1, n):
                col = np.where(a[:, p] > 0, (a[:, p] - a[:, 0]) / SM_MHZ, np.nan)
                if np.all(np.isnan(col)):
                    continue
                print(f"      {marks[p]:28s} after CTA start: median {np.nanmedian(col):7.2f}  90 % {np.nanpercentile(col, 90):7.2f}"
                      f"  max {np.nanmax(col):7.2f}   latest, absolute {np.nanmax(col + start):7.2f}")


def main() -> None:
    import torch
    ap = argparse.ArgumentParser()
    ap.add_argument("--steps", type=int, default=4)
    ap.add_argument("--workload", type=int, default=2, choices=[1, 2, 3, 4])
    args = ap.parse_args()
    binding.LIB_PATH = build_phase_library()
    lib = binding.load_library()
    lib.ficoco_phase_read.argtypes = [C.c_void_p, C.c_size_t]
    lib.ficoco_phase_read.restype = C.c_int
    dev = "cuda:0"
    batch = synth.workload(args.workload)
    rows = sum(int(t.shape[0]) for t in batch.tokens)
    ctx = binding.Context(max_tokens=rows, max_dim=batch.dim, max_batch=len(batch.tokens), device=0)
    pk = packing.pack_v(batch, dev)
    prm = binding.make_params(has_cls=batch.has_cls, back_to_back=True)
    sets = []
    for _ in range(8):                                   # 8 buffer sets: the inputs of a step are never L2-warm
        tok, att = pk.tokens.clone(), pk.attn.clone()
        res = ctx.ficoco_v_reduce(tok, att, pk.keep, pk.grid_h, pk.grid_w, pk.heads, params=prm, **pk.call_kwargs())
        sets.append((tok, att, res))

    def step(i: int) -> None:
        tok, att, res = sets[i % 8]
        ctx.ficoco_v_reduce(tok, att, pk.keep, pk.grid_h, pk.grid_w, pk.heads, params=prm, out_tokens=res.out_tokens,
                            kept_idx=res.kept_idx, pos_out=res.pos_out, **pk.call_kwargs())

    torch.cuda.synchronize()                             # a context serves one stream at a time
    stream = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(stream):
        for i in range(16):
            step(i)
        torch.cuda.synchronize()
        with torch.cuda.graph(graph, stream=stream):
            for i in range(args.steps):
                step(i)
    torch.cuda.synchronize()
    for _ in range(3):
        graph.replay()
    torch.cuda.synchronize()
    read_records(lib)
    graph.replay()
    torch.cuda.synchronize()
    report(read_records(lib), args.steps, max(0, args.steps - 2))
    assert ctx.ficoco_status() == 0
    ctx.close()


if __name__ == "__main__":
    main()
