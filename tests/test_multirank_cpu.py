"""The N > 1 path of the benchmark on CPU: two gloo ranks, each with its own shard, no
data-path collective, max-over-ranks timing and the aggregate throughput."""
import os
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def _worker(rank: int, world: int, port: int, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    from paper_2411_17686_b200 import synth
    seed = bench.shard_seed(rank)
    img = synth.vit_image(seed, 0, 4, 4, 16, "bf16", True)            # a rank's data depends on its seed only
    ms_local = 10.0 + 5.0 * rank                                        # rank 1 is the slower one
    ms = bench.max_over_ranks(ms_local, world)
    dist.barrier()
    out.put((rank, seed, int(img.astype("int64").sum()), ms, bench.aggregate_images_per_s(ms, world)))
    dist.destroy_process_group()


def test_two_ranks_shard_without_exchange_and_take_the_slowest_time():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=120) for _ in range(2))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    (r0, s0, h0, ms0, v0), (r1, s1, h1, ms1, v1) = res
    assert (r0, r1) == (0, 1) and s0 != s1 and h0 != h1          # different shards
    assert ms0 == ms1 == 15.0                                     # the slowest rank's time on both
    import bench
    assert v0 == v1 == 2 * bench.B / 15e-3                        # aggregate over both ranks


def test_bench_starts_its_own_ranks():
    """`python bench.py --gpus 2` with no launcher around it starts two ranks itself; the dry run
    takes the same path on CPU (gloo): rank 0 prints one line for n_gpus = 2 with the slowest
    rank's time and the aggregate over both shards."""
    import json
    import subprocess
    env = dict(os.environ)
    for k in ("RANK", "WORLD_SIZE", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT"):
        env.pop(k, None)
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--steps", "5", "--dry-run"],
                       capture_output=True, text=True, timeout=300, env=env)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [ln for ln in r.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1
    line = json.loads(lines[0])
    import bench
    assert line["n_gpus"] == 2 and line["dry_run"] and line["shard_seeds"] == [bench.shard_seed(0), bench.shard_seed(1)]
    assert abs(line["ms_per_step"] - 15.0 / 5) < 1e-12
    assert abs(line["value"] - 2 * bench.B / (3.0e-3)) < 1e-6
