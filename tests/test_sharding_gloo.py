"""World-size-2 CPU (gloo) test of the multi-GPU plumbing: row sharding + max-over-ranks timing.  The data path has
no collective; what is checked is that the shards tile the batch exactly, that sharded results (here computed by the
CPU oracle, since no GPU is present) concatenate to the unsharded result, and that the timing reduction works."""
import os
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_shard_rows_tiles_the_batch():
    from paper_2604_24273_b200.sharding import shard_rows

    for M in (0, 1, 7, 128, 4096, 4097):
        for world in (1, 2, 3, 8):
            spans = [shard_rows(M, world, r) for r in range(world)]
            assert spans[0][0] == 0 and sum(c for _, c in spans) == M
            for (s0, c0), (s1, _) in zip(spans, spans[1:]):
                assert s0 + c0 == s1
            counts = [c for _, c in spans]
            assert max(counts) - min(counts) <= 1


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import oracle
    from paper_2604_24273_b200 import inputs
    from paper_2604_24273_b200.sharding import max_over_ranks, shard_rows

    M, K, N = 37, 256, 128
    Wq, g = oracle.ternarize(inputs.master_weights(N, K, 1).numpy())
    x = inputs.bf16_bits(inputs.activations(M, K, 2))
    s, c = shard_rows(M, world, rank)
    mine = oracle.bitlinear(x[s:s + c], Wq, g, threads=1)["ybf16"]
    gathered = [None] * world
    dist.all_gather_object(gathered, (s, mine))
    t = max_over_ranks(10.0 + rank)
    if rank == 0:
        full = oracle.bitlinear(x, Wq, g, threads=1)["ybf16"]
        cat = np.concatenate([m for _, m in sorted(gathered, key=lambda p: p[0])], axis=0)
        out.put((bool(np.array_equal(cat, full)), t))
    dist.barrier()
    dist.destroy_process_group()


def test_two_rank_row_sharding_gloo():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 29500 + (os.getpid() % 2000)
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    ok, t = out.get(timeout=180)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert ok and t == 11.0


def test_bench_starts_its_own_ranks():
    """`python bench.py --gpus 2` with no WORLD_SIZE in the environment becomes two ranks by itself; here on CPU with the
    reference arm (rank 0 alone works and prints, the other rank exits 0): one JSON line with n_gpus = 2."""
    import json
    import subprocess

    env = {k: v for k, v in os.environ.items() if k not in ("WORLD_SIZE", "RANK", "LOCAL_RANK")}
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--impl", "reference", "--steps", "1",
                        "--warmup", "0"], env=env, cwd=ROOT, capture_output=True, text=True, timeout=600)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [l for l in r.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["n_gpus"] == 2 and d["impl"] == "reference" and d["value"] > 0
