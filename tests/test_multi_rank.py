"""N > 1 plumbing on CPU (gloo, world_size 2): the units of the path are independent, so ranks
share no data; only the timing is reduced (max over ranks) and the value aggregated."""
import os
import socket
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    from paper_2605_23200_b200 import inputs
    bench.barrier()
    got = bench.max_over_ranks(10.0 + 5.0 * rank)
    # every rank builds the same replica of a (tiny) workload: same seed, same bytes
    wl = inputs.CONFIGS[0].scaled(seq_len_min=256, seq_len_max=256, budget=64)
    cache = inputs.make_cache(wl)
    digest = torch.tensor([float(cache.k_pages.float().sum())], dtype=torch.float64)
    both = [torch.zeros_like(digest) for _ in range(world)]
    dist.all_gather(both, digest)
    out.put((rank, got, [float(x) for x in both]))
    dist.destroy_process_group()


def test_max_over_ranks_and_replicas_gloo():
    s = socket.socket(); s.bind(("127.0.0.1", 0)); port = s.getsockname()[1]; s.close()
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = [q.get(timeout=120) for _ in procs]
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, got, digests in res:
        assert got == 15.0                       # the slowest rank sets the time
        assert digests[0] == digests[1]          # replicas are identical
    # weak scaling: value = ranks * steps / max time
    assert abs(2 * 100 / (15.0 / 1e3) - 13333.333) < 1


def test_algorithmic_bytes_match_the_definition():
    sys.path.insert(0, ROOT)
    import bench
    from paper_2605_23200_b200 import inputs
    wl = inputs.CONFIGS[1]
    k_read, moved = bench.algorithmic_bytes(wl, [16384])
    assert k_read == 32 * 8 * 16384 * 256 and moved == 32 * 8 * 2048 * 1024
    assert abs((k_read + moved) / 1e9 - 1.611) < 1e-3
    wl = inputs.CONFIGS[2]
    k_read, moved = bench.algorithmic_bytes(wl, [4096, 9000])       # the first sequence is skipped
    assert k_read == 28 * 4 * 9000 * 256 and moved == 28 * 4 * 4096 * 1024


def test_bench_gpus_flag_spawns_that_many_ranks():
    """`bench.py --gpus 2` without a launcher starts two ranks itself (torch.distributed.run on 127.0.0.1);
    with the CPU plumbing arm they meet over gloo, the slowest rank sets the time and one line is printed.
    A launcher that disagrees with --gpus is refused."""
    import json
    import subprocess
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--impl", "plumbing", "--steps", "7"],
                         capture_output=True, text=True, timeout=300, env=env)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [l for l in out.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    line = json.loads(lines[0])
    assert line["n_gpus"] == 2 and line["ms_max_over_ranks"] == 20.0 and abs(line["value"] - 2 * 7 / 0.020) < 1e-6
    env2 = dict(env, WORLD_SIZE="3", RANK="0", LOCAL_RANK="0")
    bad = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--impl", "plumbing"],
                         capture_output=True, text=True, timeout=120, env=env2)
    assert bad.returncode != 0 and "--gpus 2" in (bad.stderr + bad.stdout)
