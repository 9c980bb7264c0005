"""The N > 1 path of the benchmark on CPU: two gloo ranks run the host-side replica logic (independent batch per
rank, no data-path collective; whole-job time = max over ranks, whole-job tokens = sum over ranks)."""
import os
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    sys.path.insert(0, ROOT)
    import bench
    dist.init_process_group("gloo", rank=rank, world_size=world)
    seed, lens = bench.rank_batch(rank)
    times, tokens = bench.reduce_over_ranks([0.25 + rank, 1.0 - 0.5 * rank, 2.0], float(sum(lens)), "cpu", True)
    out.put((rank, seed, lens, times, tokens))
    dist.barrier()
    dist.destroy_process_group()


def test_two_replicas_over_gloo():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    (r0, seed0, lens0, times0, tok0), (r1, seed1, lens1, times1, tok1) = res
    assert lens0 == [4326, 7827, 4142, 4287, 2539, 4429, 6355, 7218]       # rank 0 = the named batch (config 2)
    assert lens1 != lens0 and len(lens1) == 8 and all(2048 <= n <= 8192 for n in lens1)
    assert times0 == times1 == [1.25, 1.0, 2.0]                            # max over ranks, per region
    assert tok0 == tok1 == float(sum(lens0) + sum(lens1))                   # sum over ranks


def test_reference_arm_is_rank0_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    p = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "1",
                        "--warmup", "0"], env=env, capture_output=True, text=True, timeout=300)
    assert p.returncode == 0 and p.stdout.strip() == ""


def test_gpus_flag_without_a_launcher_starts_local_ranks():
    """`bench.py --gpus 2` with no WORLD_SIZE in the environment starts itself as two local ranks (one process per GPU on
    a GPU machine; here the host-only arm over gloo): rank 0 prints one line with the whole-job figures."""
    import json
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}
    p = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "hostcheck", "--gpus", "2", "--steps", "1",
                        "--warmup", "0"], env=env, capture_output=True, text=True, timeout=300)
    assert p.returncode == 0, p.stderr[-2000:]
    lines = [ln for ln in p.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1
    out = json.loads(lines[0])
    sys.path.insert(0, ROOT)
    import bench
    assert out["n_gpus"] == 2 and out["max_time"] == 2.0
    assert out["tokens"] == float(sum(bench.rank_batch(0)[1]) + sum(bench.rank_batch(1)[1]))
    assert out["seq_lens_rank0"] == bench.rank_batch(0)[1]
