"""Host logic of the N > 1 benchmark path on CPU: two gloo ranks.

The path does not shard (replicas only), so the only cross-rank steps are the barrier and the
max-over-ranks time; the reference arm must print on rank 0 only.
"""
import json
import os
import subprocess
import sys

import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _rank_main(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import bench
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    mine = 2.0 + rank                                   # rank 1 is the slow one
    slowest = bench.max_over_ranks(mine, dist, "cpu")
    dist.barrier()
    out.put((rank, slowest, bench.whole_job_tflops(10 ** 12, world, slowest)))
    dist.destroy_process_group()


def test_max_over_ranks_and_whole_job_value_with_two_gloo_ranks():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_rank_main, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert [g[1] for g in got] == [3.0, 3.0]            # every rank sees the slowest rank's time
    assert all(abs(g[2] - 2.0 / 3.0) < 1e-12 for g in got)   # 2 replicas x 1 Tflop / 3 s


def test_reference_arm_prints_on_rank_zero_only():
    def run(rank):
        env = dict(os.environ, RANK=str(rank), WORLD_SIZE="2", LOCAL_RANK=str(rank))
        return subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                               "--steps", "1", "--warmup", "0", "--workload", "c1"],
                              capture_output=True, text=True, env=env, timeout=300)
    r0, r1 = run(0), run(1)
    assert r0.returncode == 0 and r1.returncode == 0
    assert r1.stdout.strip() == ""
    line = json.loads(r0.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["n_gpus"] == 2 and line["value"] > 0
    assert line["cpu_baseline"]["kind"] == "oracle" and line["e2e"]["h2d_bytes_per_step"] == 0
