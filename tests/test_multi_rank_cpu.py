"""The N > 1 path of the benchmark on CPU: two gloo ranks.  The hot path shards by prompt with no
data-path collective, so what is distributed is only the host logic: per-rank seeds (independent
prompts), the max-over-ranks timing reduction, the aggregate, and the reference arm's "rank 0 only"."""
import json
import os
import subprocess
import sys

import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    import torch.distributed as dist
    sys.path.insert(0, ROOT)
    import bench
    from workloads import draw_lengths, get_config
    dist.init_process_group("gloo", init_method=f"tcp://127.0.0.1:{port}", rank=rank, world_size=world)
    cfg = get_config("cfg1")
    lay = draw_lengths(cfg, seed=bench.rank_seed(cfg, rank))
    times = bench.max_over_ranks([1.0 + rank, 10.0 - rank], dist)
    dist.barrier()
    out.put((rank, lay.doc_len.tolist(), times, bench.aggregate_value(2e12, times[0], world)))
    dist.destroy_process_group()


def test_two_gloo_ranks_shard_by_prompt_and_reduce_with_max():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    (_, len0, t0, v0), (_, len1, t1, v1) = res
    assert len0 != len1                          # different prompts per rank
    assert t0 == t1 == [2.0, 10.0]               # the slowest rank's time, on every rank
    assert v0 == v1 == 2 * 2e12 / 2e-3 / 1e12    # aggregate over both ranks


def test_reference_arm_runs_on_rank_zero_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "cfg0",
                        "--steps", "1", "--warmup", "0"], env=env, capture_output=True, text=True, timeout=300)
    assert r.returncode == 0 and r.stdout.strip() == ""
    env["RANK"] = "0"
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "cfg0",
                        "--steps", "1", "--warmup", "0"], env=env, capture_output=True, text=True, timeout=300)
    assert r.returncode == 0
    line = json.loads(r.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["n_gpus"] == 2 and line["value"] > 0
    assert line["cpu_baseline"]["kind"] == "oracle" and line["e2e"]["h2d_bytes_per_step"] == 0


def test_gpus_flag_starts_the_ranks_itself():
    """`bench.py --gpus 2` started as a plain script launches two ranks of itself (loopback
    rendezvous); with the reference arm, which needs no GPU, rank 0 alone prints the line."""
    sys.path.insert(0, ROOT)
    import bench
    cmd = bench.launcher_command(2, ["--gpus", "2", "--impl", "reference"])
    assert "--nproc-per-node=2" in cmd and "127.0.0.1" in cmd and cmd[-3:] == ["--gpus", "2", "--impl", "reference"][-3:]
    env = {k: v for k, v in os.environ.items() if k not in ("WORLD_SIZE", "RANK", "LOCAL_RANK")}
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--impl", "reference",
                        "--workload", "cfg0", "--steps", "1", "--warmup", "0"], env=env, capture_output=True, text=True,
                       timeout=600)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [ln for ln in r.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1                                   # rank 1 printed nothing
    line = json.loads(lines[0])
    assert line["impl"] == "reference" and line["n_gpus"] == 2
