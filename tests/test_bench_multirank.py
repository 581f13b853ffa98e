"""The N > 1 path of bench.py on CPU: two gloo ranks, one pack per rank.  The only collectives
are the max-reduction of the ranks' timings and the sum of their work, after the timed region;
the reference arm prints on rank 0 alone."""
import json
import os
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import bench
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    got = bench.max_over_ranks([1.0 + rank, 5.0 - rank, 2.0], "cpu")
    pack = bench.rank_pack(1, rank)
    got += bench.sum_over_ranks([10.0 + rank, float(pack.total_tokens)], "cpu")
    dist.barrier()
    dist.destroy_process_group()
    out.put((rank, got))


def test_max_over_ranks_two_gloo_ranks():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    results = dict(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    sys.path.insert(0, ROOT)
    import bench
    packs = [bench.rank_pack(1, r) for r in range(2)]
    assert packs[0].total_tokens != packs[1].total_tokens or list(packs[0].prefix_len) != list(packs[1].prefix_len)
    assert results[0] == results[1] == [2.0, 5.0, 2.0, 21.0, float(packs[0].total_tokens + packs[1].total_tokens)]


def test_whole_job_value_is_sum_of_the_ranks_work_over_slowest_time():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.whole_job_tflops(2e12, 1.0) == 2000.0
    assert bench.whole_job_tflops(16e12, 2.0) == 8000.0
    assert bench.max_over_ranks([3.0], "cpu") == [3.0]       # single process: identity
    assert bench.sum_over_ranks([3.0, 4.0], "cpu") == [3.0, 4.0]
    # rank 0 keeps the configuration's own pack; the others draw from the same length distribution
    from paper_2410_20305_b200 import workloads as wl
    assert list(bench.rank_pack(3, 0).cu_seqlens) == list(wl.config_pack(3).cu_seqlens)
    other = bench.rank_pack(3, 5)
    assert other.pack_len == 32768 and 0.85 * 32768 <= other.total_tokens <= 32768


def test_reference_arm_prints_one_line_on_rank_zero_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                        "--steps", "1", "--warmup", "3"], capture_output=True, text=True, env=env, timeout=600)
    assert r.returncode == 0 and r.stdout.strip() == ""
    env["RANK"] = "0"
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                        "--steps", "1", "--warmup", "3", "--workload", "4"], capture_output=True, text=True, env=env,
                       timeout=600)
    assert r.returncode == 0
    line = json.loads(r.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["cpu_baseline"]["kind"] == "oracle"
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["value"] > 0 and line["unit"] == "TFLOP/s"
