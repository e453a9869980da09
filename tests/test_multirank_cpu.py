"""Host logic of the N > 1 benchmark path, run as two gloo ranks on the CPU."""
import json
import os
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out_dir):
    sys.path.insert(0, ROOT)
    import bench
    from paper_2509_15038_b200 import synth

    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    slowest = bench.max_over_ranks(1.0 + rank, torch.device("cpu"), world)
    w = bench.rank_workload(synth.shrink(synth.CONFIGS["cfg1"], n_max=64, kv_heads=2, q_heads=2), rank)
    K, _ = synth.make_kv_element(w, 0)
    checksum = float(K.float().abs().sum())
    gathered = [None] * world
    dist.all_gather_object(gathered, (w.data_seed, checksum))
    dist.barrier()
    with open(os.path.join(out_dir, f"rank{rank}.json"), "w") as f:
        json.dump({"slowest": slowest, "gathered": gathered,
                   "value": bench.job_throughput(1000, world, slowest)}, f)
    dist.destroy_process_group()


def test_two_ranks_take_the_slowest_time_and_disjoint_data(tmp_path):
    world, port = 2, 29500 + os.getpid() % 2000
    mp.spawn(_worker, args=(world, port, str(tmp_path)), nprocs=world, join=True)
    res = [json.load(open(tmp_path / f"rank{r}.json")) for r in range(world)]
    for r in res:
        assert r["slowest"] == 2.0                       # max over ranks, on every rank
        assert r["value"] == 2 * 1000 / 2.0              # whole-job units over the slowest time
        seeds = [g[0] for g in r["gathered"]]
        sums = [g[1] for g in r["gathered"]]
        assert seeds[0] != seeds[1] and sums[0] != sums[1]   # every rank draws its own cache


def test_reference_arm_runs_on_rank_zero_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference",
                          "--workload", "cfg1", "--steps", "1", "--warmup", "0"],
                         env=env, capture_output=True, text=True, timeout=300)
    assert out.returncode == 0 and out.stdout.strip() == ""
    env["RANK"] = "0"
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference",
                          "--workload", "cfg1", "--steps", "1", "--warmup", "0"],
                         env=env, capture_output=True, text=True, timeout=300)
    line = json.loads(out.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["value"] > 0 and line["cpu_baseline"]["kind"] == "oracle"
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["gpu_launches"] == 0


def test_gpus_flag_spawns_one_rank_per_gpu_dry_run():
    """`bench.py --gpus 2` started without a launcher re-launches itself as two ranks; with --dry-run
    they run the host logic on gloo: the line says n_gpus 2, carries the slowest rank's time and the
    whole-job rate, and every rank drew its own data seed."""
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK")}
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--dry-run",
                          "--workload", "cfg2"], env=env, capture_output=True, text=True, timeout=300)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [ln for ln in out.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1                                   # rank 0 alone prints
    line = json.loads(lines[0])
    assert line["n_gpus"] == 2 and line["scaling"] == "weak"
    assert line["ms_per_step"] == 1.1                        # max over ranks of 1.0 and 1.1
    tokens = 32 * 8 * 8192
    assert line["value"] == 2 * tokens / 1.1e-3
    assert len(set(line["config"]["data_seeds"])) == 2
    one = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--dry-run", "--workload", "cfg2"],
                         env=env, capture_output=True, text=True, timeout=300)
    assert json.loads(one.stdout.strip().splitlines()[-1])["n_gpus"] == 1
