"""World-size-2 checks of the multi-process logic of bench.py on CPU (gloo):
documents are sharded one per rank with no data-path collective, the job time is
the maximum over ranks, and the oracle arm runs on rank 0 only."""
import json
import os
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)


def _worker(rank, world, port, q):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    from paper_2406_12018_b200 import workloads as wl
    w = wl.scaled(wl.CONFIGS["mistral7b_layer"], doc_tokens=64, q_heads=4, kv_heads=2, n_planted=2)
    doc = bench.rank_document(w, rank)
    mx = bench.max_over_ranks(10.0 + rank, dist, "cpu")
    q.put((rank, mx, float(doc.K.float().sum())))
    dist.barrier()
    dist.destroy_process_group()


def test_rank_sharding_and_max_time():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 29571
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in range(2))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert [r[1] for r in res] == [11.0, 11.0]           # both ranks agree on the slowest time
    assert res[0][2] != res[1][2]                          # different documents per rank


def test_reference_arm_under_torchrun_prints_one_line_from_rank0():
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2",
           "--master-addr", "127.0.0.1", "--master-port", "29572", os.path.join(ROOT, "bench.py"),
           "--impl", "reference", "--gpus", "2", "--steps", "1", "--warmup", "0"]
    r = subprocess.run(cmd, capture_output=True, text=True, timeout=600, cwd=ROOT)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [ln for ln in r.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["impl"] == "reference" and d["cpu_baseline"]["kind"] == "oracle" and d["value"] > 0
    assert d["e2e"]["h2d_bytes_per_step"] == 0 and d["unit"] == "tokens/s"


def test_gpus_flag_without_a_launcher_starts_that_many_ranks():
    # `python bench.py --gpus 2` with no launcher around it must become two ranks (one per GPU), not a silent 1-GPU
    # run: the script re-executes itself under torch.distributed.run.  --dry-run stops each rank after the set-up,
    # before any CUDA call, and prints the rank's share of the work.
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK")}
    cmd = [sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--dry-run", "--workload", "serving_mix"]
    r = subprocess.run(cmd, capture_output=True, text=True, timeout=600, cwd=ROOT, env=env)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [json.loads(ln) for ln in r.stdout.splitlines() if ln.startswith("{")]
    assert sorted(d["rank"] for d in lines) == [0, 1]
    assert all(d["n_gpus"] == 2 for d in lines)
    shares = [d["sequences_of_this_rank"] for d in sorted(lines, key=lambda d: d["rank"])]
    assert shares[0] == list(range(0, 16, 2)) and shares[1] == list(range(1, 16, 2))      # a slice of the 16 sequences each


def test_rank_sequences_partition_the_batch():
    import bench
    for world in (1, 2, 3, 8):
        parts = [bench.rank_sequences(16, r, world) for r in range(world)]
        assert sorted(x for p in parts for x in p) == list(range(16))
