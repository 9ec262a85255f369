"""Host logic of the N > 1 benchmark path on CPU: two gloo ranks.

The path does not shard with an exchange (replicas only): ranks draw different batches, the job's
time is the max over ranks and the job's throughput counts every replica's tokens."""
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
    from paper_2609_31395_b200 import synth
    dist.init_process_group("gloo", init_method=f"tcp://127.0.0.1:{port}", rank=rank, world_size=world)
    ms_local = 10.0 + 5.0 * rank                      # rank 1 is the slow one
    ms_max, value = bench.aggregate_replicas(ms_local, 280000, world, dist, torch.device("cpu"))
    wl = bench.make_workload("c1", None)
    wl.seed += 100 * rank                             # what run_ours does: every replica its own batch
    inst = synth.generate(synth.Workload("r", 1, 1, 2, [64], [4], [16], head_dim=16, page_size=4, seed=wl.seed), "cpu")
    out[rank] = (ms_max, value, float(inst.q.float().sum()))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_take_the_max_time_and_sum_the_tokens():
    mgr = mp.Manager()
    out = mgr.dict()
    mp.spawn(_worker, args=(2, 29531, out), nprocs=2, join=True)
    assert out[0][0] == out[1][0] == 15.0
    assert out[0][1] == out[1][1] == 2 * 280000 / 15e-3
    assert out[0][2] != out[1][2]                     # different seeds, different batches


def test_reference_arm_prints_on_rank_zero_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "1",
                        "--warmup", "0", "--gpus", "2"], env=env, capture_output=True, text=True, timeout=300)
    assert r.returncode == 0 and r.stdout.strip() == ""


def test_reference_arm_line_has_the_contract_keys():
    env = dict(os.environ, RANK="0", WORLD_SIZE="1", LOCAL_RANK="0")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "1",
                        "--warmup", "0", "--workload", "c1"], env=env, capture_output=True, text=True, timeout=600)
    assert r.returncode == 0, r.stderr
    d = json.loads(r.stdout.strip().splitlines()[-1])
    assert d["impl"] == "reference" and d["cpu_baseline"]["kind"] == "oracle" and d["value"] > 0
    assert d["e2e"]["h2d_bytes_per_step"] == 0 and d["unit"] == "tokens/s" and d["higher_is_better"] is True
