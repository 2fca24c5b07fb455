"""The N > 1 path of the benchmark is "replicas only" (the method has no exchange step): each rank times its own
replica and the job-level number is the sum of the work over the slowest rank's time.  This checks that host logic
with two gloo ranks on the CPU."""
import os
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    ms_local = 2.0 if rank == 0 else 3.5            # rank 1 is the slow one
    dist.barrier()
    ms, tflops = bench.aggregate_over_ranks(ms_local, 7.0e12, dist, None)
    out[rank] = (ms, tflops)
    dist.barrier()
    dist.destroy_process_group()


def test_replica_aggregation_two_gloo_ranks():
    world = 2
    mgr = mp.get_context("spawn").Manager()
    out = mgr.dict()
    mp.spawn(_worker, args=(world, 29611, out), nprocs=world, join=True)
    for rank in range(world):
        ms, tflops = out[rank]
        assert ms == 3.5                                   # max over ranks
        assert abs(tflops - 2 * 7.0e12 / 3.5e-3 / 1e12) < 1e-9   # both ranks' work over the slowest rank's time


def test_single_process_aggregation_is_identity():
    sys.path.insert(0, ROOT)
    import bench
    ms, tflops = bench.aggregate_over_ranks(4.0, 8.0e12)
    assert ms == 4.0 and abs(tflops - 8.0e12 / 4.0e-3 / 1e12) < 1e-9


def test_reference_arm_prints_one_json_line_with_the_agreed_keys():
    """`bench.py --impl reference` (the CPU oracle timed on a bounded sample) on a tiny sample: one JSON line, same metric
    and unit as the CUDA arm, the keys the measurement contract names."""
    import json
    import subprocess
    res = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "1", "--warmup", "0",
                          "--oracle-tokens", "32"], capture_output=True, text=True, cwd=ROOT, timeout=600)
    assert res.returncode == 0, res.stderr[-2000:]
    lines = [l for l in res.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["impl"] == "reference" and d["unit"] == "TFLOP/s" and d["higher_is_better"] is True and d["vs_baseline"] is None
    assert d["metric"].startswith("melded FP8-LoRA layer fwd+bwd TFLOP/s") and d["value"] > 0 and d["n_gpus"] == 1
    assert d["config"]["workload"].startswith("configs[1]") and "model" not in d["config"]
    assert d["cpu_baseline"]["kind"] == "oracle" and d["cpu_baseline"]["cores"] >= 1 and d["cpu_baseline"]["value"] == d["value"]
    assert d["e2e"] == {"value": d["value"], "unit": d["unit"], "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}
