"""Host logic of the multi-GPU benchmark path on CPU: two gloo ranks, whole-job throughput is the
units of all ranks divided by the slowest rank's time."""
import os
import sys
from pathlib import Path

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = Path(__file__).resolve().parent.parent
sys.path.insert(0, str(ROOT))


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    ms, units = bench.aggregate_over_ranks(local_ms=1.0 + rank, local_units=10.0 * (rank + 1), world=world,
                                           dist=dist, device=torch.device("cpu"))
    out[rank] = (ms, units)
    dist.barrier()
    dist.destroy_process_group()


def test_two_rank_aggregation_is_sum_of_units_over_max_time():
    world, port = 2, 29500 + os.getpid() % 2000
    out = mp.Manager().dict()
    mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
    for rank in range(world):
        ms, units = out[rank]
        assert ms == 2.0 and units == 30.0


def test_single_rank_aggregation_is_identity():
    import bench
    assert bench.aggregate_over_ranks(3.5, 7.0, 1) == (3.5, 7.0)


def test_workload_arithmetic_matches_the_encoder_layer():
    import bench
    from paper_1909_05840_b200 import synth
    wl = synth.workload(1)
    assert bench.gemm_ops(wl) == 2.0 * 4096 * (2304 * 768 + 768 * 768 + 3072 * 768 + 768 * 3072)
    # fp32 outputs dominate the traffic of three of the four GEMMs
    assert 130e6 < bench.gemm_algorithmic_bytes(wl) < 145e6


def test_reference_arm_prints_one_json_line_with_the_contract_keys():
    # `bench.py --impl reference` times the CPU oracle on a bounded sample: no GPU needed
    import json
    import subprocess
    r = subprocess.run([sys.executable, str(ROOT / "bench.py"), "--impl", "reference", "--steps", "1", "--ref-rows", "32"],
                       capture_output=True, text=True, timeout=300)
    assert r.returncode == 0, r.stderr[-500:]
    lines = [ln for ln in r.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1
    d = json.loads(lines[0])
    for key in ("impl", "metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better",
                "scaling", "vs_baseline", "dtype", "data", "config", "cpu_baseline", "e2e"):
        assert key in d, key
    assert d["impl"] == "reference" and d["value"] > 0 and d["cpu_baseline"]["kind"] == "oracle"
    assert d["e2e"]["h2d_bytes_per_step"] == 0 and d["e2e"]["d2h_bytes_per_step"] == 0
    assert d["e2e"]["value"] == d["value"] and d["vs_baseline"] is None

