"""Host-side logic of bench.py that needs no GPU: replica aggregation over ranks (gloo, world size 2),
the layer list of a denoising step, and the JSON contract of the reference arm on a tiny workload."""
import json
import os
import subprocess
import sys
import tempfile

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

import bench  # noqa: E402


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    my_ms = [3.0, 5.0][rank]                        # rank 1 is the slow replica
    slowest = bench.max_over_ranks(my_ms, dist, "cpu")
    value = bench.whole_job_tops(2.0e12, world, slowest)
    with open(os.path.join(out, f"rank{rank}.json"), "w") as f:
        json.dump([slowest, value], f)
    dist.barrier()
    dist.destroy_process_group()


def test_replica_aggregation_over_two_gloo_ranks():
    world = 2
    # Results come back through files: a manager process would be forked from this one, and a fork leaves the
    # parent's BLAS thread pool unusable for the LAPACK calls of tests that run later in the same process.
    with tempfile.TemporaryDirectory() as out:
        mp.spawn(_worker, args=(world, 29731, out), nprocs=world, join=True)
        res = {}
        for rank in range(world):
            with open(os.path.join(out, f"rank{rank}.json")) as f:
                res[rank] = tuple(json.load(f))
    for rank in range(world):
        slowest, value = res[rank]
        assert slowest == 5.0                       # every rank sees the max over ranks
        # two replicas, 2 TOP each per step, 5 ms per step -> 800 TOPS for the whole job
        assert abs(value - 800.0) < 1e-9
    assert bench.max_over_ranks(7.5, None) == 7.5   # single process: unchanged


def test_dit_step_layer_list_matches_the_workload_definition():
    shapes = bench.dit_step_layers(40)
    assert len(shapes) == 320
    assert shapes.count((5120, 5120, 32)) == 240 and shapes.count((5120, 13824, 32)) == 40 and \
        shapes.count((13824, 5120, 32)) == 40
    tera_ops = sum(2.0 * 32760 * k * n for k, n, _ in shapes) / 1e12
    assert abs(tera_ops - 783.2) < 0.5              # the per-step operation count quoted for this workload
    packed = bench.dit_step_layers(40, qkv_packed=True)   # q, k, v as one layer: same operations, 80 fewer layers
    assert len(packed) == 240 and packed.count((5120, 15360, 96)) == 40
    assert sum(k * n for k, n, _ in packed) == sum(k * n for k, n, _ in shapes)


def test_reference_arm_prints_one_contract_line_on_the_tiny_workload():
    p = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "tiny",
                        "--steps", "2", "--warmup", "1"], capture_output=True, text=True, timeout=600, cwd=ROOT)
    assert p.returncode == 0, p.stderr[-2000:]
    lines = [l for l in p.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    d = json.loads(lines[0])
    for key in ("metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better", "scaling",
                "vs_baseline", "dtype", "data", "config", "impl", "cpu_baseline", "e2e"):
        assert key in d, key
    assert d["impl"] == "reference" and d["cpu_baseline"]["kind"] == "oracle" and d["value"] > 0
    assert d["e2e"]["h2d_bytes_per_step"] == 0 and d["config"]["workload"] == "tiny"
