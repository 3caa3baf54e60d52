"""Host-side logic of bench.py that needs no GPU: the max-over-ranks reduction and the whole-job aggregate on a
world of two gloo ranks, and the reference arm (the CPU oracle timed on the bench's workload)."""
import json
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
torch = pytest.importorskip("torch")


def _rank_main(rank, world, port, out_dir):
    import torch.distributed as dist
    sys.path.insert(0, ROOT)
    import bench
    dist.init_process_group("gloo", init_method=f"tcp://127.0.0.1:{port}", rank=rank, world_size=world)
    # rank r measured (10 + r) ms for the device loop and (20 - r) ms end to end
    got = bench.max_over_ranks([10.0 + rank, 20.0 - rank], "cpu", world)
    value = bench.aggregate_value(world, 1024, 5, got[0])
    with open(os.path.join(out_dir, f"r{rank}.json"), "w") as f:
        json.dump({"got": got, "value": value}, f)
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_report_the_slowest_rank_and_the_sum_of_replicas(tmp_path):
    import torch.multiprocessing as mp
    port = 29500 + os.getpid() % 2000
    mp.spawn(_rank_main, args=(2, port, str(tmp_path)), nprocs=2, join=True)
    for r in range(2):
        d = json.load(open(tmp_path / f"r{r}.json"))
        assert d["got"] == [11.0, 20.0]                         # max over ranks, element by element
        assert abs(d["value"] - 2 * 1024 * 5 / 11e-3) < 1e-6     # both replicas' samples over the slowest time


def test_single_rank_reduction_is_the_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks([3.5, 1.25], "cpu", 1) == [3.5, 1.25]


def test_reference_arm_prints_one_json_line():
    env = dict(os.environ, RANK="0", WORLD_SIZE="1")
    out = subprocess.check_output([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference",
                                   "--workload", "mlr_tiny", "--steps", "2", "--warmup", "0"], env=env, text=True)
    lines = [l for l in out.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["impl"] == "reference" and d["unit"] == "samples/s" and d["value"] > 0
    assert d["cpu_baseline"]["kind"] == "oracle" and d["cpu_baseline"]["cores"] >= 1
    assert d["e2e"]["h2d_bytes_per_step"] == 0 and d["e2e"]["value"] == d["value"]


def test_other_ranks_of_the_reference_arm_do_nothing():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2")
    out = subprocess.check_output([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference",
                                   "--workload", "mlr_tiny", "--steps", "1", "--warmup", "0"], env=env, text=True)
    assert out.strip() == ""
