"""Host-side logic of the benchmark: max-over-ranks timing with two gloo ranks on CPU, the weak-scaling
aggregate, the bounded oracle sample and the reference arm's JSON line."""
import json
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _rank_main(rank, world, port, out):
    import torch.distributed as dist

    sys.path.insert(0, ROOT)
    import bench

    dist.init_process_group("gloo", init_method="tcp://127.0.0.1:%d" % port, rank=rank, world_size=world)
    slow = bench.max_over_ranks(1.0 + rank, world)  # rank 1 is the slow one
    rate = bench.whole_job_rate(100.0, world, slow)
    dist.barrier()
    dist.destroy_process_group()
    with open(out + ".%d" % rank, "w") as fh:
        json.dump({"slow": slow, "rate": rate}, fh)


def test_max_over_ranks_two_gloo_ranks(tmp_path):
    import torch.multiprocessing as mp

    port = 29500 + os.getpid() % 2000
    out = str(tmp_path / "r")
    mp.spawn(_rank_main, args=(2, port, out), nprocs=2, join=True)
    for rank in range(2):
        with open(out + ".%d" % rank) as fh:
            r = json.load(fh)
        assert r["slow"] == 2.0  # every rank reports the slowest rank's time
        assert r["rate"] == 100.0  # 2 ranks x 100 units in 2 s


def test_single_rank_helpers():
    sys.path.insert(0, ROOT)
    import bench
    from paper_2608_24738_b200 import workloads

    assert bench.max_over_ranks(3.5, 1) == 3.5
    assert bench.whole_job_rate(10.0, 4, 2.0) == 20.0
    w = workloads.config2(batch=4, size=64, disks=3)
    sub, k, total = bench.sample_images(w, 2 * 64 * 64)
    assert (k, total) == (2, 4) and sub.shape == (2, 1, 64, 64)
    sub, k, total = bench.sample_images(w, 1)
    assert k == 1
    assert w.io_bytes() == 5 * w.voxels


def test_reference_arm_prints_one_json_line():
    out = subprocess.run(
        [sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--config", "1", "--steps", "2",
         "--warmup", "1"], capture_output=True, text=True, check=True, cwd=ROOT)
    lines = [l for l in out.stdout.splitlines() if l.strip()]
    assert len(lines) == 1
    r = json.loads(lines[0])
    assert r["impl"] == "reference" and r["value"] > 0 and r["cpu_baseline"]["kind"] == "oracle"
    assert r["e2e"]["h2d_bytes_per_step"] == 0 and r["unit"] == "Gvoxel/s"


def test_workload_generators_are_seeded():
    from paper_2608_24738_b200 import workloads

    a, b = workloads.config1(), workloads.config1()
    assert a.sha256() == b.sha256()
    w5 = workloads.config5()
    assert w5.mask[1].all() and not w5.mask[0].all()
    assert w5.sampling == (1.0, 1.1, 1.2, 1.3, 1.4, 1.5, 1.6, 1.7)
