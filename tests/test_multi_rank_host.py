"""Host-side logic of the multi-GPU ("replicas only") path, run as two gloo ranks on CPU: the whole-job figure is
the replicas' bytes over the slowest rank's time, and only rank 0 of the reference arm works and prints."""
import json
import os
import subprocess
import sys

import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _rank_main(rank, world, port, out_dir):
    import torch.distributed as dist

    sys.path.insert(0, ROOT)
    import bench

    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        my_ms = 10.0 + 5.0 * rank            # rank 1 is the slow replica
        ms = bench.max_over_ranks(my_ms, dist, "cpu")
        gbs = bench.whole_job_gbs(1e9, 4, world, ms)
        dist.barrier()
        with open(os.path.join(out_dir, f"rank{rank}.json"), "w") as f:
            json.dump({"ms": ms, "gbs": gbs}, f)
    finally:
        dist.destroy_process_group()


def test_max_over_ranks_and_whole_job_value(tmp_path):
    world, port = 2, 29000 + os.getpid() % 2000
    mp.spawn(_rank_main, args=(world, port, str(tmp_path)), nprocs=world, join=True)
    res = [json.load(open(tmp_path / f"rank{r}.json")) for r in range(world)]
    for r in res:
        assert r["ms"] == 15.0                                  # the slowest rank's time, on every rank
        assert abs(r["gbs"] - 1e9 * 4 * 2 / 15e-3 / 1e9) < 1e-9  # both replicas' bytes over that time


def test_single_rank_passthrough():
    sys.path.insert(0, ROOT)
    import bench

    assert bench.max_over_ranks(3.5, None, "cpu") == 3.5
    assert bench.whole_job_gbs(2e9, 10, 1, 20.0) == 2e9 * 10 / 20e-3 / 1e9


def test_reference_arm_other_ranks_stay_silent():
    env = dict(os.environ, RANK="1", LOCAL_RANK="1", WORLD_SIZE="2")
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "1",
                          "--warmup", "0"], env=env, capture_output=True, text=True, timeout=300)
    assert out.returncode == 0
    assert out.stdout.strip() == ""
