"""The N > 1 path of bench.py without a GPU: replicas only, so the only multi-rank logic is the
aggregation of the per-rank timings (max) and token counts (sum), and the reference arm's rule that
only rank 0 works.  Two gloo ranks on CPU."""
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
    dist.init_process_group("gloo", init_method=f"tcp://127.0.0.1:{port}", rank=rank, world_size=world)
    # rank r "measured" (10 + r) ms and (100 * (r + 1)) tokens; second pair for the end-to-end loop
    times, counts = bench.aggregate_over_ranks([10.0 + rank, 20.0 - rank], [100.0 * (rank + 1), 7.0], world, "cpu")
    with open(os.path.join(out_dir, f"r{rank}.json"), "w") as fh:
        json.dump({"times": times, "counts": counts}, fh)
    dist.destroy_process_group()


def test_two_gloo_ranks_take_max_time_and_sum_of_tokens(tmp_path):
    world, port = 2, 29611
    mp.spawn(_rank_main, args=(world, port, str(tmp_path)), nprocs=world, join=True)
    for r in range(world):
        got = json.load(open(tmp_path / f"r{r}.json"))
        assert got["times"] == [11.0, 20.0]       # slowest rank of each loop
        assert got["counts"] == [300.0, 14.0]     # whole-job work
    # whole-job throughput as bench.py reports it
    assert 300.0 / (11.0 * 1e-3) == got["counts"][0] / (got["times"][0] * 1e-3)


def test_single_rank_needs_no_process_group():
    sys.path.insert(0, ROOT)
    import bench
    times, counts = bench.aggregate_over_ranks([3.0], [5.0], 1, "cpu")
    assert times == [3.0] and counts == [5.0]


def test_reference_arm_only_rank_zero_works():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--config", "tiny",
                          "--steps", "1", "--warmup", "3"], env=env, capture_output=True, text=True, timeout=300)
    assert out.returncode == 0 and out.stdout.strip() == ""
