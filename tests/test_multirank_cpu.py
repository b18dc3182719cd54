"""The N > 1 path of bench.py on CPU: two gloo ranks. The data path has no collective (ranks hold
independent batches); what is shared is the timing reduction and who prints."""
import json
import os
import subprocess
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)


def _worker(rank, world, port, out_dir):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    import bench
    from paper_2407_18121_b200 import workloads as wl
    dist.init_process_group("gloo", rank=rank, world_size=world)
    w = wl.WORKLOADS["tiny"]
    wr = bench.rank_workload(w, rank)
    Q, _, _ = wl.prompt_problem(wr, 0)
    times = [10.0 + rank, 5.0 - rank, 7.0]                  # rank 1 is slower on [0], rank 0 on [1]
    reduced = bench.max_over_ranks(times)
    dist.barrier()
    json.dump({"reduced": reduced, "checksum": int(Q.astype(np.int64).sum()), "seed": wr.seed,
               "value": bench.whole_job_tokens_per_s(w, world, reduced[0])},
              open(os.path.join(out_dir, f"rank{rank}.json"), "w"))
    dist.destroy_process_group()


def test_two_ranks_reduce_times_and_hold_different_batches(tmp_path):
    mp.spawn(_worker, args=(2, 29731, str(tmp_path)), nprocs=2, join=True)
    r0 = json.load(open(tmp_path / "rank0.json"))
    r1 = json.load(open(tmp_path / "rank1.json"))
    assert r0["reduced"] == r1["reduced"] == [11.0, 5.0, 7.0]           # max over ranks, element-wise
    assert r0["seed"] != r1["seed"] and r0["checksum"] != r1["checksum"]  # independent batches
    # whole-job value counts both ranks' tokens over the slower rank's time
    assert abs(r0["value"] - 1 * 32 * 2 / 11.0e-3) < 1e-6


def test_without_a_process_group_the_reduction_is_the_identity():
    import bench
    assert bench.max_over_ranks([1.5, 2.5]) == [1.5, 2.5]


def test_reference_arm_is_silent_on_other_ranks():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    p = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                        "--steps", "1", "--warmup", "0"], env=env, capture_output=True, text=True, timeout=120)
    assert p.returncode == 0 and p.stdout.strip() == ""


def test_bench_says_per_workload_whether_its_data_exceeds_l2():
    import bench
    from oracle import ec_oracle as orc
    from paper_2407_18121_b200 import workloads as wl
    big = wl.WORKLOADS["llava7b_b1"]
    small = wl.WORKLOADS["qwenvl7b_b1"]
    s_big = bench.l2_statement(big, orc.keep_count(big.prompt_len, big.keep_ratio))
    s_small = bench.l2_statement(small, orc.keep_count(small.prompt_len, small.keep_ratio))
    assert s_big.startswith("inputs larger than L2") and "168 MB" in s_big
    assert s_small.startswith("NOT larger than L2") and "84 MB" in s_small


def test_oracle_sample_is_bounded_and_scaled():
    import bench
    from paper_2407_18121_b200 import workloads as wl
    for name, w in wl.WORKLOADS.items():
        problems, steps = bench.oracle_sample_size(w)
        assert 1 <= problems <= w.N and 4 <= steps <= w.decode_steps, name
        # the sampled prompt stage stays within the multiply-add budget unless a single problem exceeds it
        per_problem = w.heads * w.prompt_len * (w.prompt_len + 1) / 2 * w.head_dim
        assert problems == 1 or problems * per_problem <= 1.0e11 + per_problem, name
