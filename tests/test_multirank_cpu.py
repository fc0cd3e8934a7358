"""The benchmark's N>1 path on CPU: two gloo ranks on 127.0.0.1.  The path does not shard (replicas only), so
what the ranks share is the reduction of their timings (maximum over ranks) and the aggregate throughput; the
reference arm runs on rank 0 alone."""
import json
import os
import socket
import subprocess
import sys

import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank_main(rank, world, port, out_dir):
    import torch.distributed as dist
    sys.path.insert(0, ROOT)
    import bench
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    per_rank = [10.0 + 3.0 * rank, 20.0 - 5.0 * rank]          # rank 1 is slower on the first, faster on the second
    got = bench.max_over_ranks(per_rank, world, "cpu")
    dist.barrier()
    dist.destroy_process_group()
    with open(os.path.join(out_dir, "r%d.json" % rank), "w") as f:
        json.dump(got, f)


def test_timings_are_reduced_to_the_maximum_over_two_gloo_ranks(tmp_path):
    port = _free_port()
    mp.spawn(_rank_main, args=(2, port, str(tmp_path)), nprocs=2, join=True)
    r0 = json.load(open(tmp_path / "r0.json"))
    r1 = json.load(open(tmp_path / "r1.json"))
    assert r0 == r1 == [13.0, 20.0]


def test_aggregate_throughput_counts_every_replica():
    sys.path.insert(0, ROOT)
    import bench
    one = bench.aggregate_tokens_per_s(32896, 1, 50.0)
    assert abs(one - 32896 / 0.05) < 1e-6
    assert abs(bench.aggregate_tokens_per_s(32896, 8, 50.0) - 8 * one) < 1e-6        # weak scaling: work per rank fixed


def test_reference_arm_runs_on_rank_zero_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    res = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "1",
                          "--warmup", "0"], env=env, capture_output=True, text=True, timeout=120)
    assert res.returncode == 0 and res.stdout.strip() == ""
