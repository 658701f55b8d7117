"""N > 1 path of bench.py on CPU: two gloo ranks, max-over-ranks timing and whole-job aggregation (replicas only)."""
import os
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import bench
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    dist.barrier()
    ms_local = 10.0 + 3.0 * rank                        # rank 1 is the slow replica
    ms = bench.max_over_ranks(ms_local, world)
    value = bench.whole_job_tokens_per_s(world, steps=100, tokens_per_step=16, ms_max=ms)
    out[rank] = (ms, value)
    dist.barrier()
    dist.destroy_process_group()


def test_two_rank_aggregation_gloo():
    world = 2
    mgr = mp.Manager()
    out = mgr.dict()
    mp.spawn(_worker, args=(world, 29611, out), nprocs=world, join=True)
    assert out[0] == out[1]
    ms, value = out[0]
    assert ms == 13.0
    assert abs(value - 2 * 100 * 16 / 13e-3) < 1e-6


def test_single_rank_needs_no_process_group():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(7.5, 1) == 7.5
    assert bench.whole_job_tokens_per_s(1, 1000, 1, 12.5) == 1000 / 12.5e-3


def test_reference_arm_idles_on_other_ranks():
    sys.path.insert(0, ROOT)
    import bench

    class Args:
        workload, steps, warmup, gpus = "decode", 1, 0, 2
    assert bench.run_reference(Args(), rank=1, world=2) is None      # no work, no output on ranks > 0


def test_workloads_follow_the_baseline_configs():
    sys.path.insert(0, ROOT)
    import bench
    from paper_2608_15383_b200 import synth
    assert bench.WORKLOADS["decode"][:2] == (1, 64) and bench.WORKLOADS["offload"][:2] == (16, 16)
    assert bench.WORKLOADS["prefill"][0] == 2048
    assert (synth.OLMOE.d_model, synth.OLMOE.d_ff, synth.OLMOE.num_experts, synth.OLMOE.top_k) == (2048, 1024, 64, 8)
