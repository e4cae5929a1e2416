"""bench.py with more than one rank: replicas only, so the multi-rank logic is a barrier, a max over the
ranks' times and the whole-job figure.  Run here as two gloo processes on CPU."""
import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    import torch.distributed as dist
    sys.path.insert(0, ROOT)
    import bench
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        local_ms = 10.0 + 5.0 * rank                   # rank 1 is the slow one
        dist.barrier()
        ms = bench.max_over_ranks(local_ms, dist, "cpu")
        out[rank] = (ms, bench.whole_job_us_per_unit(ms, 1000, world))
    finally:
        dist.destroy_process_group()


def test_two_ranks_report_the_slowest_time_and_the_whole_job_rate():
    import torch.multiprocessing as mp
    world, port = 2, 29500 + os.getpid() % 2000
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    assert res[0] == res[1]
    ms, us_per_unit = res[0]
    assert ms == 15.0
    assert us_per_unit == pytest.approx(15.0 * 1e3 / 2000)     # 2 ranks x 1000 steps in 15 ms


def test_single_rank_needs_no_process_group():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(3.5) == 3.5
    assert bench.whole_job_us_per_unit(20.0, 1000, 1) == pytest.approx(20.0)
    sh = __import__("paper_2512_12990_b200.synth", fromlist=["SHAPES"]).SHAPES["dsv2"]
    assert bench.step_bytes(sh) == 57851904            # 3 x 8-bit + 3 x 4-bit routed + 2 shared 8-bit experts


def test_prefill_flops_and_expert_bytes_are_the_stated_formulas():
    import bench
    from paper_2512_12990_b200 import synth
    sh = synth.SHAPES["qwen_prefill"]
    # 2 flops per multiply-add, three projections, top-4 routed experts of 1408 and one shared of 5632 per token
    assert bench.prefill_flops(sh, 2048) == 2 * 2048 * 3 * 2048 * (4 * 1408 + 5632) == 283467841536
    # planes used x N K / 2 + 3 bytes of (fp16 scale, u8 zero-point) per group, three matrices
    assert bench.expert_bytes(2048, 1408, 128, True) == 3 * (2048 * 1408 + 3 * 2048 * 1408 // 128) == 8853504
    assert bench.expert_bytes(2048, 1408, 128, False) == 3 * (2048 * 1408 // 2 + 3 * 2048 * 1408 // 128) == 4528128
