"""The N > 1 path of bench.py on CPU: two gloo ranks. The hot path shards by sequence with no
exchange step, so what there is to check is the host logic: every rank gets its own batch, the
timing is the MAX over ranks, the reported value is whole-job throughput, and only rank 0 of the
reference arm does any work."""
import os
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _rank_main(rank, world, port, out):
    sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        import bench
        from pask_workloads import configs as WC
        w = bench.rank_workload(WC.TINY, rank)
        slow = bench.max_over_ranks(10.0 + 5.0 * rank, "cpu")          # rank 1 is the slow one
        value = bench.whole_job_tokens_per_s(world, w.cfg.batch, 4, slow)
        out[rank] = (w.seed, w.gen_tags[0][:32].tolist(), slow, value)
        dist.barrier()
    finally:
        dist.destroy_process_group()


def test_two_ranks_own_batches_max_time_and_aggregate_value():
    world, port = 2, 29517 + os.getpid() % 500
    with mp.Manager() as m:
        out = m.dict()
        mp.spawn(_rank_main, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    (s0, t0, slow0, v0), (s1, t1, slow1, v1) = res[0], res[1]
    assert s1 == s0 + 1 and t0 != t1                      # different seeds, different tag streams
    assert slow0 == slow1 == 15.0                         # MAX over ranks, known to both
    assert v0 == v1 == 2 * 1 * 4 / 15.0e-3                # both ranks' tokens over the slowest rank's time


def test_single_rank_helpers_and_reference_arm_rank_filter(capsys):
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(3.5, "cpu") == 3.5
    assert bench.whole_job_tokens_per_s(1, 64, 20, 4000.0) == 64 * 20 / 4.0

    class A:
        config, warmup, steps, ref_seqs, cpu_seconds = bench.DEFAULT_CONFIG, 0, 1, 1, 1.0
    bench.run_reference(A, rank=1, world=2)               # ranks other than 0 print nothing and do no work
    assert capsys.readouterr().out == ""
