"""World-size-2 check (gloo, CPU) of the only multi-process logic the benchmark has: replicas + max-over-ranks timing."""
import os
import socket

import torch
import torch.distributed as dist
import torch.multiprocessing as mp


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, q):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from paper_2608_04405_b200 import replicas as R
    local_ms = 0.020 + 0.010 * rank            # rank 1 is slower
    ms = R.max_over_ranks(local_ms)
    dist.barrier()
    q.put((rank, ms, R.whole_job_tokens_per_s(4, world, ms), R.replica_salt(rank, 3)))
    dist.destroy_process_group()


def test_two_replicas_report_slowest_rank_and_aggregate_rate():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert all(abs(ms - 0.030) < 1e-12 for _, ms, _, _ in res)        # both ranks see the maximum
    assert all(abs(v - 2 * 4 / 0.030e-3) < 1e-3 for _, _, v, _ in res)  # whole-job rate over both replicas
    assert {s for _, _, _, s in res} == {3, 103}                       # replicas draw different data


def test_single_process_is_identity():
    from paper_2608_04405_b200 import replicas as R
    assert R.max_over_ranks(1.5) == 1.5
    assert R.whole_job_tokens_per_s(4, 1, 0.02) == 4 / 0.02e-3
