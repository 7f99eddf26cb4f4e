"""The N > 1 path of the benchmark is N independent replicas (the serving loop has no exchange
step); only the report is combined.  Checked here with two gloo ranks on the CPU."""
import os
import socket

import torch
import torch.distributed as dist
import torch.multiprocessing as mp


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import sys
    sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
    import bench
    ms, tokens = (100.0, 1000.0) if rank == 0 else (125.0, 1500.0)   # the slower rank sets the time
    ms_max, tok_all = bench.reduce_over_ranks(ms, tokens, torch.device("cpu"), world)
    out.put((rank, ms_max, tok_all))
    dist.barrier()
    dist.destroy_process_group()


def test_two_replicas_report_sum_of_tokens_over_slowest_time():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    got = [out.get(timeout=120) for _ in procs]
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for _, ms_max, tok_all in got:
        assert ms_max == 125.0 and tok_all == 2500.0
    assert 2500.0 / (125.0 / 1e3) == 20000.0   # whole-job tokens per second


def test_single_rank_is_identity():
    import bench
    assert bench.reduce_over_ranks(7.5, 42, torch.device("cpu"), 1) == (7.5, 42.0)
