"""The N > 1 path is N independent replicas: its only multi-process logic is the barrier and the
max-over-ranks timing.  Run here as two gloo ranks on the CPU."""
import os
import socket

import torch
import torch.multiprocessing as mp


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ.update(RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world), MASTER_ADDR="127.0.0.1",
                      MASTER_PORT=str(port))
    from paper_2601_13155_b200.replicas import Replicas
    r = Replicas(backend="gloo", device=torch.device("cpu"))
    r.barrier()
    ms = 100.0 if rank == 0 else 250.0          # rank 1 is the slow one
    out[rank] = (r.max_over_ranks(ms), r.job_throughput(32768, ms), r.rank, r.world)
    r.close()


def test_two_replicas_report_max_time_and_aggregate_throughput():
    world = 2
    port = _free_port()
    with mp.Manager() as m:
        out = m.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    assert set(res) == {0, 1}
    for rank in (0, 1):
        mx, thr, rk, w = res[rank]
        assert (rk, w) == (rank, 2)
        assert mx == 250.0
        assert abs(thr - 2 * 32768 / 0.25) < 1e-6


def test_single_process_is_a_no_op():
    for k in ("RANK", "WORLD_SIZE", "LOCAL_RANK"):
        os.environ.pop(k, None)
    from paper_2601_13155_b200.replicas import Replicas
    r = Replicas(device=torch.device("cpu"))
    r.barrier()
    assert r.world == 1 and r.max_over_ranks(3.5) == 3.5 and r.job_throughput(10, 1000.0) == 10.0
    r.close()
