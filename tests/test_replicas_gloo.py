"""The N>1 path of the benchmark (independent replicas) on two gloo ranks on CPU."""
import os
import socket

import torch.multiprocessing as mp


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _worker(rank, world, port, out):
    os.environ.update(RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world), MASTER_ADDR="127.0.0.1",
                      MASTER_PORT=str(port))
    from paper_2503_13565_b200 import replicas
    replicas.init("gloo")
    assert replicas.env_world() == (rank, rank, world)
    replicas.barrier()
    slow = replicas.max_over_ranks(1.0 + rank)            # rank 1 is the slow one
    total = replicas.sum_over_ranks(10.0)
    thr = replicas.whole_job_throughput(10.0, 1.0 + rank)
    replicas.barrier()
    replicas.shutdown()
    out.put((rank, slow, total, thr))


def test_two_replicas_report_the_slowest_time_and_the_summed_work():
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
    for rank, slow, total, thr in res:
        assert slow == 2.0 and total == 20.0 and thr == 10.0


def test_single_process_is_a_no_op():
    from paper_2503_13565_b200 import replicas
    for k in ("RANK", "LOCAL_RANK", "WORLD_SIZE"):
        os.environ.pop(k, None)
    assert replicas.env_world() == (0, 0, 1)
    replicas.init("gloo")
    replicas.barrier()
    assert replicas.max_over_ranks(3.5) == 3.5
    assert replicas.whole_job_throughput(8.0, 2.0) == 4.0
