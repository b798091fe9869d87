"""The N > 1 path of the benchmark on CPU: two gloo ranks, barrier, max over ranks, job throughput."""
import os
import socket
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def _worker(rank, world, port, out):
    os.environ.update(RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world),
                      MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    sys.path.insert(0, ROOT)
    from paper_2509_11254_b200.replicas import Replicas

    reps = Replicas("gloo", None)
    reps.barrier()
    ms = reps.max_over_ranks(10.0 + 5.0 * rank)      # rank 1 is the slow one: 15 ms
    thr = reps.job_throughput(3.0e9, ms)             # 3 GB per replica and step
    reps.barrier()
    reps.close()
    out.put((rank, ms, thr))


def test_two_gloo_ranks_agree_on_the_slowest_time():
    import torch.multiprocessing as mp

    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert [r[0] for r in res] == [0, 1]
    for _, ms, thr in res:
        assert ms == 15.0                                  # max over ranks, same on both
        assert abs(thr - 2 * 3.0e9 / 15.0e-3) < 1e-3       # both replicas' bytes over the slowest time


def test_single_process_is_a_no_op():
    sys.path.insert(0, ROOT)
    for k in ("RANK", "LOCAL_RANK", "WORLD_SIZE"):
        os.environ.pop(k, None)
    from paper_2509_11254_b200.replicas import Replicas

    reps = Replicas("gloo", None)
    reps.barrier()
    assert reps.world == 1 and reps.max_over_ranks(7.5) == 7.5
    assert reps.job_throughput(2.0, 1000.0) == 2.0
    reps.close()
