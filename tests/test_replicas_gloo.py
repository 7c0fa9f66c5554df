"""The N > 1 bookkeeping of the benchmark (replicas only, no data-path collective), run as two
gloo ranks on CPU: rendezvous, barrier, max over ranks and the whole-job throughput."""
import os
import socket

import torch.multiprocessing as mp


def _free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank: int, world: int, port: int, out):
    os.environ.update(RANK=str(rank), WORLD_SIZE=str(world), LOCAL_RANK=str(rank),
                      MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    from paper_2506_06266_b200 import replicas
    r, w, l = replicas.setup("gloo")
    assert (r, w, l) == (rank, world, rank)
    replicas.barrier(w)
    elapsed_ms = 10.0 * (rank + 1)                     # rank 1 is the slow one
    value, ms = replicas.whole_job_tokens_per_s(64 * 5, elapsed_ms, w)
    out.put((rank, value, ms, replicas.max_over_ranks(float(rank), w)))
    replicas.barrier(w)
    replicas.shutdown()


def test_two_ranks_agree_on_the_slowest_time_and_the_job_throughput():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    results = [out.get(timeout=120) for _ in procs]
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, value, ms, mx in results:
        assert ms == 20.0 and mx == 1.0
        assert abs(value - 2 * 64 * 5 / 0.020) < 1e-6


def test_single_rank_needs_no_process_group():
    from paper_2506_06266_b200 import replicas
    for k in ("RANK", "WORLD_SIZE", "LOCAL_RANK"):
        os.environ.pop(k, None)
    assert replicas.env_rank() == (0, 1, 0)
    assert replicas.max_over_ranks(3.5, 1) == 3.5
    assert replicas.whole_job_tokens_per_s(100, 50.0, 1) == (2000.0, 50.0)
