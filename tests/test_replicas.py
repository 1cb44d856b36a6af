"""World-size-2 gloo test of the replica bookkeeping (barrier, max-over-ranks timing,
whole-job throughput)."""
import os
import sys

import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    os.environ.update(RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world), MASTER_ADDR="127.0.0.1",
                      MASTER_PORT=str(port))
    from paper_2608_12385_b200 import replicas
    r, _, w = replicas.init("gloo")
    replicas.barrier()
    tput, ms = replicas.aggregate_throughput(units_this_rank=100.0 * (rank + 1), ms_this_rank=10.0 * (rank + 1))
    # a timing loop ends only when every rank says so
    agree = (replicas.all_agree(rank == 0), replicas.all_agree(True))
    out.put((r, w, tput, ms, agree))
    replicas.barrier()
    replicas.shutdown()


def test_two_replicas_aggregate_with_max_time_and_summed_units():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, 2, 29631, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, world, tput, ms, agree in res:
        assert world == 2 and ms == 20.0
        assert abs(tput - 300.0 / 0.020) < 1e-6
        assert agree == (False, True)


def test_single_process_is_identity():
    sys.path.insert(0, ROOT)
    from paper_2608_12385_b200 import replicas
    assert replicas.aggregate_throughput(50.0, 5.0) == (10000.0, 5.0)
    assert replicas.all_agree(True) and not replicas.all_agree(False)
