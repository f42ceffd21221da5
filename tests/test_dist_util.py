"""Multi-rank bookkeeping of the benchmark (weak scaling over independent prompt groups) on two gloo ranks."""
import os
import socket
import sys

import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, q):
    sys.path.insert(0, ROOT)
    os.environ.update(RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world), MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    from paper_2605_26606_b200 import dist_util
    from paper_2605_26606_b200 import workloads as wl
    import dataclasses
    r, lr, w = dist_util.init("gloo")
    dist_util.barrier()
    # every rank draws its own sampling batch
    base = wl.WORKLOADS["config0"]
    batch = wl.gen_batch(dataclasses.replace(base, data_seed=dist_util.rank_data_seed(base.data_seed, r)))
    t, u = dist_util.aggregate(10.0 + 5.0 * r, 100.0 * (r + 1))
    dist_util.barrier()
    q.put((r, w, t, u, int(batch.prompt_tokens.sum())))


def test_two_ranks_aggregate_max_time_and_total_units():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert [x[0] for x in res] == [0, 1] and all(x[1] == 2 for x in res)
    assert all(x[2] == 15.0 and x[3] == 300.0 for x in res)        # max over ranks, sum over ranks
    assert res[0][4] != res[1][4]                                  # different batches per rank


def test_single_process_passthrough():
    sys.path.insert(0, ROOT)
    from paper_2605_26606_b200 import dist_util
    assert dist_util.aggregate(3.5, 7.0) == (3.5, 7.0)
    assert dist_util.rank_data_seed(6, 0) == 6 and dist_util.rank_data_seed(6, 3) == 3006
