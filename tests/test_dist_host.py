"""Host-side multi-rank logic on CPU: gloo, world_size 2."""
import os
import socket

import torch.multiprocessing as mp

from paper_2609_38984_b200 import dist as sd
from paper_2609_38984_b200 import workloads as W


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def _worker(rank, world, port, q):
    os.environ.update(RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world), MASTER_ADDR="127.0.0.1",
                      MASTER_PORT=str(port))
    r, lr, w = sd.init("gloo")
    wl = sd.rank_workload(W.WORKLOADS["tiny"], r, w)
    sd.barrier()
    mx = sd.max_over_ranks(10.0 + r)
    sm = sd.sum_over_ranks(float(wl.batch * wl.packed_len))
    q.put((r, wl.seed, mx, sm, list(sd.sample_range(5, r, w))))
    sd.finalize()


def test_two_ranks_shard_by_sample_and_reduce_timing():
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
    assert [r[1] for r in res] == [0, 1000]                 # distinct samples per rank
    assert all(r[2] == 11.0 for r in res)                   # MAX over ranks of the per-rank time
    assert all(r[3] == 2.0 * 88 for r in res)               # units summed over ranks
    assert res[0][4] == [0, 1, 2] and res[1][4] == [3, 4]   # contiguous split, sizes differ by at most one


def test_single_process_is_a_no_op():
    assert sd.rank_workload(W.WORKLOADS["tiny"], 0, 1) is W.WORKLOADS["tiny"]
    assert sd.max_over_ranks(3.5) == 3.5 and sd.sum_over_ranks(2.0) == 2.0
    assert list(sd.sample_range(8, 0, 1)) == list(range(8))
