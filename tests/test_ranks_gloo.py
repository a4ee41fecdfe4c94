"""The multi-process plumbing on CPU: two `gloo` ranks, each with its own shard of the work.

The path shards by independent parameter-server replicas (no data-path collective), so what N > 1
adds is a barrier, the maximum of the ranks' times and disjoint input rows per rank.
"""
import os
import socket

import numpy as np
import torch.multiprocessing as mp

from paper_2406_05546_b200 import synth
from paper_2406_05546_b200.ranks import Ranks


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _rank_main(rank, world, port, q):
    os.environ.update(RANK=str(rank), WORLD_SIZE=str(world), LOCAL_RANK=str(rank),
                      MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    r = Ranks("gloo")
    r.barrier()
    # every rank reports a different time: all must agree on the slowest
    ms = r.max_over_ranks(10.0 + 5.0 * rank)
    rows = synth.batch_rows(r.batch_seed(3), 4, 8, synth.POOL_IMAGES)
    rate = r.whole_job_rate(4 * 8, ms)
    r.barrier()
    q.put((rank, ms, rate, rows.tolist()))
    r.close()


def test_two_ranks_agree_on_max_time_and_draw_disjoint_rows():
    world = 2
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_rank_main, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    out = sorted(q.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    (r0, ms0, rate0, rows0), (r1, ms1, rate1, rows1) = out
    assert (r0, r1) == (0, 1)
    assert ms0 == ms1 == 15.0                       # the slower rank's time on both
    assert rate0 == rate1 == 2 * 32 / 15e-3         # all ranks' units over that time
    assert np.array(rows0).shape == (4, 8)
    assert rows0 != rows1                           # each rank feeds its workers its own rows


def test_single_process_needs_no_group():
    for k in ("RANK", "WORLD_SIZE", "LOCAL_RANK"):
        os.environ.pop(k, None)
    r = Ranks("gloo")
    assert (r.rank, r.world) == (0, 1)
    r.barrier()
    assert r.max_over_ranks(2.5) == 2.5
    assert r.whole_job_rate(100, 50.0) == 2000.0
    r.close()
