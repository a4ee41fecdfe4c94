"""Drives the CPU oracle through a workload schedule (the counterpart of the package's harness)."""
import numpy as np

from oracle import cnn
from oracle import ps as ops
from paper_2406_05546_b200 import schedules, synth


def make_oracle(s, init_params):
    return ops.OraclePS(init_params, ring_depth=s.ring_depth, queue_slots=s.queue_slots(), ckpt_every=s.ckpt_every,
                        ckpt_slots=8, chain_len=s.chain_len, replicate_every=s.replicate_every,
                        external_store=s.external_store)


def run(s, o, pool_x, pool_y, on_tick=None, first_tick=0, last_tick=None, precision=0):
    log = []
    last_tick = s.ticks if last_tick is None else last_tick
    ids = list(range(s.W))
    for t in range(first_tick, last_tick):
        p = schedules.plan(s, t)
        events = []
        for action in p.pre:
            if action == "kill":
                o.kill(0)
            elif action == "restore":
                events.append(("restore", o.restore()))
            elif action == "failover":
                events.append(("failover", o.failover()))
        loss = None
        res = None
        if p.workers_run:
            lags = np.zeros(s.W, dtype=np.int32)
            if s.max_lag:
                lags = np.minimum(synth.lags(t, s.W, s.max_lag), o.version - o.oldest_version())
            pulled = [o.pull_snapshot(w, int(lags[w])) for w in range(s.W)]
            x, y = synth.tick_batch(pool_x, pool_y, t, s.W, s.b)
            g, l, am, z = cnn.workers_grad_step([th for _, th in pulled], ids, x, y, s.seed, t, s.dropout_p,
                                                 precision=precision)
            o.enqueue(g.astype(np.float32), ids, [v for v, _ in pulled], t)
            loss = (l, am, z)
            if p.apply:
                order = synth.arrival_order(t, s.W) if s.mode == schedules.ASYNC else None
                scale = s.replay_scale if p.catch_up else 1.0
                res = o.apply(s.mode, s.lr, scale, order)
        entry = {"tick": t, "version": o.version, "queue_len": len(o.queue), "loss": loss, "events": events,
                 "apply": res}
        log.append(entry)
        if on_tick:
            on_tick(entry)
    return log
