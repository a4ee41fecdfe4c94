"""Runs a workload schedule on the CUDA library (marshalling only: every step is a library call)."""
import numpy as np

from . import ps, schedules, synth


def make_server(s: schedules.Schedule, init_params, queue_slots=None, precision=ps.FP32):
    return ps.ParameterServer(init_params, max_workers=s.W, max_batch=s.b, ring_depth=s.ring_depth,
                              queue_slots=queue_slots or s.queue_slots(), ckpt_every=s.ckpt_every,
                              ckpt_slots=8 if s.ckpt_every else 0, chain_len=s.chain_len,
                              replicate_every=s.replicate_every, external_store=s.external_store,
                              precision=precision, dropout_p=s.dropout_p)


def clamp_lags(lags, head, oldest):
    return np.minimum(lags, head - oldest).astype(np.int32)


def run(s: schedules.Schedule, srv, pool_x, pool_y, on_tick=None, first_tick=0, last_tick=None):
    """Drives srv through ticks [first_tick, last_tick).  pool_x/pool_y: numpy image pool.
    Returns a log: per tick (version after the tick, queue length, losses or None, events)."""
    import torch
    log = []
    last_tick = s.ticks if last_tick is None else last_tick
    ids = list(range(s.W))
    for t in range(first_tick, last_tick):
        p = schedules.plan(s, t)
        events = []
        for action in p.pre:
            if action == "kill":
                srv.ps_kill(0)
            elif action == "restore":
                events.append(("restore", srv.ps_restore()))
            elif action == "failover":
                events.append(("failover", srv.ps_failover()))
        loss = None
        res = None
        if p.workers_run:
            st = srv.ps_stats()
            lags = np.zeros(s.W, dtype=np.int32)
            if s.max_lag:
                lags = clamp_lags(synth.lags(t, s.W, s.max_lag), st["version"], st["oldest_version"])
            snaps = [srv.ps_pull_snapshot(w, int(lags[w])) for w in range(s.W)]
            x, y = synth.tick_batch(pool_x, pool_y, t, s.W, s.b)
            slots = srv.ps_queue_reserve(s.W)
            loss_d, am_d = srv.workers_grad_step(snaps, ids, torch.from_numpy(x).cuda(), torch.from_numpy(y).cuda(),
                                                 s.seed, t, slot_ids=slots)
            srv.ps_enqueue(ids, [sn.version for sn in snaps], t, slot_ids=slots)
            loss = (loss_d.cpu().numpy(), am_d.cpu().numpy())
            if p.apply:
                order = synth.arrival_order(t, s.W) if s.mode == schedules.ASYNC else None
                scale = s.replay_scale if p.catch_up else 1.0
                res = srv.ps_apply(s.mode, s.lr, scale, order)
        st = srv.ps_stats()
        entry = {"tick": t, "version": st["version"], "queue_len": st["queue_len"], "loss": loss,
                 "events": events, "apply": res, "stats": st}
        log.append(entry)
        if on_tick:
            on_tick(entry)
    return log
