"""The five workload schedules as data: who runs at which tick, when the server dies and how it
comes back.  No arithmetic of the method lives here; the same plan drives the CUDA library (see
harness.py), the CPU oracle in the tests, and the benchmark.

Ticks: every live worker computes one gradient per tick; then the server, if it is up, applies.
"""
from dataclasses import dataclass, field, replace

SYNC, ASYNC, REPLAY = 0, 1, 2


@dataclass(frozen=True)
class Schedule:
    name: str
    W: int                      # logical workers
    b: int                      # batch per worker
    mode: int                   # apply mode while the server is up
    ticks: int
    ring_depth: int = 1
    ckpt_every: int = 0
    chain_len: int = 1
    replicate_every: int = 1
    external_store: bool = False
    max_lag: int = 0            # per-worker version lag drawn uniformly from 0..max_lag
    kill_at: int = -1           # the server dies before this tick's work
    recover_at: int = -1        # first tick after the outage (restore / failover happens before it)
    recover_by: str = ""        # "restore" | "failover"
    replay_scale: float = 1.0   # learning-rate scale of the catch-up replay (stateless server)
    lr: float = 0.01
    dropout_p: float = 0.25
    seed: int = 0x5EED

    def queue_slots(self):
        down = max(0, self.recover_at - self.kill_at) if self.external_store and self.kill_at >= 0 else 0
        return self.W * (down + 1)


def config(n: int) -> Schedule:
    """Full-size schedules of the five configurations."""
    if n == 1:   # sync, no failure
        return Schedule("sync", W=2, b=8, mode=SYNC, ticks=10)
    if n == 2:   # sync + checkpoint every 25 updates; killed at tick 60, down 20 ticks, restored from version 50
        return Schedule("sync-checkpoint", W=8, b=64, mode=SYNC, ticks=200, ckpt_every=25,
                        kill_at=60, recover_at=80, recover_by="restore")
    if n == 3:   # stateless; down from tick 100 to 200, 1,600 gradients buffered and replayed
        return Schedule("stateless", W=16, b=64, mode=REPLAY, ticks=300, external_store=True,
                        kill_at=100, recover_at=200, recover_by="restore")
    if n == 4:   # async, lag 0..8, every update mirrored; primary killed at tick 300, replica takes over
        return Schedule("async-chain", W=64, b=32, mode=ASYNC, ticks=400, ring_depth=9, chain_len=2,
                        replicate_every=1, max_lag=8, kill_at=300, recover_at=300, recover_by="failover")
    if n == 5:   # stateless at scale; down 200 ticks (25,600 gradients, 83 GB), 1,000 ticks in all
        return Schedule("stateless-scale", W=128, b=128, mode=REPLAY, ticks=1000, external_store=True,
                        kill_at=400, recover_at=600, recover_by="restore")
    raise ValueError("configs are numbered 1..5")


def reduced(n: int) -> Schedule:
    """The same schedules shrunk (fewer workers, smaller batches, shorter outages) so that the CPU
    oracle can follow every tick in seconds."""
    s = config(n)
    if n == 1:
        return s
    if n == 2:
        return replace(s, W=2, b=4)
    if n == 3:
        return replace(s, W=4, b=4, ticks=30, kill_at=10, recover_at=20)
    if n == 4:
        return replace(s, W=8, b=4, ticks=40, kill_at=30, recover_at=30)
    return replace(s, W=8, b=16, ticks=50, kill_at=20, recover_at=30)


@dataclass
class TickPlan:
    pre: list = field(default_factory=list)   # "kill", "restore", "failover" before the tick's work
    workers_run: bool = True
    apply: bool = True
    catch_up: bool = False                    # this tick's apply also consumes the outage's backlog


def plan(s: Schedule, t: int) -> TickPlan:
    p = TickPlan()
    if s.kill_at >= 0:
        if t == s.kill_at:
            p.pre.append("kill")
        if t == s.recover_at:
            p.pre.append(s.recover_by)
            p.catch_up = s.external_store and s.recover_at > s.kill_at
        if s.kill_at <= t < s.recover_at:
            p.apply = False
            # stateful server down: "the remaining workers are idle"; stateless: they keep going
            p.workers_run = s.external_store
    return p
