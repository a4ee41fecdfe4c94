"""Parameter-server oracle in numpy (test infrastructure only).

A plain restatement of the server side of the paper's three designs:

* synchronous / asynchronous training with checkpointing (Design, "Sync/Async
  Checkpointing"): the server applies all gradients of an iteration at once
  (sync) or one by one as they arrive (async), saves its parameters after a set
  number of weight updates, and after a failure continues from the latest
  checkpoint while the workers were idle;
* chain replication with relaxed consistency and periodic replication (Design,
  "Sync/Async Chain Replicated Parameter Servers"): every R-th weight version
  is copied to the next server, which takes over with those weights;
* the stateless server (Design, "Stateless Parameter Server" and the paper's
  pseudo-code figure): weights and the gradient queue live in an external
  store that survives the server; one server step takes all queued gradients,
  applies them to the stored weights and stores the result.

All sums are taken in double precision and rounded to fp32 once per stored
weight version.  Scaling rule (a reading of "applies all updates at once",
recorded in the design notes): SYNC steps by lr*scale/K for the K queued
gradients; ASYNC by lr*scale per gradient; REPLAY by lr*scale/W_tick where
W_tick is the number of gradients per enqueue call, so that a replay of one
tick's gradients equals the sync step.

Nothing here is shared with, or imported by, the CUDA path.
"""
import numpy as np

SYNC, ASYNC, REPLAY = 0, 1, 2


class PSError(Exception):
    def __init__(self, code, msg):
        super().__init__(f"{code}: {msg}")
        self.code = code


BAD_ARG, DOWN, QUEUE_FULL, NO_CHECKPOINT, VERSION_EVICTED, NO_REPLICA = (
    "BAD_ARG", "DOWN", "QUEUE_FULL", "NO_CHECKPOINT", "VERSION_EVICTED", "NO_REPLICA")


class OraclePS:
    def __init__(self, init_params, ring_depth=1, queue_slots=1 << 30, ckpt_every=0, ckpt_slots=4,
                 chain_len=1, replicate_every=1, external_store=False):
        theta = np.asarray(init_params, dtype=np.float32).copy()
        self.P = theta.size
        self.ring_depth = int(ring_depth)
        self.queue_slots = int(queue_slots)
        self.ckpt_every = int(ckpt_every)
        self.ckpt_slots = int(ckpt_slots)
        self.replicate_every = max(1, int(replicate_every))
        self.external_store = bool(external_store)
        self.version = 0
        self.ring = {0: theta}                      # version -> fp32 parameters
        self.replicas = [{"version": 0, "theta": theta.copy(), "alive": True}
                         for _ in range(int(chain_len) - 1)]
        self.queue = []                             # dicts: g, worker, base_version, step
        self.w_tick = 0
        self.ckpts = []                             # [(version, theta)] oldest first
        self.up = True
        self.applied_total = 0

    # -- worker-facing ---------------------------------------------------
    def head(self):
        return self.ring[self.version]

    def oldest_version(self):
        return min(self.ring)

    def pull_snapshot(self, worker, lag=0):
        """Weights of version head-lag (the worker's 'get weights' of the pseudo-code)."""
        if not self.up and not self.external_store:
            raise PSError(DOWN, "server is down and its weights died with it")
        if lag < 0:
            raise PSError(BAD_ARG, "negative lag")
        v = self.version - lag
        if v not in self.ring:
            raise PSError(VERSION_EVICTED, f"version {v} is not retained")
        return v, self.ring[v]

    def enqueue(self, grads, worker_ids, base_versions, step):
        """Workers append their gradients (the pseudo-code's append to the gradient list)."""
        if not self.up and not self.external_store:
            raise PSError(DOWN, "server is down")
        grads = np.asarray(grads, dtype=np.float32)
        n = grads.shape[0]
        if n <= 0 or grads.shape[1] != self.P:
            raise PSError(BAD_ARG, "shape")
        if len(self.queue) + n > self.queue_slots:
            raise PSError(QUEUE_FULL, "queue full")
        if self.queue and n != self.w_tick:
            raise PSError(BAD_ARG, "gradients per enqueue call changed while the queue is not empty")
        self.w_tick = n
        for i in range(n):
            self.queue.append({"g": grads[i].copy(), "worker": int(worker_ids[i]),
                               "base_version": int(base_versions[i]), "step": int(step)})

    # -- server step -------------------------------------------------------
    def _publish(self, theta32, result):
        """A new weight version exists: ring, periodic checkpoint, periodic replication."""
        self.version += 1
        self.ring[self.version] = theta32
        for v in [v for v in self.ring if v <= self.version - self.ring_depth]:
            del self.ring[v]
        if self.ckpt_every > 0 and self.version % self.ckpt_every == 0:
            self.checkpoint()
            result["checkpointed"] += 1
        if self.replicas and self.version % self.replicate_every == 0:
            self.replicate()
            result["replicated"] += 1

    def apply(self, mode, lr, scale=1.0, order=None, clip_norm=None, staleness_alpha=0.0):
        """One server step over the whole queue.

        clip_norm and staleness_alpha are the two treatments of stale gradients that the design section's closing
        remarks on the stateless server name as alternatives to a smaller learning rate (gradient clipping; an
        adaptive, here staleness-dependent, learning rate).  Readings recorded in the design notes:
          clip_norm c > 0:  every queued gradient is scaled by min(1, c / ||g||_2) (clipping by global norm, per
                            gradient, norm taken in double);
          staleness_alpha a >= 0:  gradient k is scaled by 1 / (1 + a * tau_k), tau_k = the version its update is
                            applied to minus the version its worker had read (base_version): SYNC / REPLAY apply
                            everything to the head, ASYNC applies the j-th gradient in arrival order to head + j.
        With clip_norm None and alpha 0 every factor is exactly 1."""
        if not self.up:
            raise PSError(DOWN, "server is down")
        K = len(self.queue)
        result = {"applied": 0, "new_version": self.version, "checkpointed": 0, "replicated": 0}
        if K == 0:
            return result
        idx = list(range(K)) if order is None else [int(o) for o in order]
        if sorted(idx) != list(range(K)):
            raise PSError(BAD_ARG, "order is not a permutation of the queue")
        if clip_norm is not None and not clip_norm > 0:
            raise PSError(BAD_ARG, "clip_norm must be positive")
        if staleness_alpha < 0:
            raise PSError(BAD_ARG, "staleness_alpha must be >= 0")
        lr = float(np.float32(lr))
        scale = float(np.float32(scale))
        alpha = float(np.float32(staleness_alpha))
        clip = None if clip_norm is None else float(np.float32(clip_norm))
        v0 = self.version

        def factor(k, applied_to):
            f = 1.0
            if clip is not None:
                norm = float(np.sqrt(np.sum(self.queue[k]["g"].astype(np.float64) ** 2)))
                if norm > clip:
                    f *= clip / norm
            if alpha > 0.0:
                tau = applied_to - self.queue[k]["base_version"]
                if tau < 0:
                    raise PSError(BAD_ARG, "a gradient claims a base version newer than the weights it is applied to")
                f /= 1.0 + alpha * tau
            return f

        theta = self.head()
        if mode in (SYNC, REPLAY):
            total = np.zeros(self.P, dtype=np.float64)
            for k in idx:
                total += factor(k, v0) * self.queue[k]["g"].astype(np.float64)
            div = K if mode == SYNC else self.w_tick
            new = (theta.astype(np.float64) - (lr * scale / div) * total).astype(np.float32)
            self._publish(new, result)
        elif mode == ASYNC:
            for j, k in enumerate(idx):
                new = (theta.astype(np.float64)
                       - (lr * scale * factor(k, v0 + j)) * self.queue[k]["g"].astype(np.float64)).astype(np.float32)
                self._publish(new, result)
                theta = new
        else:
            raise PSError(BAD_ARG, "mode")
        self.queue = []
        self.applied_total += K
        result["applied"] = K
        result["new_version"] = self.version
        return result

    # -- failure handling ----------------------------------------------------
    def checkpoint(self):
        self.ckpts.append((self.version, self.head().copy()))
        if len(self.ckpts) > self.ckpt_slots:
            self.ckpts.pop(0)
        return self.version

    def replicate(self):
        """One replication event.  The frontend hands its weights to the next live server and waits for that
        server's acknowledgement only (the relaxed consistency of the chain design); the hop from that server to
        the one behind it completes with the following event.  So after an event the first live server behind the
        frontend holds the frontend's version, the second what the first held before, and so on: a server further
        down the chain holds more outdated weights, as the design section says of the tertiary server."""
        live = [r for r in self.replicas if r["alive"]]
        if not live:
            raise PSError(NO_REPLICA, "no live replica")
        for i in range(len(live) - 1, 0, -1):
            live[i]["version"] = live[i - 1]["version"]
            live[i]["theta"] = live[i - 1]["theta"]
        live[0]["version"] = self.version
        live[0]["theta"] = self.head().copy()
        return self.version

    def kill(self, server=0):
        """server 0 = the current frontend; i >= 1 = the i-th LIVE server behind it (a dead server has left the
        chain: the one behind it watches the next live one in front of it instead)."""
        if server == 0:
            self.up = False
            if not self.external_store:
                self.ring = {}
                self.queue = []
        else:
            live = [r for r in self.replicas if r["alive"]]
            if server < 0 or server - 1 >= len(live):
                raise PSError(BAD_ARG, "no such server")
            live[server - 1]["alive"] = False

    def restore(self):
        """Resurrected server: latest checkpoint (stateful) or the surviving store (stateless)."""
        if self.external_store:
            self.up = True
            return self.version
        if not self.ckpts:
            raise PSError(NO_CHECKPOINT, "no checkpoint")
        v, theta = self.ckpts[-1]
        self.version = v
        self.ring = {v: theta.copy()}
        self.queue = []
        self.up = True
        return v

    def failover(self):
        """The next live server in the chain becomes the frontend with its (warm) weights."""
        while self.replicas and not self.replicas[0]["alive"]:
            self.replicas.pop(0)
        if not self.replicas:
            raise PSError(NO_REPLICA, "no live replica")
        r = self.replicas.pop(0)
        self.version = r["version"]
        self.ring = {self.version: r["theta"]}
        self.queue = []
        self.up = True
        return self.version
