"""Thin ctypes binding of libps_b200.so (argument marshalling only).

Every step of the hot path runs in the library's CUDA kernels; torch is used for device and
pinned memory and for the stream.  There is no CPU fallback: if the library is missing or no
CUDA device is present, constructing a ParameterServer raises.
"""
import ctypes as C
import os

import numpy as np

from . import build as _build

P = 813258
P_PAD = 813312
SYNC, ASYNC, REPLAY = 0, 1, 2
FP32, TF32, BF16 = 0, 1, 2

ERRORS = {-1: "PS_ERR_BAD_ARG", -2: "PS_ERR_DOWN", -3: "PS_ERR_QUEUE_FULL", -4: "PS_ERR_NO_CHECKPOINT",
          -5: "PS_ERR_VERSION_EVICTED", -6: "PS_ERR_NO_REPLICA", -7: "PS_ERR_ARENA_TOO_SMALL",
          -8: "PS_ERR_CUDA", -9: "PS_ERR_DEVICE_STATUS"}

EXPORTS = ["ps_query_bytes", "ps_create", "ps_destroy", "ps_pull_snapshot", "ps_queue_reserve", "ps_slot_ptr",
           "workers_grad_step", "workers_grad_step_summed", "ps_apply_summed", "workers_eval", "ps_dropout_mask", "ps_enqueue", "ps_apply", "ps_apply_stale", "ps_checkpoint", "ps_restore", "ps_replicate",
           "ps_kill", "ps_failover", "ps_import_params", "ps_export_params", "ps_stats", "ps_tick_host",
           "ps_tick_host_submit", "ps_tick_host_wait",
           "ps_profile", "ps_profile_read", "ps_selftest_wait_timeout", "ps_last_error", "ps_replay_sum_static", "ps_replay_sum_static_error"]


class PSError(RuntimeError):
    def __init__(self, code, msg):
        super().__init__(f"{ERRORS.get(code, code)}: {msg}")
        self.code = code
        self.name = ERRORS.get(code, str(code))


class Config(C.Structure):
    _fields_ = [("max_workers", C.c_int32), ("max_batch", C.c_int32), ("ring_depth", C.c_int32),
                ("ckpt_every", C.c_int32), ("ckpt_slots", C.c_int32), ("chain_len", C.c_int32),
                ("replicate_every", C.c_int32), ("external_store", C.c_int32), ("precision", C.c_int32),
                ("dropout_p", C.c_float), ("queue_slots", C.c_int64), ("arena", C.c_void_p),
                ("arena_bytes", C.c_uint64), ("pinned", C.c_void_p), ("pinned_bytes", C.c_uint64),
                ("stream", C.c_void_p)]


class Snapshot(C.Structure):
    _fields_ = [("version", C.c_uint64), ("dev_ptr", C.c_void_p)]


class ApplyResult(C.Structure):
    _fields_ = [("applied", C.c_int64), ("new_version", C.c_uint64), ("checkpointed", C.c_int32),
                ("replicated", C.c_int32)]


class Stats(C.Structure):
    _fields_ = [("version", C.c_uint64), ("oldest_version", C.c_uint64), ("queue_len", C.c_int64),
                ("applied_total", C.c_int64), ("up", C.c_int32), ("live_replicas", C.c_int32),
                ("checkpoints", C.c_int32), ("device_status", C.c_uint32), ("replica_version", C.c_uint64),
                ("last_ckpt_version", C.c_uint64), ("kernel_launches", C.c_int64)]


_lib = None


def load(path=None):
    """Loads the shared library (building it if its sources are newer) and declares the ABI."""
    global _lib
    if _lib is not None and path is None:
        return _lib
    L = C.CDLL(path or _build.build())
    vp, i32, i64, u64, f32 = C.c_void_p, C.c_int32, C.c_int64, C.c_uint64, C.c_float
    sig = {
        "ps_query_bytes": [C.POINTER(Config), C.POINTER(u64), C.POINTER(u64)],
        "ps_create": [C.POINTER(Config), vp, C.POINTER(vp)],
        "ps_destroy": [vp],
        "ps_pull_snapshot": [vp, i32, i32, C.POINTER(Snapshot)],
        "ps_queue_reserve": [vp, i32, vp],
        "ps_slot_ptr": [vp, i64, C.POINTER(vp)],
        "workers_grad_step": [vp, i32, i32, vp, vp, vp, vp, u64, u64, vp, vp, vp, vp],
        "workers_eval": [vp, i32, i32, vp, vp, vp, vp, vp, vp],
        "workers_grad_step_summed": [vp, i32, i32, vp, vp, vp, vp, u64, u64, vp, vp, vp],
        "ps_apply_summed": [vp, vp, i32, f32, f32, C.POINTER(ApplyResult)],
        "ps_apply_stale": [vp, i32, f32, f32, vp, f32, f32, C.POINTER(ApplyResult)],
        "ps_dropout_mask": [vp, u64, i32, u64, i32, vp],
        "ps_enqueue": [vp, i32, vp, vp, vp, vp, u64],
        "ps_apply": [vp, i32, f32, f32, vp, C.POINTER(ApplyResult)],
        "ps_checkpoint": [vp, C.POINTER(u64)],
        "ps_restore": [vp, C.POINTER(u64)],
        "ps_replicate": [vp, C.POINTER(u64)],
        "ps_kill": [vp, i32],
        "ps_failover": [vp, C.POINTER(u64)],
        "ps_import_params": [vp, vp],
        "ps_export_params": [vp, i32, vp, C.POINTER(u64)],
        "ps_stats": [vp, C.POINTER(Stats)],
        "ps_tick_host": [vp, i32, i32, vp, vp, vp, u64, u64, i32, f32, f32, vp, vp, vp, C.POINTER(ApplyResult)],
        "ps_tick_host_submit": [vp, i32, i32, vp, vp, vp, u64, u64, i32, f32, f32, vp, vp, vp],
        "ps_tick_host_wait": [vp, C.POINTER(ApplyResult)],
    }
    sig["ps_profile"] = [vp, i32]
    sig["ps_selftest_wait_timeout"] = [vp, i64]
    sig["ps_profile_read"] = [vp, i32, C.POINTER(C.c_char_p), C.POINTER(C.c_double), C.POINTER(i64)]
    for name, args in sig.items():
        fn = getattr(L, name)
        fn.argtypes = args
        fn.restype = i32
    L.ps_replay_sum_static.argtypes = [vp, i64, vp, vp, f32, vp]
    L.ps_replay_sum_static.restype = i32
    L.ps_replay_sum_static_error.argtypes = []
    L.ps_replay_sum_static_error.restype = C.c_char_p
    L.ps_last_error.argtypes = [vp]
    L.ps_last_error.restype = C.c_char_p
    if path is None:
        _lib = L
    return L


def ps_replay_sum_static(queue_dev, theta_in_dev, theta_out_dev, coef, stream=None):
    """theta_out = theta_in - coef * sum of the rows of queue_dev, for callers that may not allocate
    (the scratch is a fixed array inside the library).  queue_dev: float32 cuda tensor [K, P_PAD];
    theta_in_dev / theta_out_dev: float32 cuda tensors [P_PAD].  Runs on `stream` (torch stream) or
    torch's current stream.  Marshalling only: nothing is allocated here either."""
    import torch
    L = load()
    K = int(queue_dev.shape[0])
    for t in (queue_dev, theta_in_dev, theta_out_dev):
        assert t.is_cuda and t.dtype == torch.float32 and t.is_contiguous()
    assert queue_dev.shape[1] == P_PAD and theta_in_dev.numel() == P_PAD and theta_out_dev.numel() == P_PAD
    st = (stream or torch.cuda.current_stream()).cuda_stream
    rc = L.ps_replay_sum_static(queue_dev.data_ptr(), K, theta_in_dev.data_ptr(), theta_out_dev.data_ptr(),
                                float(coef), st)
    if rc != 0:
        raise PSError(rc, L.ps_replay_sum_static_error().decode())


def _np_ptr(a):
    return a.ctypes.data_as(C.c_void_p) if a is not None else None


class ParameterServer:
    """One server context on the current CUDA device.  Method names are the C entry points."""

    def __init__(self, init_params, max_workers, max_batch, ring_depth=1, queue_slots=None, ckpt_every=0,
                 ckpt_slots=0, chain_len=1, replicate_every=1, external_store=False, precision=FP32,
                 dropout_p=0.25, stream=None):
        import torch
        if not torch.cuda.is_available():
            raise RuntimeError("paper_2406_05546_b200 needs a CUDA device; there is no CPU path")
        self._torch = torch
        self.lib = load()
        self.W_max, self.b_max = int(max_workers), int(max_batch)
        cfg = Config()
        cfg.max_workers, cfg.max_batch, cfg.ring_depth = self.W_max, self.b_max, int(ring_depth)
        cfg.ckpt_every, cfg.ckpt_slots = int(ckpt_every), int(ckpt_slots if ckpt_slots else (8 if ckpt_every else 0))
        cfg.chain_len, cfg.replicate_every = int(chain_len), int(replicate_every)
        cfg.external_store, cfg.precision, cfg.dropout_p = int(bool(external_store)), int(precision), float(dropout_p)
        cfg.queue_slots = int(queue_slots if queue_slots else max_workers)
        a, p = C.c_uint64(), C.c_uint64()
        self._check(self.lib.ps_query_bytes(C.byref(cfg), C.byref(a), C.byref(p)))
        self.arena = torch.empty(a.value, dtype=torch.uint8, device="cuda")
        self.pinned = torch.empty(p.value, dtype=torch.uint8).pin_memory()
        self.stream = stream if stream is not None else torch.cuda.current_stream()
        cfg.arena, cfg.arena_bytes = self.arena.data_ptr(), a.value
        cfg.pinned, cfg.pinned_bytes = self.pinned.data_ptr(), p.value
        cfg.stream = self.stream.cuda_stream
        self.cfg = cfg
        init = np.ascontiguousarray(init_params, dtype=np.float32)
        assert init.shape == (P,)
        ctx = C.c_void_p()
        self._check(self.lib.ps_create(C.byref(cfg), _np_ptr(init), C.byref(ctx)))
        self.ctx = ctx

    def _check(self, rc):
        if rc != 0:
            raise PSError(rc, self.lib.ps_last_error(None).decode())

    def close(self):
        if getattr(self, "ctx", None):
            self.lib.ps_destroy(self.ctx)
            self.ctx = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # -- worker side ---------------------------------------------------------
    def ps_pull_snapshot(self, worker, lag=0):
        s = Snapshot()
        self._check(self.lib.ps_pull_snapshot(self.ctx, int(worker), int(lag), C.byref(s)))
        return s

    def ps_queue_reserve(self, n):
        ids = np.zeros(n, dtype=np.int64)
        self._check(self.lib.ps_queue_reserve(self.ctx, int(n), _np_ptr(ids)))
        return ids

    def ps_slot_ptr(self, slot):
        p = C.c_void_p()
        self._check(self.lib.ps_slot_ptr(self.ctx, int(slot), C.byref(p)))
        return p.value

    def workers_grad_step(self, snaps, worker_ids, x_dev, y_dev, seed, step, slot_ids=None, grads_dev=None,
                          loss_dev=None, argmax_dev=None):
        """x_dev [W,b,28,28] float32 cuda, y_dev [W,b] int32 cuda.  Returns (loss_dev, argmax_dev)."""
        torch = self._torch
        W, b = int(y_dev.shape[0]), int(y_dev.shape[1])
        assert x_dev.is_cuda and x_dev.dtype == torch.float32 and x_dev.is_contiguous() and x_dev.numel() == W * b * 784
        assert y_dev.is_cuda and y_dev.dtype == torch.int32 and y_dev.is_contiguous()
        arr = (Snapshot * W)(*snaps)
        wid = np.ascontiguousarray(worker_ids, dtype=np.int32)
        assert wid.shape == (W,)
        if loss_dev is None:
            loss_dev = torch.empty(W, dtype=torch.float32, device="cuda")
        if argmax_dev is None:
            argmax_dev = torch.empty((W, b), dtype=torch.int32, device="cuda")
        sid = None if slot_ids is None else np.ascontiguousarray(slot_ids, dtype=np.int64)
        if grads_dev is not None:
            assert grads_dev.is_cuda and grads_dev.dtype == torch.float32 and grads_dev.shape == (W, P_PAD) and grads_dev.is_contiguous()
        self._check(self.lib.workers_grad_step(
            self.ctx, W, b, C.cast(arr, C.c_void_p), _np_ptr(wid), x_dev.data_ptr(), y_dev.data_ptr(),
            int(seed), int(step), _np_ptr(sid), grads_dev.data_ptr() if grads_dev is not None else None,
            loss_dev.data_ptr(), argmax_dev.data_ptr()))
        return loss_dev, argmax_dev

    def workers_grad_step_summed(self, snaps, worker_ids, x_dev, y_dev, seed, step, grad_sum_dev=None, loss_dev=None,
                                 argmax_dev=None):
        """All workers on one snapshot; returns (grad_sum_dev [P_PAD], loss_dev [W], argmax_dev [W,b])."""
        torch = self._torch
        W, b = int(y_dev.shape[0]), int(y_dev.shape[1])
        assert x_dev.is_cuda and x_dev.dtype == torch.float32 and x_dev.is_contiguous() and x_dev.numel() == W * b * 784
        assert y_dev.is_cuda and y_dev.dtype == torch.int32 and y_dev.is_contiguous()
        arr = (Snapshot * W)(*snaps)
        wid = np.ascontiguousarray(worker_ids, dtype=np.int32)
        if grad_sum_dev is None:
            grad_sum_dev = torch.empty(P_PAD, dtype=torch.float32, device="cuda")
        if loss_dev is None:
            loss_dev = torch.empty(W, dtype=torch.float32, device="cuda")
        if argmax_dev is None:
            argmax_dev = torch.empty((W, b), dtype=torch.int32, device="cuda")
        self._check(self.lib.workers_grad_step_summed(
            self.ctx, W, b, C.cast(arr, C.c_void_p), _np_ptr(wid), x_dev.data_ptr(), y_dev.data_ptr(), int(seed), int(step),
            grad_sum_dev.data_ptr(), loss_dev.data_ptr(), argmax_dev.data_ptr()))
        return grad_sum_dev, loss_dev, argmax_dev

    def ps_apply_summed(self, grad_sum_dev, n_workers, lr, scale=1.0):
        res = ApplyResult()
        self._check(self.lib.ps_apply_summed(self.ctx, grad_sum_dev.data_ptr(), int(n_workers), float(lr), float(scale), C.byref(res)))
        return {"applied": res.applied, "new_version": res.new_version, "checkpointed": res.checkpointed,
                "replicated": res.replicated}

    def workers_eval(self, snaps, x_dev, y_dev):
        """Forward pass without dropout.  Returns (loss_dev [W], argmax_dev [W,b], correct_dev [W])."""
        torch = self._torch
        W, b = int(y_dev.shape[0]), int(y_dev.shape[1])
        assert x_dev.is_cuda and x_dev.dtype == torch.float32 and x_dev.is_contiguous() and x_dev.numel() == W * b * 784
        assert y_dev.is_cuda and y_dev.dtype == torch.int32 and y_dev.is_contiguous()
        arr = (Snapshot * W)(*snaps)
        loss = torch.empty(W, dtype=torch.float32, device="cuda")
        am = torch.empty((W, b), dtype=torch.int32, device="cuda")
        correct = torch.empty(W, dtype=torch.int32, device="cuda")
        self._check(self.lib.workers_eval(self.ctx, W, b, C.cast(arr, C.c_void_p), x_dev.data_ptr(), y_dev.data_ptr(),
                                          loss.data_ptr(), am.data_ptr(), correct.data_ptr()))
        return loss, am, correct

    def ps_dropout_mask(self, seed, worker_id, step, b):
        keep = self._torch.empty((b, 512), dtype=self._torch.uint8, device="cuda")
        self._check(self.lib.ps_dropout_mask(self.ctx, int(seed), int(worker_id), int(step), int(b), keep.data_ptr()))
        return keep

    def ps_enqueue(self, worker_ids, base_versions, step, slot_ids=None, grads_dev=None):
        wid = np.ascontiguousarray(worker_ids, dtype=np.int32)
        bv = np.ascontiguousarray(base_versions, dtype=np.uint64)
        n = wid.shape[0]
        sid = None if slot_ids is None else np.ascontiguousarray(slot_ids, dtype=np.int64)
        if grads_dev is not None:
            assert grads_dev.is_cuda and grads_dev.dtype == self._torch.float32 and grads_dev.shape == (n, P_PAD) and grads_dev.is_contiguous()
        self._check(self.lib.ps_enqueue(self.ctx, n, _np_ptr(sid),
                                        grads_dev.data_ptr() if grads_dev is not None else None,
                                        _np_ptr(wid), _np_ptr(bv), int(step)))

    # -- server side -----------------------------------------------------------
    def ps_apply(self, mode, lr, scale=1.0, order=None):
        res = ApplyResult()
        o = None if order is None else np.ascontiguousarray(order, dtype=np.int32)
        self._check(self.lib.ps_apply(self.ctx, int(mode), float(lr), float(scale), _np_ptr(o), C.byref(res)))
        return {"applied": res.applied, "new_version": res.new_version, "checkpointed": res.checkpointed,
                "replicated": res.replicated}

    def ps_apply_stale(self, mode, lr, scale=1.0, order=None, clip_norm=0.0, staleness_alpha=0.0):
        res = ApplyResult()
        o = None if order is None else np.ascontiguousarray(order, dtype=np.int32)
        self._check(self.lib.ps_apply_stale(self.ctx, int(mode), float(lr), float(scale), _np_ptr(o), float(clip_norm),
                                            float(staleness_alpha), C.byref(res)))
        return {"applied": res.applied, "new_version": res.new_version, "checkpointed": res.checkpointed,
                "replicated": res.replicated}

    def _version_call(self, fn):
        v = C.c_uint64()
        self._check(fn(self.ctx, C.byref(v)))
        return v.value

    def ps_checkpoint(self):
        return self._version_call(self.lib.ps_checkpoint)

    def ps_restore(self):
        return self._version_call(self.lib.ps_restore)

    def ps_replicate(self):
        return self._version_call(self.lib.ps_replicate)

    def ps_failover(self):
        return self._version_call(self.lib.ps_failover)

    def ps_kill(self, server=0):
        self._check(self.lib.ps_kill(self.ctx, int(server)))

    def ps_import_params(self, theta):
        t = np.ascontiguousarray(theta, dtype=np.float32)
        assert t.shape == (P,)
        self._check(self.lib.ps_import_params(self.ctx, _np_ptr(t)))

    def ps_export_params(self, which=0):
        out = np.zeros(P, dtype=np.float32)
        v = C.c_uint64()
        self._check(self.lib.ps_export_params(self.ctx, int(which), _np_ptr(out), C.byref(v)))
        return out, v.value

    def ps_stats(self, check=True):
        s = Stats()
        rc = self.lib.ps_stats(self.ctx, C.byref(s))
        if check:
            self._check(rc)
        return {k: getattr(s, k) for k, _ in Stats._fields_}

    def ps_tick_host(self, x_host, y_host, seed, step, apply_mode, lr, scale=1.0, lags=None, order=None,
                     loss_host=None, argmax_host=None):
        """x_host [W,b,28,28] float32 / y_host [W,b] int32: pinned torch tensors or numpy arrays."""
        W, b = int(y_host.shape[0]), int(y_host.shape[1])
        ptr = lambda t: t.data_ptr() if hasattr(t, "data_ptr") else t.ctypes.data
        if loss_host is None:
            loss_host = np.zeros(W, dtype=np.float32)
        lg = None if lags is None else np.ascontiguousarray(lags, dtype=np.int32)
        o = None if order is None else np.ascontiguousarray(order, dtype=np.int32)
        res = ApplyResult()
        self._check(self.lib.ps_tick_host(self.ctx, W, b, _np_ptr(lg), ptr(x_host), ptr(y_host), int(seed), int(step),
                                          int(apply_mode), float(lr), float(scale), _np_ptr(o), ptr(loss_host),
                                          ptr(argmax_host) if argmax_host is not None else None, C.byref(res)))
        return loss_host, {"applied": res.applied, "new_version": res.new_version,
                           "checkpointed": res.checkpointed, "replicated": res.replicated}

    def ps_tick_host_submit(self, x_host, y_host, seed, step, apply_mode, lr, scale=1.0, lags=None, order=None,
                            loss_host=None, argmax_host=None):
        """Enqueues a whole tick and returns at once; the buffers must stay alive until ps_tick_host_wait."""
        W, b = int(y_host.shape[0]), int(y_host.shape[1])
        ptr = lambda t: t.data_ptr() if hasattr(t, "data_ptr") else t.ctypes.data
        if loss_host is None:
            loss_host = np.zeros(W, dtype=np.float32)
        lg = None if lags is None else np.ascontiguousarray(lags, dtype=np.int32)
        o = None if order is None else np.ascontiguousarray(order, dtype=np.int32)
        self._check(self.lib.ps_tick_host_submit(self.ctx, W, b, _np_ptr(lg), ptr(x_host), ptr(y_host), int(seed), int(step),
                                                 int(apply_mode), float(lr), float(scale), _np_ptr(o), ptr(loss_host),
                                                 ptr(argmax_host) if argmax_host is not None else None))
        self._inflight = getattr(self, "_inflight", []) + [(x_host, y_host, loss_host, argmax_host, lg, o)]
        return loss_host

    def ps_tick_host_wait(self):
        res = ApplyResult()
        self._check(self.lib.ps_tick_host_wait(self.ctx, C.byref(res)))
        if getattr(self, "_inflight", None):
            self._inflight.pop(0)
        return {"applied": res.applied, "new_version": res.new_version,
                "checkpointed": res.checkpointed, "replicated": res.replicated}

    def ps_selftest_wait_timeout(self, limit_cycles=20000):
        self._check(self.lib.ps_selftest_wait_timeout(self.ctx, int(limit_cycles)))

    def ps_profile(self, enable):
        self._check(self.lib.ps_profile(self.ctx, int(bool(enable))))

    def ps_profile_read(self):
        """{kernel name: (total ms, launches)} since profiling was switched on."""
        out = {}
        k = 0
        while True:
            name, ms, n = C.c_char_p(), C.c_double(), C.c_int64()
            if self.lib.ps_profile_read(self.ctx, k, C.byref(name), C.byref(ms), C.byref(n)) != 0:
                break
            out[name.value.decode()] = (ms.value, n.value)
            k += 1
        return out

    # -- helpers for tests (plain copies through torch, no arithmetic) ----------
    def slot_tensor(self, slot):
        """A [P_PAD] float32 cuda view of a queue slot (borrowed memory)."""
        torch = self._torch
        off = self.ps_slot_ptr(slot) - self.arena.data_ptr()
        return self.arena[off:off + P_PAD * 4].view(torch.float32)
