"""ctypes wrapper of oracle/cnn_oracle.c (test infrastructure only)."""
import ctypes as C

import numpy as np

from . import build as _build

P = 813258
IMG = 28
HID = 512
NCLS = 10

# name -> (offset, shape), canonical order (model endnote of the paper + design readings)
TENSORS = {
    "conv1.w": (0, (16, 1, 3, 3)),
    "conv1.b": (144, (16,)),
    "conv2.w": (160, (32, 16, 3, 3)),
    "conv2.b": (4768, (32,)),
    "fc1.w": (4800, (512, 1568)),
    "fc1.b": (807616, (512,)),
    "fc2.w": (808128, (10, 512)),
    "fc2.b": (813248, (10,)),
}

_lib = None


def lib():
    global _lib
    if _lib is None:
        L = C.CDLL(_build.build())
        L.oracle_param_count.restype = C.c_int64
        L.oracle_philox4x32_10.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p]
        L.oracle_philox4x32_10.restype = None
        L.oracle_dropout_keep.argtypes = [C.c_uint64, C.c_uint32, C.c_uint64, C.c_int32, C.c_double, C.c_void_p]
        L.oracle_dropout_keep.restype = None
        L.oracle_grad_step_f64.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.c_void_p,
                                           C.c_double, C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
        L.oracle_grad_step_f64.restype = C.c_int32
        L.oracle_grad_step_f64_diag.argtypes = L.oracle_grad_step_f64.argtypes + [C.c_void_p]
        L.oracle_grad_step_f64_diag.restype = C.c_int32
        L.oracle_workers_grad_step.argtypes = [C.c_int32, C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p,
                                               C.c_void_p, C.c_uint64, C.c_uint64, C.c_double, C.c_int32,
                                               C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
        L.oracle_workers_grad_step.restype = C.c_int32
        L.oracle_num_threads.restype = C.c_int32
        L.oracle_round_operand.argtypes = [C.c_double, C.c_int32]
        L.oracle_round_operand.restype = C.c_double
        assert L.oracle_param_count() == P
        _lib = L
    return _lib


def _ptr(a):
    return a.ctypes.data_as(C.c_void_p) if a is not None else None


def philox4x32_10(ctr, key):
    c = np.asarray(ctr, dtype=np.uint32).copy()
    k = np.asarray(key, dtype=np.uint32).copy()
    out = np.zeros(4, dtype=np.uint32)
    lib().oracle_philox4x32_10(_ptr(c), _ptr(k), _ptr(out))
    return out


def dropout_keep(seed, worker, step, b, p):
    keep = np.zeros(b * HID, dtype=np.uint8)
    lib().oracle_dropout_keep(int(seed), int(worker), int(step), int(b), float(p), _ptr(keep))
    return keep.reshape(b, HID)


class _Diag(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in ("p1", "a2", "p2", "u", "dh", "code2", "on", "flip")]


def grad_step_f64(theta, x, y, keep=None, drop_p=0.25, precision=0, diag=False, flips=None):
    """One worker, everything double.  Returns (grad[P], loss, argmax[b], logits[b,10]).
    precision 1: ReLU/pooling decisions are taken on a TF32-operand forward pass (values stay exact);
    precision 2: the same with BF16 operands in the second convolution (the 512-unit layer stays TF32).
    diag=True appends a dict of the exact pass's per-sample intermediates: p1 [b,16,14,14], a2 [b,32,14,14],
    p2 [b,1568], u [b,512] (pre-activations of the 512-unit layer), dh [b,512] (gradient w.r.t. that layer's
    output after ReLU, dropout applied), code2 [b,1568] and on [b,512] (the decisions that were used).
    flips (needs diag=True): [(sample, unit), ...] whose ReLU decision is taken the other way."""
    theta = np.ascontiguousarray(theta, dtype=np.float64)
    x = np.ascontiguousarray(x, dtype=np.float64)
    y = np.ascontiguousarray(y, dtype=np.int32)
    b = y.shape[0]
    assert theta.shape == (P,) and x.size == b * IMG * IMG
    if keep is not None:
        keep = np.ascontiguousarray(keep, dtype=np.uint8)
        assert keep.size == b * HID
    grad = np.zeros(P, dtype=np.float64)
    loss = np.zeros(1, dtype=np.float64)
    am = np.zeros(b, dtype=np.int32)
    logits = np.zeros((b, NCLS), dtype=np.float64)
    d, dstruct = None, None
    if diag:
        d = {"p1": np.zeros((b, 16, 14, 14)), "a2": np.zeros((b, 32, 14, 14)), "p2": np.zeros((b, 1568)),
             "u": np.zeros((b, HID)), "dh": np.zeros((b, HID)), "code2": np.zeros((b, 1568), dtype=np.int32),
             "on": np.zeros((b, HID), dtype=np.int32)}
        flip = np.zeros((b, HID), dtype=np.uint8)
        for i, j in (flips or []):
            flip[int(i), int(j)] = 1
        dstruct = _Diag(*[d[n].ctypes.data for n, _ in _Diag._fields_ if n != "flip"], flip.ctypes.data if flips else None)
    rc = lib().oracle_grad_step_f64_diag(_ptr(theta), _ptr(x), _ptr(y), b, _ptr(keep), float(drop_p), int(precision),
                                         _ptr(grad), _ptr(loss), _ptr(am), _ptr(logits),
                                         C.addressof(dstruct) if diag else None)
    if rc != 0:
        raise ValueError("oracle_grad_step_f64: bad argument")
    if diag:
        return grad, float(loss[0]), am, logits, d
    return grad, float(loss[0]), am, logits


def worker_grad_step_diag(theta32, worker_id, x, y, seed, step, drop_p=0.25, precision=0, flips=None):
    """One worker of workers_grad_step (fp32 snapshot and images widened to double, Philox keep mask of
    (seed, worker_id, step)) with the intermediates of grad_step_f64(diag=True)."""
    y = np.ascontiguousarray(y, dtype=np.int32)
    keep = dropout_keep(seed, worker_id, step, y.shape[0], drop_p) if drop_p > 0 else None
    return grad_step_f64(np.asarray(theta32, dtype=np.float32).astype(np.float64),
                         np.asarray(x, dtype=np.float32).astype(np.float64), y, keep, drop_p, precision, diag=True,
                         flips=flips)


def workers_grad_step(thetas, worker_ids, x, y, seed, step, drop_p=0.25, precision=0):
    """W workers with fp32 snapshots.  thetas: list of W float32 arrays [P] (may repeat).
    x [W,b,28,28] float32, y [W,b] int32.  Returns (grads[W,P] f64, loss[W] f64,
    argmax[W,b] i32, logits[W,b,10] f64)."""
    W = len(thetas)
    x = np.ascontiguousarray(x, dtype=np.float32)
    y = np.ascontiguousarray(y, dtype=np.int32)
    b = y.shape[1]
    assert x.shape[0] == W and y.shape[0] == W and x.size == W * b * IMG * IMG
    keepalive = [np.ascontiguousarray(t, dtype=np.float32) for t in thetas]
    for t in keepalive:
        assert t.shape == (P,)
    ptrs = (C.c_void_p * W)(*[t.ctypes.data for t in keepalive])
    wid = np.ascontiguousarray(worker_ids, dtype=np.int32)
    grads = np.zeros((W, P), dtype=np.float64)
    loss = np.zeros(W, dtype=np.float64)
    am = np.zeros((W, b), dtype=np.int32)
    logits = np.zeros((W, b, NCLS), dtype=np.float64)
    rc = lib().oracle_workers_grad_step(W, b, C.cast(ptrs, C.c_void_p), _ptr(wid), _ptr(x), _ptr(y),
                                        int(seed), int(step), float(drop_p), int(precision), _ptr(grads), _ptr(loss),
                                        _ptr(am), _ptr(logits))
    if rc != 0:
        raise ValueError("oracle_workers_grad_step: bad argument")
    return grads, loss, am, logits


def workers_eval(thetas, x, y, precision=0):
    """Evaluation pass (the paper's metric exporter: accuracy and loss while training): the forward pass of
    workers_grad_step without dropout (every unit kept, no rescaling).  Returns (loss[W] f64, argmax[W,b] i32,
    correct[W] i64 = samples whose argmax equals the label, logits[W,b,10] f64).  The gradient the C routine also
    computes is not returned."""
    W = len(thetas)
    _, loss, am, logits = workers_grad_step(thetas, list(range(W)), x, y, 0, 0, drop_p=0.0, precision=precision)
    correct = (am == np.asarray(y, dtype=np.int32)).sum(axis=1)
    return loss, am, correct, logits


def round_operand(v, precision):
    return float(lib().oracle_round_operand(float(v), int(precision)))


def num_threads():
    return int(lib().oracle_num_threads())
