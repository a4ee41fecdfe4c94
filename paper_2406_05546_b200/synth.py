"""Seeded synthetic inputs shared by the CUDA tests, the oracle tests and the benchmark.

This module holds none of the method's arithmetic: only random images, labels,
initial weights, worker lags and arrival orders, all drawn from numpy's PCG64
generator with the seeds stated below.  The images stand in for FashionMNIST
(1x28x28 grey images, 10 classes, a 60,000-image training pool), which the
paper trains on and which is not available offline.
"""
import numpy as np

P = 813258
IMG = 28
POOL_IMAGES = 60000

# (name, offset, shape, fan_in) in the canonical flat order
_LAYOUT = [
    ("conv1.w", 0, (16, 1, 3, 3), 9),
    ("conv1.b", 144, (16,), 0),
    ("conv2.w", 160, (32, 16, 3, 3), 144),
    ("conv2.b", 4768, (32,), 0),
    ("fc1.w", 4800, (512, 1568), 1568),
    ("fc1.b", 807616, (512,), 0),
    ("fc2.w", 808128, (10, 512), 512),
    ("fc2.b", 813248, (10,), 0),
]


def layout():
    """[(name, offset, shape)] of the eight parameter tensors."""
    return [(n, o, s) for n, o, s, _ in _LAYOUT]


def init_params(seed: int = 1, bias_scale: float = 0.0) -> np.ndarray:
    """Kaiming-uniform weights U(-sqrt(6/fan_in), +sqrt(6/fan_in)); biases zero
    (or U(-bias_scale, bias_scale) when bias_scale > 0, used by tests that want
    every parameter to matter)."""
    rng = np.random.Generator(np.random.PCG64(seed))
    theta = np.zeros(P, dtype=np.float32)
    for _, off, shape, fan_in in _LAYOUT:
        n = int(np.prod(shape))
        if fan_in > 0:
            lim = np.sqrt(6.0 / fan_in)
            theta[off:off + n] = rng.uniform(-lim, lim, size=n).astype(np.float32)
        elif bias_scale > 0:
            theta[off:off + n] = rng.uniform(-bias_scale, bias_scale, size=n).astype(np.float32)
    return theta


def image_pool(n: int = POOL_IMAGES, seed: int = 0):
    """n images with pixels i.i.d. U[0,1) (float32) and labels uniform over 10 classes."""
    rng = np.random.Generator(np.random.PCG64(seed))
    x = rng.random((n, IMG, IMG), dtype=np.float32)
    y = rng.integers(0, 10, size=n, dtype=np.int32)
    return x, y


def batch_rows(tick: int, W: int, b: int, n_pool: int) -> np.ndarray:
    """Pool rows of the batch of every worker at a tick: ((tick*W + w)*b + i) mod n_pool, shape [W,b]."""
    w = np.arange(W, dtype=np.int64)[:, None]
    i = np.arange(b, dtype=np.int64)[None, :]
    return ((tick * W + w) * b + i) % n_pool


def tick_batch(pool_x, pool_y, tick: int, W: int, b: int):
    rows = batch_rows(tick, W, b, pool_x.shape[0])
    return np.ascontiguousarray(pool_x[rows]), np.ascontiguousarray(pool_y[rows])


def lags(tick: int, W: int, max_lag: int = 8, seed: int = 2) -> np.ndarray:
    """Per-worker version lag, uniform over 0..max_lag, keyed by (seed, tick)."""
    rng = np.random.Generator(np.random.PCG64([seed, tick]))
    return rng.integers(0, max_lag + 1, size=W, dtype=np.int32)


def arrival_order(tick: int, W: int, seed: int = 3) -> np.ndarray:
    """Permutation of the W workers giving the order in which their gradients reach the server."""
    rng = np.random.Generator(np.random.PCG64([seed, tick]))
    return rng.permutation(W).astype(np.int32)


def random_gradients(K: int, seed: int = 4, scale: float = 1e-2) -> np.ndarray:
    """K synthetic fp32 'gradients' [K,P] ~ N(0, scale^2) for server-side tests that need no CNN."""
    rng = np.random.Generator(np.random.PCG64(seed))
    return (rng.standard_normal((K, P), dtype=np.float32) * np.float32(scale)).astype(np.float32)
