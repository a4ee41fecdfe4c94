"""How far the exact pass's integer decisions are from flipping, and how far operand rounding can move them.

Used by the tests that compare the tensor-core path with the plain definition (decisions taken on exact
values): a reduced-precision product can only decide differently where the exact margin of the decision is
smaller than the error its rounded operands can cause.  Everything here is computed from the oracle's own
intermediates (oracle.cnn.grad_step_f64(diag=True)); nothing comes from the CUDA path.

Bounds (u = unit roundoff of one operand; a product of two rounded operands is off by at most about 2u):
  second convolution, BF16 operands (8 significant bits, u = 2^-9):  |error of a sum| <= 2^-8 * sum |w * p|
  512-unit layer, TF32 operands (11 significant bits, u = 2^-12 .. 2^-11): <= 2^-10 * sum |W * p2|, plus what the
      second convolution's error does to p2.  Summing the latter's worst cases over 1568 inputs would flag every
      unit, so it enters as four times the root of the sum of squares (independent rounding errors), which the
      CPU pins check against the decisions the oracle itself takes on rounded operands.
"""
import numpy as np
import torch

EPS_CONV_BF16 = 2.0 ** -8
EPS_DENSE_TF32 = 2.0 ** -10
RSS_FACTOR = 4.0


def decision_margins(theta, diag):
    """theta [P] (float64 or float32), diag from the exact pass of one worker.  Returns a dict:
    pool_margin, pool_bound [b,1568]; relu_margin, relu_bound [b,512]; pool_uncertain, relu_uncertain (bool)."""
    th = np.asarray(theta, dtype=np.float64)
    w2 = torch.from_numpy(th[160:4768].reshape(32, 16, 3, 3))
    W1 = th[4800:807616].reshape(512, 1568)
    p1 = torch.from_numpy(diag["p1"])
    a2 = diag["a2"]
    b = a2.shape[0]
    # sum |w| * |p| behind every pre-activation of the second convolution
    A2 = torch.nn.functional.conv2d(p1.abs(), w2.abs(), padding=1).numpy()
    win = a2.reshape(b, 32, 7, 2, 7, 2).transpose(0, 1, 2, 4, 3, 5).reshape(b, 32, 7, 7, 4)
    Aw = A2.reshape(b, 32, 7, 2, 7, 2).transpose(0, 1, 2, 4, 3, 5).reshape(b, 32, 7, 7, 4)
    srt = np.sort(win, axis=-1)
    best, second = srt[..., 3], srt[..., 2]
    live = best > 0
    pool_margin = np.where(live, np.minimum(best - second, best), -best).reshape(b, 1568)
    pool_bound = (2.0 * EPS_CONV_BF16 * Aw.max(axis=-1)).reshape(b, 1568)      # two candidates, each off by its bound
    value_bound = (EPS_CONV_BF16 * Aw.max(axis=-1)).reshape(b, 1568)           # error of the pooled value itself
    p2 = diag["p2"]
    A1 = np.abs(p2) @ np.abs(W1).T
    prop = np.sqrt((value_bound ** 2) @ (W1.T ** 2))
    relu_margin = np.abs(diag["u"])
    relu_bound = EPS_DENSE_TF32 * A1 + RSS_FACTOR * prop
    return {"pool_margin": pool_margin, "pool_bound": pool_bound, "relu_margin": relu_margin,
            "relu_bound": relu_bound, "pool_uncertain": pool_margin <= pool_bound,
            "relu_uncertain": relu_margin <= relu_bound}


def unit_contributions(diag, j):
    """Rows of what sample i adds to row j of the 512-unit layer's weight gradient (and to its bias gradient, last
    column) when the unit is on: dh[i, j] * [p2[i, :], 1].  Shape [b, 1569]."""
    return diag["dh"][:, j:j + 1] * np.concatenate([diag["p2"], np.ones((diag["p2"].shape[0], 1))], axis=1)


def explain_row_by_flips(diff_row, contrib, candidates, tol_abs):
    """Is diff_row (got - ref for row j of fc1.w with the fc1.b entry appended) a signed sum of the contributions of
    some candidate samples (each flipped once: +1 switched on, -1 switched off) up to tol_abs?  Returns the list of
    (sample, sign) or None."""
    cand = list(candidates)
    if not cand:
        return None
    A = contrib[cand].T                                      # [1569, n]
    coef, *_ = np.linalg.lstsq(A, diff_row, rcond=None)
    signs = np.rint(coef)
    if np.any(np.abs(signs) > 1):
        return None
    resid = diff_row - A @ signs
    if np.abs(resid).max() > tol_abs:
        return None
    return [(cand[k], int(signs[k])) for k in range(len(cand)) if signs[k] != 0]
