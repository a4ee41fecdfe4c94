"""Comparison helpers shared by the GPU parity tests (no method arithmetic)."""
import numpy as np

from paper_2406_05546_b200 import synth

TOL_FP32 = 1e-4     # max error relative to the tensor's max-abs, FP32 path (stated target)
TOL_TENSOR = 2e-2   # same, tensor-core path (BF16 products in the convolutions, TF32 in the 512-unit layer)


def tensor_rel_errors(got, ref):
    """Per parameter tensor: max|got-ref| / max|ref| (both flat [P] arrays)."""
    out = {}
    for name, off, shape in synth.layout():
        n = int(np.prod(shape))
        r = np.asarray(ref[off:off + n], dtype=np.float64)
        g = np.asarray(got[off:off + n], dtype=np.float64)
        denom = np.abs(r).max()
        err = np.abs(g - r).max()
        out[name] = err / denom if denom > 0 else err
    return out


def assert_params_close(got, ref, tol, what=""):
    errs = tensor_rel_errors(got, ref)
    bad = {k: v for k, v in errs.items() if not v <= tol}
    assert not bad, f"{what}: relative error above {tol}: {bad} (all: {errs})"
    return errs


def assert_sum_close(got, parts, tol, what=""):
    """got [P] against the sum of parts [W, P] (one gradient per worker): each worker's gradient is allowed tol times its
    own tensor's max-abs, so their sum is allowed the sum of those allowances (the workers' errors add at worst), which is
    what is checked per tensor.  Returns the errors relative to the SUM's max-abs, for the record."""
    parts = np.asarray(parts, dtype=np.float64)
    ref = parts.sum(axis=0)
    errs, bad = {}, {}
    for name, off, shape in synth.layout():
        n = int(np.prod(shape))
        err = np.abs(np.asarray(got[off:off + n], dtype=np.float64) - ref[off:off + n]).max()
        allowed = tol * np.abs(parts[:, off:off + n]).max(axis=1).sum()
        errs[name] = err / max(np.abs(ref[off:off + n]).max(), 1e-300)
        if not err <= allowed:
            bad[name] = (err, allowed)
    assert not bad, f"{what}: error above the summed allowance: {bad} (relative to the sum: {errs})"
    return errs


def assert_params_close_up_to_unit_flips(got, ref, tol, theta, diag, what="", recompute=None):
    """As assert_params_close, except that ReLU decisions of the 512-unit layer that sit within rounding distance of
    zero may have come out the other way.  What is admitted, and checked:
    (1) a row of fc1.w (with its fc1.b entry) that is off must belong to a unit whose EXACT pre-activation lies within
        the operand-rounding bound of zero (tests/margins.py) in some sample, and
    (2) the row's difference must equal, within the tolerance, the signed sum of exactly such samples' contributions
        dh[i, j] * p2[i, :] (least squares over the candidate samples, coefficients rounded to -1 / 0 / +1);
    (3) with `recompute` (a function: list of (sample, unit) -> the oracle's gradient with those decisions taken the
        other way), EVERY tensor must then be within the tolerance of that recomputed gradient: a flip also moves the
        layers below through the back-propagated signal, visibly so at small batches.  Without `recompute` every other
        tensor must be within the tolerance of `ref` as it stands.
    `theta` are the worker's weights and `diag` the oracle's intermediates of the pass that produced `ref`.
    Returns the list of (unit, [(sample, sign), ...])."""
    from tests import margins
    errs = tensor_rel_errors(got, ref)
    lay = {name: (off, shape) for name, off, shape in synth.layout()}
    off_w, shape_w = lay["fc1.w"]
    off_b, _ = lay["fc1.b"]
    n = int(np.prod(shape_w))
    gw = np.asarray(got[off_w:off_w + n], dtype=np.float64).reshape(shape_w)
    rw = np.asarray(ref[off_w:off_w + n], dtype=np.float64).reshape(shape_w)
    gb = np.asarray(got[off_b:off_b + shape_w[0]], dtype=np.float64)
    rb = np.asarray(ref[off_b:off_b + shape_w[0]], dtype=np.float64)
    w_scale, b_scale = np.abs(rw).max(), np.abs(rb).max()
    unit_err = np.maximum(np.abs(gw - rw).max(axis=1) / w_scale, np.abs(gb - rb) / b_scale)
    flagged = np.where(unit_err > tol)[0]
    explained = []
    if flagged.size:
        m = margins.decision_margins(theta, diag)
        for j in flagged:
            cand = np.where(m["relu_uncertain"][:, j])[0]
            assert cand.size, f"{what}: hidden unit {j} is off by {unit_err[j]:.2e} and no sample has it near zero"
            contrib = margins.unit_contributions(diag, j)
            # bias column rescaled so that one absolute tolerance serves the whole row
            k = w_scale / b_scale
            contrib[:, -1] *= k
            diff = np.concatenate([gw[j] - rw[j], [(gb[j] - rb[j]) * k]])
            flips = margins.explain_row_by_flips(diff, contrib, cand, tol * w_scale)
            assert flips, (f"{what}: hidden unit {j} is off by {unit_err[j]:.2e} and no set of near-zero samples "
                           f"({cand.tolist()}) explains the difference of its row")
            explained.append((int(j), flips))
    if explained and recompute is not None:
        new_ref = recompute([(i, j) for j, fl in explained for i, _ in fl])
        assert_params_close(got, new_ref, tol, what + ", against the gradient under the decisions it took")
        return explained
    bad = {k: v for k, v in errs.items() if not v <= tol and k not in ("fc1.w", "fc1.b")}
    assert not bad, f"{what}: relative error above {tol}: {bad} (all: {errs})"
    return explained


def assert_argmax_valid(got, ref_logits, tol):
    """Labels must equal the oracle's wherever its top-2 margin exceeds tol*max|logit|; elsewhere
    the chosen class must be one of the near-maximal ones.  Returns the number of ambiguous rows."""
    z = np.asarray(ref_logits, dtype=np.float64).reshape(-1, 10)
    got = np.asarray(got).reshape(-1)
    top = np.sort(z, axis=1)
    margin = top[:, -1] - top[:, -2]
    slack = tol * np.abs(z).max(axis=1)
    clear = margin > slack
    ref = z.argmax(axis=1)
    assert (got[clear] == ref[clear]).all(), "argmax differs where the oracle's margin is clear"
    amb = np.where(~clear)[0]
    for r in amb:
        assert z[r, got[r]] >= top[r, -1] - slack[r]
    return int(amb.size)
