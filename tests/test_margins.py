"""CPU checks of the decision-margin rule (tests/margins.py) and of the unit-flip explanation used by the
tensor-core parity tests.  Mistakes are planted on the CPU, in copies of the oracle's own results."""
import numpy as np
import pytest

from oracle import cnn
from paper_2406_05546_b200 import synth
from tests import margins
from tests.parity import assert_params_close_up_to_unit_flips

OFF_F1W, OFF_F1B = 4800, 807616


def _case(seed, b):
    rng = np.random.default_rng(seed)
    theta = synth.init_params(1, bias_scale=0.05)
    x = rng.random((b, 28, 28), dtype=np.float32)
    y = rng.integers(0, 10, (b,)).astype(np.int32)
    return theta, x, y


@pytest.mark.parametrize("seed,b", [(0, 8), (1, 16)])
def test_rounded_operands_change_decisions_only_inside_the_margin_bound(seed, b):
    """The oracle's own reduced-precision decision pass (BF16 operands in the second convolution, TF32 in the
    512-unit layer) may differ from the exact decisions only where the exact margin is below the stated bound;
    and it does differ somewhere, so the statement is not empty."""
    theta, x, y = _case(seed, b)
    g0, _, _, _, d0 = cnn.worker_grad_step_diag(theta, 0, x, y, 5, 7, 0.25, precision=0)
    g2, _, _, _, d2 = cnn.worker_grad_step_diag(theta, 0, x, y, 5, 7, 0.25, precision=2)
    m = margins.decision_margins(theta, d0)
    pool_diff = d0["code2"] != d2["code2"]
    relu_diff = d0["on"] != d2["on"]
    assert pool_diff.sum() > 0 and relu_diff.sum() > 0
    assert not (pool_diff & ~m["pool_uncertain"]).any()
    assert not (relu_diff & ~m["relu_uncertain"]).any()
    # the exact intermediates do not depend on which decisions were used afterwards
    assert (d0["a2"] == d2["a2"]).all() and (d0["p1"] == d2["p1"]).all()
    # margins are what they say: a live pooled value equals the exact winner, a dead one is zero
    live = d0["code2"] < 4
    assert (d0["p2"][live] > 0).all() and (d0["p2"][~live] == 0).all()


def test_margin_definitions_on_hand_made_windows():
    """pool_margin: distance to the runner-up or to zero, whichever is nearer; dead windows: distance of the
    largest element to zero.  Checked on a crafted a2 through the same code path."""
    b = 1
    diag = {"p1": np.zeros((b, 16, 14, 14)), "a2": np.full((b, 32, 14, 14), -1.0), "p2": np.zeros((b, 1568)),
            "u": np.zeros((b, 512))}
    diag["a2"][0, 0, 0:2, 0:2] = [[0.5, 0.2], [-3.0, 0.45]]       # live: runner-up 0.05 away
    diag["a2"][0, 0, 0:2, 2:4] = [[0.03, -2.0], [-3.0, -1.0]]     # live: zero 0.03 away
    diag["a2"][0, 0, 0:2, 4:6] = [[-0.25, -2.0], [-3.0, -1.0]]    # dead: largest is 0.25 below zero
    m = margins.decision_margins(np.zeros(cnn.P), diag)
    np.testing.assert_allclose(m["pool_margin"][0, :3], [0.05, 0.03, 0.25], atol=1e-15)
    assert (m["pool_bound"] == 0).all()                          # all-zero weights: nothing can move


def test_flip_explanation_accepts_real_flips_and_rejects_anything_else():
    theta, x, y = _case(3, 12)
    g, _, _, _, d = cnn.worker_grad_step_diag(theta, 0, x, y, 5, 7, 0.25, precision=0)
    m = margins.decision_margins(theta, d)
    # the uncertain (sample, unit) with the largest contribution, so that every planted change is well above the tolerance
    i, j = [int(v) for v in np.unravel_index(np.argmax(np.where(m["relu_uncertain"], np.abs(d["dh"]), 0)), d["dh"].shape)]

    def with_flip(i, j, base=None):
        out = (g if base is None else base).copy()
        sign = -1.0 if d["on"][i, j] else 1.0
        out[OFF_F1W + j * 1568:OFF_F1W + (j + 1) * 1568] += sign * d["dh"][i, j] * d["p2"][i]
        out[OFF_F1B + j] += sign * d["dh"][i, j]
        return out, sign

    got, sign = with_flip(i, j)
    found = assert_params_close_up_to_unit_flips(got, g, 2e-2, theta, d, "planted flip")
    assert found == [(j, [(i, int(sign))])]
    # the same flip in a sample whose pre-activation is far from zero is not admissible
    far = np.where(~m["relu_uncertain"].any(axis=0)[None, :], np.abs(d["dh"]), 0)
    i2, j2 = [int(v) for v in np.unravel_index(np.argmax(far), far.shape)]
    bad, _ = with_flip(i2, j2)
    assert np.abs(bad - g).max() > 2e-2 * np.abs(g[OFF_F1W:OFF_F1B]).max()
    with pytest.raises(AssertionError, match="no sample has it near zero"):
        assert_params_close_up_to_unit_flips(bad, g, 2e-2, theta, d, "flip far from zero")
    # a corrupted row of an uncertain unit is not a flip
    junk = g.copy()
    junk[OFF_F1W + j * 1568:OFF_F1W + (j + 1) * 1568] += np.random.default_rng(0).normal(0, 0.1 * np.abs(g[OFF_F1W:OFF_F1B]).max(), 1568)
    with pytest.raises(AssertionError, match="explains the difference"):
        assert_params_close_up_to_unit_flips(junk, g, 2e-2, theta, d, "corrupted row")
    # half a contribution is not a flip either
    half = g.copy()
    half[OFF_F1W + j * 1568:OFF_F1W + (j + 1) * 1568] += 0.5 * d["dh"][i, j] * d["p2"][i]
    assert np.abs(half - g).max() > 2e-2 * np.abs(g[OFF_F1W:OFF_F1B]).max()
    with pytest.raises(AssertionError):
        assert_params_close_up_to_unit_flips(half, g, 2e-2, theta, d, "half a flip")
    # and an error in another tensor still fails
    other = got.copy()
    other[160] += 1.0
    with pytest.raises(AssertionError, match="conv2.w"):
        assert_params_close_up_to_unit_flips(other, g, 2e-2, theta, d, "other tensor")
