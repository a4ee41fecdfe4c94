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


def test_a_forced_decision_changes_exactly_what_a_flip_changes():
    """The oracle's decision override (used to ask for the exact gradient under the other, equally valid choice at a
    unit near zero): the unit's row of fc1.w moves by the sample's contribution dh * p2 and its fc1.b entry by dh, no
    other row of the layer moves, the output layer's gradient moves only through the forward value (which a unit near
    zero barely changes), overriding twice is the identity, and the result is what torch's autograd gives when the
    unit's ReLU is replaced by the identity (switched on) or by zero (switched off)."""
    import torch
    theta, x, y = _case(4, 6)
    g, loss, _, _, d = cnn.worker_grad_step_diag(theta, 0, x, y, 5, 7, 0.25, precision=0)
    m = margins.decision_margins(theta, d)
    i, j = [int(v) for v in np.unravel_index(np.argmax(np.where(m["relu_uncertain"], np.abs(d["dh"]), 0)), d["dh"].shape)]
    g1, _, _, _, d1 = cnn.worker_grad_step_diag(theta, 0, x, y, 5, 7, 0.25, precision=0, flips=[(i, j)])
    assert d1["on"][i, j] != d["on"][i, j] and (np.delete(d1["on"].ravel(), i * 512 + j) == np.delete(d["on"].ravel(), i * 512 + j)).all()
    dw = (g1 - g)[OFF_F1W:OFF_F1B].reshape(512, 1568)
    sign = -1.0 if d["on"][i, j] else 1.0
    # the contribution that appears or disappears is the one of the pass in which the unit is on (the forward pass, and
    # with it dh, differs between the two passes by what u[i, j], a value near zero, does to the logits)
    dh_on = d["dh"][i, j] if d["on"][i, j] else d1["dh"][i, j]
    assert np.abs(dw[j] - sign * dh_on * d["p2"][i]).max() <= 1e-9 * np.abs(dw[j]).max() + 1e-15
    assert np.abs(np.delete(dw, j, axis=0)).max() <= 1e-2 * np.abs(dw[j]).max()
    assert abs((g1 - g)[OFF_F1B + j] - sign * dh_on) <= 1e-9 * abs(dh_on) + 1e-15
    g2 = cnn.worker_grad_step_diag(theta, 0, x, y, 5, 7, 0.25, precision=0, flips=[(i, j), (i, j)])[0]
    assert np.array_equal(g2, g1)                   # the list marks units; marking one twice is marking it once
    # torch: the same graph with that one unit's ReLU replaced
    t = torch.tensor(theta.astype(np.float64), requires_grad=True)
    seg = lambda name: t[cnn.TENSORS[name][0]:cnn.TENSORS[name][0] + int(np.prod(cnn.TENSORS[name][1]))].reshape(cnn.TENSORS[name][1])
    F = torch.nn.functional
    keep = torch.tensor(cnn.dropout_keep(5, 0, 7, 6, 0.25).astype(np.float64))
    h = torch.tensor(x.astype(np.float64)).reshape(6, 1, 28, 28)
    h = F.max_pool2d(F.relu(F.conv2d(h, seg("conv1.w"), seg("conv1.b"), padding=1)), 2)
    h = F.max_pool2d(F.relu(F.conv2d(h, seg("conv2.w"), seg("conv2.b"), padding=1)), 2)
    u = F.linear(h.flatten(1), seg("fc1.w"), seg("fc1.b"))
    gate = (u > 0).to(u.dtype).detach()
    gate[i, j] = 1.0 - gate[i, j]
    z = F.linear(u * gate * keep / 0.75, seg("fc2.w"), seg("fc2.b"))
    F.cross_entropy(z, torch.tensor(y.astype(np.int64))).backward()
    assert np.abs(t.grad.numpy() - g1).max() <= 1e-11
