"""The allocation-free reduce-and-apply entry point against the context-based replay.

ps_replay_sum_static serves callers that cannot allocate device memory when they call (their
application's pool owns the GPU, or an allocation's device-wide stall is not acceptable); its
partial sums live in a fixed array inside the library.  This file is named to be collected last,
so that a run stopping at the first failure has already run every other test.  It passes on its
own in a fresh process and after the rest of the suite.
"""
import numpy as np
import pytest

from paper_2406_05546_b200 import synth

pytestmark = pytest.mark.gpu

TOL = 1e-6      # same bound as the other server-side parity tests: relative to the tensor's max-abs


def _existing_path(theta, grads_dev, lr):
    """The context-based replay of the same queue (one enqueue call of K gradients, so the divisor is K)."""
    from paper_2406_05546_b200 import ps
    K = grads_dev.shape[0]
    srv = ps.ParameterServer(theta, max_workers=1, max_batch=1, queue_slots=K, external_store=True)
    # the enqueue call carries K gradients; max_workers only bounds the grad step, not the queue
    srv.ps_enqueue(list(range(K)), [0] * K, 0, grads_dev=grads_dev)
    res = srv.ps_apply(ps.REPLAY, lr)
    assert res["applied"] == K
    out = srv.ps_export_params()[0]
    srv.close()
    return out


def test_static_replay_matches_context_replay_twice_in_a_row():
    import torch
    from paper_2406_05546_b200 import ps
    from tests.parity import assert_params_close
    theta = synth.init_params(seed=1, bias_scale=0.05)
    theta_pad = np.zeros(ps.P_PAD, dtype=np.float32)
    theta_pad[:ps.P] = theta
    lr = 0.01
    # second call: shorter queue with different data, so stale partial sums from the first would show
    for K, seed in [(300, 41), (37, 42)]:
        g = np.zeros((K, ps.P_PAD), dtype=np.float32)
        g[:, :ps.P] = synth.random_gradients(K, seed=seed)
        gd = torch.from_numpy(g).cuda()
        tin = torch.from_numpy(theta_pad).cuda()
        tout = torch.full((ps.P_PAD,), float("nan"), device="cuda")
        coef = float(np.float32(lr) / np.float32(K))
        ps.ps_replay_sum_static(gd, tin, tout, coef)
        torch.cuda.synchronize()
        got = tout.cpu().numpy()
        want = _existing_path(theta, gd, lr)
        assert_params_close(got[:ps.P], want, TOL, f"static replay, K={K}")
        assert (got[ps.P:] == 0).all()
        step_w = want.astype(np.float64) - theta
        step_g = got[:ps.P].astype(np.float64) - theta
        assert np.abs(step_g - step_w).max() <= 2e-3 * np.abs(step_w).max()


def test_static_replay_rejects_sizes_beyond_the_maximum():
    import torch
    from paper_2406_05546_b200 import ps
    L = ps.load()
    t = torch.zeros(ps.P_PAD, device="cuda")
    for K in (0, 65537):
        rc = L.ps_replay_sum_static(t.data_ptr(), K, t.data_ptr(), t.data_ptr(), 0.0, None)
        assert rc == -1 and b"65536" in L.ps_replay_sum_static_error()
    assert L.ps_replay_sum_static(None, 1, t.data_ptr(), t.data_ptr(), 0.0, None) == -1
