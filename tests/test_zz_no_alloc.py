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


def _oracle_replay(theta, grads, lr):
    """The definition: theta - lr / K * (sum of the gradients in double), rounded once (oracle/ps.py, REPLAY with
    one enqueue call of K gradients)."""
    from oracle import ps as ops
    K = grads.shape[0]
    o = ops.OraclePS(theta, external_store=True)
    o.enqueue(grads, range(K), [0] * K, 0)
    assert o.apply(ops.REPLAY, lr)["applied"] == K
    return o.head()


def test_static_replay_matches_context_replay_twice_in_a_row():
    """Calls in a row on the one shared scratch array: a long queue, then shorter ones with other data (stale partial
    sums of an earlier call would show), among them K = 2 and K = 5, which leave some of the array's four ranges
    empty; one call in place (output buffer = input buffer) and one on a side stream.  Every result is compared
    with the context-based replay (the existing entry point) and with the CPU oracle.  From the second call on the
    device's free memory must not move: nothing is allocated."""
    import torch
    from paper_2406_05546_b200 import ps
    from tests.parity import assert_params_close
    theta = synth.init_params(seed=1, bias_scale=0.05)
    theta_pad = np.zeros(ps.P_PAD, dtype=np.float32)
    theta_pad[:ps.P] = theta
    lr = 0.01
    side = torch.cuda.Stream()
    cases = [(300, 41, "plain"), (37, 42, "plain"), (2, 43, "plain"), (5, 44, "in place"), (64, 45, "side stream")]
    inputs = []
    for K, seed, how in cases:          # every buffer exists before the calls whose memory use is watched
        g = np.zeros((K, ps.P_PAD), dtype=np.float32)
        g[:, :ps.P] = synth.random_gradients(K, seed=seed)
        inputs.append((g, torch.from_numpy(g).cuda(), torch.from_numpy(theta_pad).cuda(),
                       torch.full((ps.P_PAD,), float("nan"), device="cuda")))
    torch.cuda.synchronize()
    free_after_first = None
    for (K, seed, how), (g, gd, tin, tout) in zip(cases, inputs):
        coef = float(np.float32(lr) / np.float32(K))
        if how == "in place":
            ps.ps_replay_sum_static(gd, tin, tin, coef)
            out = tin
        elif how == "side stream":
            side.wait_stream(torch.cuda.current_stream())
            ps.ps_replay_sum_static(gd, tin, tout, coef, stream=side)
            side.synchronize()
            out = tout
        else:
            ps.ps_replay_sum_static(gd, tin, tout, coef)
            out = tout
        torch.cuda.synchronize()
        free_now = torch.cuda.mem_get_info()[0]
        if free_after_first is None:
            free_after_first = free_now          # the first call on a device sets the array up
        else:
            assert free_now == free_after_first, "a later call changed the device's free memory"
        got = out.cpu().numpy()
        assert (got[ps.P:] == 0).all()
        for name, want in (("context replay", _existing_path(theta, gd, lr)), ("oracle", _oracle_replay(theta, g[:, :ps.P], lr))):
            assert_params_close(got[:ps.P], want, TOL, f"static replay vs {name}, K={K}, {how}")
            step_w = want.astype(np.float64) - theta
            step_g = got[:ps.P].astype(np.float64) - theta
            assert np.abs(step_g - step_w).max() <= 2e-3 * np.abs(step_w).max(), (name, K, how)
        free_after_first = torch.cuda.mem_get_info()[0]      # the comparison paths above allocate through torch


def test_static_replay_rejects_sizes_beyond_the_maximum():
    import torch
    from paper_2406_05546_b200 import ps
    L = ps.load()
    t = torch.zeros(ps.P_PAD, device="cuda")
    for K in (0, 65537):
        rc = L.ps_replay_sum_static(t.data_ptr(), K, t.data_ptr(), t.data_ptr(), 0.0, None)
        assert rc == -1 and b"65536" in L.ps_replay_sum_static_error()
    assert L.ps_replay_sum_static(None, 1, t.data_ptr(), t.data_ptr(), 0.0, None) == -1
