"""GPU parity: server-side reduce/apply/replay, checkpoint rollback and chain mirror vs the oracle."""
import numpy as np
import pytest

from paper_2406_05546_b200 import synth
from tests.parity import assert_params_close

pytestmark = pytest.mark.gpu

# theta' = theta - c * sum(g): the oracle sums in double and rounds once; the kernel sums in fp32.
# With |g| ~ 1e-2 and c <= 1e-2 the difference is far below one part in 1e6 of max|theta|.
TOL_APPLY = 1e-6


def _pad(g):
    import torch
    from paper_2406_05546_b200 import ps
    out = np.zeros((g.shape[0], ps.P_PAD), dtype=np.float32)
    out[:, :ps.P] = g
    return torch.from_numpy(out).cuda()


def _pair(**kw):
    from oracle import ps as ops
    from paper_2406_05546_b200 import ps
    theta = synth.init_params(seed=1, bias_scale=0.05)
    okw = dict(kw)
    okw.pop("max_workers", None)
    gkw = dict(kw)
    gkw.setdefault("max_workers", 8)
    o = ops.OraclePS(theta, **okw)
    g = ps.ParameterServer(theta, max_batch=1, **gkw)
    return ops, ps, o, g


def _both_enqueue(o, g, grads, step=0, base=None):
    n = grads.shape[0]
    base = [o.version] * n if base is None else base
    o.enqueue(grads, range(n), base, step)
    g.ps_enqueue(list(range(n)), base, step, grads_dev=_pad(grads))


@pytest.mark.parametrize("K", [1, 7, 8, 37])
def test_sync_apply(K):
    ops, ps, o, g = _pair(queue_slots=64, max_workers=64)
    grads = synth.random_gradients(K, seed=K)
    _both_enqueue(o, g, grads)
    ro = o.apply(ops.SYNC, 0.01)
    rg = g.ps_apply(ps.SYNC, 0.01)
    assert ro == rg
    th, v = g.ps_export_params()
    assert v == o.version == 1
    assert_params_close(th, o.head(), TOL_APPLY, "sync")
    assert g.ps_stats()["queue_len"] == 0
    g.close()


def test_replay_long_queue_two_stage_sum_and_scale():
    ops, ps, o, g = _pair(queue_slots=400, external_store=True, max_workers=4)
    o.kill(); g.ps_kill()
    T, W = 75, 4          # K = 300: the split reduction path, with a ragged last split
    for t in range(T):
        _both_enqueue(o, g, synth.random_gradients(W, seed=1000 + t), step=t, base=[0] * W)
    assert g.ps_stats()["queue_len"] == T * W
    with pytest.raises(ps.PSError) as e:
        g.ps_apply(ps.REPLAY, 0.01)
    assert e.value.name == "PS_ERR_DOWN"
    assert o.restore() == g.ps_restore() == 0
    ro = o.apply(ops.REPLAY, 0.01, scale=0.5)
    rg = g.ps_apply(ps.REPLAY, 0.01, scale=0.5)
    assert ro == rg and rg["applied"] == T * W and rg["new_version"] == 1
    th, _ = g.ps_export_params()
    assert_params_close(th, o.head(), TOL_APPLY, "replay")
    # the update itself (theta' - theta), not just theta', must match: compare the step taken
    theta0 = synth.init_params(seed=1, bias_scale=0.05)
    step_o = o.head().astype(np.float64) - theta0
    step_g = th.astype(np.float64) - theta0
    assert np.abs(step_g - step_o).max() <= 1e-3 * np.abs(step_o).max()
    g.close()


def test_replay_zero_downtime_equals_sync_on_gpu():
    ops, ps, _, a = _pair(queue_slots=8, external_store=True)
    _, _, _, c = _pair(queue_slots=8)
    for t in range(3):
        grads = _pad(synth.random_gradients(5, seed=10 + t))
        a.ps_enqueue(range(5), [t] * 5, t, grads_dev=grads)
        c.ps_enqueue(range(5), [t] * 5, t, grads_dev=grads)
        a.ps_apply(ps.REPLAY, 0.01)
        c.ps_apply(ps.SYNC, 0.01)
    ta, va = a.ps_export_params()
    tc, vc = c.ps_export_params()
    assert va == vc == 3 and (ta == tc).all()
    a.close(); c.close()


def test_async_ordered_apply_ring_and_mirror():
    ops, ps, o, g = _pair(queue_slots=64, ring_depth=9, chain_len=2, replicate_every=1, max_workers=64)
    for tick in range(3):
        K = [20, 5, 64][tick]
        grads = synth.random_gradients(K, seed=30 + tick)
        order = synth.arrival_order(tick, K)
        _both_enqueue(o, g, grads, step=tick)
        ro = o.apply(ops.ASYNC, 0.01, order=order)
        rg = g.ps_apply(ps.ASYNC, 0.01, order=order)
        assert ro == rg
        st = g.ps_stats()
        assert st["version"] == o.version and st["oldest_version"] == o.oldest_version()
        assert st["replica_version"] == o.replicas[0]["version"] == o.version
        # every retained version matches the oracle's (the ring serves the stale readers)
        import torch
        for lag in range(min(9, o.version + 1)):
            s = g.ps_pull_snapshot(0, lag)
            v, th_o = o.pull_snapshot(0, lag)
            assert s.version == v
            off = s.dev_ptr - g.arena.data_ptr()
            th_g = g.arena[off:off + ps.P * 4].view(torch.float32).cpu().numpy()
            assert_params_close(th_g, th_o, TOL_APPLY, f"version {v}")
        head, _ = g.ps_export_params(0)
        rep, rv = g.ps_export_params(-1)
        assert rv == o.version and (rep == head).all()        # mirror is bit-identical to the head
    with pytest.raises(ps.PSError) as e:
        g.ps_pull_snapshot(0, 9)
    assert e.value.name == "PS_ERR_VERSION_EVICTED"
    g.close()


def test_async_equals_sequential_single_updates_bit_for_bit():
    ops, ps, _, a = _pair(queue_slots=16, ring_depth=4, max_workers=16)
    _, _, _, c = _pair(queue_slots=16, ring_depth=1, max_workers=16)
    grads = synth.random_gradients(11, seed=3)
    order = synth.arrival_order(0, 11)
    a.ps_enqueue(range(11), [0] * 11, 0, grads_dev=_pad(grads))
    a.ps_apply(ps.ASYNC, 0.01, order=order)
    for k in order:
        c.ps_enqueue([0], [0], 0, grads_dev=_pad(grads[k:k + 1]))
        c.ps_apply(ps.ASYNC, 0.01)
    ta, va = a.ps_export_params()
    tc, vc = c.ps_export_params()
    assert va == vc == 11 and (ta == tc).all()
    a.close(); c.close()


def test_periodic_replication_and_failover():
    ops, ps, o, g = _pair(queue_slots=8, ring_depth=9, chain_len=2, replicate_every=3)
    for tick in range(4):
        grads = synth.random_gradients(4, seed=20 + tick)
        order = synth.arrival_order(tick, 4)
        _both_enqueue(o, g, grads, step=tick)
        assert o.apply(ops.ASYNC, 0.01, order=order) == g.ps_apply(ps.ASYNC, 0.01, order=order)
        assert g.ps_stats()["replica_version"] == o.replicas[0]["version"] == (o.version // 3) * 3
    rep_o = o.replicas[0]["theta"].copy()
    o.kill(); g.ps_kill()
    with pytest.raises(ps.PSError) as e:
        g.ps_pull_snapshot(0)
    assert e.value.name == "PS_ERR_DOWN"
    assert o.failover() == g.ps_failover() == 15
    th, v = g.ps_export_params()
    assert v == 15
    assert_params_close(th, rep_o, TOL_APPLY, "failover weights")
    st = g.ps_stats()
    assert st["version"] == st["oldest_version"] == 15 and st["live_replicas"] == 0 and st["up"] == 1
    # training continues on the new frontend, without a replica
    grads = synth.random_gradients(2, seed=99)
    _both_enqueue(o, g, grads, step=5)
    assert o.apply(ops.ASYNC, 0.01) == g.ps_apply(ps.ASYNC, 0.01)
    assert_params_close(g.ps_export_params()[0], o.head(), TOL_APPLY, "after failover")
    g.ps_kill()
    with pytest.raises(ps.PSError) as e:
        g.ps_failover()
    assert e.value.name == "PS_ERR_NO_REPLICA"
    g.close()


def test_explicit_replicate_and_sync_mirror():
    ops, ps, o, g = _pair(queue_slots=8, chain_len=2, replicate_every=2)
    for t in range(3):
        _both_enqueue(o, g, synth.random_gradients(3, seed=t), step=t)
        assert o.apply(ops.SYNC, 0.01) == g.ps_apply(ps.SYNC, 0.01)
    assert g.ps_stats()["replica_version"] == 2
    assert g.ps_replicate() == o.replicate() == 3
    head, _ = g.ps_export_params(0)
    rep, rv = g.ps_export_params(-1)
    assert rv == 3 and (head == rep).all()
    g.close()


def test_checkpoint_rollback_schedule_config2_shape():
    # checkpoint every 25 updates, kill before tick 60, 20 idle ticks, restore -> version 50, end 170
    ops, ps, o, g = _pair(queue_slots=4, ckpt_every=25, ckpt_slots=8)
    ck = []
    at50 = None
    for tick in range(200):
        if tick == 60:
            o.kill(); g.ps_kill()
        if 60 <= tick < 80:
            for fn in (lambda: g.ps_pull_snapshot(0), lambda: g.ps_apply(ps.SYNC, 0.01), lambda: g.ps_queue_reserve(1)):
                with pytest.raises(ps.PSError) as e:
                    fn()
                assert e.value.name == "PS_ERR_DOWN"
            continue
        if tick == 80:
            assert o.restore() == g.ps_restore() == 50
            th, v = g.ps_export_params()
            assert v == 50 and (th == at50).all()          # the rollback reproduces the checkpoint bytes
            st = g.ps_stats()
            assert st["queue_len"] == 0 and st["oldest_version"] == 50
        grads = synth.random_gradients(2, seed=100 + tick)
        _both_enqueue(o, g, grads, step=tick)
        ro, rg = o.apply(ops.SYNC, 0.01), g.ps_apply(ps.SYNC, 0.01)
        assert ro == rg
        if rg["checkpointed"]:
            ck.append(rg["new_version"])
            th_c, v_c = g.ps_export_params(1000)
            assert v_c == rg["new_version"] and (th_c == g.ps_export_params()[0]).all()
        if rg["new_version"] == 50 and at50 is None:
            at50 = g.ps_export_params()[0]
    assert ck == [25, 50, 75, 100, 125, 150]
    st = g.ps_stats()
    assert st["version"] == o.version == 170 and st["last_ckpt_version"] == 150
    assert_params_close(g.ps_export_params()[0], o.head(), 1e-5, "after 170 updates")
    g.close()


def test_async_checkpoint_mid_apply_and_errors():
    ops, ps, o, g = _pair(queue_slots=8, ring_depth=2, ckpt_every=4, ckpt_slots=2)
    with pytest.raises(ps.PSError) as e:
        g.ps_restore()
    assert e.value.name == "PS_ERR_NO_CHECKPOINT"
    grads = synth.random_gradients(6, seed=8)
    _both_enqueue(o, g, grads)
    assert o.apply(ops.ASYNC, 0.01) == g.ps_apply(ps.ASYNC, 0.01)
    th_c, v_c = g.ps_export_params(1000)
    assert v_c == 4
    assert_params_close(th_c, o.ckpts[-1][1], TOL_APPLY, "mid-apply checkpoint")
    with pytest.raises(ps.PSError) as e:
        g.ps_enqueue(range(8), [0] * 8, 0, grads_dev=_pad(synth.random_gradients(8)))
        g.ps_enqueue(range(8), [0] * 8, 0, grads_dev=_pad(synth.random_gradients(8)))
    assert e.value.name == "PS_ERR_QUEUE_FULL"
    with pytest.raises(ps.PSError) as e:
        g.ps_apply(ps.ASYNC, 0.01, order=[0, 0, 1, 2, 3, 4, 5, 6])
    assert e.value.name == "PS_ERR_BAD_ARG"
    g.close()


def _steps(o, g, ops, ps, n, seed0, W=2, mode=None):
    for t in range(n):
        _both_enqueue(o, g, synth.random_gradients(W, seed=seed0 + t), step=t)
        assert o.apply(ops.SYNC if mode is None else mode, 0.01) == g.ps_apply(ps.SYNC if mode is None else mode, 0.01)


def _chain_matches(o, g, what):
    live = [r for r in o.replicas if r["alive"]]
    assert g.ps_stats()["live_replicas"] == len(live)
    for i, r in enumerate(live):
        th, v = g.ps_export_params(-(i + 1))
        assert v == r["version"], (what, i)
        assert_params_close(th, r["theta"], TOL_APPLY, f"{what}: server {i + 1} behind the frontend")


def test_chain_of_three_double_failure():
    """Frontend and secondary die; the tertiary, one replication event behind, takes over (design section on chain
    replication).  Sync and async applies, R = 2."""
    for mode_name in ("SYNC", "ASYNC"):
        ops, ps, o, g = _pair(queue_slots=8, ring_depth=4, chain_len=3, replicate_every=2)
        mode_o, mode_g = getattr(ops, mode_name), getattr(ps, mode_name)
        for t in range(5):
            W = 1 if mode_name == "SYNC" else [1, 3, 2, 1, 2][t]
            _both_enqueue(o, g, synth.random_gradients(W, seed=40 + t), step=t)
            assert o.apply(mode_o, 0.01) == g.ps_apply(mode_g, 0.01)
            _chain_matches(o, g, f"{mode_name} step {t}")
        o.kill(0); g.ps_kill(0)
        o.kill(1); g.ps_kill(1)
        v = o.failover()
        assert g.ps_failover() == v and o.replicas == []
        th, vg = g.ps_export_params()
        assert vg == v
        assert_params_close(th, o.head(), TOL_APPLY, "tertiary's weights")
        st = g.ps_stats()
        assert st["live_replicas"] == 0 and st["version"] == st["oldest_version"] == v and st["up"] == 1
        _steps(o, g, ops, ps, 1, 60)
        assert_params_close(g.ps_export_params()[0], o.head(), TOL_APPLY, "after the double failure")
        g.ps_kill(0)
        with pytest.raises(ps.PSError) as e:
            g.ps_failover()
        assert e.value.name == "PS_ERR_NO_REPLICA"
        g.close()


def test_async_segment_with_many_replication_events_fills_the_chain():
    # R = 1 and a 20-gradient ordered apply: 20 events in one launch; the servers behind the frontend end up with the
    # last, the one before last and the one before that
    ops, ps, o, g = _pair(queue_slots=32, ring_depth=9, chain_len=4, replicate_every=1, max_workers=32)
    for tick, K in enumerate([20, 2, 1]):
        grads = synth.random_gradients(K, seed=70 + tick)
        _both_enqueue(o, g, grads, step=tick)
        order = synth.arrival_order(tick, K)
        assert o.apply(ops.ASYNC, 0.01, order=order) == g.ps_apply(ps.ASYNC, 0.01, order=order)
        assert [r["version"] for r in o.replicas] == [o.version, o.version - 1, o.version - 2]
        _chain_matches(o, g, f"tick {tick}")
    g.close()


def test_killing_a_server_behind_the_frontend():
    ops, ps, o, g = _pair(queue_slots=4, chain_len=4, replicate_every=1)
    _steps(o, g, ops, ps, 3, 70)
    o.kill(2); g.ps_kill(2)
    _steps(o, g, ops, ps, 1, 80)
    assert [r["version"] for r in o.replicas if r["alive"]] == [4, 3]
    _chain_matches(o, g, "after the middle server died")
    o.kill(2); g.ps_kill(2)
    with pytest.raises(ps.PSError) as e:
        g.ps_kill(2)
    assert e.value.name == "PS_ERR_BAD_ARG"
    with pytest.raises(ops.PSError):
        o.kill(2)
    _steps(o, g, ops, ps, 1, 90)
    _chain_matches(o, g, "one server left behind the frontend")
    g.close()
    # failover skips dead servers in front of the first live one
    ops, ps, o, g = _pair(queue_slots=4, chain_len=3, replicate_every=1)
    _steps(o, g, ops, ps, 2, 90)
    for srv in (1, 0):
        o.kill(srv); g.ps_kill(srv)
    assert o.failover() == g.ps_failover() == 1
    assert_params_close(g.ps_export_params()[0], o.head(), TOL_APPLY, "the last server's weights")
    g.close()


def test_periodic_replication_rollback_to_last_replicated_version():
    ops, ps, o, g = _pair(queue_slots=4, chain_len=2, replicate_every=4)
    _steps(o, g, ops, ps, 7, 100)
    o.kill(0); g.ps_kill(0)
    assert o.failover() == g.ps_failover() == 4
    assert_params_close(g.ps_export_params()[0], o.head(), TOL_APPLY, "rolled back to version 4")
    _steps(o, g, ops, ps, 2, 200)
    assert g.ps_stats()["version"] == o.version == 6
    assert_params_close(g.ps_export_params()[0], o.head(), TOL_APPLY, "after the rollback")
    g.close()


def test_checkpoint_slots_keep_the_most_recent_ones():
    ops, ps, o, g = _pair(queue_slots=4, ckpt_every=2, ckpt_slots=3)
    heads = {}
    for t in range(9):
        _steps(o, g, ops, ps, 1, 300 + t)
        heads[o.version] = g.ps_export_params()[0]
    assert [v for v, _ in o.ckpts] == [4, 6, 8]
    st = g.ps_stats()
    assert st["checkpoints"] == 3 and st["last_ckpt_version"] == 8
    for j, v in enumerate([8, 6, 4]):
        th, vg = g.ps_export_params(1000 + j)
        assert vg == v and (th == heads[v]).all()
    with pytest.raises(ps.PSError) as e:
        g.ps_export_params(1003)
    assert e.value.name == "PS_ERR_NO_CHECKPOINT"
    o.kill(0); g.ps_kill(0)
    assert o.restore() == g.ps_restore() == 8
    assert (g.ps_export_params()[0] == heads[8]).all()
    g.close()


@pytest.mark.parametrize("K", [5, 300])
def test_apply_in_place_with_a_ring_of_depth_one(K):
    # ring_depth 1 (the benchmark's configuration): the new head overwrites the old one in the same buffer
    ops, ps, o, g = _pair(queue_slots=K, ring_depth=1, external_store=True, max_workers=8)
    grads = synth.random_gradients(K, seed=11)
    o.enqueue(grads, range(K), [0] * K, 0)
    g.ps_enqueue(list(range(K)), [0] * K, 0, grads_dev=_pad(grads))
    assert o.apply(ops.REPLAY, 0.01, scale=1.0 / 8) == g.ps_apply(ps.REPLAY, 0.01, scale=1.0 / 8)
    assert_params_close(g.ps_export_params()[0], o.head(), TOL_APPLY, "in-place apply")
    g.close()


def test_a_bounded_wait_that_runs_out_is_reported_and_nothing_hangs():
    """The give-up path of the tensor-core kernels' waits: a probe kernel waits about 10 microseconds on a barrier
    nobody arrives at, records the time-out in the status word and returns; ps_stats reports it; the device and a
    fresh context work as before."""
    import torch
    ops, ps, o, g = _pair(queue_slots=4)
    assert g.ps_stats()["device_status"] == 0
    g.ps_selftest_wait_timeout(20000)
    with pytest.raises(ps.PSError) as e:
        g.ps_stats()
    assert e.value.name == "PS_ERR_DEVICE_STATUS"
    assert g.ps_stats(check=False)["device_status"] == 2
    with pytest.raises(ps.PSError) as e:
        g.ps_selftest_wait_timeout(0)
    assert e.value.name == "PS_ERR_BAD_ARG"
    # the context still computes (its status word keeps the flag) ...
    _both_enqueue(o, g, synth.random_gradients(2, seed=1))
    assert o.apply(ops.SYNC, 0.01) == g.ps_apply(ps.SYNC, 0.01)
    assert_params_close(g.ps_export_params()[0], o.head(), TOL_APPLY, "apply after the probe")
    g.close()
    # ... and a fresh context runs a tensor-core tick with a clean status
    theta = synth.init_params(1)
    srv = ps.ParameterServer(theta, max_workers=2, max_batch=4, queue_slots=2, precision=ps.BF16)
    rng = np.random.default_rng(0)
    x = rng.random((2, 4, 28, 28), dtype=np.float32)
    y = rng.integers(0, 10, (2, 4)).astype(np.int32)
    loss, res = srv.ps_tick_host(x, y, 0x5EED, 0, ps.SYNC, 0.01)
    st = srv.ps_stats()
    assert st["device_status"] == 0 and st["version"] == 1 and np.isfinite(loss).all()
    srv.close()
    torch.cuda.synchronize()


# ---- treatments of stale gradients ------------------------------------------------------------------------------------

def _known_norm_grads(norms, seed):
    rng = np.random.default_rng(seed)
    g = synth.random_gradients(len(norms), seed=seed)
    for k, nrm in enumerate(norms):
        g[k] *= np.float32(nrm / np.linalg.norm(g[k].astype(np.float64)))
    return g


@pytest.mark.parametrize("mode_name,K", [("SYNC", 6), ("REPLAY", 300), ("ASYNC", 9)])
def test_clipping_by_global_norm(mode_name, K):
    ops, ps, o, g = _pair(queue_slots=max(K, 8), ring_depth=3, external_store=(mode_name == "REPLAY"), max_workers=64)
    norms = np.random.default_rng(K).uniform(0.2, 5.0, size=K)
    norms[0], norms[-1] = 0.01, 50.0
    grads = _known_norm_grads(norms, seed=K)
    _both_enqueue(o, g, grads)
    order = synth.arrival_order(0, K) if mode_name == "ASYNC" else None
    ro = o.apply(getattr(ops, mode_name), 0.01, order=order, clip_norm=1.0)
    rg = g.ps_apply_stale(getattr(ps, mode_name), 0.01, order=order, clip_norm=1.0)
    assert ro == rg
    theta0 = synth.init_params(seed=1, bias_scale=0.05)
    th = g.ps_export_params()[0]
    assert_params_close(th, o.head(), TOL_APPLY, f"clipped {mode_name}")
    step_o, step_g = o.head().astype(np.float64) - theta0, th.astype(np.float64) - theta0
    assert np.abs(step_g - step_o).max() <= 2e-3 * np.abs(step_o).max()
    # and the clipping did something: the plain step is far from this one
    _, _, o2, _g2 = _pair(queue_slots=max(K, 8), ring_depth=3, external_store=(mode_name == "REPLAY"), max_workers=64)
    o2.enqueue(grads, range(K), [0] * K, 0)
    o2.apply(getattr(ops, mode_name), 0.01, order=order)
    assert np.abs((o2.head().astype(np.float64) - theta0) - step_o).max() > 0.1 * np.abs(step_o).max()
    _g2.close(); g.close()


@pytest.mark.parametrize("mode_name", ["SYNC", "REPLAY", "ASYNC"])
def test_staleness_scaled_learning_rate(mode_name):
    ops, ps, o, g = _pair(queue_slots=16, ring_depth=9, external_store=(mode_name == "REPLAY"), max_workers=16)
    _steps(o, g, ops, ps, 5, 800)                           # head is version 5
    K = 8
    grads = synth.random_gradients(K, seed=33)
    base = [5, 0, 3, 5, 1, 4, 2, 0]
    _both_enqueue(o, g, grads, step=9, base=base)
    order = synth.arrival_order(2, K) if mode_name == "ASYNC" else None
    before = o.head().astype(np.float64)
    ro = o.apply(getattr(ops, mode_name), 0.01, order=order, staleness_alpha=0.5, clip_norm=3.0)
    rg = g.ps_apply_stale(getattr(ps, mode_name), 0.01, order=order, staleness_alpha=0.5, clip_norm=3.0)
    assert ro == rg
    th = g.ps_export_params()[0]
    assert_params_close(th, o.head(), TOL_APPLY, f"staleness-scaled {mode_name}")
    step_o, step_g = o.head().astype(np.float64) - before, th.astype(np.float64) - before
    assert np.abs(step_g - step_o).max() <= 2e-3 * np.abs(step_o).max()
    # both treatments off is the plain apply, bit for bit
    _both_enqueue(o, g, grads, step=10)
    h0 = g.ps_export_params()[0]
    rg = g.ps_apply_stale(getattr(ps, mode_name), 0.01, order=order)
    plain = g.ps_export_params()[0]
    _, _, _, g2 = _pair(queue_slots=16, ring_depth=9, external_store=(mode_name == "REPLAY"), max_workers=16)
    g2.ps_import_params(h0)
    g2.ps_enqueue(list(range(K)), [0] * K, 10, grads_dev=_pad(grads))
    g2.ps_apply(getattr(ps, mode_name), 0.01, order=order)
    assert (g2.ps_export_params()[0] == plain).all()
    # a base version from the future is refused
    g.ps_enqueue([0], [10 ** 6], 11, grads_dev=_pad(grads[:1]))
    with pytest.raises(ps.PSError) as e:
        g.ps_apply_stale(getattr(ps, mode_name), 0.01, staleness_alpha=0.5)
    assert e.value.name == "PS_ERR_BAD_ARG"
    g2.close(); g.close()


def test_two_failures_in_one_run():
    """The schedule of the paper's second accuracy experiment, two server failures in one run, on both recovery
    designs: checkpointing (each restore rolls back to the latest checkpoint, the updates since are lost and redone
    with new gradients) and a chain of three (each failover moves to the next server, the second one to older weights)."""
    ops, ps, o, g = _pair(queue_slots=4, ckpt_every=10, ckpt_slots=4)
    _steps(o, g, ops, ps, 13, 1000)
    o.kill(0); g.ps_kill(0)
    assert o.restore() == g.ps_restore() == 10
    _steps(o, g, ops, ps, 14, 1100)                     # 10 -> 24, checkpoint at 20
    o.kill(0); g.ps_kill(0)
    assert o.restore() == g.ps_restore() == 20
    _steps(o, g, ops, ps, 3, 1200)
    st = g.ps_stats()
    assert st["version"] == o.version == 23 and st["last_ckpt_version"] == 20 and st["checkpoints"] == 2
    assert [v for v, _ in o.ckpts] == [10, 20]
    assert_params_close(g.ps_export_params()[0], o.head(), 1e-5, "after two rollbacks")
    g.close()
    ops, ps, o, g = _pair(queue_slots=4, chain_len=3, replicate_every=3)
    _steps(o, g, ops, ps, 8, 1300)                      # events at 3 and 6: the servers hold 6 and 3
    o.kill(0); g.ps_kill(0)
    assert o.failover() == g.ps_failover() == 6
    _steps(o, g, ops, ps, 2, 1400)                      # 7, 8: no event yet, the last server still holds 3
    o.kill(0); g.ps_kill(0)
    assert o.failover() == g.ps_failover() == 3
    _steps(o, g, ops, ps, 2, 1500)
    assert g.ps_stats()["version"] == o.version == 5 and g.ps_stats()["live_replicas"] == 0
    assert_params_close(g.ps_export_params()[0], o.head(), 1e-5, "after two failovers")
    g.close()
