"""Pins for the parameter-server oracle: invariants and closed forms that follow from the
paper's description of the sync, async, checkpointing, chain-replicated and stateless servers."""
import numpy as np
import pytest

from oracle import cnn
from oracle import ps as ops
from paper_2406_05546_b200 import synth

P = cnn.P


def _small_grads(K, seed=4):
    return synth.random_gradients(K, seed=seed)


def test_sync_W_workers_equals_one_worker_with_concatenated_batch():
    # "aggregating gradients from all workers before updating weights": with a mean loss per worker
    # and a mean over workers, W workers x batch b is one worker x batch W*b (masks concatenated).
    rng = np.random.default_rng(0)
    W, b = 3, 2
    theta = synth.init_params(seed=1, bias_scale=0.05)
    x = rng.random((W, b, 28, 28), dtype=np.float32)
    y = rng.integers(0, 10, (W, b)).astype(np.int32)
    keep = (rng.random((W, b, 512)) >= 0.25).astype(np.uint8)
    t64 = theta.astype(np.float64)
    gs = [cnn.grad_step_f64(t64, x[w].astype(np.float64), y[w], keep[w], 0.25)[0] for w in range(W)]
    big = cnn.grad_step_f64(t64, x.reshape(W * b, 28, 28).astype(np.float64), y.reshape(-1),
                            keep.reshape(W * b, 512), 0.25)[0]
    assert np.abs(np.mean(gs, axis=0) - big).max() < 1e-13
    s = ops.OraclePS(theta)
    s.enqueue(np.asarray(gs, dtype=np.float32), range(W), [0] * W, 0)
    s.apply(ops.SYNC, 0.01)
    one = ops.OraclePS(theta)
    one.enqueue(big.astype(np.float32)[None], [0], [0], 0)
    one.apply(ops.SYNC, 0.01)
    # the two differ only by the fp32 rounding of the stored gradients and of the stored weights (|theta| < 1)
    assert np.abs(s.head() - one.head()).max() <= 2.0 ** -24


def test_sync_closed_form_and_version():
    theta = synth.init_params(1)
    g = _small_grads(4)
    s = ops.OraclePS(theta)
    s.enqueue(g, range(4), [0] * 4, 0)
    r = s.apply(ops.SYNC, 0.01)
    expect = (theta.astype(np.float64) - np.float64(np.float32(0.01)) / 4 * g.astype(np.float64).sum(0)).astype(np.float32)
    assert (s.head() == expect).all()
    assert r == {"applied": 4, "new_version": 1, "checkpointed": 0, "replicated": 0}
    assert s.queue == [] and s.version == 1


def test_replay_with_zero_downtime_equals_sync():
    theta = synth.init_params(1)
    a = ops.OraclePS(theta, external_store=True)
    c = ops.OraclePS(theta)
    for t in range(3):
        g = _small_grads(5, seed=10 + t)
        a.enqueue(g, range(5), [t] * 5, t)
        c.enqueue(g, range(5), [t] * 5, t)
        a.apply(ops.REPLAY, 0.01)
        c.apply(ops.SYNC, 0.01)
        assert (a.head() == c.head()).all() and a.version == c.version == t + 1


def test_replay_is_order_independent_and_equals_sum_of_frozen_sync_steps():
    theta = synth.init_params(1)
    T, W = 6, 4
    g = _small_grads(T * W, seed=7)
    a = ops.OraclePS(theta, external_store=True)
    b = ops.OraclePS(theta, external_store=True)
    a.kill(); b.kill()
    for t in range(T):
        a.enqueue(g[t * W:(t + 1) * W], range(W), [0] * W, t)
        b.enqueue(g[t * W:(t + 1) * W], range(W), [0] * W, t)
    a.restore(); b.restore()
    perm = np.random.default_rng(3).permutation(T * W)
    ra = a.apply(ops.REPLAY, 0.01)
    b.apply(ops.REPLAY, 0.01, order=perm)
    assert ra["applied"] == T * W and ra["new_version"] == 1
    assert np.abs(a.head().astype(np.float64) - b.head()).max() <= 1.2e-7 * np.abs(theta).max()
    # K = T*W gradients computed on frozen weights: theta - lr/W * sum_k g_k
    expect = theta.astype(np.float64) - np.float64(np.float32(0.01)) / W * g.astype(np.float64).sum(0)
    assert (a.head() == expect.astype(np.float32)).all()
    # learning-rate scale-down for many pending gradients is the `scale` factor
    c = ops.OraclePS(theta, external_store=True)
    for t in range(T):
        c.enqueue(g[t * W:(t + 1) * W], range(W), [0] * W, t)
    c.apply(ops.REPLAY, 0.01, scale=0.5)
    expect = theta.astype(np.float64) - np.float64(np.float32(0.01)) * 0.5 / W * g.astype(np.float64).sum(0)
    assert (c.head() == expect.astype(np.float32)).all()


def test_async_single_gradient_equals_sync_single_worker_and_ordered_closed_form():
    theta = synth.init_params(1)
    g = _small_grads(5, seed=2)
    a = ops.OraclePS(theta, ring_depth=9)
    s = ops.OraclePS(theta)
    a.enqueue(g[:1], [0], [0], 0); s.enqueue(g[:1], [0], [0], 0)
    a.apply(ops.ASYNC, 0.01); s.apply(ops.SYNC, 0.01)
    assert (a.head() == s.head()).all()
    # ordered application: version v0+j is theta - lr * sum of the first j gradients in arrival order
    a = ops.OraclePS(theta, ring_depth=9)
    a.enqueue(g, range(5), [0] * 5, 0)
    order = [3, 0, 4, 1, 2]
    r = a.apply(ops.ASYNC, 0.01, order=order)
    assert r["applied"] == 5 and a.version == 5
    run = theta.astype(np.float64)
    for j, k in enumerate(order):
        run = run - np.float64(np.float32(0.01)) * g[k].astype(np.float64)
        v, th = a.pull_snapshot(0, lag=5 - (j + 1))
        assert v == j + 1
        assert np.abs(th - run).max() <= 6e-8 * (j + 1) * np.abs(theta).max()
    # a different arrival order gives the same final weights up to rounding, not bit for bit in general
    b = ops.OraclePS(theta, ring_depth=9)
    b.enqueue(g, range(5), [0] * 5, 0)
    b.apply(ops.ASYNC, 0.01)
    assert np.abs(b.head() - a.head()).max() <= 1e-6


def test_version_ring_retains_exactly_ring_depth_versions():
    theta = synth.init_params(1)
    s = ops.OraclePS(theta, ring_depth=9)
    g = _small_grads(12, seed=5)
    s.enqueue(g, range(12), [0] * 12, 0)
    s.apply(ops.ASYNC, 0.01)
    assert s.version == 12 and s.oldest_version() == 4 and len(s.ring) == 9
    assert s.pull_snapshot(0, 8)[0] == 4
    with pytest.raises(ops.PSError) as e:
        s.pull_snapshot(0, 9)
    assert e.value.code == ops.VERSION_EVICTED


def test_checkpoint_rollback_schedule():
    # checkpoint every 25 updates; killed before tick 60, down for 20 ticks (workers idle),
    # restored from the version-50 checkpoint, then 120 more updates: final version 170.
    theta = synth.init_params(1)
    s = ops.OraclePS(theta, ckpt_every=25, ckpt_slots=8)
    seen_ckpts = []
    at50 = None
    for tick in range(200):
        if tick == 60:
            s.kill()
        if 60 <= tick < 80:
            with pytest.raises(ops.PSError) as e:
                s.pull_snapshot(0)
            assert e.value.code == ops.DOWN
            with pytest.raises(ops.PSError):
                s.apply(ops.SYNC, 0.01)
            continue
        if tick == 80:
            assert s.restore() == 50
            assert s.version == 50 and (s.head() == at50).all() and s.queue == []
        g = _small_grads(2, seed=100 + tick) * np.float32(0.1)
        s.enqueue(g, [0, 1], [s.version] * 2, tick)
        r = s.apply(ops.SYNC, 0.01)
        if r["checkpointed"]:
            seen_ckpts.append(s.version)
        if s.version == 50 and at50 is None:
            at50 = s.head().copy()
    assert s.version == 170
    assert seen_ckpts == [25, 50, 75, 100, 125, 150]
    with pytest.raises(ops.PSError) as e:
        ops.OraclePS(theta).restore()
    assert e.value.code == ops.NO_CHECKPOINT


def test_async_checkpoint_captures_the_intermediate_version():
    theta = synth.init_params(1)
    s = ops.OraclePS(theta, ring_depth=2, ckpt_every=4)
    g = _small_grads(6, seed=8)
    s.enqueue(g, range(6), [0] * 6, 0)
    r = s.apply(ops.ASYNC, 0.01)
    assert r["checkpointed"] == 1 and s.ckpts[-1][0] == 4
    run = theta
    for k in range(4):
        run = (run.astype(np.float64) - np.float64(np.float32(0.01)) * g[k].astype(np.float64)).astype(np.float32)
    assert (s.ckpts[-1][1] == run).all()


def test_chain_mirror_and_failover():
    theta = synth.init_params(1)
    for R in (1, 3):
        s = ops.OraclePS(theta, ring_depth=9, chain_len=2, replicate_every=R)
        hist = {0: theta.copy()}
        for tick in range(4):
            g = _small_grads(4, seed=20 + tick)
            s.enqueue(g, range(4), [s.version] * 4, tick)
            s.apply(ops.ASYNC, 0.01, order=synth.arrival_order(tick, 4))
            hist[s.version] = s.head().copy()
            last = (s.version // R) * R
            assert s.replicas[0]["version"] == last
            if last == s.version:
                assert (s.replicas[0]["theta"] == s.head()).all()
        rep_v, rep_t = s.replicas[0]["version"], s.replicas[0]["theta"].copy()
        s.kill()
        with pytest.raises(ops.PSError):
            s.pull_snapshot(0)
        assert s.failover() == rep_v
        assert s.version == rep_v and (s.head() == rep_t).all() and s.oldest_version() == rep_v
        with pytest.raises(ops.PSError) as e:
            s.kill(); s.failover()
        assert e.value.code == ops.NO_REPLICA


def test_stateless_server_keeps_store_while_down():
    theta = synth.init_params(1)
    s = ops.OraclePS(theta, external_store=True)
    g = _small_grads(6, seed=9)
    s.enqueue(g[:2], [0, 1], [0, 0], 0)
    s.apply(ops.REPLAY, 0.01)
    before = s.head().copy()
    s.kill()
    v, th = s.pull_snapshot(0)              # workers keep reading the stored weights
    assert v == 1 and (th == before).all()
    s.enqueue(g[2:4], [0, 1], [1, 1], 1)    # and keep appending gradients
    s.enqueue(g[4:6], [0, 1], [1, 1], 2)
    with pytest.raises(ops.PSError):
        s.apply(ops.REPLAY, 0.01)
    assert s.restore() == 1 and len(s.queue) == 4
    r = s.apply(ops.REPLAY, 0.01)
    assert r["applied"] == 4 and s.version == 2 and s.queue == []
    with pytest.raises(ops.PSError) as e:
        s.enqueue(g[:2], [0, 1], [2, 2], 3); s.enqueue(g[:3], [0, 1, 2], [2] * 3, 3)
    assert e.value.code == ops.BAD_ARG


def test_queue_capacity():
    s = ops.OraclePS(synth.init_params(1), queue_slots=3)
    g = _small_grads(2)
    s.enqueue(g, [0, 1], [0, 0], 0)
    with pytest.raises(ops.PSError) as e:
        s.enqueue(g, [0, 1], [0, 0], 1)
    assert e.value.code == ops.QUEUE_FULL


def _steps(s, n, seed0, W=2):
    for t in range(n):
        s.enqueue(_small_grads(W, seed=seed0 + t), range(W), [s.version] * W, t)
        s.apply(ops.SYNC, 0.01)


def test_chain_of_three_tertiary_holds_older_weights_and_survives_a_double_failure():
    # Design, chain replication: the frontend waits for the next server only, so the server behind that one is one
    # replication event behind; when frontend and secondary both fail, the tertiary recovers with older weights.
    theta = synth.init_params(1)
    R = 2
    s = ops.OraclePS(theta, chain_len=3, replicate_every=R)
    hist = {0: theta.copy()}
    for t in range(5):
        _steps(s, 1, 40 + t)
        hist[s.version] = s.head().copy()
        first = (s.version // R) * R
        assert s.replicas[0]["version"] == first
        assert s.replicas[1]["version"] == max(first - R, 0)
        assert (s.replicas[0]["theta"] == hist[first]).all() and (s.replicas[1]["theta"] == hist[max(first - R, 0)]).all()
    assert s.version == 5
    s.kill(0)
    s.kill(1)                                   # the secondary dies too
    assert s.failover() == 2                    # the tertiary takes over, one event (R versions) behind the secondary's 4
    assert (s.head() == hist[2]).all() and s.oldest_version() == 2 and s.replicas == []
    _steps(s, 1, 60)                            # training goes on without a replica
    assert s.version == 3
    s.kill(0)
    with pytest.raises(ops.PSError) as e:
        s.failover()
    assert e.value.code == ops.NO_REPLICA


def test_killing_a_server_behind_the_frontend_shortens_the_chain():
    theta = synth.init_params(1)
    s = ops.OraclePS(theta, chain_len=4, replicate_every=1)
    _steps(s, 3, 70)
    assert [r["version"] for r in s.replicas] == [3, 2, 1]
    s.kill(2)                                   # the second live server behind the frontend
    assert [r["alive"] for r in s.replicas] == [True, False, True]
    _steps(s, 1, 80)
    # the dead server is skipped: the last one now follows the first, and the dead one keeps what it had
    assert [r["version"] for r in s.replicas] == [4, 2, 3]
    s.kill(2)                                   # now the second LIVE one is the last server
    assert [r["alive"] for r in s.replicas] == [True, False, False]
    with pytest.raises(ops.PSError) as e:
        s.kill(2)
    assert e.value.code == ops.BAD_ARG
    s.kill(1)
    s.kill(0)
    with pytest.raises(ops.PSError) as e:
        s.failover()
    assert e.value.code == ops.NO_REPLICA
    # failover skips dead servers in front of the first live one
    s = ops.OraclePS(theta, chain_len=3, replicate_every=1)
    _steps(s, 2, 90)
    th1 = s.replicas[1]["theta"].copy()
    s.kill(1); s.kill(0)
    assert s.failover() == 1 and (s.head() == th1).all() and s.replicas == []


def test_periodic_replication_rolls_back_to_the_last_replicated_version():
    # R > 1: updates since the last replication event are lost with the frontend
    theta = synth.init_params(1)
    s = ops.OraclePS(theta, chain_len=2, replicate_every=4)
    seen = {}
    for t in range(7):
        _steps(s, 1, 100 + t)
        seen[s.version] = s.head().copy()
    assert s.version == 7 and s.replicas[0]["version"] == 4
    s.kill(0)
    assert s.failover() == 4 and (s.head() == seen[4]).all()
    _steps(s, 1, 200)
    assert s.version == 5 and not (s.head() == seen[5]).all()      # a different fifth update than the lost one


def test_checkpoint_slots_keep_the_most_recent_ones():
    theta = synth.init_params(1)
    s = ops.OraclePS(theta, ckpt_every=2, ckpt_slots=3)
    kept = {}
    for t in range(9):
        _steps(s, 1, 300 + t)
        if s.version % 2 == 0:
            kept[s.version] = s.head().copy()
    assert [v for v, _ in s.ckpts] == [4, 6, 8]                     # 2 was overwritten by 8
    for v, th in s.ckpts:
        assert (th == kept[v]).all()
    s.kill(0)
    assert s.restore() == 8 and (s.head() == kept[8]).all()


# ---- treatments of stale gradients (design section, closing remarks on the stateless server) ----------------------

def _unit_grads(norms, P=P, seed=0):
    """Gradients of exactly known Euclidean norm: a few +-1 entries scaled."""
    rng = np.random.default_rng(seed)
    out = np.zeros((len(norms), P), dtype=np.float32)
    for k, nrm in enumerate(norms):
        pos = rng.choice(P, size=16, replace=False)
        out[k, pos] = np.float32(nrm / 4.0) * rng.choice([-1.0, 1.0], size=16).astype(np.float32)   # sqrt(16) = 4
    return out


def test_clipping_by_global_norm_closed_form():
    theta = synth.init_params(1)
    norms = [0.5, 2.0, 8.0, 1.0]           # powers of two: every scaled entry is exact in fp32
    g = _unit_grads(norms)
    s = ops.OraclePS(theta, external_store=True)
    s.enqueue(g, range(4), [0] * 4, 0)
    s.apply(ops.REPLAY, 0.5, clip_norm=1.0)
    clipped = np.stack([g[k].astype(np.float64) * min(1.0, 1.0 / norms[k]) for k in range(4)])
    expect = (theta.astype(np.float64) - 0.5 / 4 * clipped.sum(0)).astype(np.float32)
    assert (s.head() == expect).all()
    for k in range(4):                      # what was applied has norm min(norm, c)
        assert abs(np.linalg.norm(clipped[k]) - min(norms[k], 1.0)) < 1e-12
    # a bound above every norm changes nothing, bit for bit
    a = ops.OraclePS(theta, external_store=True); a.enqueue(g, range(4), [0] * 4, 0); a.apply(ops.REPLAY, 0.5, clip_norm=100.0)
    b = ops.OraclePS(theta, external_store=True); b.enqueue(g, range(4), [0] * 4, 0); b.apply(ops.REPLAY, 0.5)
    assert (a.head() == b.head()).all()
    with pytest.raises(ops.PSError):
        a.enqueue(g, range(4), [1] * 4, 0); a.apply(ops.REPLAY, 0.5, clip_norm=0.0)


def test_staleness_scaling_closed_forms():
    theta = synth.init_params(1)
    g = _small_grads(6, seed=12)
    lr32 = np.float64(np.float32(0.01))
    # replay after an outage: every queued gradient was computed on the stored version, so they are all equally stale
    # and the treatment is a plain learning-rate scale of 1 / (1 + alpha * tau)
    s = ops.OraclePS(theta, external_store=True)
    _steps(s, 3, 400)                                   # head is version 3
    s.enqueue(g, range(6), [1] * 6, 0)                  # read at version 1: tau = 2
    t = ops.OraclePS(s.head(), external_store=True)
    t.enqueue(g, range(6), [0] * 6, 0)
    s.apply(ops.REPLAY, 0.01, staleness_alpha=0.5)
    t.apply(ops.REPLAY, 0.01, scale=0.5)                # 1 / (1 + 0.5 * 2)
    assert (s.head() == t.head()).all()
    # alpha = 0 is the plain step
    a = ops.OraclePS(theta); a.enqueue(g, range(6), [0] * 6, 0); a.apply(ops.SYNC, 0.01, staleness_alpha=0.0)
    b = ops.OraclePS(theta); b.enqueue(g, range(6), [0] * 6, 0); b.apply(ops.SYNC, 0.01)
    assert (a.head() == b.head()).all()
    # async: the j-th update in arrival order is applied to version v0 + j; mixed base versions
    s = ops.OraclePS(theta, ring_depth=4)
    _steps(s, 2, 500)                                   # v0 = 2
    base = [2, 0, 1, 2, 0, 1]
    order = [4, 1, 0, 5, 2, 3]
    s.enqueue(g, range(6), base, 0)
    run = s.head().astype(np.float64)
    v0 = s.version
    s.apply(ops.ASYNC, 0.01, order=order, staleness_alpha=0.25)
    for j, k in enumerate(order):
        run = (run - lr32 / (1.0 + np.float64(0.25) * (v0 + j - base[k])) * g[k].astype(np.float64)).astype(np.float32).astype(np.float64)
    assert (s.head() == run.astype(np.float32)).all() and s.version == v0 + 6
    # a base version from the future is refused
    s.enqueue(g[:1], [0], [s.version + 1], 0)
    with pytest.raises(ops.PSError):
        s.apply(ops.SYNC, 0.01, staleness_alpha=0.1)


def test_clipping_and_staleness_compose():
    theta = synth.init_params(1)
    g = _unit_grads([4.0, 0.25], seed=3)
    s = ops.OraclePS(theta)
    _steps(s, 4, 600)
    th0 = s.head().astype(np.float64)
    s.enqueue(g, [0, 1], [4, 2], 0)                     # tau = 0 and 2
    s.apply(ops.SYNC, 1.0, clip_norm=1.0, staleness_alpha=1.0)
    expect = th0 - 1.0 / 2 * (g[0].astype(np.float64) * 0.25 * 1.0 + g[1].astype(np.float64) * 1.0 / 3.0)
    assert np.abs(s.head() - expect).max() <= 2.0 ** -24 * max(1.0, np.abs(expect).max())
