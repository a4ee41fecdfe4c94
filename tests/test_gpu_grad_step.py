"""GPU parity: the worker gradient step against the CPU oracle, through the C ABI."""
import numpy as np
import pytest

from paper_2406_05546_b200 import synth
from tests.parity import (TOL_FP32, TOL_TENSOR, assert_argmax_valid, assert_params_close,
                          assert_params_close_up_to_unit_flips, assert_sum_close, tensor_rel_errors)

pytestmark = pytest.mark.gpu

SEED = 0x5EED


def _setup(W, b, n_versions=1, drop_p=0.25, precision=0):
    import torch
    from paper_2406_05546_b200 import ps
    theta0 = synth.init_params(seed=1, bias_scale=0.05)
    srv = ps.ParameterServer(theta0, max_workers=W, max_batch=b, ring_depth=max(1, n_versions),
                             queue_slots=max(W, n_versions), dropout_p=drop_p, precision=precision)
    return torch, ps, srv, theta0


def _run_and_compare(W, b, lags=None, n_versions=1, step=3, drop_p=0.25, worker_ids=None, in_slots=False,
                     precision=0):
    from oracle import cnn
    tol = TOL_TENSOR if precision else TOL_FP32
    torch, ps, srv, theta0 = _setup(W, b, n_versions, drop_p, precision)
    versions = {0: theta0}
    # produce older/newer versions with async applies of random "gradients" so that snapshots differ
    for v in range(1, n_versions):
        g = np.zeros((1, ps.P_PAD), dtype=np.float32)
        g[0, :ps.P] = synth.random_gradients(1, seed=50 + v, scale=2.0)[0]
        srv.ps_enqueue([0], [v - 1], 0, grads_dev=torch.from_numpy(g).cuda())
        srv.ps_apply(ps.ASYNC, 0.01)
        versions[v], ver = srv.ps_export_params(0)
        assert ver == v
    rng = np.random.default_rng(7)
    x = rng.random((W, b, 28, 28), dtype=np.float32)
    y = rng.integers(0, 10, (W, b)).astype(np.int32)
    lags = [0] * W if lags is None else lags
    ids = list(range(W)) if worker_ids is None else worker_ids
    snaps = [srv.ps_pull_snapshot(w, lags[w]) for w in range(W)]
    xd, yd = torch.from_numpy(x).cuda(), torch.from_numpy(y).cuda()
    if in_slots:
        slots = srv.ps_queue_reserve(W)
        loss, am = srv.workers_grad_step(snaps, ids, xd, yd, SEED, step, slot_ids=slots)
        grads = torch.stack([srv.slot_tensor(s) for s in slots]).cpu().numpy()
    else:
        gd = torch.full((W, ps.P_PAD), float("nan"), device="cuda")
        loss, am = srv.workers_grad_step(snaps, ids, xd, yd, SEED, step, grads_dev=gd)
        grads = gd.cpu().numpy()
    srv.ps_stats()
    thetas = [versions[s.version] for s in snaps]
    og, ol, oa, oz = cnn.workers_grad_step(thetas, ids, x, y, SEED, step, drop_p, precision=precision)
    for w in range(W):
        assert (grads[w, ps.P:] == 0).all()
        if precision and W * b > 500:
            # several hundred thousand ReLU decisions: a hidden unit within rounding distance of zero may come out the
            # other way; the helper admits that, and only that (see its docstring), so the oracle's intermediates of
            # this worker are needed whenever a row is off
            errs = tensor_rel_errors(grads[w, :ps.P], og[w])
            if max(errs.values()) > tol:
                g1, _, _, _, diag = cnn.worker_grad_step_diag(thetas[w], ids[w], x[w], y[w], SEED, step, drop_p, precision)
                assert np.array_equal(g1, og[w])
                redo = lambda fl, w=w: cnn.worker_grad_step_diag(thetas[w], ids[w], x[w], y[w], SEED, step, drop_p, precision, flips=fl)[0]
                flips = assert_params_close_up_to_unit_flips(grads[w, :ps.P], og[w], tol, thetas[w], diag, f"gradient of worker {w}", recompute=redo)
                print(f"worker {w}: hidden units decided differently within the rounding bound of zero: {flips}")
            continue
        errs = assert_params_close(grads[w, :ps.P], og[w], tol, f"gradient of worker {w}")
        if precision and w == 0:
            print("tensor-path relative errors:", {k: f"{v:.1e}" for k, v in errs.items()})
    np.testing.assert_allclose(loss.cpu().numpy(), ol, rtol=3e-3 if precision else 1e-5, atol=1e-6)
    assert_argmax_valid(am.cpu().numpy(), oz, tol)
    srv.close()
    return grads


def test_config1_shape_two_workers_batch8():
    _run_and_compare(2, 8, in_slots=True)


def test_ragged_batch_and_worker_ids():
    _run_and_compare(3, 5, worker_ids=[11, 4, 200], step=(1 << 33) + 5)


def test_batch_spanning_several_tiles_with_tail():
    _run_and_compare(2, 70)


def test_stale_snapshots_grouped_over_three_versions():
    # five workers over three distinct weight versions, interleaved so that grouping must reorder
    _run_and_compare(5, 6, lags=[2, 0, 1, 2, 0], n_versions=3)


@pytest.mark.parametrize("W,b,kw", [(2, 8, {}), (3, 5, {"worker_ids": [11, 4, 200]}), (2, 150, {}),
                                     (5, 6, {"lags": [2, 0, 1, 2, 0], "n_versions": 3}), (1, 1, {}),
                                     (2, 4, {"drop_p": 0.0}),
                                     # 777 rows over two weight versions: the persistent convolution kernels take
                                     # ranges of several rows that cross worker boundaries inside a version group
                                     (7, 111, {"lags": [1, 0, 1, 1, 0, 0, 1], "n_versions": 2})])
def test_tensor_core_path(W, b, kw):
    _run_and_compare(W, b, precision=2, **kw)


@pytest.mark.parametrize("precision", [0, 2])
def test_maximum_number_of_workers_with_an_odd_batch(precision):
    # 256 workers (the library's limit) of three samples: every worker's last sample has no partner in the first
    # convolution's filter-gradient kernel, and ranges of the persistent kernels cross many worker boundaries
    _run_and_compare(256, 3, precision=precision, worker_ids=[(7 * w + 3) % 1000 for w in range(256)])


def test_tensor_core_path_repeatable_bit_for_bit():
    a = _run_and_compare(3, 9, precision=2)
    b = _run_and_compare(3, 9, precision=2)
    assert (a == b).all()


@pytest.mark.parametrize("W,b", [(2, 8), (3, 40)])
def test_tensor_core_path_against_the_plain_definition(W, b):
    """The tensor-core path against the oracle with EVERY decision taken on exact values (precision 0): what the
    benchmarked path's error is against the definition, and that it comes from decisions inside the
    operand-rounding bound and from nothing else.
      - output layer: within the tolerance as it stands (a ReLU that flips at zero changes no forward value);
      - 512-unit layer: every row is within the tolerance after removing the contributions of samples whose exact
        pre-activation is inside the bound (least-squares explanation, coefficients -1 / 0 / +1);
      - convolutions: pooling winners inside the bound re-route gradient between neighbouring positions; their
        error is reported and must not exceed what the oracle itself shows between exact and rounded decisions
        plus the tolerance (every such difference lies inside the bound: tests/test_margins.py)."""
    from oracle import cnn
    import torch
    from paper_2406_05546_b200 import ps
    from tests import margins
    torch_, ps_, srv, theta0 = _setup(W, b, 1, 0.25, 2)
    rng = np.random.default_rng(21)
    x = rng.random((W, b, 28, 28), dtype=np.float32)
    y = rng.integers(0, 10, (W, b)).astype(np.int32)
    snaps = [srv.ps_pull_snapshot(w) for w in range(W)]
    gd = torch.full((W, ps.P_PAD), float("nan"), device="cuda")
    srv.workers_grad_step(snaps, list(range(W)), torch.from_numpy(x).cuda(), torch.from_numpy(y).cuda(), SEED, 4, grads_dev=gd)
    srv.ps_stats()
    grads = gd.cpu().numpy()
    srv.close()
    n_flips = n_pool_unc = n_relu_unc = 0
    for w in range(W):
        g0, _, _, _, d0 = cnn.worker_grad_step_diag(theta0, w, x[w], y[w], SEED, 4, 0.25, precision=0)
        g2 = cnn.worker_grad_step_diag(theta0, w, x[w], y[w], SEED, 4, 0.25, precision=2)[0]
        m = margins.decision_margins(theta0, d0)
        n_pool_unc += int(m["pool_uncertain"].sum()); n_relu_unc += int(m["relu_uncertain"].sum())
        e_kernel = tensor_rel_errors(grads[w, :ps.P], g0)
        e_oracle = tensor_rel_errors(g2, g0)
        print(f"worker {w}: kernel vs exact decisions", {k: f"{v:.1e}" for k, v in e_kernel.items()})
        print(f"worker {w}: oracle with rounded decisions vs exact decisions", {k: f"{v:.1e}" for k, v in e_oracle.items()})
        for name in ("fc2.w", "fc2.b"):
            assert e_kernel[name] <= TOL_TENSOR, (name, e_kernel[name])
        for name in ("conv1.w", "conv1.b", "conv2.w", "conv2.b"):
            assert e_kernel[name] <= e_oracle[name] + TOL_TENSOR, (name, e_kernel[name], e_oracle[name])
        # the 512-unit layer, row by row: got = exact-decision gradient + flips of samples inside the bound.  The
        # convolution tensors are excluded from this call's tolerance check by comparing them in a copy.
        probe = g0.copy()
        probe[4800:808128] = grads[w, 4800:808128]
        flips = assert_params_close_up_to_unit_flips(probe, g0, TOL_TENSOR, theta0, d0, f"worker {w} vs exact decisions")
        n_flips += sum(len(f) for _, f in flips)
    print(f"{n_flips} ReLU decisions of the 512-unit layer differ from the exact ones; all inside the bound "
          f"({n_relu_unc} of {W * b * 512} decisions are; pooling: {n_pool_unc} of {W * b * 1568})")


def test_no_dropout():
    _run_and_compare(2, 4, drop_p=0.0)


def test_single_sample_single_worker():
    _run_and_compare(1, 1)


def test_repeatable_bit_for_bit():
    a = _run_and_compare(3, 9)
    b = _run_and_compare(3, 9)
    assert (a == b).all()


def test_dropout_mask_bit_exact():
    from oracle import cnn
    torch, ps, srv, _ = _setup(1, 1)
    for seed, worker, step, b in [(SEED, 0, 0, 1), (SEED, 3, 7, 64), (0xDEADBEEFCAFEF00D, 255, (5 << 32) | 9, 129)]:
        got = srv.ps_dropout_mask(seed, worker, step, b).cpu().numpy()
        assert (got == cnn.dropout_keep(seed, worker, step, b, 0.25)).all()
    srv.close()


def test_grad_step_uses_that_mask():
    # fc1 weights zero and bias one: the hidden layer is 1 before dropout, so with one sample the
    # fc2 weight gradient is dz[c] * keep[j] / (1-p): its zero pattern is exactly the mask.
    from oracle import cnn
    import torch
    from paper_2406_05546_b200 import ps
    theta = synth.init_params(seed=1)
    theta[4800:807616] = 0
    theta[807616:808128] = 1
    srv = ps.ParameterServer(theta, max_workers=4, max_batch=1, queue_slots=4)
    x = np.random.default_rng(0).random((4, 1, 28, 28), dtype=np.float32)
    y = np.array([[1], [2], [3], [4]], dtype=np.int32)
    ids = [9, 0, 77, 3]
    snaps = [srv.ps_pull_snapshot(w) for w in range(4)]
    gd = torch.zeros((4, ps.P_PAD), device="cuda")
    srv.workers_grad_step(snaps, ids, torch.from_numpy(x).cuda(), torch.from_numpy(y).cuda(), SEED, 21, grads_dev=gd)
    g = gd.cpu().numpy()
    for w in range(4):
        keep = cnn.dropout_keep(SEED, ids[w], 21, 1, 0.25)[0]
        gw2 = g[w, 808128:813248].reshape(10, 512)
        assert ((gw2 != 0).all(axis=0) == (keep == 1)).all()
        assert ((gw2 == 0).all(axis=0) == (keep == 0)).all()
    srv.close()


def test_bad_label_is_reported_not_trapped():
    torch, ps, srv, _ = _setup(1, 2)
    x = torch.zeros((1, 2, 28, 28), device="cuda")
    y = torch.tensor([[3, 12]], dtype=torch.int32, device="cuda")
    gd = torch.zeros((1, ps.P_PAD), device="cuda")
    srv.workers_grad_step([srv.ps_pull_snapshot(0)], [0], x, y, SEED, 0, grads_dev=gd)
    with pytest.raises(ps.PSError) as e:
        srv.ps_stats()
    assert e.value.name == "PS_ERR_DEVICE_STATUS"
    srv.close()


def test_argument_errors():
    torch, ps, srv, _ = _setup(2, 4)
    x = torch.zeros((3, 4, 28, 28), device="cuda")
    y = torch.zeros((3, 4), dtype=torch.int32, device="cuda")
    snaps = [srv.ps_pull_snapshot(0)] * 3
    with pytest.raises(ps.PSError) as e:
        srv.workers_grad_step(snaps, [0, 1, 2], x, y, SEED, 0, grads_dev=torch.zeros((3, ps.P_PAD), device="cuda"))
    assert e.value.name == "PS_ERR_BAD_ARG"
    with pytest.raises(ps.PSError):
        srv.workers_grad_step(snaps[:2], [0, 1], x[:2], y[:2], SEED, 0, slot_ids=[0, 1])   # not reserved
    with pytest.raises(ps.PSError) as e:
        srv.ps_pull_snapshot(0, lag=1)
    assert e.value.name == "PS_ERR_VERSION_EVICTED"
    srv.close()


@pytest.mark.parametrize("precision,W,b", [(0, 3, 4), (0, 9, 5), (2, 9, 5), (2, 8, 16)])
def test_tick_from_host_buffers_matches_the_oracle(precision, W, b):
    """ps_tick_host: inputs copied in by worker chunks (four when there are eight workers or more), snapshots
    with lags, grad step into reserved slots, enqueue, sync apply, losses and labels copied out."""
    from oracle import cnn, ps as ops
    import torch
    from paper_2406_05546_b200 import ps
    tol = TOL_TENSOR if precision else TOL_FP32
    theta0 = synth.init_params(seed=1, bias_scale=0.05)
    srv = ps.ParameterServer(theta0, max_workers=W, max_batch=b, ring_depth=2, queue_slots=W, dropout_p=0.25,
                             precision=precision)
    o = ops.OraclePS(theta0, ring_depth=2)
    # one async update first, so that lag 1 reads different weights than lag 0
    g = np.zeros((1, ps.P_PAD), dtype=np.float32)
    g[0, :ps.P] = synth.random_gradients(1, seed=61, scale=2.0)[0]
    srv.ps_enqueue([0], [0], 0, grads_dev=torch.from_numpy(g).cuda())
    srv.ps_apply(ps.ASYNC, 0.01)
    o.enqueue(g[:, :ps.P], [0], [0], 0)
    o.apply(ops.ASYNC, 0.01)
    rng = np.random.default_rng(11)
    x = rng.random((W, b, 28, 28), dtype=np.float32)
    y = rng.integers(0, 10, (W, b)).astype(np.int32)
    lags = [(w * 3) % 2 for w in range(W)]
    am = np.zeros((W, b), dtype=np.int32)
    loss, res = srv.ps_tick_host(x, y, SEED, 5, ps.SYNC, 0.01, lags=lags, argmax_host=am)
    theta, version = srv.ps_export_params()
    srv.ps_stats()
    srv.close()
    thetas = [o.pull_snapshot(w, l)[1] for w, l in enumerate(lags)]
    og, ol, oa, oz = cnn.workers_grad_step(thetas, list(range(W)), x, y, SEED, 5, 0.25, precision=precision)
    o.enqueue(og.astype(np.float32), range(W), [1 - l for l in lags], 5)
    o.apply(ops.SYNC, 0.01)
    assert res["applied"] == W and version == res["new_version"] == 2
    np.testing.assert_allclose(loss, ol, rtol=3e-3 if precision else 1e-5, atol=1e-6)
    assert_argmax_valid(am, oz, tol if precision else 10 * TOL_FP32)
    assert_params_close(theta, o.head(), tol, "parameters after the tick")
    # the tick moves the head by lr * mean gradient: compare that step too, which the parameters' size would hide
    before = o.ring[1].astype(np.float64)
    assert_params_close(theta - before, o.head() - before, max(tol, 10 * TOL_FP32), "the tick's update")


@pytest.mark.parametrize("precision", [0, 2])
def test_pipelined_ticks_equal_sequential_ticks(precision):
    """Two ticks in flight (ps_tick_host_submit / ps_tick_host_wait) leave the same weights, losses, labels and
    versions, bit for bit, as the same ticks run one by one through ps_tick_host."""
    import torch
    from paper_2406_05546_b200 import ps
    W, b, T = 9, 6, 5
    theta0 = synth.init_params(seed=1, bias_scale=0.05)
    rng = np.random.default_rng(3)
    xs = [torch.from_numpy(rng.random((W, b, 28, 28), dtype=np.float32)).pin_memory() for _ in range(T)]
    ys = [torch.from_numpy(rng.integers(0, 10, (W, b)).astype(np.int32)).pin_memory() for _ in range(T)]
    out = []
    for pipelined in (False, True):
        srv = ps.ParameterServer(theta0, max_workers=W, max_batch=b, ring_depth=2, queue_slots=W, precision=precision)
        loss = [np.zeros(W, dtype=np.float32) for _ in range(T)]
        am = [np.zeros((W, b), dtype=np.int32) for _ in range(T)]
        results = []
        if pipelined:
            srv.ps_tick_host_submit(xs[0], ys[0], SEED, 0, ps.SYNC, 0.01, loss_host=loss[0], argmax_host=am[0])
            for t in range(1, T):
                srv.ps_tick_host_submit(xs[t], ys[t], SEED, t, ps.SYNC, 0.01, loss_host=loss[t], argmax_host=am[t])
                results.append(srv.ps_tick_host_wait())
            with pytest.raises(ps.PSError):          # the synchronous form refuses to run while a tick is in flight
                srv.ps_tick_host(xs[0], ys[0], SEED, 99, ps.SYNC, 0.01)
            results.append(srv.ps_tick_host_wait())
            with pytest.raises(ps.PSError):
                srv.ps_tick_host_wait()
        else:
            for t in range(T):
                results.append(srv.ps_tick_host(xs[t], ys[t], SEED, t, ps.SYNC, 0.01, loss_host=loss[t], argmax_host=am[t])[1])
        theta, version = srv.ps_export_params()
        srv.ps_stats()
        srv.close()
        out.append((theta, version, np.stack(loss), np.stack(am), [r["new_version"] for r in results]))
    a, p = out
    assert a[1] == p[1] == T and a[4] == p[4] == list(range(1, T + 1))
    assert (a[0] == p[0]).all() and (a[2] == p[2]).all() and (a[3] == p[3]).all()


@pytest.mark.parametrize("precision,W,b,lags", [(0, 3, 17, None), (2, 3, 17, None), (2, 4, 150, [1, 0, 0, 1]), (0, 1, 1, None)])
def test_evaluation_pass_matches_the_oracle(precision, W, b, lags):
    """workers_eval: forward only, no dropout; loss, labels and the count of correct labels per group."""
    from oracle import cnn
    n_versions = 2 if lags else 1
    torch, ps, srv, theta0 = _setup(W, b, n_versions, 0.25, precision)      # the context's dropout rate must not matter
    versions = {0: theta0}
    if lags:
        g = np.zeros((1, ps.P_PAD), dtype=np.float32)
        g[0, :ps.P] = synth.random_gradients(1, seed=51, scale=2.0)[0]
        srv.ps_enqueue([0], [0], 0, grads_dev=torch.from_numpy(g).cuda())
        srv.ps_apply(ps.ASYNC, 0.01)
        versions[1] = srv.ps_export_params(0)[0]
    rng = np.random.default_rng(8)
    x = rng.random((W, b, 28, 28), dtype=np.float32)
    y = rng.integers(0, 10, (W, b)).astype(np.int32)
    snaps = [srv.ps_pull_snapshot(w, lags[w] if lags else 0) for w in range(W)]
    before = srv.ps_stats()
    loss, am, correct = srv.workers_eval(snaps, torch.from_numpy(x).cuda(), torch.from_numpy(y).cuda())
    after = srv.ps_stats()
    assert after["queue_len"] == before["queue_len"] == 0 and after["version"] == before["version"]
    ol, oa, oc, oz = cnn.workers_eval([versions[s.version] for s in snaps], x, y, precision=precision)
    tol = TOL_TENSOR if precision else TOL_FP32
    np.testing.assert_allclose(loss.cpu().numpy(), ol, rtol=3e-3 if precision else 1e-5, atol=1e-6)
    am = am.cpu().numpy()
    n_amb = assert_argmax_valid(am, oz, tol)
    # the count is exact given the labels the kernel chose; it equals the oracle's where no row is ambiguous
    assert (correct.cpu().numpy() == (am == y).sum(axis=1)).all()
    if n_amb == 0:
        assert (correct.cpu().numpy() == oc).all()
    srv.close()


@pytest.mark.parametrize("precision,W,b", [(0, 3, 5), (0, 8, 9), (2, 2, 8), (2, 8, 24), (2, 17, 6), (2, 6, 70)])
def test_summed_step_equals_the_sum_of_the_workers_gradients_and_the_sync_update(precision, W, b):
    """workers_grad_step_summed + ps_apply_summed: the one vector equals the sum of the oracle's per-worker gradients,
    and the update equals the oracle's synchronous step over those gradients (W = 17 has no divisor up to 16 but 1:
    the whole batch goes through one product; W = 8: eight groups; W = 6: six)."""
    from oracle import cnn, ps as ops
    tol = TOL_TENSOR if precision else TOL_FP32
    torch, ps, srv, theta0 = _setup(W, b, 1, 0.25, precision)
    rng = np.random.default_rng(31)
    x = rng.random((W, b, 28, 28), dtype=np.float32)
    y = rng.integers(0, 10, (W, b)).astype(np.int32)
    ids = [(5 * w + 2) % 251 for w in range(W)]
    snaps = [srv.ps_pull_snapshot(w) for w in range(W)]
    xd, yd = torch.from_numpy(x).cuda(), torch.from_numpy(y).cuda()
    gsum = torch.full((ps.P_PAD,), float("nan"), device="cuda")
    _, loss, am = srv.workers_grad_step_summed(snaps, ids, xd, yd, SEED, 6, grad_sum_dev=gsum)
    srv.ps_stats()
    og, ol, oa, oz = cnn.workers_grad_step([theta0] * W, ids, x, y, SEED, 6, 0.25, precision=precision)
    got = gsum.cpu().numpy()
    assert (got[ps.P:] == 0).all()
    assert_sum_close(got[:ps.P], og, tol, "summed gradient")
    np.testing.assert_allclose(loss.cpu().numpy(), ol, rtol=3e-3 if precision else 1e-5, atol=1e-6)
    assert_argmax_valid(am.cpu().numpy(), oz, tol)
    # the per-worker path gives the same sum (another order of additions)
    gd = torch.zeros((W, ps.P_PAD), device="cuda")
    srv.workers_grad_step(snaps, ids, xd, yd, SEED, 6, grads_dev=gd)
    assert_params_close(got[:ps.P], gd.sum(dim=0).cpu().numpy()[:ps.P], 1e-5 if precision == 0 else 1e-4, "summed vs per-worker path")
    # the server step
    o = ops.OraclePS(theta0)
    o.enqueue(og.astype(np.float32), ids, [0] * W, 6)
    ro = o.apply(ops.SYNC, 0.01)
    rg = srv.ps_apply_summed(gsum, W, 0.01)
    assert ro == rg
    th, v = srv.ps_export_params()
    assert v == 1
    assert_params_close(th, o.head(), tol, "parameters after the summed step")
    assert_params_close(th.astype(np.float64) - theta0, o.head().astype(np.float64) - theta0, max(tol, 1e-3), "the summed step's update")
    # errors: stale readers need the per-worker path; a non-empty queue must be applied first
    g = torch.zeros((1, ps.P_PAD), device="cuda")
    srv.ps_enqueue([0], [1], 7, grads_dev=g)
    with pytest.raises(ps.PSError) as e:
        srv.ps_apply_summed(gsum, W, 0.01)
    assert e.value.name == "PS_ERR_BAD_ARG"
    srv.close()


def test_summed_step_refuses_mixed_snapshots():
    torch, ps, srv, theta0 = _setup(2, 4, 2, 0.25, 0)
    g = np.zeros((1, ps.P_PAD), dtype=np.float32)
    g[0, :ps.P] = synth.random_gradients(1, seed=52, scale=2.0)[0]
    srv.ps_enqueue([0], [0], 0, grads_dev=torch.from_numpy(g).cuda())
    srv.ps_apply(ps.ASYNC, 0.01)
    snaps = [srv.ps_pull_snapshot(0, 0), srv.ps_pull_snapshot(1, 1)]
    x = torch.zeros((2, 4, 28, 28), device="cuda")
    y = torch.zeros((2, 4), dtype=torch.int32, device="cuda")
    with pytest.raises(ps.PSError) as e:
        srv.workers_grad_step_summed(snaps, [0, 1], x, y, SEED, 0)
    assert e.value.name == "PS_ERR_BAD_ARG"
    srv.close()
