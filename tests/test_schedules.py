"""CPU checks of the schedule tables and of the oracle driven through them (no GPU)."""
import numpy as np

from paper_2406_05546_b200 import schedules, synth
from tests import oracle_driver


def test_full_size_tables_match_the_stated_workloads():
    s2, s3, s4, s5 = (schedules.config(n) for n in (2, 3, 4, 5))
    assert (s2.W, s2.b, s2.ticks, s2.ckpt_every, s2.kill_at, s2.recover_at) == (8, 64, 200, 25, 60, 80)
    assert (s3.W, s3.b) == (16, 64) and s3.W * (s3.recover_at - s3.kill_at) == 1600
    assert (s4.W, s4.b, s4.ring_depth, s4.max_lag, s4.chain_len, s4.replicate_every) == (64, 32, 9, 8, 2, 1)
    assert (s5.W, s5.b, s5.ticks) == (128, 128, 1000) and s5.W * (s5.recover_at - s5.kill_at) == 25600
    assert abs(25600 * 813258 * 4 / 1e9 - 83.3) < 0.1 and abs(1600 * 813258 * 4 / 1e9 - 5.2) < 0.01
    # stateful outage: workers idle; stateless outage: workers keep producing, nothing applied
    assert not schedules.plan(s2, 70).workers_run and not schedules.plan(s2, 70).apply
    assert schedules.plan(s3, 150).workers_run and not schedules.plan(s3, 150).apply
    assert schedules.plan(s3, 200).pre == ["restore"] and schedules.plan(s3, 200).catch_up
    assert schedules.plan(s4, 300).pre == ["kill", "failover"] and schedules.plan(s4, 300).apply


def test_oracle_follows_reduced_schedules_with_the_expected_counters():
    px, py = synth.image_pool(512, seed=0)
    theta = synth.init_params(1)
    # stateless: 10 ticks of backlog (W=4) consumed by one replay; versions count server steps
    s = schedules.reduced(3)
    o = oracle_driver.make_oracle(s, theta)
    log = oracle_driver.run(s, o, px, py)
    assert [e["queue_len"] for e in log[9:21]] == [0, 4, 8, 12, 16, 20, 24, 28, 32, 36, 40, 0]
    assert log[20]["apply"]["applied"] == 44 and log[-1]["version"] == 20
    # async chain: 8 versions per tick, failover at tick 30 keeps the mirrored head (R = 1)
    s = schedules.reduced(4)
    o = oracle_driver.make_oracle(s, theta)
    log = oracle_driver.run(s, o, px, py)
    assert log[29]["version"] == 240 and log[30]["events"] == [("failover", 240)] and log[-1]["version"] == 320
    assert np.isfinite(o.head()).all()


def test_lags_and_orders_are_seeded_and_in_range():
    l = synth.lags(7, 64, 8)
    assert (l == synth.lags(7, 64, 8)).all() and l.min() >= 0 and l.max() <= 8 and len(set(l)) > 4
    o = synth.arrival_order(7, 64)
    assert sorted(o) == list(range(64)) and (o != synth.arrival_order(8, 64)).any()
