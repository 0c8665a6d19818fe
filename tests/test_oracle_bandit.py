"""Pins of the UCBSpec / EXP3Spec checker: hand-worked trajectories, identities from the
regret proofs, library softmax, Monte-Carlo unbiasedness."""
import math

import numpy as np
import pytest

from conftest import golden_lines
from oracle import bandit as ob


def test_ucbspec_round_robin_prefix():
    for K in (1, 2, 5):
        u = ob.UCBSpec(3, list(range(1, K + 1)))
        for t in range(K):
            arm, gamma, _ = u.select()
            assert (arm == t).all() and (gamma == t + 1).all()
            u.update(arm, np.full(3, 1 + t % 2))


def test_ucbspec_hand_worked_radius_and_monotonicity():
    # (L/2) sqrt((1+n)/n^2 (1 + 2 ln(K t^2 sqrt(1+n)/delta))) at L=4, K=2, t=2, n=1, delta=.5:
    # 2 * sqrt(2 * (1 + 2 ln(2*4*1.414214/0.5))) = 2 * sqrt(2 * 7.238369) = 7.609638
    assert abs(ob.confidence_radius(4, 2, 2, 1, 0.5) - 7.609638) < 1e-6
    for t in (5, 50, 5000):
        cr = [ob.confidence_radius(8, 4, t, n, 0.5) for n in range(1, 60)]
        assert all(a > b for a, b in zip(cr, cr[1:]))            # shrinks with pulls
    assert ob.confidence_radius(8, 4, 100, 3, 0.5) > ob.confidence_radius(8, 4, 10, 3, 0.5)  # grows with t
    assert abs(ob.confidence_radius(8, 4, 9, 3, 0.5) / ob.confidence_radius(4, 4, 9, 3, 0.5) - 2) < 1e-12


def test_ucbspec_scripted_trajectory():
    rows = golden_lines("ucbspec_scripted.txt")
    u = ob.UCBSpec(1, [2, 4, 6], delta=0.5)
    assert u.L == 6
    for f in rows:
        arm, _, flagged = u.select()
        assert int(arm[0]) == int(f[1]), f
        if f[3] != "rr":
            want = np.array([float(x) for x in f[3:6]])
            assert np.allclose(u.last_index[0], want, atol=2e-6), f
        u.update(arm, np.array([int(f[2])]))
    assert list(u.n[0]) == [4, 4, 4] and list(u.sumY[0]) == [9, 15, 11] and u.t[0] == 12


def test_ucbspec_equal_counts_follow_the_mean_and_ties_go_low():
    u = ob.UCBSpec(1, [1, 2, 3])
    u.n[:] = 5; u.sumY[0] = [10, 14, 12]; u.t[:] = 15
    assert int(u.select()[0][0]) == 1
    u.sumY[0] = [14, 14, 12]
    arm, _, flagged = u.select()
    assert int(arm[0]) == 0 and not flagged[0]


def test_ucbspec_finds_the_best_arm_eventually():
    rng = np.random.default_rng(0)
    u = ob.UCBSpec(1, [2, 4, 8])
    means = [1.5, 2.5, 6.0]
    pulls = np.zeros(3)
    for t in range(6000):
        arm, _, _ = u.select()
        a = int(arm[0]); pulls[a] += 1
        y = int(np.clip(round(rng.normal(means[a], 1.0)), 1, 9))
        u.update(arm, np.array([y]))
    assert pulls[2] > 0.6 * pulls.sum()


def test_exp3spec_scripted_trajectory():
    rows = golden_lines("exp3spec_scripted.txt")
    e = ob.EXP3Spec(1, [2, 4])
    us = [0.3, 0.9, 0.5, 0.2, 0.7]
    for f, u_arm in zip(rows, us):
        t = int(f[0])
        assert abs(e.learning_rate(t) - float(f[1])) < 1e-6
        arm, _, _ = e.select(np.array([u_arm]))
        assert np.allclose(e.last_p[0], [float(f[2]), float(f[3])], atol=1e-6)
        assert int(arm[0]) == int(f[4])
        y = int(f[5])
        assert abs(e.loss_estimate(0, int(arm[0]), y) - float(f[6])) < 1e-6
        e.update(arm, np.array([y]))
        assert np.allclose(e.S[0], [float(f[7]), float(f[8])], atol=1e-6)


def test_exp3spec_probabilities_are_the_ftrl_softmax():
    """p_1 is uniform; p_t = softmax(-eta_t * S_{t-1}) (the FTRL/negentropy view in the
    proof of Theorem 3), compared with scipy's softmax; sums to one."""
    from scipy.special import softmax
    rng = np.random.default_rng(1)
    for K in (1, 2, 4, 7):
        e = ob.EXP3Spec(2, list(range(1, K + 1)))
        assert np.allclose(e.probabilities(0), np.full(K, 1.0 / K), atol=1e-15)
        for t in range(1, 40):
            u = rng.random(2)
            arm, _, _ = e.select(u)
            for b in range(2):
                eta = math.sqrt(math.log(K) / (t * K))
                assert np.allclose(e.last_p[b], softmax(-eta * e.S[b]), atol=1e-12)
                assert abs(e.last_p[b].sum() - 1.0) < 1e-12
            e.update(arm, rng.integers(1, K + 2, size=2))
        assert (e.t == 39).all()


def test_exp3spec_loss_identity_every_round():
    """p_t^T Zhat_t = (L + 1 - y_t) / L  (first display in the proof of Theorem 3)."""
    rng = np.random.default_rng(2)
    e = ob.EXP3Spec(1, [1, 3, 5, 8])
    for t in range(200):
        arm, _, _ = e.select(rng.random(1))
        y = int(rng.integers(1, e.L + 2))
        zhat = np.zeros(4); zhat[int(arm[0])] = e.loss_estimate(0, int(arm[0]), y)
        assert abs(e.last_p[0] @ zhat - (e.L + 1 - y) / e.L) < 1e-12
        before = e.S.copy()
        e.update(arm, np.array([y]))
        changed = np.nonzero(e.S[0] != before[0])[0]
        assert set(changed) <= {int(arm[0])}                      # indicator: other arms untouched


def test_exp3spec_loss_estimate_is_unbiased():
    """E[Zhat_{i,t}] = z_{i,t} = 1 - (y_{i,t} - 1)/L over the draw of the arm."""
    rng = np.random.default_rng(3)
    K, L = 3, 6
    y_of_arm = np.array([2, 7, 4])
    S0 = np.array([0.5, 3.0, 1.2])
    n = 60000
    acc = np.zeros(K); sq = np.zeros(K)
    e = ob.EXP3Spec(1, [2, 4, 6])
    for _ in range(n):
        e.S[0] = S0; e.t[0] = 7
        arm, _, _ = e.select(rng.random(1))
        a = int(arm[0])
        z = e.loss_estimate(0, a, int(y_of_arm[a]))
        acc[a] += z; sq[a] += z * z
    mean = acc / n
    sd = np.sqrt(np.maximum(sq / n - mean ** 2, 1e-12) / n)
    want = 1.0 - (y_of_arm - 1) / L
    assert (np.abs(mean - want) < 5 * sd + 1e-9).all()


def test_exp3spec_arm_draw_frequencies():
    rng = np.random.default_rng(4)
    e = ob.EXP3Spec(1, [1, 2, 3, 4])
    e.S[0] = [0.0, 2.0, 1.0, 5.0]; e.t[0] = 3
    p = e.probabilities(0)
    n = 40000
    hist = np.zeros(4)
    for _ in range(n):
        hist[int(e.select(rng.random(1))[0][0])] += 1
    assert (np.abs(hist / n - p) < 5 * np.sqrt(p * (1 - p) / n)).all()
    # inverse CDF edges: strict crossing
    c = np.cumsum(p)
    assert int(e.select(np.array([c[0] - 1e-7]))[0][0]) == 0
    assert int(e.select(np.array([c[0] + 1e-7]))[0][0]) == 1
    assert int(e.select(np.array([1 - 1e-12]))[0][0]) == 3


def test_single_arm_configurations():
    e = ob.EXP3Spec(2, [5])
    arm, gamma, _ = e.select(np.array([0.3, 0.9]))
    assert (arm == 0).all() and (gamma == 5).all() and e.learning_rate(3) == 0.0
    e.update(arm, np.array([3, 6]))
    assert np.allclose(e.S[:, 0], [(6 - 3) / 5, 0.0])
    u = ob.UCBSpec(2, [5])
    for _ in range(4):
        arm, gamma, _ = u.select()
        assert (arm == 0).all()
        u.update(arm, np.array([2, 3]))


def test_active_mask_freezes_sequences():
    u = ob.UCBSpec(2, [1, 2])
    act = np.array([True, False])
    arm, gamma, _ = u.select(act)
    assert arm[1] == -1 and gamma[1] == 0
    u.update(arm, np.array([2, 2]), act)
    assert u.t[0] == 1 and u.t[1] == 0 and u.n[1].sum() == 0


# ---- UCBSpec with a real reward (Section 6.2) ----------------------------------------------------

def test_ucbspec_reward_scripted_trajectory():
    rows = golden_lines("ucbspec_reward_scripted.txt")
    u = ob.UCBSpecReward(1, [0, 3], width=10.0, delta=0.5)
    for f in rows:
        arm, gamma, _ = u.select()
        assert int(arm[0]) == int(f[1]) and int(gamma[0]) == [0, 3][int(f[1])], f
        if f[3] != "rr":
            assert np.allclose(u.last_index[0], [float(f[3]), float(f[4])], atol=2e-6), f
        u.update(arm, np.array([float(f[2])]))
    assert list(u.n[0]) == [4, 4] and list(u.sumR[0]) == [13.25, 13.5] and u.t[0] == 8


def test_ucbspec_reward_with_accepted_lengths_plays_ucbspec():
    """W = L and reward = accepted length - 1 (the accepted length lives in [1, L+1], an interval of
    width L): the listing of UCBSpec with every mean lowered by one, so the same arms."""
    rng = np.random.default_rng(3)
    gam = [1, 2, 4, 6]
    a, r = ob.UCBSpec(5, gam, delta=0.5), ob.UCBSpecReward(5, gam, width=6.0, delta=0.5)
    for t in range(300):
        arm_a, g_a, fl = a.select()
        arm_r, g_r, _ = r.select()
        same = arm_a == arm_r
        assert (same | fl).all() and (g_a[same] == g_r[same]).all()
        if t >= 4:
            assert np.allclose(a.last_index, r.last_index + 1.0, rtol=0, atol=1e-12)
        y = np.array([rng.integers(1, gam[i] + 2) for i in arm_a])
        a.update(arm_a, y)
        r.update(arm_a, (y - 1).astype(np.float64))
    assert np.array_equal(a.n, r.n) and np.array_equal((a.sumY - a.n).astype(np.float64), r.sumR)


def test_ucbspec_reward_scale_and_shift_leave_the_arms_unchanged():
    """Index = mean + (W/2) f(n, t): scaling rewards and W by c scales every index by c; adding a
    constant to every reward adds it to every index.  Either way the arg-max stays."""
    rng = np.random.default_rng(4)
    gam = [0, 1, 2, 3, 4]
    base = ob.UCBSpecReward(1, gam, width=8.0)
    scaled = ob.UCBSpecReward(1, gam, width=8.0 * 4.0)               # powers of two: exact scaling
    shifted = ob.UCBSpecReward(1, gam, width=8.0)
    means = np.array([2.0, 2.6, 3.1, 2.9, 2.2])
    for t in range(400):
        arm, _, flagged = base.select()
        a2, a3 = scaled.select()[0], shifted.select()[0]
        assert (arm == a2).all()
        assert (arm == a3).all() or flagged.any()
        if t >= 5:
            assert np.array_equal(scaled.last_index, 4.0 * base.last_index)
            assert np.allclose(shifted.last_index, base.last_index + 0.5, rtol=0, atol=1e-12)
        r = np.clip(means[arm] + rng.normal(0, 0.7, size=1), 0.0, 7.0)
        r = np.round(r * 64) / 64                                    # dyadic rewards: sums are exact
        base.update(arm, r); scaled.update(arm, 4.0 * r); shifted.update(arm, r + 0.5)
    assert base.n[0].argmax() == 2                                   # and it has found the best arm


def test_ucbspec_reward_clamps_into_the_declared_range():
    u = ob.UCBSpecReward(1, [0, 1], width=5.0)
    for r in (7.5, -1.0, float("nan"), 2.0):
        arm, _, _ = u.select() if u.t[0] < 2 else (np.array([0]), None, None)
        u.update(np.array([0]), np.array([r]))
    assert u.sumR[0, 0] == 5.0 + 0.0 + 0.0 + 2.0 and u.n[0, 0] == 4


def test_throughput_reward_closed_forms():
    y = np.array([3, 1, 2, 5])
    assert list(ob.throughput_reward(y, 0.5, whole_batch=False)) == [6.0, 2.0, 4.0, 10.0]
    assert list(ob.throughput_reward(y, 0.5, whole_batch=True)) == [22.0] * 4
    act = np.array([1, 0, 1, 1], dtype=bool)
    assert list(ob.throughput_reward(y, 0.25, whole_batch=False, active=act)) == [12.0, 0.0, 8.0, 20.0]
    assert list(ob.throughput_reward(y, 0.25, whole_batch=True, active=act)) == [40.0, 0.0, 40.0, 40.0]
    # gamma = 0 everywhere (canonical decoding): one token per sequence and round
    assert list(ob.throughput_reward(np.ones(3, dtype=np.int64), 2.0, whole_batch=True)) == [1.5] * 3
