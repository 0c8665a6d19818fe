"""UCBSpec on the round's throughput (Section 6.2) through the C ABI against the CPU oracle
(needs a B200): arms bit-exact except at flagged near-ties of the index, rewards and reward sums
bit-exact (integer totals, one fp64 division, the same additions in the same order)."""
import numpy as np
import pytest
import torch

from oracle import bandit as ob
from paper_2505_15141_b200 import workloads as wl
import parity

pytestmark = pytest.mark.gpu
DEV = "cuda"


def test_closed_loop_tiny_tput_per_sequence_rewards(lib):
    w = wl.WORKLOADS["tiny_tput"]
    t = parity.closed_loop(lib, w, w.rounds, DEV)
    assert t.sequences == w.B * w.rounds and t.flagged_arm <= 2


def test_closed_loop_llama3_tput_full_size(lib):
    """48 sequences share the reward: their bandits stay together, the batch has one speculation
    length per round, canonical decoding (gamma = 0) is one of the arms."""
    w = wl.WORKLOADS["llama3_tput"]
    carry = {}
    t = parity.closed_loop(lib, w, 40, DEV, sample=[0, 23, 47], carry=carry)
    t2 = parity.closed_loop(lib, w, w.rounds - 40, DEV, sample=[], first_round=41, carry=carry)
    assert t.flagged_arm + t2.flagged_arm <= 2
    st = lib.bs_bandit_read(carry["state"], lib.BS_UCB_REWARD, w.B, w.K)
    assert (st["n"] == st["n"][0]).all() and (st["t"] == w.rounds).all()      # one trajectory for the whole batch
    n, mean = st["n"][0], st["S"][0] / st["n"][0]
    assert n.min() >= 1 and n.sum() == w.rounds
    assert (mean > 0).all() and (mean <= w.reward_width).all()
    assert n[mean.argmin()] <= n[mean.argmax()]                              # the worst observed arm is not the favourite


def test_indices_match_the_oracle_and_inactive_sequences_are_frozen(lib):
    rng = np.random.default_rng(11)
    B, gam, W = 37, [0, 2, 3, 5, 8, 1], 40.0
    K = len(gam)
    state = lib.new_bandit(lib.BS_UCB_REWARD, B, gam, 0.3, DEV, reward_width=W)
    o = ob.UCBSpecReward(B, gam, W, 0.3)
    arm_d = torch.zeros(B, dtype=torch.int32, device=DEV); gam_d = torch.zeros(B, dtype=torch.int32, device=DEV)
    idx_d = torch.zeros(B, K, dtype=torch.float64, device=DEV)
    means = rng.uniform(5, 30, size=(B, K))
    for t in range(200):
        act = rng.random(B) < 0.8
        act_d = torch.as_tensor(act.astype(np.uint8), device=DEV)
        lib.bs_bandit_select(state, lib.BS_UCB_REWARD, B, K, None, act_d, arm_d, gam_d, idx_d)
        arm_ref, gam_ref, flagged = o.select(act)
        arm = arm_d.cpu().numpy().astype(np.int64)
        assert ((arm == arm_ref) | flagged).all() and (arm[~act] == -1).all()
        assert (gam_d.cpu().numpy()[arm == arm_ref] == gam_ref[arm == arm_ref]).all()
        past = act & (o.t >= K)
        if past.any():
            assert np.allclose(idx_d.cpu().numpy()[past], o.last_index[past], rtol=1e-13, atol=0)
        # rewards stray outside [0, W] and are sometimes NaN: both sides clamp
        r = means[np.arange(B), np.maximum(arm, 0)] + rng.normal(0, 12, size=B)
        r[rng.random(B) < 0.02] = np.nan
        lib.bs_bandit_update_reward(state, B, K, arm_d, torch.as_tensor(r, device=DEV), act_d)
        o.update(arm, r, act)
    st = lib.bs_bandit_read(state, lib.BS_UCB_REWARD, B, K)
    assert (st["n"] == o.n).all() and np.array_equal(st["S"], o.sumR) and (st["t"] == o.t).all()
    assert st["S"].min() >= 0 and (st["S"] <= W * st["n"]).all()


@pytest.mark.parametrize("B", [1, 50, 4096])
def test_throughput_reward_matches_the_oracle(lib, B):
    rng = np.random.default_rng(B)
    y = rng.integers(1, 9, size=B).astype(np.int32)
    act = rng.random(B) < 0.7
    y_d = torch.as_tensor(y, device=DEV); act_d = torch.as_tensor(act.astype(np.uint8), device=DEV)
    out = torch.full((B,), -1.0, dtype=torch.float64, device=DEV)
    for whole in (False, True):
        for a_np, a_d in ((None, None), (act, act_d)):
            lib.bs_throughput_reward(y_d, a_d, B, 0.0371, whole, out)
            assert np.array_equal(out.cpu().numpy(), ob.throughput_reward(y, 0.0371, whole, a_np))


def test_reward_calls_reject_what_they_cannot_use(lib):
    B, K = 4, 3
    state = lib.new_bandit(lib.BS_UCB_REWARD, B, [0, 1, 2], 0.5, DEV, reward_width=10.0)
    arm = torch.zeros(B, dtype=torch.int32, device=DEV); y = torch.ones(B, dtype=torch.int32, device=DEV)
    r = torch.zeros(B, dtype=torch.float64, device=DEV)
    with pytest.raises(lib.BanditSpecError):
        lib.bs_bandit_init(state, lib.BS_UCB_REWARD, B, K, [0, 1, 2], 0.5)          # no reward range
    with pytest.raises(lib.BanditSpecError):
        lib.bs_bandit_update(state, lib.BS_UCB_REWARD, B, K, arm, y)                # integer update on real sums
    for width in (0.0, -1.0, float("inf"), float("nan")):
        with pytest.raises(lib.BanditSpecError):
            lib.bs_bandit_init_reward(state, B, K, [0, 1, 2], 0.5, width)
    for seconds in (0.0, -2.0, float("inf"), float("nan")):
        with pytest.raises(lib.BanditSpecError):
            lib.bs_throughput_reward(y, None, B, seconds, True, r)
    lib.bs_bandit_init_reward(state, B, K, [0, 0, 0], 0.5, 3.0)                     # canonical decoding only: allowed
    torch.cuda.synchronize()


@pytest.mark.parametrize("name,rounds", [("tiny_ucb", 64), ("tiny_tput", 120), ("llama3_ucb", 30), ("qwen_exp3", 30)])
def test_closed_loop_with_the_fused_bandit_step(lib, name, rounds):
    """bs_bandit_step (update of round t + select of round t + 1 in one launch) against the oracle's two
    steps: same arms, same statistics."""
    w = wl.WORKLOADS[name]
    sample = None if w.B <= 8 else [0, w.B // 2, w.B - 1]
    t = parity.closed_loop(lib, w, rounds, DEV, sample=sample, fused_step=True)
    assert t.flagged_arm <= 2


def test_bandit_step_equals_update_then_select(lib):
    rng = np.random.default_rng(5)
    B, gam = 70, [1, 2, 4, 7, 3]
    K = len(gam)
    for alg in (lib.BS_UCB, lib.BS_EXP3):
        sa = lib.new_bandit(alg, B, gam, 0.5, DEV); sb = lib.new_bandit(alg, B, gam, 0.5, DEV)
        arm_a = torch.zeros(B, dtype=torch.int32, device=DEV); arm_b = torch.zeros(B, dtype=torch.int32, device=DEV)
        g_a = torch.zeros(B, dtype=torch.int32, device=DEV); g_b = torch.zeros(B, dtype=torch.int32, device=DEV)
        ia = torch.zeros(B, K, dtype=torch.float64, device=DEV); ib = torch.zeros(B, K, dtype=torch.float64, device=DEV)
        u = torch.as_tensor(rng.random(B).astype(np.float32), device=DEV)
        act = torch.as_tensor((rng.random(B) < 0.85).astype(np.uint8), device=DEV)
        lib.bs_bandit_select(sa, alg, B, K, u, act, arm_a, g_a)
        lib.bs_bandit_select(sb, alg, B, K, u, act, arm_b, g_b)
        for t in range(60):
            y = torch.as_tensor(rng.integers(1, 9, size=B).astype(np.int32), device=DEV)
            u = torch.as_tensor(rng.random(B).astype(np.float32), device=DEV)
            lib.bs_bandit_update(sa, alg, B, K, arm_a, y, act)
            lib.bs_bandit_select(sa, alg, B, K, u, act, arm_a, g_a, ia)
            lib.bs_bandit_step(sb, alg, B, K, y, u, act, arm_b, g_b, ib)
            assert torch.equal(arm_a, arm_b) and torch.equal(g_a, g_b)
            assert torch.equal(torch.nan_to_num(ia, nan=-1.0), torch.nan_to_num(ib, nan=-1.0))
        assert torch.equal(sa, sb)                                        # the whole state blob, bit for bit
