"""CPU checker for the arm-selection algorithms UCBSpec and EXP3Spec.  TEST INFRASTRUCTURE.

Plain fp64 Python/NumPy written from Algorithm 4 / Algorithm 8 (UCBSpec) and
Algorithm 5 / Algorithm 9 (EXP3Spec).  Nothing in the product path may import
it and it imports nothing from the product.  One independent bandit instance
per sequence; the history H_t is reduced to its sufficient statistics.

Readings where the paper is silent or its two listings differ (all listed in
the design notes): L is the largest speculation length of the configuration and
is the same for every arm; delta is a parameter (0.5 in the regret proof);
`t` inside the confidence radius is the number of completed rounds; rounds
1..K play arms 1..K in order; arg-max ties go to the lowest index; log is
natural; EXP3Spec follows the full listing (Algorithm 9): the probability
vector that draws I_t is the one that divides the loss estimate of round t, and
eta_t uses the current round index t >= 1; exp(-eta * S) is evaluated after
subtracting min S (same distribution); I_t ~ p_t is drawn by inverse CDF from
one uniform, smallest i whose cumulative probability strictly exceeds u.

UCBSpecReward is UCBSpec fed a real-valued reward (Section 6.2 takes the current
throughput, generated tokens per second, as the reward and gives no formula).  Reading: the
listing of Algorithm 8 is kept, the history holds the real rewards, and the factor L/2 of the
confidence radius -- half the width of the interval [1, L+1] the accepted length lives in --
becomes half the width W of the interval [0, W] the caller declares for its reward.
throughput_reward is the reward itself: tokens emitted in the round over the seconds the round
took, per sequence or for the whole batch.  Their pins: UCBSpecReward with W = L and the
accepted length as reward plays UCBSpec's arms; scaling rewards and W together, or shifting
every reward, leaves the arms unchanged; a hand-worked trajectory (tests/golden).

Pins (tests/test_oracle_bandit.py): the round-robin prefix, hand-worked arm
sequences for scripted rewards (tests/golden), a hand-worked radius value,
monotonicity of the radius, p_1 uniform and sum p = 1, p_t against
scipy.special.softmax(-eta_t * S), the identity p_t^T Zhat_t = (L+1-y_t)/L from
the proof of Theorem 3, and unbiasedness of Zhat by Monte Carlo.
"""
from __future__ import annotations

import math
from typing import Optional, Sequence

import numpy as np

UCB_TIE = 1e-9     # top-two index values closer than this (and not bit-equal): flagged
ARM_CDF_TIE = 1e-9  # u_arm within this of an EXP3 CDF edge: flagged


def confidence_radius(L: float, K: int, t: int, n: int, delta: float) -> float:
    """cr_{i,t} of Algorithm 4: (L/2) sqrt( (1+n)/n^2 * (1 + 2 log(K t^2 (1+n)^(1/2) / delta)) )."""
    return (L / 2.0) * math.sqrt((1.0 + n) / (n * n)
                                 * (1.0 + 2.0 * math.log(K * t * t * math.sqrt(1.0 + n) / delta)))


class UCBSpec:
    """Algorithm 8 for B independent sequences."""

    def __init__(self, B: int, arm_gamma: Sequence[int], delta: float = 0.5):
        self.B, self.K = B, len(arm_gamma)
        self.arm_gamma = np.asarray(arm_gamma, dtype=np.int64)
        self.L = int(max(arm_gamma))
        self.delta = float(delta)
        self.n = np.zeros((B, self.K), dtype=np.int64)       # n_{i,t}
        self.sumY = np.zeros((B, self.K), dtype=np.int64)    # sum_s Y_{i,s} 1{I_s = i}
        self.t = np.zeros(B, dtype=np.int64)                 # completed rounds
        self.last_index = np.full((B, self.K), np.nan)       # UCB_{i,t-1} used by the last select

    def index_values(self, b: int) -> np.ndarray:
        t = int(self.t[b])
        out = np.empty(self.K)
        for i in range(self.K):
            n = int(self.n[b, i])
            out[i] = self.sumY[b, i] / n + confidence_radius(self.L, self.K, t, n, self.delta)
        return out

    def select(self, active: Optional[np.ndarray] = None):
        """Returns (arm[B], gamma[B], flagged[B]); inactive sequences get arm -1, gamma 0."""
        arm = np.full(self.B, -1, dtype=np.int64)
        flagged = np.zeros(self.B, dtype=bool)
        for b in range(self.B):
            if active is not None and not active[b]:
                continue
            t = int(self.t[b])
            if t < self.K:                       # round-robin over the first K rounds
                arm[b] = t
                continue
            ucb = self.index_values(b)
            self.last_index[b] = ucb
            a = int(np.argmax(ucb))              # first maximum = lowest index
            arm[b] = a
            if self.K > 1:
                second = np.partition(ucb, -2)[-2]
                flagged[b] = (ucb[a] - second) < UCB_TIE and ucb[a] != second
        gamma = np.where(arm >= 0, self.arm_gamma[np.maximum(arm, 0)], 0)
        return arm, gamma, flagged

    def update(self, arm: np.ndarray, y: np.ndarray, active: Optional[np.ndarray] = None):
        for b in range(self.B):
            if active is not None and not active[b]:
                continue
            a = int(arm[b])
            self.n[b, a] += 1
            self.sumY[b, a] += int(y[b])
            self.t[b] += 1


class EXP3Spec:
    """Algorithm 9 for B independent sequences."""

    def __init__(self, B: int, arm_gamma: Sequence[int]):
        self.B, self.K = B, len(arm_gamma)
        self.arm_gamma = np.asarray(arm_gamma, dtype=np.int64)
        self.L = int(max(arm_gamma))
        self.S = np.zeros((B, self.K), dtype=np.float64)     # sum_{s<t} Zhat_{i,s}
        self.t = np.zeros(B, dtype=np.int64)                 # completed rounds
        self.p_sel = np.ones(B, dtype=np.float64)            # p_{t, I_t} of the pending round
        self.last_p = np.full((B, self.K), np.nan)

    def learning_rate(self, t: int) -> float:
        """eta_t = sqrt(log K / (t K)), t >= 1."""
        return math.sqrt(math.log(self.K) / (t * self.K))

    def probabilities(self, b: int) -> np.ndarray:
        """p_{t,i} proportional to exp(-eta_t * sum_{s<t} Zhat_{i,s}), for the round t = completed + 1."""
        eta = self.learning_rate(int(self.t[b]) + 1)
        s = self.S[b]
        w = np.array([math.exp(-eta * (s[i] - s.min())) for i in range(self.K)])
        tot = 0.0
        for i in range(self.K):
            tot += w[i]
        return w / tot

    def select(self, u_arm: np.ndarray, active: Optional[np.ndarray] = None):
        arm = np.full(self.B, -1, dtype=np.int64)
        flagged = np.zeros(self.B, dtype=bool)
        for b in range(self.B):
            if active is not None and not active[b]:
                continue
            p = self.probabilities(b)
            self.last_p[b] = p
            u = float(u_arm[b])
            c = 0.0
            a = self.K - 1                       # last arm if rounding leaves the sum below u
            for i in range(self.K):
                c += p[i]
                if abs(c - u) < ARM_CDF_TIE and i < self.K - 1:
                    flagged[b] = True
                if c > u:
                    a = i
                    break
            arm[b] = a
            self.p_sel[b] = p[a]
        gamma = np.where(arm >= 0, self.arm_gamma[np.maximum(arm, 0)], 0)
        return arm, gamma, flagged

    def loss_estimate(self, b: int, arm: int, y: int) -> float:
        """Zhat_{I_t,t} = (L + 1 - y) / (L p_{t,I_t})."""
        return (self.L + 1 - int(y)) / (self.L * self.p_sel[b])

    def update(self, arm: np.ndarray, y: np.ndarray, active: Optional[np.ndarray] = None):
        for b in range(self.B):
            if active is not None and not active[b]:
                continue
            a = int(arm[b])
            self.S[b, a] += self.loss_estimate(b, a, int(y[b]))
            self.t[b] += 1


class UCBSpecReward:
    """Algorithm 8 with a real reward in [0, W] in place of the accepted length (Section 6.2: the
    reward is the current throughput; arms are speculation lengths, gamma = 0 being canonical
    decoding, Algorithm 1)."""

    def __init__(self, B: int, arm_gamma: Sequence[int], width: float, delta: float = 0.5):
        self.B, self.K = B, len(arm_gamma)
        self.arm_gamma = np.asarray(arm_gamma, dtype=np.int64)
        self.W = float(width)
        self.delta = float(delta)
        self.n = np.zeros((B, self.K), dtype=np.int64)
        self.sumR = np.zeros((B, self.K), dtype=np.float64)  # sum of the rewards of arm i, in the order received
        self.t = np.zeros(B, dtype=np.int64)
        self.last_index = np.full((B, self.K), np.nan)

    def index_values(self, b: int) -> np.ndarray:
        t = int(self.t[b])
        out = np.empty(self.K)
        for i in range(self.K):
            n = int(self.n[b, i])
            out[i] = self.sumR[b, i] / n + confidence_radius(self.W, self.K, t, n, self.delta)
        return out

    def select(self, active: Optional[np.ndarray] = None):
        arm = np.full(self.B, -1, dtype=np.int64)
        flagged = np.zeros(self.B, dtype=bool)
        for b in range(self.B):
            if active is not None and not active[b]:
                continue
            t = int(self.t[b])
            if t < self.K:
                arm[b] = t
                continue
            ucb = self.index_values(b)
            self.last_index[b] = ucb
            a = int(np.argmax(ucb))
            arm[b] = a
            if self.K > 1:
                second = np.partition(ucb, -2)[-2]
                flagged[b] = (ucb[a] - second) < UCB_TIE * max(1.0, self.W) and ucb[a] != second
        gamma = np.where(arm >= 0, self.arm_gamma[np.maximum(arm, 0)], 0)
        return arm, gamma, flagged

    def update(self, arm: np.ndarray, reward: np.ndarray, active: Optional[np.ndarray] = None):
        """Rewards outside [0, W] are clamped into it; NaN counts as 0."""
        for b in range(self.B):
            if active is not None and not active[b]:
                continue
            a = int(arm[b])
            r = float(reward[b])
            r = 0.0 if math.isnan(r) else min(max(r, 0.0), self.W)
            self.n[b, a] += 1
            self.sumR[b, a] += r
            self.t[b] += 1


def throughput_reward(y: np.ndarray, seconds: float, whole_batch: bool,
                      active: Optional[np.ndarray] = None) -> np.ndarray:
    """Tokens per second of the round (Section 6.2).  y[b]: tokens sequence b emitted in the round
    (accepted drafts plus the resampled or bonus token).  Per sequence: y[b] / seconds.  Whole
    batch: (sum of y over the active sequences) / seconds for every active sequence, so bandits
    started together stay together and the batch shares one speculation length.  Inactive: 0."""
    y = np.asarray(y, dtype=np.int64)
    act = np.ones(len(y), dtype=bool) if active is None else np.asarray(active, dtype=bool)
    out = np.zeros(len(y), dtype=np.float64)
    if whole_batch:
        total = int(y[act].sum())
        out[act] = float(total) / float(seconds)
    else:
        for b in range(len(y)):
            if act[b]:
                out[b] = float(int(y[b])) / float(seconds)
    return out
