"""Parity helpers: compare the CUDA round with the CPU oracle under the flagged-tie rules.

Floating point decides three integers: the accept flag, the inverse-CDF token and the arm.
The oracle works in fp64, the kernels in fp32 (fp64 for the bandits), so a decision may
differ only where the oracle says it is a near-tie:
  accept   |u - min(1, p/q)| < 1e-5 at the first position where the two disagree
  token    u within 1e-6 (normalised CDF units) of an edge of the oracle token's interval, and
           the CUDA token has positive mass and an interval that meets [u - 1e-6, u + 1e-6]
  arm      top two UCB values within 1e-9 (not bit-equal), or u_arm within 1e-9 of a CDF edge
  fallback the residual's total mass is below 2^-17 and the CUDA token is the one the target row gives
Every such event is counted; anything else must match exactly.  After a flagged divergence the
oracle is re-synchronised to the CUDA outcome so that one tie does not derail a trajectory.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import List, Optional, Sequence

import numpy as np
import torch

from oracle import bandit as ob
from oracle import verify as ov
from paper_2505_15141_b200 import workloads as wl

P_TOL = 1e-5
RESIDUAL_FLOOR = 2.0 ** -18     # residual totals at or below this are "no mass" on the device (reading c5)
# EXP3Spec's cumulative loss estimates, fp64 on both sides.  The two exp() routines differ in the
# last bit, and a difference d in S_i moves p_i by about eta * d * p_i, hence the next estimate
# (L+1-y)/(L p_i) by eta * d relative: every pull multiplies the difference by about
# 1 + eta * Z (measured: 1e-16 grows to 9e-7 over 1000 rounds of the 4-armed workload).  So the
# states are compared over stretches of at most a few hundred rounds, within S_RTOL, and a
# trajectory that is carried into another stretch restarts the oracle from the CUDA state.
S_RTOL = 1e-10


@dataclass
class Tally:
    sequences: int = 0
    positions: int = 0
    flagged_accept: int = 0
    flagged_token: int = 0
    flagged_arm: int = 0
    flagged_fallback: int = 0
    max_p_err: float = 0.0
    max_S_rel: float = 0.0
    sum_y: int = 0

    def merge(self, o: "Tally") -> None:
        for k in ("sequences", "positions", "flagged_accept", "flagged_token", "flagged_arm", "flagged_fallback", "sum_y"):
            setattr(self, k, getattr(self, k) + getattr(o, k))
        self.max_p_err = max(self.max_p_err, o.max_p_err)


def to_np(t: torch.Tensor) -> np.ndarray:
    return t.detach().float().cpu().numpy() if t.is_floating_point() else t.detach().cpu().numpy()


def check_sequence(ref: ov.SequenceResult, tau_gpu: int, out_tokens_gpu: np.ndarray, out_len_gpu: int,
                   p_gpu: np.ndarray, q_gpu: np.ndarray, *, target_rows, draft_rows, tokens, gamma: int,
                   u_accept, u_resample: float, temperature: float, tally: Tally, where="",
                   walk: bool = False) -> ov.SequenceResult:
    """Checks one sequence; returns the oracle result the trajectory should continue from.
    walk: the early-exit path examines positions up to the first rejection only, so its token
    probabilities are compared there and must be zero behind it."""
    G1 = len(out_tokens_gpu)
    tally.sequences += 1
    tally.positions += gamma
    greedy = temperature == 0.0
    seen = min(tau_gpu + 1, gamma) if walk else gamma            # positions whose probabilities were formed
    if not greedy and seen:
        err = max(np.abs(p_gpu[:seen] - ref.p_tok[:seen]).max(), np.abs(q_gpu[:seen] - ref.q_tok[:seen]).max())
        tally.max_p_err = max(tally.max_p_err, float(err))
        assert err <= P_TOL, f"{where}: token probability off by {err}"
    assert (p_gpu[seen:] == 0).all() and (q_gpu[seen:] == 0).all(), f"{where}: padded p/q not zero"
    if tau_gpu != ref.tau:
        j = min(tau_gpu, ref.tau)                      # first position where the decisions differ
        assert not greedy, f"{where}: greedy accept_len {tau_gpu} != {ref.tau}"
        assert 0 <= tau_gpu <= gamma and abs(ref.accept_margin[j]) < ov.ACCEPT_TIE, \
            f"{where}: accept_len {tau_gpu} != {ref.tau} and position {j} is no tie (margin {ref.accept_margin[j]})"
        tally.flagged_accept += 1
        ref = ov.verify_sequence(target_rows, draft_rows, tokens, gamma, u_accept, u_resample, temperature,
                                 keep_mass=True, forced_tau=tau_gpu)
    tau = ref.tau
    assert out_len_gpu == tau + 1, f"{where}: out_len {out_len_gpu} != {tau + 1}"
    assert list(out_tokens_gpu[:tau]) == [int(t) for t in tokens[:tau]], f"{where}: accepted tokens differ"
    assert (out_tokens_gpu[tau + 1:] == -1).all(), f"{where}: padding of out_tokens is not -1"
    tok = int(out_tokens_gpu[tau])
    if (tok != ref.token and not greedy and tau < gamma and not ref.used_fallback
            and ref.mass.sum() < 2 * RESIDUAL_FLOOR):
        # P and Q are normalised, so the residual's total is the probability of stopping here; the
        # kernels count a total at or below RESIDUAL_FLOOR as "no mass" and draw from the target row
        alt, lo, hi = ov.inverse_cdf(ov.softmax_row(target_rows[tau], temperature), float(u_resample))
        if tok == alt:
            tally.flagged_fallback += 1
            ref.token, ref.cdf_lo, ref.cdf_hi, ref.used_fallback = tok, lo, hi, True
            ref.out_tokens[-1] = tok
    if tok != ref.token:
        assert not greedy, f"{where}: greedy token {tok} != {ref.token}"
        u = float(u_resample)
        near = min(u - ref.cdf_lo, ref.cdf_hi - u) < ov.CDF_TIE
        mass = ref.mass
        assert mass is not None
        c = np.cumsum(mass) / mass.sum()
        lo, hi = (c[tok - 1] if tok > 0 else 0.0), c[tok]
        ok = near and mass[tok] > 0 and lo <= u + ov.CDF_TIE and hi >= u - ov.CDF_TIE
        assert ok, (f"{where}: token {tok} != {ref.token}; u={u} oracle interval [{ref.cdf_lo}, {ref.cdf_hi}) "
                    f"cuda interval [{lo}, {hi}) mass {mass[tok]}")
        tally.flagged_token += 1
        ref.token = tok
        ref.out_tokens[-1] = tok
    tally.sum_y += tau + 1
    return ref


def check_round(out, rnd: wl.RoundInputs, temperature: float, tally: Tally,
                seqs: Optional[Sequence[int]] = None, where="", walk: bool = False) -> List[Optional[ov.SequenceResult]]:
    """Compares a RoundOutput with the oracle on the sequences `seqs` (default: all)."""
    B = rnd.target.shape[0]
    seqs = range(B) if seqs is None else seqs
    tau = to_np(out.accept_len); ot = to_np(out.out_tokens); ol = to_np(out.out_len)
    pg = to_np(out.p_tok); qg = to_np(out.q_tok)
    toks = to_np(rnd.tokens)
    res: List[Optional[ov.SequenceResult]] = [None] * B
    for b in seqs:
        g = int(rnd.gamma[b])
        t_rows = rnd.target[b, :g + 1].float().cpu().numpy()
        d_rows = None if temperature == 0.0 else rnd.draft[b, :g].float().cpu().numpy()
        ref = ov.verify_sequence(t_rows, d_rows, toks[b], g, rnd.uniforms.u_accept[b],
                                 float(rnd.uniforms.u_resample[b]), temperature, keep_mass=True)
        res[b] = check_sequence(ref, int(tau[b]), ot[b], int(ol[b]), pg[b], qg[b],
                                target_rows=t_rows, draft_rows=d_rows, tokens=toks[b], gamma=g,
                                u_accept=rnd.uniforms.u_accept[b], u_resample=float(rnd.uniforms.u_resample[b]),
                                temperature=temperature, tally=tally, where=f"{where} b={b}", walk=walk)
    return res


def gpu_round(bs, rnd: wl.RoundInputs, temperature: float, workspace=None):
    """Run one verification round through the binding on the device of rnd.target."""
    dev = rnd.target.device
    return bs.verify_round(rnd.target, None if temperature == 0.0 else rnd.draft, rnd.tokens,
                           torch.as_tensor(np.asarray(rnd.gamma, dtype=np.int32), device=dev),
                           torch.as_tensor(rnd.uniforms.u_accept, device=dev),
                           torch.as_tensor(rnd.uniforms.u_resample, device=dev), temperature,
                           workspace=workspace)


def closed_loop(bs, w: wl.Workload, rounds: int, device, sample: Optional[Sequence[int]] = None,
                first_round: int = 1, state=None, oracle_bandit=None, carry: Optional[dict] = None,
                fused_step: bool = False) -> Tally:
    """select -> make inputs for the chosen arms -> verify -> resample -> update, on the GPU and in
    the oracle side by side.  `sample`: sequences whose verification the oracle replays (default
    all); the oracle bandit of the others is fed the CUDA reward (teacher forcing).  fused_step: the
    update of a round and the select of the next go through bs_bandit_step (one launch)."""
    B, K, G, V = w.B, w.K, w.Gmax, w.V
    alg = {None: None, "ucb": bs.BS_UCB, "exp3": bs.BS_EXP3, "ucb_reward": bs.BS_UCB_REWARD}[w.alg]
    tally = Tally()
    ws = bs.new_workspace(B, G, V, device)
    if carry is not None and "state" in carry:           # continue a trajectory started by an earlier call
        state, oracle_bandit = carry["state"], carry["oracle_bandit"]
    if alg is not None and state is None:
        if w.alg == "ucb_reward":
            state = bs.new_bandit(alg, B, w.arm_gamma, w.delta, device, reward_width=w.reward_width)
            oracle_bandit = ob.UCBSpecReward(B, w.arm_gamma, w.reward_width, w.delta)
        else:
            state = bs.new_bandit(alg, B, w.arm_gamma, w.delta, device)
            oracle_bandit = ob.UCBSpec(B, w.arm_gamma, w.delta) if w.alg == "ucb" else ob.EXP3Spec(B, w.arm_gamma)
    if carry is not None:
        carry["state"], carry["oracle_bandit"] = state, oracle_bandit
    arm_d = torch.zeros(B, dtype=torch.int32, device=device)
    gamma_d = torch.full((B,), w.arm_gamma[0], dtype=torch.int32, device=device)
    for rnd_i in range(first_round, first_round + rounds):
        un = wl.round_uniforms(w.seed, rnd_i, B, G)
        if alg is not None:
            u_arm_d = torch.as_tensor(un.u_arm, device=device)
            if not fused_step or rnd_i == first_round:       # later rounds: chosen by the step call of the round before
                bs.bs_bandit_select(state, alg, B, K, u_arm_d, None, arm_d, gamma_d)
            arm_gpu = to_np(arm_d).astype(np.int64)
            if w.alg in ("ucb", "ucb_reward"):
                arm_ref, _, flagged = oracle_bandit.select()
            else:
                arm_ref, _, flagged = oracle_bandit.select(un.u_arm)
            diff = np.nonzero(arm_gpu != arm_ref)[0]
            for b in diff:
                assert flagged[b], f"round {rnd_i} b={b}: arm {arm_gpu[b]} != {arm_ref[b]} without a tie"
                tally.flagged_arm += 1
                if w.alg == "exp3":
                    oracle_bandit.p_sel[b] = oracle_bandit.last_p[b][arm_gpu[b]]
            arm = arm_gpu
            assert (to_np(gamma_d) == np.asarray(w.arm_gamma)[arm]).all()
        else:
            arm = np.zeros(B, dtype=np.int64)
        rnd = wl.make_round(w, rnd_i, arm, device=device)
        out = gpu_round(bs, rnd, w.temperature, ws)
        status = bs.bs_get_device_status(ws, B, G, V)
        assert (status & ~bs.BS_DEV_RESIDUAL_FALLBACK == 0).all(), f"round {rnd_i}: device status {status}"
        refs = check_round(out, rnd, w.temperature, tally, seqs=sample, where=f"round {rnd_i}")
        y_gpu = to_np(out.out_len).astype(np.int64)
        y = y_gpu.copy()
        for b, r in enumerate(refs):
            if r is not None:
                y[b] = r.y                       # equal to the CUDA value unless the check failed
        assert (y == y_gpu).all()
        if w.alg == "ucb_reward":
            # the round's throughput as the reward; the duration is the workload's stand-in for a measurement
            seconds = wl.step_seconds(w, np.asarray(w.arm_gamma)[arm])
            rew_d = torch.empty(B, dtype=torch.float64, device=device)
            bs.bs_throughput_reward(out.out_len, None, B, seconds, w.whole_batch, rew_d)
            rew = ob.throughput_reward(y, seconds, w.whole_batch)
            assert np.array_equal(rew_d.cpu().numpy(), rew), f"round {rnd_i}: throughput reward differs"
            assert rew.max() <= w.reward_width
            if fused_step and rnd_i + 1 < first_round + rounds:
                bs.bs_bandit_step(state, alg, B, K, rew_d, None, None, arm_d, gamma_d)
            else:
                bs.bs_bandit_update_reward(state, B, K, arm_d, rew_d)
            oracle_bandit.update(arm, rew)
        elif alg is not None:
            if fused_step and rnd_i + 1 < first_round + rounds:
                u_next = torch.as_tensor(wl.round_uniforms(w.seed, rnd_i + 1, B, G).u_arm, device=device)
                bs.bs_bandit_step(state, alg, B, K, out.out_len, u_next, None, arm_d, gamma_d)
            else:
                bs.bs_bandit_update(state, alg, B, K, arm_d, out.out_len)
            oracle_bandit.update(arm, y)
    if alg is not None:
        st = bs.bs_bandit_read(state, alg, B, K)
        assert (st["t"] == oracle_bandit.t).all()
        if w.alg == "ucb":
            assert (st["n"] == oracle_bandit.n).all() and (st["sumY"] == oracle_bandit.sumY).all()
        elif w.alg == "ucb_reward":                      # the same fp64 additions in the same order
            assert (st["n"] == oracle_bandit.n).all() and np.array_equal(st["S"], oracle_bandit.sumR)
        else:
            rel = np.abs(st["S"] - oracle_bandit.S) / np.maximum(np.abs(oracle_bandit.S), 1e-12)
            tally.max_S_rel = max(tally.max_S_rel, float(rel.max()))
            assert rel.max() <= S_RTOL, f"cumulative losses off by {rel.max()} (relative) after round {oracle_bandit.t.max()}"
            if carry is not None:
                oracle_bandit.S[...] = st["S"]
    return tally
