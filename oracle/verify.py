"""CPU checker for one speculative-decoding verification round.  TEST INFRASTRUCTURE.

Plain, slow, fp64 NumPy.  It exists to check the CUDA path and to be timed as
the CPU baseline; nothing in the product path may import it, and it imports
nothing from the product.  Every function follows one passage of the paper:

* softmax with temperature                      -- Section 2 (LLM decoding)
* accept test r <= min{1, P/Q}, first rejection -- Algorithm 6, the for-loop
* residual Norm([P - Q]_+) and its definitions  -- Algorithm 6 (else-branch) and
                                                   the notation paragraph above it
* bonus token from P when all drafts pass       -- Algorithm 6, the line after the loop
* drafted token x~ ~ Q                          -- Algorithm 6, the first line
* greedy decoding as temperature -> 0           -- Section 2
* accepted length counts the bonus token, y = tau + 1 in [1, L+1]  -- Section 3

Where the paper is silent the readings are (all listed in the design notes):
rows are 0-based, row j of either model is conditioned on the first j drafted
tokens; a categorical is sampled from ONE uniform by inverse CDF in vocabulary
order, emitting the smallest v whose cumulative mass strictly exceeds u * total;
Q(x)=0 counts as ratio = +inf (accept); a residual of total mass 0 falls back
to the target row; the arg-max tie-break is the lowest index; in greedy mode
the drafted token is taken to be the draft's arg-max, so only "token == target
arg-max" is tested.

Pins (tests/test_oracle_verify.py): a hand-worked 3-token example, the
distribution of the emitted token against the target by chi-square, the
closed-form acceptance probability sum_v min(p, q), the truncated geometric law
of the accepted length, q == p, brute-force greedy, and numpy.searchsorted for
the categorical special case.  Parity unpinned: the identity of the emitted
token when u lies within rounding of a CDF edge (fixed only by the inverse-CDF
reading above).
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import List, Optional

import numpy as np

ACCEPT_TIE = 1e-5      # |u - min(1, p/q)| below this: the accept decision is flagged
CDF_TIE = 1e-6         # u within this of an edge of the token's CDF interval: flagged


def softmax_row(logits: np.ndarray, temperature: float) -> np.ndarray:
    """softmax(logits / T) of one row, fp64 (Section 2)."""
    z = np.asarray(logits, dtype=np.float64) / float(temperature)
    z = z - z.max()
    e = np.exp(z)
    return e / e.sum()


def argmax_lowest(row: np.ndarray) -> int:
    """Index of the largest logit, lowest index among equals (greedy decoding, Section 2)."""
    return int(np.argmax(np.asarray(row)))  # numpy returns the first maximum


def positive_part(f: np.ndarray) -> np.ndarray:
    """[f]_+ = max{0, f} (notation paragraph before Algorithm 6)."""
    return np.maximum(f, 0.0)


def inverse_cdf(mass: np.ndarray, u: float):
    """Sample Norm(mass) with one uniform: smallest v with sum_{w<=v} mass_w > u * sum(mass).

    Returns (v, lo, hi): the token and the edges of its interval in normalised
    CDF units, lo <= u < hi in exact arithmetic.
    """
    c = np.cumsum(np.asarray(mass, dtype=np.float64))
    total = c[-1]
    v = int(np.searchsorted(c, float(u) * total, side="right"))
    if v >= len(c):                       # u * total == total can only come from rounding
        v = int(np.nonzero(mass > 0)[0][-1])
    lo = (c[v - 1] if v > 0 else 0.0) / total
    hi = c[v] / total
    return v, lo, hi


def draft_token(draft_row: np.ndarray, u: float, temperature: float):
    """Drafting step, Algorithm 6, first line: x~ ~ Q(. | pt, x~_{1:j}) with Q = softmax(draft row / T),
    drawn from ONE uniform by the inverse-CDF reading above; at temperature 0 the arg-max
    (Section 2).  Returns (token, lo, hi) with the token's CDF interval (0, 1 in greedy mode)."""
    if temperature == 0.0:
        return argmax_lowest(draft_row), 0.0, 1.0
    return inverse_cdf(softmax_row(draft_row, temperature), u)


@dataclass
class SequenceResult:
    tau: int                       # number of accepted drafted tokens
    y: int                         # accepted length including the resampled/bonus token
    token: int                     # the resampled (tau < gamma) or bonus (tau == gamma) token
    out_tokens: List[int]          # drafted tokens 1..tau, then `token`
    p_tok: np.ndarray              # [gamma] target probability of each drafted token
    q_tok: np.ndarray              # [gamma] draft probability of each drafted token
    accept_margin: np.ndarray      # [gamma] u_j - min(1, p/q)   (<= 0 means accept)
    cdf_lo: float = 0.0            # CDF interval of `token` (normalised), sampling mode
    cdf_hi: float = 1.0
    used_fallback: bool = False    # residual had zero total mass
    mass: Optional[np.ndarray] = field(default=None, repr=False)   # the sampled mass vector


def verify_sequence(target_rows: np.ndarray, draft_rows: Optional[np.ndarray],
                    tokens: np.ndarray, gamma: int, u_accept: np.ndarray,
                    u_resample: float, temperature: float,
                    keep_mass: bool = False, forced_tau: Optional[int] = None) -> SequenceResult:
    """One sequence of one round: Algorithm 6 from its second line on, given the logits.

    target_rows [>= gamma+1, V], draft_rows [>= gamma, V] (not read when T == 0),
    tokens [>= gamma], u_accept [>= gamma].  `forced_tau` replays the resampling
    step at a given stopping position (used to re-synchronise after a flagged tie).
    """
    gamma = int(gamma)
    if temperature == 0.0:
        return _verify_sequence_greedy(target_rows, tokens, gamma, forced_tau)

    # target and draft distributions of every drafted position ("in parallel")
    Ps = [softmax_row(target_rows[j], temperature) for j in range(gamma)]
    Qs = [softmax_row(draft_rows[j], temperature) for j in range(gamma)]
    p_tok = np.array([Ps[j][int(tokens[j])] for j in range(gamma)], dtype=np.float64)
    q_tok = np.array([Qs[j][int(tokens[j])] for j in range(gamma)], dtype=np.float64)
    margin = np.full(gamma, np.nan)
    for j in range(gamma):
        ratio = np.inf if q_tok[j] == 0.0 else p_tok[j] / q_tok[j]
        margin[j] = float(u_accept[j]) - min(1.0, ratio)

    tau = 0
    stopped = False
    for j in range(gamma):                                   # for k = 1..L
        accept = margin[j] <= 0.0                            # r <= min{1, P/Q}
        if forced_tau is not None:
            accept = j < forced_tau
        if accept:
            tau = j + 1
        else:
            stopped = True
            break
    used_fallback = False
    if stopped:                                              # rejected at row tau
        mass = positive_part(Ps[tau] - Qs[tau])              # [P - Q]_+
        if not mass.sum() > 0.0:
            mass = Ps[tau]
            used_fallback = True
    else:                                                    # tau == gamma: bonus token
        mass = softmax_row(target_rows[gamma], temperature)
    v, lo, hi = inverse_cdf(mass, u_resample)
    return SequenceResult(tau=tau, y=tau + 1, token=v,
                          out_tokens=[int(t) for t in tokens[:tau]] + [v],
                          p_tok=p_tok, q_tok=q_tok, accept_margin=margin,
                          cdf_lo=lo, cdf_hi=hi, used_fallback=used_fallback,
                          mass=mass if keep_mass else None)


def _verify_sequence_greedy(target_rows, tokens, gamma, forced_tau=None) -> SequenceResult:
    """Temperature -> 0 (Section 2): both models are point masses on their arg-max, so the
    drafted token passes iff it is the target's arg-max, and the emitted token at the stop
    (or the bonus token) is the target's arg-max of that row."""
    tau = 0
    for j in range(gamma):
        ok = int(tokens[j]) == argmax_lowest(target_rows[j])
        if forced_tau is not None:
            ok = j < forced_tau
        if ok:
            tau = j + 1
        else:
            break
    v = argmax_lowest(target_rows[tau])
    z = np.zeros(gamma)
    return SequenceResult(tau=tau, y=tau + 1, token=v,
                          out_tokens=[int(t) for t in tokens[:tau]] + [v],
                          p_tok=z, q_tok=z.copy(), accept_margin=np.full(gamma, np.nan))


def verify_round(target: np.ndarray, draft: Optional[np.ndarray], tokens: np.ndarray,
                 gamma: np.ndarray, u_accept: np.ndarray, u_resample: np.ndarray,
                 temperature: float, keep_mass: bool = False) -> List[SequenceResult]:
    """The batch: sequences are independent (Algorithm 3 runs one decoding stream each)."""
    B = target.shape[0]
    return [verify_sequence(target[b], None if draft is None else draft[b], tokens[b],
                            int(gamma[b]), u_accept[b], float(u_resample[b]), temperature,
                            keep_mass=keep_mass)
            for b in range(B)]


def acceptance_probability(P: np.ndarray, Q: np.ndarray) -> float:
    """P(accept) when x ~ Q and r ~ U[0,1]: sum_x Q(x) min{1, P(x)/Q(x)} = sum_x min{P, Q}."""
    return float(np.minimum(P, Q).sum())


def truncated_geometric_pmf(alpha: float, L: int) -> np.ndarray:
    """Law of the accepted length on {1..L+1} (Section 4, truncated geometric distribution):
    alpha^(x-1) (1 - alpha) for x <= L and alpha^L for x = L+1."""
    x = np.arange(1, L + 1)
    return np.concatenate([alpha ** (x - 1) * (1 - alpha), [alpha ** L]])
