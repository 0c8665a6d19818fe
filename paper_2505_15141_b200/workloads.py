"""Seeded synthetic inputs for the batched speculative-verification round.

This module only *makes inputs*: logits, drafted tokens and the uniform random
numbers a round consumes.  It contains none of the verification or bandit
arithmetic and loads no native code, so the CUDA path and the CPU checker can
both be fed from it without sharing anything else.

The inputs stand in for LLM decoding traffic (real models and prompt sets are
not available here): batch sizes 4..256, vocabularies 1024 / 32000 / 128256 /
152064, speculation lengths up to 8, bf16 or fp32 logits.

Random numbers
--------------
All uniforms come from Philox4x32-10 (Salmon et al., "Parallel random numbers:
as easy as 1, 2, 3", SC'11), a counter-based generator:

    key     = (seed & 0xffffffff, seed >> 32)
    counter = (round, sequence b, block, stream tag)
    u       = ((word >> 9) + 0.5) * 2**-23      in (0, 1), exact in fp32 (24 significant bits)

Stream tags: 0 = accept uniforms (position j uses word j%4 of block j//4),
1 = resample uniform (block 0, word 0), 2 = arm uniform (block 0, word 0),
3 = drafting uniforms (same indexing as tag 0).
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Optional, Sequence, Tuple

import numpy as np
import torch

TAG_ACCEPT, TAG_RESAMPLE, TAG_ARM, TAG_DRAFT = 0, 1, 2, 3

_M0 = np.uint64(0xD2511F53)
_M1 = np.uint64(0xCD9E8D57)
_W0 = 0x9E3779B9
_W1 = 0xBB67AE85
_LO = np.uint64(0xFFFFFFFF)
_S32 = np.uint64(32)


def philox4x32_10(counter: np.ndarray, key: Tuple[int, int]) -> np.ndarray:
    """Philox4x32 with 10 rounds.

    counter: integer array [..., 4] (each word < 2**32); key: two 32-bit words.
    Returns uint32 array [..., 4].
    """
    c = np.asarray(counter).astype(np.uint64)
    c0, c1, c2, c3 = c[..., 0], c[..., 1], c[..., 2], c[..., 3]
    k0, k1 = int(key[0]) & 0xFFFFFFFF, int(key[1]) & 0xFFFFFFFF
    for _ in range(10):
        p0 = _M0 * c0
        p1 = _M1 * c2
        hi0, lo0 = p0 >> _S32, p0 & _LO
        hi1, lo1 = p1 >> _S32, p1 & _LO
        c0, c1, c2, c3 = hi1 ^ c1 ^ np.uint64(k0), lo1, hi0 ^ c3 ^ np.uint64(k1), lo0
        k0 = (k0 + _W0) & 0xFFFFFFFF
        k1 = (k1 + _W1) & 0xFFFFFFFF
    return np.stack([c0, c1, c2, c3], axis=-1).astype(np.uint32)


def words_to_uniform(words: np.ndarray) -> np.ndarray:
    """Map 32-bit words to fp32 uniforms strictly inside (0, 1)."""
    return ((words >> np.uint32(9)).astype(np.float64) + 0.5).astype(np.float32) * np.float32(2.0 ** -23)


def _stream(seed: int, rnd: int, B: int, n: int, tag: int) -> np.ndarray:
    """n uniforms per sequence from the stream `tag`: array [B, n] fp32."""
    nblk = max(1, (n + 3) // 4)
    ctr = np.zeros((B, nblk, 4), dtype=np.uint64)
    ctr[..., 0] = rnd & 0xFFFFFFFF
    ctr[..., 1] = np.arange(B, dtype=np.uint64)[:, None]
    ctr[..., 2] = np.arange(nblk, dtype=np.uint64)[None, :]
    ctr[..., 3] = tag
    w = philox4x32_10(ctr, (seed & 0xFFFFFFFF, (seed >> 32) & 0xFFFFFFFF))
    return words_to_uniform(w.reshape(B, nblk * 4)[:, :n])


@dataclass
class RoundUniforms:
    u_accept: np.ndarray    # [B, Gmax] fp32
    u_resample: np.ndarray  # [B] fp32
    u_arm: np.ndarray       # [B] fp32
    u_draft: np.ndarray     # [B, Gmax] fp32


def round_uniforms(seed: int, rnd: int, B: int, Gmax: int) -> RoundUniforms:
    """All uniforms round `rnd` consumes, for every sequence."""
    g = max(Gmax, 1)
    return RoundUniforms(
        u_accept=_stream(seed, rnd, B, g, TAG_ACCEPT)[:, :Gmax].copy(),
        u_resample=_stream(seed, rnd, B, 1, TAG_RESAMPLE)[:, 0].copy(),
        u_arm=_stream(seed, rnd, B, 1, TAG_ARM)[:, 0].copy(),
        u_draft=_stream(seed, rnd, B, g, TAG_DRAFT)[:, :Gmax].copy(),
    )


# --------------------------------------------------------------------------
# Workload presets
# --------------------------------------------------------------------------

@dataclass(frozen=True)
class Workload:
    name: str
    B: int
    V: int
    arm_gamma: Tuple[int, ...]      # speculation length of each arm
    dtype: str                      # "f32" | "bf16"
    temperature: float              # 0.0 = greedy
    rounds: int
    seed: int
    alg: Optional[str]              # "ucb" | "exp3" | "ucb_reward" (throughput as the reward) | None (fixed arm 0)
    target_std: float = 3.0
    boost_prob: float = 0.05        # Bernoulli probability of a +boost entry
    boost: float = 8.0
    sigma: str = "fixed"            # "fixed" | "per_seq" | "per_arm_phase"
    sigma_fixed: float = 1.0
    sigma_range: Tuple[float, float] = (0.3, 2.0)
    sigma_arms: Tuple[float, ...] = (0.3, 0.8, 1.5, 3.0)
    phase_len: int = 200
    delta: float = 0.5
    # "ucb_reward" only: a stand-in for the measured duration of a decoding step, which the paper
    # measures and this harness has no models to measure: one target pass plus gamma draft passes
    step_target_s: float = 0.025
    step_draft_s: float = 0.0015
    step_verify_s: float = 0.0004   # extra per drafted position inside the target pass
    whole_batch: bool = True        # the batch shares one reward (and so one speculation length)

    @property
    def reward_width(self) -> float:
        """Upper end of the reward range: every sequence emits gamma_max + 1 tokens in the shortest step."""
        per_seq = (self.Gmax + 1) / self.step_target_s
        return per_seq * self.B if self.whole_batch else per_seq

    @property
    def K(self) -> int:
        return len(self.arm_gamma)

    @property
    def Gmax(self) -> int:
        return max(self.arm_gamma)

    @property
    def torch_dtype(self) -> torch.dtype:
        return torch.float32 if self.dtype == "f32" else torch.bfloat16

    @property
    def elem_size(self) -> int:
        return 4 if self.dtype == "f32" else 2


WORKLOADS = {
    # tiny: iid N(0, 2^2) target, no boosted entries, draft = target + N(0, 0.5^2)
    "tiny_ucb": Workload("tiny_ucb", B=4, V=1024, arm_gamma=(2, 4, 6), dtype="f32",
                         temperature=1.0, rounds=64, seed=0, alg="ucb",
                         target_std=2.0, boost_prob=0.0, sigma_fixed=0.5),
    "tiny_ucb_greedy": Workload("tiny_ucb_greedy", B=4, V=1024, arm_gamma=(2, 4, 6), dtype="f32",
                                temperature=0.0, rounds=64, seed=0, alg="ucb",
                                target_std=2.0, boost_prob=0.0, sigma_fixed=0.5),
    # 32000-entry vocabulary, fixed speculation length 5
    "llama2_fixed": Workload("llama2_fixed", B=32, V=32000, arm_gamma=(5,), dtype="bf16",
                             temperature=0.7, rounds=200, seed=1, alg=None),
    # 128256-entry vocabulary, UCBSpec over four speculation lengths, ragged per sequence
    "llama3_ucb": Workload("llama3_ucb", B=64, V=128256, arm_gamma=(2, 4, 6, 8), dtype="bf16",
                           temperature=1.0, rounds=500, seed=2, alg="ucb", sigma="per_seq"),
    # 152064-entry vocabulary, EXP3Spec, draft quality per arm rotates every 200 rounds
    "qwen_exp3": Workload("qwen_exp3", B=256, V=152064, arm_gamma=(1, 3, 5, 8), dtype="f32",
                          temperature=1.0, rounds=1000, seed=4, alg="exp3", sigma="per_arm_phase"),
    # 128256-entry vocabulary, UCBSpec over the speculation lengths 0..4 (0 = canonical decoding) with the
    # round's throughput as the reward; 48 sequences that share the reward
    "llama3_tput": Workload("llama3_tput", B=48, V=128256, arm_gamma=(0, 1, 2, 3, 4), dtype="bf16",
                            temperature=1.0, rounds=300, seed=6, alg="ucb_reward", sigma_fixed=1.2),
    "tiny_tput": Workload("tiny_tput", B=6, V=1024, arm_gamma=(0, 1, 2, 3), dtype="f32",
                          temperature=1.0, rounds=120, seed=7, alg="ucb_reward", whole_batch=False,
                          target_std=2.0, boost_prob=0.0, sigma_fixed=0.7),
}


def step_seconds(w: Workload, gamma: np.ndarray) -> float:
    """Stand-in for the measured duration of one decoding step of the batch: the draft model runs
    max(gamma) times, the target model once over max(gamma) + 1 positions."""
    g = int(np.max(gamma)) if len(gamma) else 0
    return w.step_target_s + g * (w.step_draft_s + w.step_verify_s)


def torch_generator(seed: int, rnd: int, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed((seed * 1_000_003 + rnd * 7919 + 12345) & 0x7FFFFFFFFFFFFFFF)
    return g


def per_sequence_sigma(w: Workload) -> np.ndarray:
    """Draft-noise scale per sequence for sigma == "per_seq" (fixed for the run)."""
    rs = np.random.RandomState(w.seed + 977)
    lo, hi = w.sigma_range
    return rs.uniform(lo, hi, size=w.B).astype(np.float32)


def round_sigma(w: Workload, rnd: int, arm: Optional[np.ndarray]) -> np.ndarray:
    """Draft-noise scale of every sequence in round `rnd` (1-based) given its arm."""
    if w.sigma == "fixed":
        return np.full(w.B, w.sigma_fixed, dtype=np.float32)
    if w.sigma == "per_seq":
        return per_sequence_sigma(w)
    if w.sigma == "per_arm_phase":
        assert arm is not None
        phase = (rnd - 1) // w.phase_len
        tab = np.asarray(w.sigma_arms, dtype=np.float32)
        return tab[(np.asarray(arm) + phase) % len(tab)]
    raise ValueError(w.sigma)


def make_logits(w: Workload, rnd: int, sigma: np.ndarray, device="cpu",
                B: Optional[int] = None) -> Tuple[torch.Tensor, torch.Tensor]:
    """Target logits [B, Gmax+1, V] and draft logits [B, Gmax, V] in w's dtype.

    target = N(0, std^2) + boost * Bernoulli(boost_prob)   (fp32, then rounded)
    draft  = (fp32 target before rounding) + sigma_b * N(0, 1), then rounded
    """
    B = w.B if B is None else B
    G, V = w.Gmax, w.V
    g = torch_generator(w.seed, rnd, device)
    t = torch.empty(B, G + 1, V, dtype=torch.float32, device=device)
    t.normal_(0.0, w.target_std, generator=g)
    if w.boost_prob > 0.0:
        mask = torch.empty(B, G + 1, V, dtype=torch.float32, device=device).uniform_(generator=g)
        t += w.boost * (mask < w.boost_prob).to(torch.float32)
        del mask
    d = torch.empty(B, G, V, dtype=torch.float32, device=device)
    d.normal_(0.0, 1.0, generator=g)
    s = torch.as_tensor(np.asarray(sigma, dtype=np.float32)[:B], device=device).view(B, 1, 1)
    d.mul_(s).add_(t[:, :G, :])
    return t.to(w.torch_dtype), d.to(w.torch_dtype)


def draw_draft_tokens(draft_logits: torch.Tensor, temperature: float,
                      u_draft: np.ndarray) -> torch.Tensor:
    """Drafted tokens [B, Gmax] int32: position j is drawn from softmax(draft row j / T)
    by inverse CDF with the uniform u_draft[b, j]; at temperature 0 it is the row argmax.
    (Input generation only: rows are independent "contexts", see make_logits.)"""
    B, G, V = draft_logits.shape
    if G == 0:
        return torch.zeros(B, 0, dtype=torch.int32, device=draft_logits.device)
    if temperature == 0.0:
        return draft_logits.float().argmax(dim=-1).to(torch.int32)
    dev = draft_logits.device
    acc = torch.float64 if dev.type == "cpu" else torch.float32
    out = torch.empty(B, G, dtype=torch.int32, device=dev)
    u = torch.as_tensor(np.asarray(u_draft, dtype=np.float32), device=dev).to(acc)
    for j in range(G):  # one position at a time bounds the temporary to [B, V]
        pr = torch.softmax(draft_logits[:, j, :].to(acc) / temperature, dim=-1)
        cdf = torch.cumsum(pr, dim=-1)
        tgt = (u[:, j] * cdf[:, -1]).unsqueeze(-1)
        idx = torch.searchsorted(cdf, tgt, right=True).squeeze(-1).clamp_(max=V - 1)
        out[:, j] = idx.to(torch.int32)
    return out


@dataclass
class RoundInputs:
    target: torch.Tensor        # [B, Gmax+1, V]
    draft: torch.Tensor         # [B, Gmax, V]
    tokens: torch.Tensor        # [B, Gmax] int32
    gamma: np.ndarray           # [B] int32
    uniforms: RoundUniforms
    sigma: np.ndarray = field(default_factory=lambda: np.zeros(0, np.float32))


def make_round(w: Workload, rnd: int, arm: Optional[np.ndarray] = None,
               device="cpu", B: Optional[int] = None) -> RoundInputs:
    """Everything one verification round reads, for round `rnd` (1-based).
    `arm` [B] is the arm each sequence plays (None = arm 0 for all).  `B` overrides the batch
    size (the first B sequences' arms / noise scales / uniforms; fresh logits)."""
    if arm is None:
        arm = np.zeros(w.B, dtype=np.int32)
    arm = np.asarray(arm, dtype=np.int32)
    gamma = np.asarray(w.arm_gamma, dtype=np.int32)[arm]
    sig = round_sigma(w, rnd, arm)
    nb = w.B if B is None else B
    t, d = make_logits(w, rnd, sig, device=device, B=nb)
    un = round_uniforms(w.seed, rnd, nb, w.Gmax)
    gamma, sig = gamma[:nb], sig[:nb]
    tok = draw_draft_tokens(d, w.temperature, un.u_draft)
    return RoundInputs(target=t, draft=d, tokens=tok, gamma=gamma, uniforms=un, sigma=sig)


# --------------------------------------------------------------------------
# Inputs of the fused LM-head path
# --------------------------------------------------------------------------

@dataclass(frozen=True)
class LmHeadWorkload:
    name: str
    B: int
    gamma: int                      # fixed speculation length (= Gmax)
    V: int
    d_t: int                        # hidden size of the target model
    d_d: int                        # hidden size of the draft model
    temperature: float
    seed: int


LMHEAD_WORKLOADS = {
    # 128256-entry vocabulary, 4096-wide target and 2048-wide draft model, 16 sequences
    "lmhead_llama3": LmHeadWorkload("lmhead_llama3", B=16, gamma=4, V=128256, d_t=4096, d_d=2048,
                                    temperature=1.0, seed=3),
    # the same model pair at a batch where the products stop being bound by streaming W
    "lmhead_llama3_b128": LmHeadWorkload("lmhead_llama3_b128", B=128, gamma=4, V=128256, d_t=4096, d_d=2048,
                                         temperature=1.0, seed=3),
}


@dataclass
class LmHeadInputs:
    H_t: torch.Tensor          # [B*(G+1), d_t] bf16, N(0, 1)
    W_t: torch.Tensor          # [d_t, V] bf16, N(0, 1/d_t)
    H_d: torch.Tensor          # [B*G, d_d] bf16
    W_d: torch.Tensor          # [d_d, V] bf16, N(0, 1/d_d)
    tokens: torch.Tensor       # [B, G] int32 drafted tokens
    gamma: np.ndarray          # [B] int32
    uniforms: RoundUniforms


def make_lmhead_inputs(w: LmHeadWorkload, rnd: int = 1, device="cpu", gamma: Optional[np.ndarray] = None,
                       weights: Optional[Tuple[torch.Tensor, torch.Tensor]] = None) -> LmHeadInputs:
    """Hidden states N(0,1) and output embeddings N(0, 1/d), rounded to bf16.  The drafted tokens
    are drawn from softmax(H_d W_d / T) with torch's matmul (input generation only).
    `weights` re-uses (W_t, W_d) from an earlier call: the embeddings are fixed across rounds."""
    B, G, V = w.B, w.gamma, w.V
    g = torch_generator(w.seed, rnd, device)
    if weights is None:
        gw = torch_generator(w.seed, 0, device)
        W_t = torch.empty(w.d_t, V, dtype=torch.float32, device=device).normal_(0.0, w.d_t ** -0.5, generator=gw)
        W_t = W_t.to(torch.bfloat16)
        W_d = torch.empty(w.d_d, V, dtype=torch.float32, device=device).normal_(0.0, w.d_d ** -0.5, generator=gw)
        W_d = W_d.to(torch.bfloat16)
    else:
        W_t, W_d = weights
    H_t = torch.empty(B * (G + 1), w.d_t, dtype=torch.float32, device=device).normal_(generator=g).to(torch.bfloat16)
    H_d = torch.empty(B * G, w.d_d, dtype=torch.float32, device=device).normal_(generator=g).to(torch.bfloat16)
    un = round_uniforms(w.seed, rnd, B, G)
    if G > 0:
        if torch.device(device).type == "cpu":
            d_logits = (H_d.float() @ W_d.float()).view(B, G, V)
        else:
            d_logits = (H_d @ W_d).float().view(B, G, V)
        tok = draw_draft_tokens(d_logits, w.temperature, un.u_draft)
        del d_logits
    else:
        tok = torch.zeros(B, 0, dtype=torch.int32, device=device)
    gam = np.full(B, G, dtype=np.int32) if gamma is None else np.asarray(gamma, dtype=np.int32)
    return LmHeadInputs(H_t=H_t, W_t=W_t, H_d=H_d, W_d=W_d, tokens=tok.contiguous(), gamma=gam, uniforms=un)


# --------------------------------------------------------------------------
# Inputs of the greedy tree-verification path: tree shapes as arms
# --------------------------------------------------------------------------

@dataclass(frozen=True)
class TreeWorkload:
    name: str
    B: int
    V: int
    dtype: str                      # "bf16" | "f32"
    shapes: Tuple[Tuple[int, ...], ...]   # per arm: parent of node 1..n (0 = the prompt)
    p_right: float                  # probability that a drafted node carries the target's arg-max at its parent
    seed: int
    delta: float = 0.5

    @property
    def K(self) -> int:
        return len(self.shapes)

    @property
    def Nmax(self) -> int:
        return max(len(s) for s in self.shapes)

    @property
    def depths(self) -> Tuple[int, ...]:
        out = []
        for s in self.shapes:
            d = [0]
            for par in s:
                d.append(d[par] + 1)
            out.append(max(d))
        return tuple(out)

    @property
    def elem_size(self) -> int:
        return 2 if self.dtype == "bf16" else 4


TREE_WORKLOADS = {
    # LLaMA-3 vocabulary, 64 sequences, three shapes: a chain of 5, a binary tree of depth 3, a 3 x 3 tree of depth 2
    "llama3_tree": TreeWorkload("llama3_tree", B=64, V=128256, dtype="bf16",
                                shapes=((0, 1, 2, 3, 4), (0, 0, 1, 1, 2, 2, 3, 3, 4, 4, 5, 5, 6, 6),
                                        (0, 0, 0, 1, 1, 1, 2, 2, 2, 3, 3, 3)), p_right=0.75, seed=6),
    "tiny_tree": TreeWorkload("tiny_tree", B=4, V=1024, dtype="f32",
                              shapes=((0, 1, 2), (0, 0, 1, 1, 2, 2), (0, 0, 0)), p_right=0.75, seed=7),
}


@dataclass
class TreeInputs:
    target: torch.Tensor       # [B, Nmax+1, V]: row n = the target's logits after the path to node n
    tokens: torch.Tensor       # [K, B, Nmax] int32: the drafted tokens if sequence b uses shape k
    shape_parent: torch.Tensor  # [K, Nmax] int32
    shape_nodes: torch.Tensor   # [K] int32


def make_tree_inputs(w: TreeWorkload, rnd: int = 1, device="cpu") -> TreeInputs:
    """Target rows as in the chain workloads (N(0, 3^2) with 5 % of the entries raised by 8).  There is no draft
    model here: a drafted node carries the target's arg-max at its parent with probability p_right and a uniformly
    drawn token otherwise, for every shape a sequence might be given (the shape is chosen on the device)."""
    B, V, N, K = w.B, w.V, w.Nmax, w.K
    g = torch_generator(w.seed, rnd, device)
    t = torch.empty(B, N + 1, V, dtype=torch.float32, device=device).normal_(0.0, 3.0, generator=g)
    t += 8.0 * (torch.rand(B, N + 1, V, generator=g, device=device) < 0.05)
    t = t.to(torch.bfloat16 if w.dtype == "bf16" else torch.float32)
    am = t.float().argmax(dim=-1)                                   # [B, N+1]
    sp = torch.zeros(K, N, dtype=torch.int32)
    sn = torch.zeros(K, dtype=torch.int32)
    for k, s in enumerate(w.shapes):
        sp[k, :len(s)] = torch.tensor(s, dtype=torch.int32)
        sn[k] = len(s)
    sp, sn = sp.to(device), sn.to(device)
    right = torch.rand(K, B, N, generator=g, device=device) < w.p_right
    rnd_tok = torch.randint(0, V, (K, B, N), generator=g, device=device)
    at_parent = torch.stack([am.gather(1, sp[k].long().unsqueeze(0).expand(B, N)) for k in range(K)])   # [K, B, N]
    tok = torch.where(right, at_parent, rnd_tok).to(torch.int32)
    return TreeInputs(target=t.contiguous(), tokens=tok.contiguous(), shape_parent=sp, shape_nodes=sn)
