"""ctypes binding of libbanditspec.so: the same entry points as include/banditspec.h.

Argument marshalling only: tensors are passed as raw device pointers, every step of the
round runs in the library's CUDA kernels on torch's current stream.  PyTorch is used for
device memory and streams.  Importing this module loads the CUDA library and raises if it is
missing -- there is no CPU fallback.
"""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass
from typing import Optional, Sequence

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libbanditspec.so")
if not os.path.exists(LIB_PATH):
    raise ImportError(f"{LIB_PATH} is missing: build it with `python __graft_entry__.py` "
                      "(the CUDA library is required; there is no fallback path)")
_lib = C.CDLL(LIB_PATH)

BS_OK = 0
BS_ERR_INVALID_ARG, BS_ERR_CUDA, BS_ERR_UNSUPPORTED, BS_ERR_WORKSPACE, BS_ERR_TIMEOUT, BS_ERR_DEVICE_DATA = 1, 2, 3, 4, 5, 6
BS_F32, BS_BF16 = 0, 1
BS_UCB, BS_EXP3, BS_UCB_REWARD = 0, 1, 2
BS_DEV_BAD_GAMMA, BS_DEV_BAD_TOKEN, BS_DEV_NONFINITE, BS_DEV_RESIDUAL_FALLBACK, BS_DEV_DRAFT_MISSING = 1, 2, 4, 8, 16
BS_DEV_BAD_TREE = 32
BS_MAX_GAMMA, BS_MAX_ARMS, BS_MAX_BATCH = 31, 32, 4096

_vp, _i, _f, _d, _sz = C.c_void_p, C.c_int, C.c_float, C.c_double, C.c_size_t

# name -> (restype, argtypes); must list every symbol the header declares
SIGNATURES = {
    "bs_status_string": (C.c_char_p, [_i]),
    "bs_last_cuda_error": (C.c_char_p, []),
    "bs_workspace_bytes": (_sz, [_i, _i, _i]),
    "bs_workspace_init": (_i, [_vp, _sz, _vp]),
    "bs_get_device_status": (_i, [_vp, _sz, _i, _i, _i, _vp, _vp]),
    "bs_softmax_verify": (_i, [_vp, _vp, _i, _vp, _vp, _vp, _f, _i, _i, _i, _vp, _vp, _vp, _vp, _sz, _vp]),
    "bs_residual_sample": (_i, [_vp, _vp, _i, _vp, _vp, _vp, _vp, _f, _i, _i, _i, _vp, _vp, _vp, _sz, _vp]),
    "bs_softmax_verify_noalloc": (_i, [_vp, _vp, _i, _vp, _vp, _vp, _f, _i, _i, _i, _vp, _vp, _vp, _vp]),
    "bs_verify_walk": (_i, [_vp, _vp, _i, _vp, _vp, _vp, _vp, _f, _i, _i, _i, _vp, _vp, _vp, _vp, _vp, _vp, _sz, _vp]),
    "bs_verify_walk_drafted": (_i, [_vp, _vp, _i, _vp, _vp, _vp, _vp, _f, _i, _i, _i, _vp, _vp, _vp, _vp, _vp, _vp, _sz,
                                    _vp]),
    "bs_draft_sample": (_i, [_vp, _i, _i, _vp, _vp, _f, _i, _i, _i, _vp, _vp, _sz, _vp]),
    "bs_softmax_verify_drafted": (_i, [_vp, _vp, _i, _vp, _vp, _vp, _f, _i, _i, _i, _vp, _vp, _vp, _vp, _sz, _vp]),
    "bs_tree_verify_greedy": (_i, [_vp, _i, _vp, _vp, _vp, _i, _i, _i, _vp, _vp, _vp, _vp, _vp, _sz, _vp]),
    "bs_tree_expand_shapes": (_i, [_vp, _vp, _vp, _i, _i, _i, _vp, _vp, _vp]),
    "bs_lmhead_workspace_bytes": (_sz, [_i, _i, _i]),
    "bs_lmhead_verify": (_i, [_vp, _vp, _i, _vp, _vp, _i, _vp, _vp, _vp, _f, _i, _i, _i, _vp, _vp, _vp, _vp, _vp,
                              _vp, _sz, _vp]),
    "bs_bandit_state_bytes": (_sz, [_i, _i, _i]),
    "bs_bandit_init": (_i, [_vp, _sz, _i, _i, _i, _vp, _d, _vp]),
    "bs_bandit_select": (_i, [_vp, _sz, _i, _i, _i, _vp, _vp, _vp, _vp, _vp, _vp]),
    "bs_bandit_update": (_i, [_vp, _sz, _i, _i, _i, _vp, _vp, _vp, _vp]),
    "bs_bandit_read": (_i, [_vp, _sz, _i, _i, _i, _vp, _vp, _vp, _vp, _vp]),
    "bs_bandit_step": (_i, [_vp, _sz, _i, _i, _i, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp]),
    "bs_bandit_init_reward": (_i, [_vp, _sz, _i, _i, _vp, _d, _d, _vp]),
    "bs_bandit_update_reward": (_i, [_vp, _sz, _i, _i, _vp, _vp, _vp, _vp]),
    "bs_throughput_reward": (_i, [_vp, _vp, _i, _d, _i, _vp, _vp]),
}
for _name, (_res, _args) in SIGNATURES.items():
    _fn = getattr(_lib, _name)
    _fn.restype, _fn.argtypes = _res, _args


class BanditSpecError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        detail = f" [{_lib.bs_last_cuda_error().decode()}]" if code == BS_ERR_CUDA else ""
        super().__init__(f"{where}: {_lib.bs_status_string(code).decode()} (bs_status {code}){detail}")


def _check(code: int, where: str) -> None:
    if code != BS_OK:
        raise BanditSpecError(code, where)


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    if t is None:
        return None
    assert t.is_contiguous(), "tensors must be contiguous"
    return t.data_ptr()


def _stream(stream=None) -> int:
    s = torch.cuda.current_stream() if stream is None else stream
    return s.cuda_stream


def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return BS_F32
    if t.dtype == torch.bfloat16:
        return BS_BF16
    raise TypeError(f"logits must be float32 or bfloat16, got {t.dtype}")


# ---- workspace ---------------------------------------------------------------------

def bs_workspace_bytes(B: int, Gmax: int, V: int) -> int:
    return int(_lib.bs_workspace_bytes(B, Gmax, V))


def bs_workspace_init(workspace: torch.Tensor, stream=None) -> None:
    _check(_lib.bs_workspace_init(_ptr(workspace), workspace.numel() * workspace.element_size(), _stream(stream)),
           "bs_workspace_init")


def new_workspace(B: int, Gmax: int, V: int, device="cuda") -> torch.Tensor:
    """Allocate (through torch) and clear a workspace for the given limits."""
    n = bs_workspace_bytes(B, Gmax, V)
    if n == 0:
        raise BanditSpecError(BS_ERR_UNSUPPORTED, "bs_workspace_bytes")
    ws = torch.empty(n, dtype=torch.uint8, device=device)
    bs_workspace_init(ws)
    return ws


def bs_get_device_status(workspace: torch.Tensor, B: int, Gmax: int, V: int, stream=None) -> np.ndarray:
    """Per-sequence status bits of the last verify/residual pair (synchronises)."""
    host = np.zeros(B, dtype=np.int32)
    code = _lib.bs_get_device_status(_ptr(workspace), workspace.numel(), B, Gmax, V,
                                     host.ctypes.data_as(_vp), _stream(stream))
    if code not in (BS_OK, BS_ERR_DEVICE_DATA):
        raise BanditSpecError(code, "bs_get_device_status")
    return host


# ---- verification ---------------------------------------------------------------------

def bs_softmax_verify(target_logits, draft_logits, draft_tokens, gamma, u_accept, temperature: float,
                      accept_len, p_tok, q_tok, workspace, stream=None) -> None:
    B, G1, V = target_logits.shape
    _check(_lib.bs_softmax_verify(_ptr(target_logits), _ptr(draft_logits), _dtype_code(target_logits),
                                  _ptr(draft_tokens), _ptr(gamma), _ptr(u_accept), float(temperature),
                                  B, G1 - 1, V, _ptr(accept_len), _ptr(p_tok), _ptr(q_tok),
                                  _ptr(workspace), workspace.numel(), _stream(stream)), "bs_softmax_verify")


def bs_residual_sample(target_logits, draft_logits, draft_tokens, gamma, accept_len, u_resample,
                       temperature: float, out_tokens, out_len, workspace, stream=None) -> None:
    B, G1, V = target_logits.shape
    _check(_lib.bs_residual_sample(_ptr(target_logits), _ptr(draft_logits), _dtype_code(target_logits),
                                   _ptr(draft_tokens), _ptr(gamma), _ptr(accept_len), _ptr(u_resample),
                                   float(temperature), B, G1 - 1, V, _ptr(out_tokens), _ptr(out_len),
                                   _ptr(workspace), workspace.numel(), _stream(stream)), "bs_residual_sample")


BS_NOALLOC_SCRATCH_BYTES = 2 << 20


def bs_softmax_verify_noalloc(target_logits, draft_logits, draft_tokens, gamma, u_accept, temperature: float,
                              accept_len, p_tok, q_tok, stream=None) -> None:
    """bs_softmax_verify on the scratch array built into the library: for callers that cannot
    allocate device memory (fixed memory pools, buffer-only plugins, no-cudaMalloc paths).
    Sizes whose workspace exceeds BS_NOALLOC_SCRATCH_BYTES raise BS_ERR_WORKSPACE; calls that
    overlap on one GPU race on the shared array."""
    B, G1, V = target_logits.shape
    _check(_lib.bs_softmax_verify_noalloc(_ptr(target_logits), _ptr(draft_logits), _dtype_code(target_logits),
                                          _ptr(draft_tokens), _ptr(gamma), _ptr(u_accept), float(temperature),
                                          B, G1 - 1, V, _ptr(accept_len), _ptr(p_tok), _ptr(q_tok),
                                          _stream(stream)), "bs_softmax_verify_noalloc")


@dataclass
class RoundOutput:
    accept_len: torch.Tensor   # [B] int32, tau
    p_tok: torch.Tensor        # [B, Gmax] fp32
    q_tok: torch.Tensor        # [B, Gmax] fp32
    out_tokens: torch.Tensor   # [B, Gmax+1] int32
    out_len: torch.Tensor      # [B] int32, y = tau + 1
    workspace: torch.Tensor


def verify_round(target_logits, draft_logits, draft_tokens, gamma, u_accept, u_resample,
                 temperature: float, workspace: Optional[torch.Tensor] = None) -> RoundOutput:
    """Allocates the outputs and calls bs_softmax_verify then bs_residual_sample."""
    B, G1, V = target_logits.shape
    G = G1 - 1
    dev = target_logits.device
    if workspace is None:
        workspace = new_workspace(B, G, V, dev)
    accept_len = torch.empty(B, dtype=torch.int32, device=dev)
    p_tok = torch.empty(B, G, dtype=torch.float32, device=dev)
    q_tok = torch.empty(B, G, dtype=torch.float32, device=dev)
    out_tokens = torch.empty(B, G + 1, dtype=torch.int32, device=dev)
    out_len = torch.empty(B, dtype=torch.int32, device=dev)
    bs_softmax_verify(target_logits, draft_logits, draft_tokens, gamma, u_accept, temperature,
                      accept_len, p_tok, q_tok, workspace)
    bs_residual_sample(target_logits, draft_logits, draft_tokens, gamma, accept_len, u_resample,
                       temperature, out_tokens, out_len, workspace)
    return RoundOutput(accept_len, p_tok, q_tok, out_tokens, out_len, workspace)


def bs_verify_walk(target_logits, draft_logits, draft_tokens, gamma, u_accept, u_resample, temperature: float,
                   accept_len, p_tok, q_tok, out_tokens, out_len, workspace, stream=None) -> None:
    """Verification with early exit and resampling in one launch."""
    B, G1, V = target_logits.shape
    _check(_lib.bs_verify_walk(_ptr(target_logits), _ptr(draft_logits), _dtype_code(target_logits),
                               _ptr(draft_tokens), _ptr(gamma), _ptr(u_accept), _ptr(u_resample), float(temperature),
                               B, G1 - 1, V, _ptr(accept_len), _ptr(p_tok), _ptr(q_tok), _ptr(out_tokens),
                               _ptr(out_len), _ptr(workspace), workspace.numel(), _stream(stream)), "bs_verify_walk")


def bs_verify_walk_drafted(target_logits, draft_logits, draft_tokens, gamma, u_accept, u_resample, temperature: float,
                           accept_len, p_tok, q_tok, out_tokens, out_len, workspace, stream=None) -> None:
    """bs_verify_walk on the statistics bs_draft_sample left in the workspace: target rows only."""
    B, G1, V = target_logits.shape
    _check(_lib.bs_verify_walk_drafted(_ptr(target_logits), _ptr(draft_logits), _dtype_code(target_logits),
                                       _ptr(draft_tokens), _ptr(gamma), _ptr(u_accept), _ptr(u_resample),
                                       float(temperature), B, G1 - 1, V, _ptr(accept_len), _ptr(p_tok), _ptr(q_tok),
                                       _ptr(out_tokens), _ptr(out_len), _ptr(workspace), workspace.numel(),
                                       _stream(stream)), "bs_verify_walk_drafted")


def verify_round_walk(target_logits, draft_logits, draft_tokens, gamma, u_accept, u_resample,
                      temperature: float, workspace: Optional[torch.Tensor] = None) -> RoundOutput:
    """Allocates the outputs and calls bs_verify_walk."""
    B, G1, V = target_logits.shape
    G = G1 - 1
    dev = target_logits.device
    if workspace is None:
        workspace = new_workspace(B, G, V, dev)
    accept_len = torch.full((B,), -9, dtype=torch.int32, device=dev)
    p_tok = torch.full((B, G), -1.0, dtype=torch.float32, device=dev)
    q_tok = torch.full((B, G), -1.0, dtype=torch.float32, device=dev)
    out_tokens = torch.full((B, G + 1), -9, dtype=torch.int32, device=dev)
    out_len = torch.full((B,), -9, dtype=torch.int32, device=dev)
    bs_verify_walk(target_logits, draft_logits, draft_tokens, gamma, u_accept, u_resample, temperature,
                   accept_len, p_tok, q_tok, out_tokens, out_len, workspace)
    return RoundOutput(accept_len, p_tok, q_tok, out_tokens, out_len, workspace)


# ---- drafting on the device ------------------------------------------------------------

def bs_draft_sample(draft_logits, position: int, gamma, u_draft, temperature: float, draft_tokens, workspace,
                    stream=None) -> None:
    """Drafted token of `position` for every sequence with position < gamma_b, into draft_tokens[b, position]."""
    B, G, V = draft_logits.shape
    assert draft_tokens.shape == (B, G) and draft_tokens.dtype == torch.int32
    _check(_lib.bs_draft_sample(_ptr(draft_logits), _dtype_code(draft_logits), int(position), _ptr(gamma),
                                _ptr(u_draft), float(temperature), B, G, V, _ptr(draft_tokens),
                                _ptr(workspace), workspace.numel(), _stream(stream)), "bs_draft_sample")


def bs_softmax_verify_drafted(target_logits, draft_logits, draft_tokens, gamma, u_accept, temperature: float,
                              accept_len, p_tok, q_tok, workspace, stream=None) -> None:
    B, G1, V = target_logits.shape
    _check(_lib.bs_softmax_verify_drafted(_ptr(target_logits), _ptr(draft_logits), _dtype_code(target_logits),
                                          _ptr(draft_tokens), _ptr(gamma), _ptr(u_accept), float(temperature),
                                          B, G1 - 1, V, _ptr(accept_len), _ptr(p_tok), _ptr(q_tok),
                                          _ptr(workspace), workspace.numel(), _stream(stream)),
           "bs_softmax_verify_drafted")


# ---- greedy verification of a tree of drafts ---------------------------------------------------

def bs_tree_verify_greedy(target_logits, node_parent, node_tokens, n_nodes, accept_len, out_nodes, out_tokens,
                          out_len, workspace, stream=None) -> None:
    """target_logits [B, Nmax+1, V]: row n = the target's logits after the path to node n (row 0: the prompt)."""
    B, N1, V = target_logits.shape
    _check(_lib.bs_tree_verify_greedy(_ptr(target_logits), _dtype_code(target_logits), _ptr(node_parent),
                                      _ptr(node_tokens), _ptr(n_nodes), B, N1 - 1, V, _ptr(accept_len),
                                      _ptr(out_nodes), _ptr(out_tokens), _ptr(out_len), _ptr(workspace),
                                      workspace.numel(), _stream(stream)), "bs_tree_verify_greedy")


def bs_tree_expand_shapes(shape_parent, shape_nodes, arm, node_parent, n_nodes, stream=None) -> None:
    K, Nmax = shape_parent.shape
    B = arm.shape[0]
    _check(_lib.bs_tree_expand_shapes(_ptr(shape_parent), _ptr(shape_nodes), _ptr(arm), K, B, Nmax,
                                      _ptr(node_parent), _ptr(n_nodes), _stream(stream)), "bs_tree_expand_shapes")


# ---- fused LM head ----------------------------------------------------------------------

def bs_lmhead_workspace_bytes(B: int, Gmax: int, V: int) -> int:
    return int(_lib.bs_lmhead_workspace_bytes(B, Gmax, V))


def new_lmhead_workspace(B: int, Gmax: int, V: int, device="cuda") -> torch.Tensor:
    n = bs_lmhead_workspace_bytes(B, Gmax, V)
    if n == 0:
        raise BanditSpecError(BS_ERR_UNSUPPORTED, "bs_lmhead_workspace_bytes")
    ws = torch.empty(n, dtype=torch.uint8, device=device)
    bs_workspace_init(ws)
    return ws


def bs_lmhead_verify(H_t, W_t, H_d, W_d, draft_tokens, gamma, u_accept, temperature: float, B: int, Gmax: int,
                     logits_t_out, logits_d_out, accept_len, p_tok, q_tok, workspace, stream=None) -> None:
    """H_t [B*(Gmax+1), d_t], W_t [d_t, V], H_d [B*Gmax, d_d], W_d [d_d, V] bf16; logits out fp32."""
    d_t, V = W_t.shape
    assert H_t.shape == (B * (Gmax + 1), d_t) and H_t.dtype == torch.bfloat16 and W_t.dtype == torch.bfloat16
    d_d = 0
    if W_d is not None:
        d_d = W_d.shape[0]
        assert W_d.shape[1] == V and H_d.shape == (B * Gmax, d_d)
        assert H_d.dtype == torch.bfloat16 and W_d.dtype == torch.bfloat16
    assert logits_t_out.dtype == torch.float32 and logits_t_out.numel() == B * (Gmax + 1) * V
    _check(_lib.bs_lmhead_verify(_ptr(H_t), _ptr(W_t), d_t, _ptr(H_d), _ptr(W_d), d_d, _ptr(draft_tokens),
                                 _ptr(gamma), _ptr(u_accept), float(temperature), B, Gmax, V,
                                 _ptr(logits_t_out), _ptr(logits_d_out), _ptr(accept_len), _ptr(p_tok), _ptr(q_tok),
                                 _ptr(workspace), workspace.numel(), _stream(stream)), "bs_lmhead_verify")


# ---- bandits ---------------------------------------------------------------------------

def bs_bandit_state_bytes(alg: int, B: int, K: int) -> int:
    return int(_lib.bs_bandit_state_bytes(alg, B, K))


def bs_bandit_init(state: torch.Tensor, alg: int, B: int, K: int, arm_gamma: Sequence[int],
                   delta: float = 0.5, stream=None) -> None:
    ag = np.ascontiguousarray(arm_gamma, dtype=np.int32)
    assert ag.shape == (K,)
    _check(_lib.bs_bandit_init(_ptr(state), state.numel(), alg, B, K, ag.ctypes.data_as(_vp),
                               float(delta), _stream(stream)), "bs_bandit_init")


def bs_bandit_select(state, alg: int, B: int, K: int, u_arm, active, arm, gamma, index_out=None,
                     stream=None) -> None:
    _check(_lib.bs_bandit_select(_ptr(state), state.numel(), alg, B, K, _ptr(u_arm), _ptr(active),
                                 _ptr(arm), _ptr(gamma), _ptr(index_out), _stream(stream)), "bs_bandit_select")


def bs_bandit_update(state, alg: int, B: int, K: int, arm, reward_y, active=None, stream=None) -> None:
    _check(_lib.bs_bandit_update(_ptr(state), state.numel(), alg, B, K, _ptr(arm), _ptr(reward_y),
                                 _ptr(active), _stream(stream)), "bs_bandit_update")


def bs_bandit_step(state, alg: int, B: int, K: int, reward, u_arm_next, active, arm, gamma, index_out=None,
                   stream=None) -> None:
    """Update with this round's reward (int32 accepted lengths, or fp64 rewards for BS_UCB_REWARD) and
    select the next round's arms, in one launch; `arm` is read and overwritten."""
    ry, rr = (None, reward) if alg == BS_UCB_REWARD else (reward, None)
    assert (rr.dtype == torch.float64) if rr is not None else (ry.dtype == torch.int32)
    _check(_lib.bs_bandit_step(_ptr(state), state.numel(), alg, B, K, _ptr(ry), _ptr(rr), _ptr(u_arm_next),
                               _ptr(active), _ptr(arm), _ptr(gamma), _ptr(index_out), _stream(stream)),
           "bs_bandit_step")


def bs_bandit_read(state, alg: int, B: int, K: int, stream=None) -> dict:
    """Sufficient statistics as host arrays: UCBSpec {n, sumY, t}; EXP3Spec {S, n, t}; real-reward
    UCBSpec {S (the reward sums), n, t}."""
    t = np.zeros(B, dtype=np.int64)
    if alg == BS_UCB:
        n = np.zeros((B, K), dtype=np.int64)
        sy = np.zeros((B, K), dtype=np.int64)
        _check(_lib.bs_bandit_read(_ptr(state), state.numel(), alg, B, K, n.ctypes.data_as(_vp),
                                   sy.ctypes.data_as(_vp), None, t.ctypes.data_as(_vp), _stream(stream)),
               "bs_bandit_read")
        return {"n": n, "sumY": sy, "t": t}
    S = np.zeros((B, K), dtype=np.float64)
    n = np.zeros((B, K), dtype=np.int64)
    _check(_lib.bs_bandit_read(_ptr(state), state.numel(), alg, B, K, n.ctypes.data_as(_vp), None,
                               S.ctypes.data_as(_vp), t.ctypes.data_as(_vp), _stream(stream)), "bs_bandit_read")
    return {"S": S, "n": n, "t": t}


def bs_bandit_init_reward(state: torch.Tensor, B: int, K: int, arm_gamma: Sequence[int], delta: float,
                          reward_width: float, stream=None) -> None:
    ag = np.ascontiguousarray(np.asarray(arm_gamma, dtype=np.int32))
    assert ag.shape == (K,)
    _check(_lib.bs_bandit_init_reward(_ptr(state), state.numel(), B, K, ag.ctypes.data_as(_vp), float(delta),
                                      float(reward_width), _stream(stream)), "bs_bandit_init_reward")


def bs_bandit_update_reward(state, B: int, K: int, arm, reward, active=None, stream=None) -> None:
    assert reward.dtype == torch.float64
    _check(_lib.bs_bandit_update_reward(_ptr(state), state.numel(), B, K, _ptr(arm), _ptr(reward), _ptr(active),
                                        _stream(stream)), "bs_bandit_update_reward")


def bs_throughput_reward(out_len, active, B: int, seconds: float, whole_batch: bool, reward, stream=None) -> None:
    assert out_len.dtype == torch.int32 and reward.dtype == torch.float64
    _check(_lib.bs_throughput_reward(_ptr(out_len), _ptr(active), B, float(seconds), int(bool(whole_batch)),
                                     _ptr(reward), _stream(stream)), "bs_throughput_reward")


def new_bandit(alg: int, B: int, arm_gamma: Sequence[int], delta: float = 0.5, device="cuda",
               reward_width: Optional[float] = None) -> torch.Tensor:
    K = len(arm_gamma)
    n = bs_bandit_state_bytes(alg, B, K)
    if n == 0:
        raise BanditSpecError(BS_ERR_UNSUPPORTED, "bs_bandit_state_bytes")
    state = torch.empty(n, dtype=torch.uint8, device=device)
    if alg == BS_UCB_REWARD:
        bs_bandit_init_reward(state, B, K, arm_gamma, delta, reward_width)
    else:
        bs_bandit_init(state, alg, B, K, arm_gamma, delta)
    return state
