"""Fused LM head (tensor-core product + softmax statistics + accept scan) against the CPU oracle,
through the C ABI (needs a B200).

Logits are compared with the fp64 product of the same bf16 inputs.  The verification that
follows is compared with the oracle run on the logits the GPU wrote (a logit that differs in the
last fp32 bits may legitimately move an accept decision, so both sides must see the same logits).
"""
import numpy as np
import pytest
import torch

from oracle import lmhead as ol
from paper_2505_15141_b200 import workloads as wl
import parity

pytestmark = pytest.mark.gpu
DEV = "cuda"
LOGIT_RTOL = 2e-2          # bound stated for the bf16 product
LOGIT_ATOL_SEEN = 2e-3     # what fp32 accumulation of exact bf16 products should stay well inside


def run_lmhead(lib, inp, B, G, V, T):
    ws = lib.new_lmhead_workspace(B, G, V, DEV)
    lt = torch.full((B, G + 1, V), float("nan"), dtype=torch.float32, device=DEV)
    ld = torch.full((B, max(G, 1), V), float("nan"), dtype=torch.float32, device=DEV)[:, :G].contiguous()
    accept_len = torch.full((B,), -7, dtype=torch.int32, device=DEV)
    p_tok = torch.zeros(B, G, dtype=torch.float32, device=DEV)
    q_tok = torch.zeros(B, G, dtype=torch.float32, device=DEV)
    out_tokens = torch.zeros(B, G + 1, dtype=torch.int32, device=DEV)
    out_len = torch.zeros(B, dtype=torch.int32, device=DEV)
    gamma_d = torch.as_tensor(inp.gamma, device=DEV)
    u_acc = torch.as_tensor(inp.uniforms.u_accept, device=DEV)
    u_res = torch.as_tensor(inp.uniforms.u_resample, device=DEV)
    greedy = T == 0.0
    need_draft = not greedy and G > 0
    lib.bs_lmhead_verify(inp.H_t, inp.W_t, inp.H_d if need_draft else None, inp.W_d if need_draft else None,
                         inp.tokens, gamma_d, u_acc, T, B, G, lt, ld if need_draft else None,
                         accept_len, p_tok, q_tok, ws)
    lib.bs_residual_sample(lt, ld if need_draft else None, inp.tokens, gamma_d, accept_len, u_res, T,
                           out_tokens, out_len, ws)
    torch.cuda.synchronize()
    st = lib.bs_get_device_status(ws, B, G, V)
    assert (st & ~lib.BS_DEV_RESIDUAL_FALLBACK == 0).all(), st
    return lib.RoundOutput(accept_len, p_tok, q_tok, out_tokens, out_len, ws), lt, ld


def check_logits(got: torch.Tensor, H: torch.Tensor, W: torch.Tensor, rows, where):
    """Rows `rows` of got [M, V] against the fp64 product."""
    Hn = H[rows].float().cpu().numpy()
    Wn = W.float().cpu().numpy()
    want = ol.lmhead_logits(Hn, Wn)
    g = got[rows].double().cpu().numpy()
    assert np.isfinite(g).all(), f"{where}: non-finite logits"
    err = np.abs(g - want)
    scale = np.maximum(np.abs(want), np.sqrt((want ** 2).mean()))
    assert (err <= LOGIT_RTOL * scale).all(), f"{where}: max relative error {(err / scale).max()}"
    assert err.max() <= LOGIT_ATOL_SEEN * max(1.0, np.abs(want).max()), f"{where}: max abs error {err.max()}"
    return float(err.max())


def check_verify(lib, out, lt, ld, inp, T, where):
    rnd = wl.RoundInputs(target=lt, draft=ld, tokens=inp.tokens, gamma=inp.gamma, uniforms=inp.uniforms)
    tally = parity.Tally()
    parity.check_round(out, rnd, T, tally, where=where)
    return tally


@pytest.mark.parametrize("B,G,V,d_t,d_d", [
    (3, 2, 1000, 136, 64),        # one row tile, ragged vocabulary tile, ragged k-block
    (2, 1, 256, 64, 64),          # exactly one tile, one k-block
    (5, 3, 2056, 320, 192),       # nine column tiles with a tail of 8 columns
    (40, 4, 1544, 256, 128),      # M = 200 / 160: two row tiles, the second ragged
])
def test_lmhead_small_shapes(lib, B, G, V, d_t, d_d):
    w = wl.LmHeadWorkload("t", B=B, gamma=G, V=V, d_t=d_t, d_d=d_d, temperature=1.0, seed=B * 1000 + V)
    rng = np.random.default_rng(V)
    gam = rng.integers(0, G + 1, size=B).astype(np.int32)
    gam[0] = G
    inp = wl.make_lmhead_inputs(w, 1, DEV, gamma=gam)
    # scale the hidden states up so that the distributions are peaked enough to reject sometimes
    inp.H_t = (inp.H_t.float() * 2.0).to(torch.bfloat16)
    out, lt, ld = run_lmhead(lib, inp, B, G, V, 1.0)
    check_logits(lt.view(-1, V), inp.H_t, inp.W_t, slice(None), "target")
    check_logits(ld.view(-1, V), inp.H_d, inp.W_d, slice(None), "draft")
    t = check_verify(lib, out, lt, ld, inp, 1.0, f"lmhead B={B} V={V}")
    assert t.sequences == B


def test_lmhead_greedy(lib):
    B, G, V = 6, 3, 1288
    w = wl.LmHeadWorkload("g", B=B, gamma=G, V=V, d_t=128, d_d=64, temperature=0.0, seed=5)
    inp = wl.make_lmhead_inputs(w, 1, DEV)
    # drafted tokens: the target arg-max, except where flipped
    ref = (inp.H_t.float() @ inp.W_t.float()).view(B, G + 1, V)
    tok = ref[:, :G].argmax(dim=-1).to(torch.int32)
    tok[1, 1] = (tok[1, 1] + 1) % V
    tok[4, 0] = (tok[4, 0] + 3) % V
    inp.tokens = tok.contiguous()
    out, lt, ld = run_lmhead(lib, inp, B, G, V, 0.0)
    check_logits(lt.view(-1, V), inp.H_t, inp.W_t, slice(None), "target")
    t = check_verify(lib, out, lt, lt[:, :G].contiguous(), inp, 0.0, "lmhead greedy")
    assert t.flagged_accept == 0 and t.flagged_token == 0
    assert int(out.accept_len[1]) == 1 and int(out.accept_len[4]) == 0


def test_lmhead_rejects_unsupported_shapes(lib):
    B, G, V = 2, 1, 1004                       # V not a multiple of 8
    H = torch.zeros(B * (G + 1), 64, dtype=torch.bfloat16, device=DEV)
    W = torch.zeros(64, V, dtype=torch.bfloat16, device=DEV)
    Hd = torch.zeros(B * G, 64, dtype=torch.bfloat16, device=DEV)
    ws = torch.zeros(1 << 20, dtype=torch.uint8, device=DEV)
    lt = torch.zeros(B, G + 1, V, device=DEV); ld = torch.zeros(B, G, V, device=DEV)
    z = torch.zeros(B, G, dtype=torch.int32, device=DEV); gm = torch.ones(B, dtype=torch.int32, device=DEV)
    u = torch.full((B, G), 0.5, device=DEV); al = torch.zeros(B, dtype=torch.int32, device=DEV)
    with pytest.raises(lib.BanditSpecError) as e:
        lib.bs_lmhead_verify(H, W, Hd, W, z, gm, u, 1.0, B, G, lt, ld, al, None, None, ws)
    assert e.value.code == lib.BS_ERR_UNSUPPORTED
    small = torch.zeros(256, dtype=torch.uint8, device=DEV)
    V2 = 1008
    W2 = torch.zeros(64, V2, dtype=torch.bfloat16, device=DEV)
    lt2 = torch.zeros(B, G + 1, V2, device=DEV); ld2 = torch.zeros(B, G, V2, device=DEV)
    with pytest.raises(lib.BanditSpecError) as e:
        lib.bs_lmhead_verify(H, W2, Hd, W2, z, gm, u, 1.0, B, G, lt2, ld2, al, None, None, small)
    assert e.value.code == lib.BS_ERR_WORKSPACE


def test_lmhead_full_size(lib):
    """16 sequences, speculation length 4, 128256-entry vocabulary, 4096 / 2048-wide models: sampled
    rows of both products against the fp64 product, all sequences' verification against the oracle."""
    w = wl.LMHEAD_WORKLOADS["lmhead_llama3"]
    B, G, V = w.B, w.gamma, w.V
    inp = wl.make_lmhead_inputs(w, 1, DEV)
    out, lt, ld = run_lmhead(lib, inp, B, G, V, w.temperature)
    e1 = check_logits(lt.view(-1, V), inp.H_t, inp.W_t, [0, 37, 79], "target")
    e2 = check_logits(ld.view(-1, V), inp.H_d, inp.W_d, [0, 21, 63], "draft")
    assert max(e1, e2) < 1e-3
    # every row is finite and has the spread N(0,1) logits should have
    assert torch.isfinite(lt).all() and torch.isfinite(ld).all()
    assert 0.9 < float(lt.std()) < 1.1 and 0.9 < float(ld.std()) < 1.1
    t = check_verify(lib, out, lt, ld, inp, w.temperature, "lmhead full size")
    assert t.sequences == B and t.flagged_accept + t.flagged_token <= 2
    # a second call on the same inputs is bit-identical
    out2, lt2, ld2 = run_lmhead(lib, inp, B, G, V, w.temperature)
    assert torch.equal(lt, lt2) and torch.equal(ld, ld2) and torch.equal(out.out_tokens, out2.out_tokens)


def _lm_shapes(n, seed):
    rng = np.random.default_rng(seed)
    return [(int(rng.integers(1, 60)), int(rng.integers(0, 6)), int(rng.choice([8, 264, 1000, 2056, 4104, 8200])),
             int(rng.choice([8, 72, 200, 264, 520])), int(rng.choice([8, 64, 136, 328]))) for _ in range(n)]


@pytest.mark.parametrize("B,G,V,d_t,d_d", _lm_shapes(12, 7))
def test_lmhead_random_shapes(lib, B, G, V, d_t, d_d):
    """Row counts on both sides of one and two 128-row tiles, k-extents that are not multiples of the
    64-deep stage, vocabularies that end inside a tile, speculation length 0 (no draft product)."""
    w = wl.LmHeadWorkload("r", B=B, gamma=G, V=V, d_t=d_t, d_d=d_d, temperature=1.0, seed=B * 100 + V)
    rng = np.random.default_rng(B + V + d_t)
    gam = rng.integers(0, G + 1, size=B).astype(np.int32)
    inp = wl.make_lmhead_inputs(w, 1, DEV, gamma=gam)
    out, lt, ld = run_lmhead(lib, inp, B, G, V, 1.0)
    check_logits(lt.view(-1, V), inp.H_t, inp.W_t, slice(None), "target")
    if G > 0:
        check_logits(ld.view(-1, V), inp.H_d, inp.W_d, slice(None), "draft")
    t = check_verify(lib, out, lt, ld, inp, 1.0, f"lmhead random B={B} G={G} V={V}")
    assert t.sequences == B
