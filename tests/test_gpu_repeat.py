"""The same round launched again and again must give the same bits (needs a B200).

Every kernel of the path reduces in a fixed order, so nothing in its results may depend on timing.
At the full batch sizes, where ring slots are refilled at full speed, a slot handed back to the bulk
copy before a consumer's loads had finished showed up as a residual piece mass that changed in about
one launch per thousand (one per hundred in the early-exit kernel); this test repeats a round often
enough to see that."""
import numpy as np
import pytest
import torch

from paper_2505_15141_b200 import workloads as wl

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _inputs(name, round_index):
    w = wl.WORKLOADS[name]
    arm = np.random.default_rng(round_index).integers(0, max(w.K, 1), size=w.B)
    rnd = wl.make_round(w, round_index, arm, device=DEV)
    gam = torch.as_tensor(np.asarray(rnd.gamma, dtype=np.int32), device=DEV)
    return w, rnd, gam, torch.as_tensor(rnd.uniforms.u_accept, device=DEV), torch.as_tensor(rnd.uniforms.u_resample, device=DEV)


@pytest.mark.parametrize("name,reps", [("qwen_exp3", 2500), ("llama3_ucb", 1500)])
def test_two_call_round_repeats_bit_for_bit(lib, name, reps):
    w, rnd, gam, ua, ur = _inputs(name, 61)
    ws = lib.new_workspace(w.B, w.Gmax, w.V, DEV)
    ref = lib.verify_round(rnd.target, rnd.draft, rnd.tokens, gam, ua, ur, w.temperature, ws)
    ref_ws = ws.clone()
    flush = torch.empty(48 << 20, dtype=torch.float32, device=DEV)
    bad = torch.zeros((), dtype=torch.int64, device=DEV)
    for i in range(reps):
        if i % 3 == 1:
            flush.zero_()                                   # vary what the round finds in L2
        o = lib.verify_round(rnd.target, rnd.draft, rnd.tokens, gam, ua, ur, w.temperature, ws)
        # the workspace holds the row statistics, the segment partials and every residual piece mass
        same = ((ws == ref_ws).all() & (o.accept_len == ref.accept_len).all() & (o.out_tokens == ref.out_tokens).all()
                & (o.p_tok == ref.p_tok).all() & (o.q_tok == ref.q_tok).all() & (o.out_len == ref.out_len).all())
        bad += (~same).to(torch.int64)
    assert int(bad) == 0, f"{int(bad)} of {reps} repetitions differ from the first"


def test_walk_round_repeats_bit_for_bit(lib):
    w, rnd, gam, ua, ur = _inputs("qwen_exp3", 62)
    ws = lib.new_workspace(w.B, w.Gmax, w.V, DEV)
    ref = lib.verify_round_walk(rnd.target, rnd.draft, rnd.tokens, gam, ua, ur, w.temperature, ws)
    ref_ws = ws.clone()                                     # positions are examined in order: what is written is fixed too
    bad = torch.zeros((), dtype=torch.int64, device=DEV)
    reps = 1500
    for i in range(reps):
        o = lib.verify_round_walk(rnd.target, rnd.draft, rnd.tokens, gam, ua, ur, w.temperature, ws)
        same = ((ws == ref_ws).all() & (o.accept_len == ref.accept_len).all() & (o.out_tokens == ref.out_tokens).all()
                & (o.p_tok == ref.p_tok).all() & (o.q_tok == ref.q_tok).all() & (o.out_len == ref.out_len).all())
        bad += (~same).to(torch.int64)
    assert int(bad) == 0, f"{int(bad)} of {reps} repetitions differ from the first"


@pytest.mark.parametrize("name,reps", [("lmhead_llama3", 400), ("lmhead_llama3_b128", 150)])
def test_lmhead_round_repeats_bit_for_bit(lib, name, reps):
    """Both tile shapes of the fused LM head (rows <= 128 and > 128): logits, statistics, accepted
    lengths and the tokens resampled from those logits."""
    w = wl.LMHEAD_WORKLOADS[name]
    B, G, V = w.B, w.gamma, w.V
    inp = wl.make_lmhead_inputs(w, 2, DEV)
    ws = lib.new_lmhead_workspace(B, G, V, DEV)
    gam = torch.as_tensor(inp.gamma, device=DEV)
    ua = torch.as_tensor(inp.uniforms.u_accept, device=DEV); ur = torch.as_tensor(inp.uniforms.u_resample, device=DEV)

    def run():
        lt = torch.empty(B, G + 1, V, dtype=torch.float32, device=DEV)
        ld = torch.empty(B, G, V, dtype=torch.float32, device=DEV)
        acc = torch.empty(B, dtype=torch.int32, device=DEV)
        p = torch.empty(B, G, dtype=torch.float32, device=DEV); q = torch.empty(B, G, dtype=torch.float32, device=DEV)
        ot = torch.empty(B, G + 1, dtype=torch.int32, device=DEV); ol = torch.empty(B, dtype=torch.int32, device=DEV)
        lib.bs_lmhead_verify(inp.H_t, inp.W_t, inp.H_d, inp.W_d, inp.tokens, gam, ua, w.temperature, B, G,
                             lt, ld, acc, p, q, ws)
        lib.bs_residual_sample(lt, ld, inp.tokens, gam, acc, ur, w.temperature, ot, ol, ws)
        return lt, ld, acc, p, q, ot, ol

    ref = run()
    ref_ws = ws.clone()
    bad = torch.zeros((), dtype=torch.int64, device=DEV)
    for i in range(reps):
        o = run()
        same = (ws == ref_ws).all()
        for a, b in zip(o, ref):
            same = same & (a == b).all()
        bad += (~same).to(torch.int64)
        del o
    assert int(bad) == 0, f"{int(bad)} of {reps} repetitions differ from the first"
    st = lib.bs_get_device_status(ws, B, G, V)
    assert (st & ~lib.BS_DEV_RESIDUAL_FALLBACK == 0).all()


def test_drafted_round_repeats_bit_for_bit(lib):
    """Drafting on the device (one call per position), verification on the drafting statistics, resampling:
    the drafted tokens, the outputs and the workspace repeat."""
    w = wl.WORKLOADS["llama3_ucb"]
    B, G, V, T = w.B, w.Gmax, w.V, w.temperature
    _, rnd, gam, ua, ur = _inputs("llama3_ucb", 63)
    ud = torch.as_tensor(rnd.uniforms.u_draft, device=DEV)
    ws = lib.new_workspace(B, G, V, DEV)

    def run():
        tok = torch.full((B, G), -1, dtype=torch.int32, device=DEV)
        for j in range(G):
            lib.bs_draft_sample(rnd.draft, j, gam, ud, T, tok, ws)
        acc = torch.empty(B, dtype=torch.int32, device=DEV)
        p = torch.empty(B, G, dtype=torch.float32, device=DEV); q = torch.empty(B, G, dtype=torch.float32, device=DEV)
        ot = torch.empty(B, G + 1, dtype=torch.int32, device=DEV); ol = torch.empty(B, dtype=torch.int32, device=DEV)
        lib.bs_softmax_verify_drafted(rnd.target, rnd.draft, tok, gam, ua, T, acc, p, q, ws)
        lib.bs_residual_sample(rnd.target, rnd.draft, tok, gam, acc, ur, T, ot, ol, ws)
        return tok, acc, p, q, ot, ol

    ref = run()
    ref_ws = ws.clone()
    bad = torch.zeros((), dtype=torch.int64, device=DEV)
    reps = 300
    for i in range(reps):
        o = run()
        same = (ws == ref_ws).all()
        for a, b in zip(o, ref):
            same = same & (a == b).all()
        bad += (~same).to(torch.int64)
    assert int(bad) == 0, f"{int(bad)} of {reps} repetitions differ from the first"
    st = lib.bs_get_device_status(ws, B, G, V)
    assert (st & ~lib.BS_DEV_RESIDUAL_FALLBACK == 0).all()


def test_two_streams_with_their_own_workspaces_do_not_disturb_each_other(lib):
    """Two batches in flight at once (two-call path, two streams, a workspace each) give what each gives alone."""
    wa, rnda, gama, uaa, ura = _inputs("llama3_ucb", 64)
    wb, rndb, gamb, uab, urb = _inputs("llama2_fixed", 65)
    wsa = lib.new_workspace(wa.B, wa.Gmax, wa.V, DEV); wsb = lib.new_workspace(wb.B, wb.Gmax, wb.V, DEV)
    refa = lib.verify_round(rnda.target, rnda.draft, rnda.tokens, gama, uaa, ura, wa.temperature, wsa)
    refb = lib.verify_round(rndb.target, rndb.draft, rndb.tokens, gamb, uab, urb, wb.temperature, wsb)
    torch.cuda.synchronize()
    ref_wsa, ref_wsb = wsa.clone(), wsb.clone()
    sa, sb = torch.cuda.Stream(), torch.cuda.Stream()
    for i in range(200):
        with torch.cuda.stream(sa):
            oa = lib.verify_round(rnda.target, rnda.draft, rnda.tokens, gama, uaa, ura, wa.temperature, wsa)
        with torch.cuda.stream(sb):
            ob = lib.verify_round(rndb.target, rndb.draft, rndb.tokens, gamb, uab, urb, wb.temperature, wsb)
            if i % 2:                                           # the shorter round twice: the overlap shifts
                ob = lib.verify_round(rndb.target, rndb.draft, rndb.tokens, gamb, uab, urb, wb.temperature, wsb)
        sa.synchronize(); sb.synchronize()
        assert torch.equal(oa.out_tokens, refa.out_tokens) and torch.equal(oa.accept_len, refa.accept_len)
        assert torch.equal(oa.p_tok, refa.p_tok) and torch.equal(wsa, ref_wsa), f"iteration {i}: first batch differs"
        assert torch.equal(ob.out_tokens, refb.out_tokens) and torch.equal(ob.accept_len, refb.accept_len)
        assert torch.equal(ob.p_tok, refb.p_tok) and torch.equal(wsb, ref_wsb), f"iteration {i}: second batch differs"
