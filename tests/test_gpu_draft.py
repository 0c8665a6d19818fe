"""Drafting on the device (bs_draft_sample) and the verification that re-uses its statistics
(bs_softmax_verify_drafted) against the CPU oracle, through the C ABI (needs a B200).

Tokens: oracle.verify.draft_token on the same row and uniform; a token may differ only where the
uniform lies within CDF_TIE of an edge of the oracle token's interval (the rule of the resampling
step).  The drafted verification must reproduce bs_softmax_verify exactly: it uses the same
statistics kernels, only on fewer rows.
"""
import numpy as np
import pytest
import torch

from oracle import verify as ov
from paper_2505_15141_b200 import workloads as wl
import parity

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _logits(seed, B, G, V, dtype, std=3.0, sigma=1.0):
    g = torch.Generator(device="cpu"); g.manual_seed(seed)
    t = torch.randn(B, G + 1, V, generator=g) * std
    d = t[:, :G] + sigma * torch.randn(B, G, V, generator=g)
    return t.to(dtype).to(DEV), d.to(dtype).to(DEV)


def _draft_all(lib, d, gamma_d, u_d, T, ws):
    B, G, V = d.shape
    tok = torch.full((B, G), -5, dtype=torch.int32, device=DEV)
    for j in range(G):
        lib.bs_draft_sample(d, j, gamma_d, None if T == 0.0 else u_d, T, tok, ws)
    torch.cuda.synchronize()
    return tok


def _check_tokens(tok, d, gamma, u, T):
    """Every drafted position against the oracle; returns the number of flagged near-ties."""
    B, G, V = d.shape
    flagged = 0
    dn = d.float().cpu().numpy(); tk = tok.cpu().numpy()
    for b in range(B):
        for j in range(G):
            if j >= gamma[b]:
                assert tk[b, j] == -5, "positions that are not drafted must be left alone"
                continue
            want, lo, hi = ov.draft_token(dn[b, j], float(u[b, j]), T)
            if tk[b, j] != want:
                assert T != 0.0, f"greedy draft b={b} j={j}: {tk[b, j]} != {want}"
                near = min(float(u[b, j]) - lo, hi - float(u[b, j])) < ov.CDF_TIE
                q = ov.softmax_row(dn[b, j], T); c = np.cumsum(q)
                v = int(tk[b, j])
                assert near and 0 <= v < V and q[v] > 0 and (c[v - 1] if v else 0.0) <= u[b, j] + ov.CDF_TIE \
                    and c[v] >= u[b, j] - ov.CDF_TIE, f"b={b} j={j}: token {v} != {want}, u={u[b, j]} in [{lo},{hi})"
                flagged += 1
    return flagged


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("V", [8, 1000, 8200, 40000])
def test_draft_tokens_match_the_oracle(lib, dtype, V):
    rng = np.random.default_rng(V)
    B, G = 7, 5
    for T in (1.0, 0.6, 0.0):
        _, d = _logits(V + int(T * 10), B, G, V, dtype)
        gamma = rng.integers(0, G + 1, size=B).astype(np.int32); gamma[0] = G; gamma[1] = 0
        u = rng.random((B, G)).astype(np.float32) * 0.999 + 0.0005
        ws = lib.new_workspace(B, G, V, DEV)
        tok = _draft_all(lib, d, torch.as_tensor(gamma, device=DEV), torch.as_tensor(u, device=DEV), T, ws)
        assert _check_tokens(tok, d, gamma, u, T) <= 1
        st = lib.bs_get_device_status(ws, B, G, V)
        assert (st == 0).all()


def test_drafted_round_equals_plain_round_and_the_oracle(lib):
    """draft -> verify_drafted -> resample gives exactly what verify -> resample gives on the same
    tokens, and both match the oracle; two rounds in a row on one workspace."""
    rng = np.random.default_rng(3)
    B, G, V, T = 9, 6, 32000, 0.8
    ws = lib.new_workspace(B, G, V, DEV)
    ws2 = lib.new_workspace(B, G, V, DEV)
    for rnd in range(2):
        t, d = _logits(100 + rnd, B, G, V, torch.bfloat16)
        gamma = rng.integers(0, G + 1, size=B).astype(np.int32); gamma[0] = G
        un = wl.round_uniforms(11, rnd + 1, B, G)
        gamma_d = torch.as_tensor(gamma, device=DEV)
        u_acc = torch.as_tensor(un.u_accept, device=DEV); u_res = torch.as_tensor(un.u_resample, device=DEV)
        tok = _draft_all(lib, d, gamma_d, torch.as_tensor(un.u_draft, device=DEV), T, ws)
        assert _check_tokens(tok, d, gamma, un.u_draft, T) <= 1
        tok = torch.where(tok < 0, torch.zeros_like(tok), tok).contiguous()      # padded entries are never read
        out = {}
        for name, fn, w_ in (("drafted", lib.bs_softmax_verify_drafted, ws), ("plain", lib.bs_softmax_verify, ws2)):
            acc = torch.zeros(B, dtype=torch.int32, device=DEV)
            p = torch.zeros(B, G, device=DEV); q = torch.zeros(B, G, device=DEV)
            ot = torch.zeros(B, G + 1, dtype=torch.int32, device=DEV); ol = torch.zeros(B, dtype=torch.int32, device=DEV)
            fn(t, d, tok, gamma_d, u_acc, T, acc, p, q, w_)
            lib.bs_residual_sample(t, d, tok, gamma_d, acc, u_res, T, ot, ol, w_)
            torch.cuda.synchronize()
            assert (lib.bs_get_device_status(w_, B, G, V) & ~lib.BS_DEV_RESIDUAL_FALLBACK == 0).all()
            out[name] = lib.RoundOutput(acc, p, q, ot, ol, w_)
        a, b_ = out["drafted"], out["plain"]
        assert torch.equal(a.accept_len, b_.accept_len) and torch.equal(a.out_tokens, b_.out_tokens)
        assert torch.allclose(a.p_tok, b_.p_tok, atol=1e-6, rtol=0) and torch.allclose(a.q_tok, b_.q_tok, atol=1e-6, rtol=0)
        rin = wl.RoundInputs(target=t, draft=d, tokens=tok, gamma=gamma, uniforms=un)
        tally = parity.Tally()
        parity.check_round(a, rin, T, tally, where=f"drafted round {rnd}")
        assert tally.sequences == B


def test_verify_drafted_without_drafting_is_reported(lib):
    B, G, V, T = 4, 3, 4096, 1.0
    t, d = _logits(5, B, G, V, torch.float32)
    gamma = np.array([3, 2, 0, 3], np.int32); gamma_d = torch.as_tensor(gamma, device=DEV)
    un = wl.round_uniforms(2, 1, B, G)
    ws = lib.new_workspace(B, G, V, DEV)
    tok = torch.zeros(B, G, dtype=torch.int32, device=DEV)
    # only positions 0 and 1 are drafted: sequences with gamma = 3 miss position 2
    for j in range(2):
        lib.bs_draft_sample(d, j, gamma_d, torch.as_tensor(un.u_draft, device=DEV), T, tok, ws)
    acc = torch.full((B,), -1, dtype=torch.int32, device=DEV)
    lib.bs_softmax_verify_drafted(t, d, tok, gamma_d, torch.as_tensor(un.u_accept, device=DEV), T, acc, None, None, ws)
    st = lib.bs_get_device_status(ws, B, G, V)
    assert st[0] & lib.BS_DEV_DRAFT_MISSING and st[3] & lib.BS_DEV_DRAFT_MISSING and int(acc[0]) == 0 and int(acc[3]) == 0
    assert st[1] == 0 and st[2] == 0 and int(acc[2]) == 0
    # rows that are not 16-byte aligned are refused, not mis-read
    d_odd = torch.zeros(2, 2, 1001, device=DEV)
    with pytest.raises(lib.BanditSpecError) as e:
        lib.bs_draft_sample(d_odd, 0, torch.ones(2, dtype=torch.int32, device=DEV), torch.full((2, 2), 0.5, device=DEV),
                            1.0, torch.zeros(2, 2, dtype=torch.int32, device=DEV), lib.new_workspace(2, 2, 1001, DEV))
    assert e.value.code == lib.BS_ERR_UNSUPPORTED


def test_drafted_round_full_size(lib):
    """64 sequences, 128256-entry vocabulary, bf16, ragged speculation lengths up to 8 (the launch
    configuration the benchmark's --drafted round times): drafted tokens of sampled sequences against
    the oracle, the drafted verification against the plain one for every sequence."""
    w = wl.WORKLOADS["llama3_ucb"]
    B, G, V, T = w.B, w.Gmax, w.V, w.temperature
    arm = np.arange(B) % w.K
    rnd = wl.make_round(w, 5, arm, device=DEV)
    gamma_d = torch.as_tensor(rnd.gamma, device=DEV)
    ws = lib.new_workspace(B, G, V, DEV); ws2 = lib.new_workspace(B, G, V, DEV)
    tok = _draft_all(lib, rnd.draft, gamma_d, torch.as_tensor(rnd.uniforms.u_draft, device=DEV), T, ws)
    sample = [0, 3, 17, 42, 63]
    sub = torch.as_tensor(sample, device=DEV)
    assert _check_tokens(tok[sub], rnd.draft[sub], rnd.gamma[sample], rnd.uniforms.u_draft[sample], T) <= 1
    tk = tok.cpu().numpy()
    for b in range(B):
        assert ((tk[b, :rnd.gamma[b]] >= 0) & (tk[b, :rnd.gamma[b]] < V)).all() and (tk[b, rnd.gamma[b]:] == -5).all()
    tok = torch.where(tok < 0, torch.zeros_like(tok), tok).contiguous()
    u_acc = torch.as_tensor(rnd.uniforms.u_accept, device=DEV)
    res = []
    for fn, w_ in ((lib.bs_softmax_verify_drafted, ws), (lib.bs_softmax_verify, ws2)):
        acc = torch.zeros(B, dtype=torch.int32, device=DEV); p = torch.zeros(B, G, device=DEV); q = torch.zeros(B, G, device=DEV)
        fn(rnd.target, rnd.draft, tok, gamma_d, u_acc, T, acc, p, q, w_)
        torch.cuda.synchronize()
        assert (lib.bs_get_device_status(w_, B, G, V) == 0).all()
        res.append((acc, p, q))
    assert torch.equal(res[0][0], res[1][0])
    assert torch.allclose(res[0][1], res[1][1], atol=1e-6, rtol=0) and torch.allclose(res[0][2], res[1][2], atol=1e-6, rtol=0)


def test_drafted_walk_equals_plain_walk_and_the_oracle(lib):
    """draft -> bs_verify_walk_drafted against bs_verify_walk on the same tokens and against the oracle;
    two rounds on one workspace; an undrafted position is reported."""
    rng = np.random.default_rng(8)
    B, G, V, T = 10, 5, 40000, 0.9
    ws = lib.new_workspace(B, G, V, DEV); ws2 = lib.new_workspace(B, G, V, DEV)
    for rnd_i in range(2):
        t, d = _logits(300 + rnd_i, B, G, V, torch.float32, sigma=0.6)
        gamma = rng.integers(0, G + 1, size=B).astype(np.int32); gamma[0] = G
        un = wl.round_uniforms(13, rnd_i + 1, B, G)
        gamma_d = torch.as_tensor(gamma, device=DEV)
        u_acc = torch.as_tensor(un.u_accept, device=DEV); u_res = torch.as_tensor(un.u_resample, device=DEV)
        tok = _draft_all(lib, d, gamma_d, torch.as_tensor(un.u_draft, device=DEV), T, ws)
        tok = torch.where(tok < 0, torch.zeros_like(tok), tok).contiguous()
        outs = []
        for fn, w_ in ((lib.bs_verify_walk_drafted, ws), (lib.bs_verify_walk, ws2)):
            acc = torch.zeros(B, dtype=torch.int32, device=DEV); p = torch.zeros(B, G, device=DEV); q = torch.zeros(B, G, device=DEV)
            ot = torch.zeros(B, G + 1, dtype=torch.int32, device=DEV); ol = torch.zeros(B, dtype=torch.int32, device=DEV)
            fn(t, d, tok, gamma_d, u_acc, u_res, T, acc, p, q, ot, ol, w_)
            torch.cuda.synchronize()
            assert (lib.bs_get_device_status(w_, B, G, V) & ~lib.BS_DEV_RESIDUAL_FALLBACK == 0).all()
            outs.append(lib.RoundOutput(acc, p, q, ot, ol, w_))
        a, b_ = outs
        assert torch.equal(a.accept_len, b_.accept_len) and torch.equal(a.out_tokens, b_.out_tokens)
        assert torch.allclose(a.p_tok, b_.p_tok, atol=1e-6, rtol=0) and torch.allclose(a.q_tok, b_.q_tok, atol=1e-6, rtol=0)
        rin = wl.RoundInputs(target=t, draft=d, tokens=tok, gamma=gamma, uniforms=un)
        tally = parity.Tally()
        parity.check_round(a, rin, T, tally, where=f"drafted walk round {rnd_i}", walk=True)
    # nothing drafted this time: every sequence with gamma > 0 is reported and accepts nothing
    acc = torch.full((B,), -1, dtype=torch.int32, device=DEV)
    ot = torch.zeros(B, G + 1, dtype=torch.int32, device=DEV); ol = torch.zeros(B, dtype=torch.int32, device=DEV)
    lib.bs_verify_walk_drafted(t, d, tok, gamma_d, u_acc, u_res, T, acc, None, None, ot, ol, ws)
    st = lib.bs_get_device_status(ws, B, G, V)
    for b in range(B):
        assert bool(st[b] & lib.BS_DEV_DRAFT_MISSING) == (gamma[b] > 0) and (gamma[b] == 0 or int(acc[b]) == 0)


@pytest.mark.parametrize("walk", [False, True])
def test_a_draft_row_that_cannot_be_sampled_is_reported_by_the_verification(lib, walk):
    """A draft row with a NaN has no finite normaliser: the drafting pass cannot sample it (it emits token 0) and
    says so through the drafted-positions word, the verification call that follows reports BS_DEV_NONFINITE for
    that sequence -- whichever of the two drafted verification entry points is used -- and the other sequences
    are untouched."""
    B, G, V, T = 4, 3, 8192, 1.0
    t, d = _logits(17, B, G, V, torch.float32)
    d[1, 1, 77] = float("nan")
    gamma = np.array([3, 3, 2, 3], np.int32); gamma_d = torch.as_tensor(gamma, device=DEV)
    un = wl.round_uniforms(5, 1, B, G)
    u_d = torch.as_tensor(un.u_draft, device=DEV)
    ws = lib.new_workspace(B, G, V, DEV)
    tok = _draft_all(lib, d, gamma_d, u_d, T, ws)
    assert 0 <= int(tok[1, 1]) < V
    acc = torch.full((B,), -1, dtype=torch.int32, device=DEV)
    p = torch.zeros(B, G, device=DEV); q = torch.zeros(B, G, device=DEV)
    ot = torch.zeros(B, G + 1, dtype=torch.int32, device=DEV); ol = torch.zeros(B, dtype=torch.int32, device=DEV)
    ua = torch.as_tensor(un.u_accept, device=DEV); ur = torch.as_tensor(un.u_resample, device=DEV)
    if walk:
        lib.bs_verify_walk_drafted(t, d, tok, gamma_d, ua, ur, T, acc, p, q, ot, ol, ws)
    else:
        lib.bs_softmax_verify_drafted(t, d, tok, gamma_d, ua, T, acc, p, q, ws)
        lib.bs_residual_sample(t, d, tok, gamma_d, acc, ur, T, ot, ol, ws)
    torch.cuda.synchronize()
    st = lib.bs_get_device_status(ws, B, G, V)
    assert st[1] & lib.BS_DEV_NONFINITE, st
    assert (st[[0, 2, 3]] & ~lib.BS_DEV_RESIDUAL_FALLBACK == 0).all(), st
    # the healthy sequences against the oracle
    rin = wl.RoundInputs(target=t, draft=d, tokens=tok, gamma=gamma, uniforms=un)
    out = lib.RoundOutput(acc, p, q, ot, ol, ws)
    parity.check_round(out, rin, T, parity.Tally(), seqs=[0, 2, 3], where="beside a NaN draft row", walk=walk)
