"""bs_verify_walk (verification with early exit + resampling in one launch) against the CPU oracle,
through the C ABI (needs a B200).  Same rules as the two-call path: accepted lengths and tokens
bit-exact except at flagged near-ties, probabilities of the examined positions within 1e-5."""
import numpy as np
import pytest
import torch

from paper_2505_15141_b200 import workloads as wl
import parity

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _round(rng, B, G, V, dtype, T, sigma=1.0, gamma=None, std=3.0):
    g = torch.Generator(device="cpu"); g.manual_seed(int(rng.integers(1 << 30)))
    t = torch.randn(B, G + 1, V, generator=g) * std
    d = t[:, :G] + sigma * torch.randn(B, G, V, generator=g)
    t, d = t.to(dtype).to(DEV), d.to(dtype).to(DEV)
    gamma = rng.integers(0, G + 1, size=B).astype(np.int32) if gamma is None else np.asarray(gamma, np.int32)
    un = wl.RoundUniforms(rng.random((B, G)).astype(np.float32) * 0.999 + 0.0005,
                          rng.random(B).astype(np.float32) * 0.999 + 0.0005,
                          rng.random(B).astype(np.float32), rng.random((B, G)).astype(np.float32) * 0.999 + 0.0005)
    tok = wl.draw_draft_tokens(d, T, un.u_draft)
    return wl.RoundInputs(target=t, draft=d, tokens=tok.contiguous(), gamma=gamma, uniforms=un)


def _walk(lib, rnd, T, ws=None):
    dev = rnd.target.device
    out = lib.verify_round_walk(rnd.target, rnd.draft, rnd.tokens,
                                torch.as_tensor(np.asarray(rnd.gamma, np.int32), device=dev),
                                torch.as_tensor(rnd.uniforms.u_accept, device=dev),
                                torch.as_tensor(rnd.uniforms.u_resample, device=dev), T, workspace=ws)
    torch.cuda.synchronize()
    return out


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("B,G,V", [(5, 4, 1000), (3, 6, 40000), (40, 3, 8200), (700, 2, 256), (2, 8, 128256),
                                   (1500, 1, 16504), (2600, 1, 16504)])
def test_walk_parity(lib, dtype, B, G, V):
    """One CTA per sequence, several CTAs per sequence, several sequences per CTA; one and many segments; batches
    that fill the clusters' sequence slots and batches beyond them (the kernel that goes through the workspace)."""
    rng = np.random.default_rng(B * 7 + V)
    tally = parity.Tally()
    for T in (1.0, 0.6):
        rnd = _round(rng, B, G, V, dtype, T, sigma=0.7)
        out = _walk(lib, rnd, T)
        st = lib.bs_get_device_status(out.workspace, B, G, V)
        assert (st & ~lib.BS_DEV_RESIDUAL_FALLBACK == 0).all(), st
        seqs = range(B) if B <= 64 else list(range(0, B, 23))
        parity.check_round(out, rnd, T, tally, seqs=seqs, where=f"walk B={B} V={V} T={T}", walk=True)
        y = out.out_len.cpu().numpy(); tau = out.accept_len.cpu().numpy()
        assert ((y == tau + 1) & (tau >= 0) & (tau <= rnd.gamma)).all()
    assert tally.flagged_accept + tally.flagged_token <= 2 + tally.sequences // 100


@pytest.mark.parametrize("B,G,V,dtype", [(6, 12, 40000, torch.float32), (330, 12, 40000, torch.float32),
                                         (3, 31, 65536, torch.bfloat16)])
def test_walk_long_accepted_runs(lib, B, G, V, dtype):
    """Runs of up to 32 positions: a sequence is streamed ahead of its decisions through a few mailboxes that
    are reused every fourth position -- with one sequence per cluster (far ahead) and with several (one ahead).
    Half of the sequences have q == p, so every draft passes and the bonus row is sampled."""
    rng = np.random.default_rng(B + G)
    rnd = _round(rng, B, G, V, dtype, 1.0, sigma=0.25, gamma=rng.integers(G - 2, G + 1, size=B))
    same = np.arange(B) % 2 == 0
    rnd.draft[torch.as_tensor(same, device=DEV)] = rnd.target[torch.as_tensor(same, device=DEV), :G]
    rnd.tokens = wl.draw_draft_tokens(rnd.draft, 1.0, rnd.uniforms.u_draft).contiguous()
    ws = lib.new_workspace(B, G, V, DEV)
    tally = parity.Tally()
    out = _walk(lib, rnd, 1.0, ws)
    assert (lib.bs_get_device_status(ws, B, G, V) & ~lib.BS_DEV_RESIDUAL_FALLBACK == 0).all()
    tau = out.accept_len.cpu().numpy()
    assert (tau[same] == rnd.gamma[same]).all()                          # r <= min{1, 1} always holds
    assert B < 6 or tau[~same].max() >= 4                                # the mailboxes were reused by a rejecting run too
    seqs = range(B) if B <= 8 else list(range(0, B, 37)) + [1]
    parity.check_round(out, rnd, 1.0, tally, seqs=seqs, where=f"walk long runs B={B}", walk=True)
    ref = parity.gpu_round(lib, rnd, 1.0, ws)                            # the two-call path on the same workspace
    differ = [b for b in range(B) if int(ref.accept_len[b]) != int(out.accept_len[b])
              or not torch.equal(ref.out_tokens[b], out.out_tokens[b])]
    parity.check_round(ref, rnd, 1.0, tally, seqs=differ, where="two-call long runs")
    parity.check_round(out, rnd, 1.0, tally, seqs=differ, where="walk long runs", walk=True)
    assert len(differ) <= tally.flagged_accept + tally.flagged_token


def test_walk_edge_cases_and_reuse(lib):
    rng = np.random.default_rng(17)
    B, G, V = 8, 6, 3000
    rnd = _round(rng, B, G, V, torch.float32, 1.0, gamma=[0, G, G, G, 3, 3, 2, 1])
    rnd.draft[2] = rnd.target[2, :G]                                     # q == p: everything passes, bonus row
    rnd.draft[3] = -rnd.target[3, :G] * 3                                # far apart: stops at once
    rnd.target[5] = 1.25; rnd.draft[5] = -0.5                            # constant rows
    rnd.tokens = wl.draw_draft_tokens(rnd.draft, 1.0, rnd.uniforms.u_draft).contiguous()
    ws = lib.new_workspace(B, G, V, DEV)
    tally = parity.Tally()
    out = _walk(lib, rnd, 1.0, ws)
    refs = parity.check_round(out, rnd, 1.0, tally, where="walk edge", walk=True)
    assert refs[0].y == 1 and refs[2].tau == G and refs[3].tau <= 1
    # the same workspace again, and then the two-call path on it: counters were left clean
    out2 = _walk(lib, rnd, 1.0, ws)
    assert torch.equal(out.out_tokens, out2.out_tokens) and torch.equal(out.p_tok, out2.p_tok)
    out3 = parity.gpu_round(lib, rnd, 1.0, ws)
    assert torch.equal(out3.accept_len, out.accept_len) and torch.equal(out3.out_tokens, out.out_tokens)
    # data errors are reported, not fatal
    rnd.tokens[4, 1] = V + 3
    rnd.gamma = np.array([0, G, G, G, 3, 3, 99, 1], np.int32)
    out4 = _walk(lib, rnd, 1.0, ws)
    st = lib.bs_get_device_status(ws, B, G, V)
    assert st[4] & lib.BS_DEV_BAD_TOKEN and int(out4.accept_len[4]) <= 1
    assert st[6] & lib.BS_DEV_BAD_GAMMA and int(out4.out_len[6]) == 1
    parity.check_round(out4, rnd, 1.0, tally, seqs=[0, 1, 2, 3, 5, 7], where="walk after errors", walk=True)
    # rows that are not 16-byte aligned are refused on the host
    odd = _round(rng, 2, 2, 1001, torch.float32, 1.0)
    with pytest.raises(lib.BanditSpecError) as e:
        _walk(lib, odd, 1.0)
    assert e.value.code == lib.BS_ERR_UNSUPPORTED


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_walk_greedy_with_ties(lib, dtype):
    """Temperature 0: a draft passes iff it is the arg-max of its target row (lowest index among equal
    maxima), the emitted token is the arg-max of the stop row; bit-exact, no flags."""
    rng = np.random.default_rng(23)
    tally = parity.Tally()
    for B, G, V in ((6, 5, 4096), (3, 4, 33336), (300, 2, 512)):
        # coarse values -> many exact ties for the arg-max
        t = torch.as_tensor(rng.integers(-4, 5, size=(B, G + 1, V)).astype(np.float32)).to(dtype).to(DEV)
        gamma = rng.integers(0, G + 1, size=B).astype(np.int32)
        tok = t[:, :G].float().argmax(dim=-1).to(torch.int32)
        flip = torch.as_tensor(rng.random((B, G)) < 0.3, device=DEV)
        tok = torch.where(flip, (tok + 1) % V, tok).to(torch.int32).contiguous()
        rnd = wl.RoundInputs(target=t, draft=t[:, :G].contiguous(), tokens=tok, gamma=gamma,
                             uniforms=wl.round_uniforms(1, 1, B, G))
        ws = lib.new_workspace(B, G, V, DEV)
        out = _walk(lib, rnd, 0.0, ws)
        assert (lib.bs_get_device_status(ws, B, G, V) == 0).all()
        seqs = range(B) if B <= 16 else list(range(0, B, 17))
        parity.check_round(out, rnd, 0.0, tally, seqs=seqs, where=f"walk greedy V={V}", walk=True)
        ref = parity.gpu_round(lib, rnd, 0.0, ws)            # the two-call path on the same workspace
        assert torch.equal(ref.accept_len, out.accept_len) and torch.equal(ref.out_tokens, out.out_tokens)
        assert torch.equal(ref.out_len, out.out_len)
    assert tally.flagged_accept == 0 and tally.flagged_token == 0


def test_walk_full_size(lib):
    """The launch configurations the benchmark times: 64 x 128256 bf16 (four CTAs per sequence) and
    256 x 152064 fp32 (one CTA per sequence); sampled sequences against the oracle, all against
    the invariants, and accepted lengths against the two-call path."""
    for name, sample in (("llama3_ucb", [0, 1, 17, 40, 63]), ("qwen_exp3", [0, 100, 255])):
        w = wl.WORKLOADS[name]
        arm = np.arange(w.B) % w.K
        rnd = wl.make_round(w, 7, arm, device=DEV)
        out = _walk(lib, rnd, w.temperature)
        st = lib.bs_get_device_status(out.workspace, w.B, w.Gmax, w.V)
        assert (st & ~lib.BS_DEV_RESIDUAL_FALLBACK == 0).all()
        tally = parity.Tally()
        parity.check_round(out, rnd, w.temperature, tally, seqs=sample, where=f"walk {name}", walk=True)
        ref = parity.gpu_round(lib, rnd, w.temperature)
        # the two paths merge statistics in different orders: they may differ at near-ties only, and the
        # oracle says for every differing sequence whether it is one
        agree = (ref.accept_len == out.accept_len) & (ref.out_tokens == out.out_tokens).all(dim=1)
        differ = [int(b) for b in torch.nonzero(~agree).flatten().cpu().numpy()]
        assert len(differ) <= 6, differ
        ties = parity.Tally()
        parity.check_round(ref, rnd, w.temperature, ties, seqs=differ, where=f"two-call {name}")
        parity.check_round(out, rnd, w.temperature, ties, seqs=differ, where=f"walk {name}", walk=True)
        assert (ties.flagged_accept + ties.flagged_token >= 1) == bool(differ)
        y = out.out_len.cpu().numpy(); tau = out.accept_len.cpu().numpy(); ot = out.out_tokens.cpu().numpy()
        assert ((y == tau + 1) & (tau <= rnd.gamma)).all()
        for b in range(w.B):
            assert 0 <= ot[b, tau[b]] < w.V and (ot[b, y[b]:] == -1).all()


def test_walk_wait_that_cannot_end_is_reported_and_the_context_survives(lib):
    """The CTAs that share a sequence wait for its decision word.  With the sequence's arrival counter
    spoilt beforehand (the workspace's first B words are those counters) no finisher ever completes
    the count, so nobody decides: the producers' bounded wait must give up after about a second, the
    kernel must drain, bs_get_device_status must say BS_ERR_TIMEOUT, and after bs_workspace_init the
    same workspace must work again."""
    rng = np.random.default_rng(41)
    B, G, V = 4, 3, 4096
    rnd = _round(rng, B, G, V, torch.float32, 1.0, gamma=[3, 2, 3, 1])
    ws = lib.new_workspace(B, G, V, DEV)
    ws.view(torch.int32)[2] = 5                                  # sequence 2 can never reach its count
    out = _walk(lib, rnd, 1.0, ws)                               # returns: every wait is bounded
    with pytest.raises(lib.BanditSpecError) as e:
        lib.bs_get_device_status(ws, B, G, V)
    assert e.value.code == lib.BS_ERR_TIMEOUT
    # the other sequences were finished all the same
    tally = parity.Tally()
    parity.check_round(out, rnd, 1.0, tally, seqs=[0, 1, 3], where="walk beside a stuck sequence", walk=True)
    lib.bs_workspace_init(ws)
    out2 = _walk(lib, rnd, 1.0, ws)
    assert (lib.bs_get_device_status(ws, B, G, V) == 0).all()
    parity.check_round(out2, rnd, 1.0, tally, where="walk after re-initialising the workspace", walk=True)
