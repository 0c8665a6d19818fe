"""CUDA path against the CPU oracle, element by element, through the C ABI (needs a B200)."""
import numpy as np
import pytest
import torch

from oracle import bandit as ob
from oracle import verify as ov
from paper_2505_15141_b200 import workloads as wl
import parity

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _random_round(rng, B, G, V, dtype, T, sigma=1.0, gamma=None, std=3.0):
    g = torch.Generator(device="cpu"); g.manual_seed(int(rng.integers(1 << 30)))
    t = torch.randn(B, G + 1, V, generator=g) * std
    d = t[:, :G] + sigma * torch.randn(B, G, V, generator=g)
    t, d = t.to(dtype).to(DEV), d.to(dtype).to(DEV)
    gamma = rng.integers(0, G + 1, size=B).astype(np.int32) if gamma is None else np.asarray(gamma, np.int32)
    un = wl.RoundUniforms(rng.random((B, G)).astype(np.float32) * 0.999 + 0.0005,
                          rng.random(B).astype(np.float32) * 0.999 + 0.0005,
                          rng.random(B).astype(np.float32), rng.random((B, G)).astype(np.float32) * 0.999 + 0.0005)
    tok = wl.draw_draft_tokens(d, T, un.u_draft)
    return wl.RoundInputs(target=t, draft=d, tokens=tok, gamma=gamma, uniforms=un)


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("V", [1, 7, 1000, 1001, 8192, 8193, 20011, 40000])
def test_unit_parity_ragged_vocab(lib, dtype, V):
    """Several tiles and ragged tails: V below / at / above one segment, odd V (rows not 16-byte aligned)."""
    rng = np.random.default_rng(V)
    tally = parity.Tally()
    for T in (1.0, 0.6):
        rnd = _random_round(rng, B=5, G=4, V=V, dtype=dtype, T=T)
        out = parity.gpu_round(lib, rnd, T)
        parity.check_round(out, rnd, T, tally, where=f"V={V} T={T}")
        st = lib.bs_get_device_status(out.workspace, 5, 4, V)
        assert (st & ~lib.BS_DEV_RESIDUAL_FALLBACK == 0).all()
    assert tally.sequences == 10


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_greedy_parity_with_ties(lib, dtype):
    rng = np.random.default_rng(3)
    tally = parity.Tally()
    for V in (5, 4096, 33333):
        B, G = 6, 5
        # coarse values -> many exact ties for the arg-max
        t = torch.as_tensor(rng.integers(-4, 5, size=(B, G + 1, V)).astype(np.float32)).to(dtype).to(DEV)
        gamma = rng.integers(0, G + 1, size=B).astype(np.int32)
        tok = t[:, :G].float().argmax(dim=-1).to(torch.int32)           # the right token ...
        flip = torch.as_tensor(rng.random((B, G)) < 0.3, device=DEV)
        tok = torch.where(flip, (tok + 1) % V, tok).to(torch.int32)      # ... except where flipped
        un = wl.round_uniforms(1, 1, B, G)
        rnd = wl.RoundInputs(target=t, draft=t[:, :G].contiguous(), tokens=tok.contiguous(), gamma=gamma, uniforms=un)
        out = parity.gpu_round(lib, rnd, 0.0)
        parity.check_round(out, rnd, 0.0, tally, where=f"greedy V={V}")
    assert tally.flagged_accept == 0 and tally.flagged_token == 0


def test_edge_cases(lib):
    rng = np.random.default_rng(11)
    tally = parity.Tally()
    B, G, V = 8, 6, 3000
    # gamma = 0 (canonical decoding), gamma = Gmax, identical models (accept all),
    # hopeless drafts (reject at first), tokens at 0 and V-1, extreme logits, identical logits
    rnd = _random_round(rng, B, G, V, torch.float32, 1.0, gamma=[0, G, G, G, 3, 3, 2, 1])
    rnd.draft[2] = rnd.target[2, :G]                                     # q == p
    rnd.draft[3] = -rnd.target[3, :G] * 3                                # far apart
    rnd.target[4] *= 26.0; rnd.draft[4] *= 26.0                          # logits up to about +-80
    rnd.target[5] = 1.25; rnd.draft[5] = -0.5                            # constant rows
    tok = wl.draw_draft_tokens(rnd.draft, 1.0, rnd.uniforms.u_draft)
    tok[6, 0] = 0; tok[6, 1] = V - 1
    rnd.tokens = tok.contiguous()
    out = parity.gpu_round(lib, rnd, 1.0)
    refs = parity.check_round(out, rnd, 1.0, tally, where="edge")
    assert refs[0].y == 1 and refs[2].tau == G and refs[2].y == G + 1
    assert refs[3].tau <= 1
    st = lib.bs_get_device_status(out.workspace, B, G, V)
    assert (st & ~lib.BS_DEV_RESIDUAL_FALLBACK == 0).all()
    # Gmax = 0: a batch of canonical-decoding steps
    rnd0 = _random_round(rng, 3, 0, 5000, torch.bfloat16, 0.9)
    out0 = parity.gpu_round(lib, rnd0, 0.9)
    parity.check_round(out0, rnd0, 0.9, tally, where="Gmax=0")
    # the largest supported speculation length
    rndL = _random_round(rng, 2, lib.BS_MAX_GAMMA, 600, torch.float32, 1.0, sigma=0.2,
                         gamma=[lib.BS_MAX_GAMMA, 17])
    outL = parity.gpu_round(lib, rndL, 1.0)
    parity.check_round(outL, rndL, 1.0, tally, where="Gmax=31")


def test_device_data_errors_are_reported_not_fatal(lib):
    rng = np.random.default_rng(12)
    B, G, V = 4, 3, 500
    rnd = _random_round(rng, B, G, V, torch.float32, 1.0, gamma=[3, 3, 3, 3])
    rnd.tokens[1, 1] = V + 7                       # token out of range -> position rejected
    rnd.gamma = np.array([3, 3, 9, 3], np.int32)   # gamma out of range -> processed as gamma 0
    rnd.target[3, 0, 5] = float("nan")             # non-finite normaliser
    out = parity.gpu_round(lib, rnd, 1.0)
    st = lib.bs_get_device_status(out.workspace, B, G, V)
    assert st[0] == 0
    assert st[1] & lib.BS_DEV_BAD_TOKEN and int(out.accept_len[1]) <= 1
    assert st[2] & lib.BS_DEV_BAD_GAMMA and int(out.accept_len[2]) == 0 and int(out.out_len[2]) == 1
    assert st[3] & lib.BS_DEV_NONFINITE
    # the context is still usable and sequence 0 is still right
    tally = parity.Tally()
    parity.check_round(out, rnd, 1.0, tally, seqs=[0], where="after errors")


@pytest.mark.parametrize("dtype,V", [(torch.float32, 4096), (torch.bfloat16, 32000), (torch.float32, 1001),
                                     (torch.bfloat16, 20011)])
def test_zero_mass_residual_falls_back_to_the_target_row(lib, dtype, V):
    """Algorithm 6's else-branch when [P - Q]_+ has no mass.  With draft == target nothing is ever
    rejected, so the stop is forced through bs_residual_sample's accept_len input: the residual at the
    stop row is exactly zero on both sides, the token must be the one the oracle draws from the stop
    row's target distribution, and the status word must say that the fallback was taken.  Aligned
    rows take the pipelined kernels, odd V the generic ones."""
    rng = np.random.default_rng(V + 5)
    B, G, T = 6, 4, 0.8
    rnd = _random_round(rng, B, G, V, dtype, T, gamma=[4, 4, 3, 2, 1, 4])
    rnd.draft = rnd.target[:, :G].clone().contiguous()
    forced = np.array([0, 3, 1, 1, 0, 4], np.int32)              # the last sequence keeps everything: bonus row
    dev = rnd.target.device
    ws = lib.new_workspace(B, G, V, dev)
    acc = torch.empty(B, dtype=torch.int32, device=dev)
    p = torch.empty(B, G, device=dev); q = torch.empty(B, G, device=dev)
    ot = torch.empty(B, G + 1, dtype=torch.int32, device=dev); ol = torch.empty(B, dtype=torch.int32, device=dev)
    gamma_d = torch.as_tensor(rnd.gamma, device=dev)
    lib.bs_softmax_verify(rnd.target, rnd.draft, rnd.tokens, gamma_d, torch.as_tensor(rnd.uniforms.u_accept, device=dev),
                          T, acc, p, q, ws)
    assert (acc.cpu().numpy() == rnd.gamma).all() and torch.allclose(p, q, atol=1e-6, rtol=0)   # q == p accepts everything
    lib.bs_residual_sample(rnd.target, rnd.draft, rnd.tokens, gamma_d, torch.as_tensor(forced, device=dev),
                           torch.as_tensor(rnd.uniforms.u_resample, device=dev), T, ot, ol, ws)
    st = lib.bs_get_device_status(ws, B, G, V)
    assert (st[:5] == lib.BS_DEV_RESIDUAL_FALLBACK).all() and st[5] == 0, st
    toks = rnd.tokens.cpu().numpy()
    flagged = 0
    for b in range(B):
        t_rows = rnd.target[b].float().cpu().numpy()
        u = float(rnd.uniforms.u_resample[b])
        ref = ov.verify_sequence(t_rows, t_rows[:G], toks[b], int(rnd.gamma[b]), rnd.uniforms.u_accept[b], u, T,
                                 keep_mass=True, forced_tau=int(forced[b]))
        assert ref.used_fallback == (b < 5) and ref.tau == forced[b]
        assert int(ol[b]) == forced[b] + 1 and list(ot[b, :forced[b]].cpu().numpy()) == list(toks[b, :forced[b]])
        tok = int(ot[b, forced[b]])
        if tok != ref.token:                                     # only at an edge of the token's interval
            c = np.cumsum(ref.mass) / ref.mass.sum()
            lo, hi = (c[tok - 1] if tok > 0 else 0.0), c[tok]
            assert min(u - ref.cdf_lo, ref.cdf_hi - u) < ov.CDF_TIE and ref.mass[tok] > 0
            assert lo <= u + ov.CDF_TIE and hi >= u - ov.CDF_TIE
            flagged += 1
    assert flagged <= 1


def test_same_inputs_twice_are_bit_identical(lib):
    rng = np.random.default_rng(13)
    rnd = _random_round(rng, 16, 5, 32000, torch.bfloat16, 0.7)
    ws = lib.new_workspace(16, 5, 32000, DEV)
    a = parity.gpu_round(lib, rnd, 0.7, ws)
    a = [x.clone() for x in (a.accept_len, a.p_tok, a.q_tok, a.out_tokens, a.out_len)]
    b = parity.gpu_round(lib, rnd, 0.7, ws)
    for x, y in zip(a, (b.accept_len, b.p_tok, b.q_tok, b.out_tokens, b.out_len)):
        assert torch.equal(x, y)


def test_batch_split_equals_whole_batch(lib):
    """Sequences are independent: two half batches give exactly the whole batch's result."""
    rng = np.random.default_rng(14)
    rnd = _random_round(rng, 8, 4, 9000, torch.float32, 1.0)
    whole = parity.gpu_round(lib, rnd, 1.0)
    for lo, hi in ((0, 4), (4, 8)):
        part = wl.RoundInputs(rnd.target[lo:hi].contiguous(), rnd.draft[lo:hi].contiguous(),
                              rnd.tokens[lo:hi].contiguous(), rnd.gamma[lo:hi],
                              wl.RoundUniforms(rnd.uniforms.u_accept[lo:hi], rnd.uniforms.u_resample[lo:hi],
                                               rnd.uniforms.u_arm[lo:hi], rnd.uniforms.u_draft[lo:hi]))
        o = parity.gpu_round(lib, part, 1.0)
        assert torch.equal(o.accept_len, whole.accept_len[lo:hi])
        assert torch.equal(o.out_tokens, whole.out_tokens[lo:hi])
        assert torch.equal(o.p_tok, whole.p_tok[lo:hi])


# ---- bandits -------------------------------------------------------------------------------

@pytest.mark.parametrize("alg_name", ["ucb", "exp3"])
def test_bandit_trajectories_match_the_oracle(lib, alg_name):
    rng = np.random.default_rng(21)
    B, arm_gamma = 37, (1, 3, 5, 8)
    K = len(arm_gamma)
    alg = lib.BS_UCB if alg_name == "ucb" else lib.BS_EXP3
    state = lib.new_bandit(alg, B, arm_gamma, 0.5, DEV)
    ref = ob.UCBSpec(B, arm_gamma, 0.5) if alg_name == "ucb" else ob.EXP3Spec(B, arm_gamma)
    arm_d = torch.empty(B, dtype=torch.int32, device=DEV); gam_d = torch.empty_like(arm_d)
    idx_d = torch.empty(B, K, dtype=torch.float64, device=DEV)
    flagged_total = 0
    for t in range(300):
        u = rng.random(B).astype(np.float32)
        lib.bs_bandit_select(state, alg, B, K, torch.as_tensor(u, device=DEV), None, arm_d, gam_d, idx_d)
        arm = arm_d.cpu().numpy().astype(np.int64)
        a_ref, g_ref, flagged = (ref.select() if alg_name == "ucb" else ref.select(u))
        shown = idx_d.cpu().numpy()
        if alg_name == "exp3":
            assert np.allclose(shown, ref.last_p, rtol=1e-9, atol=1e-15)
        elif t >= K:
            assert np.allclose(shown, ref.last_index, rtol=1e-11)
        bad = (arm != a_ref) & ~flagged
        assert not bad.any(), (t, np.nonzero(bad))
        for b in np.nonzero(arm != a_ref)[0]:
            flagged_total += 1
            if alg_name == "exp3":
                ref.p_sel[b] = ref.last_p[b][arm[b]]
        assert (gam_d.cpu().numpy() == np.asarray(arm_gamma)[arm]).all()
        y = np.minimum(1 + rng.geometric(0.4, size=B) * (arm + 1) // 2, np.asarray(arm_gamma)[arm] + 1).astype(np.int32)
        lib.bs_bandit_update(state, alg, B, K, arm_d, torch.as_tensor(y, device=DEV))
        ref.update(arm, y)
    st = lib.bs_bandit_read(state, alg, B, K)
    assert (st["t"] == 300).all()
    if alg_name == "ucb":
        assert (st["n"] == ref.n).all() and (st["sumY"] == ref.sumY).all()
    else:
        assert np.allclose(st["S"], ref.S, rtol=1e-10)
    assert flagged_total <= 2


def test_exp3spec_thousand_rounds_without_restart(lib):
    """Algorithm 9 over the 1000 rounds of the 4-armed adversarial workload (256 sequences, arms
    gamma = 1, 3, 5, 8, the arms' acceptance rates rotating every 200 rounds) with NO re-synchronisation
    of the cumulative loss estimates: the oracle keeps its own S throughout and is only told which arm
    the device played.  Both sides are fp64; their exp() routines differ in the last bit and the
    difference compounds (a difference d in S_i moves the next estimate by eta * d relative), so S
    drifts apart -- measured here, bounded below.  What the drift may change is an arm choice whose
    uniform falls between the two sides' CDF edges; every differing choice must be exactly that, and
    the two probability vectors must differ by no more than the drift in S explains."""
    rng = np.random.default_rng(4)
    B, arm_gamma, rounds = 256, (1, 3, 5, 8), 1000
    K, L = len(arm_gamma), max(arm_gamma)
    rate = np.array([0.85, 0.65, 0.45, 0.2])                     # acceptance rate of the draft qualities 0.3 .. 3.0
    state = lib.new_bandit(lib.BS_EXP3, B, arm_gamma, 0.5, DEV)
    ref = ob.EXP3Spec(B, arm_gamma)
    arm_d = torch.empty(B, dtype=torch.int32, device=DEV); gam_d = torch.empty_like(arm_d)
    p_d = torch.empty(B, K, dtype=torch.float64, device=DEV)
    differ, between, worst_p, drift = 0, 0, 0.0, 0.0
    for t in range(1, rounds + 1):
        u = wl.round_uniforms(4, t, B, L).u_arm
        lib.bs_bandit_select(state, lib.BS_EXP3, B, K, torch.as_tensor(u, device=DEV), None, arm_d, gam_d, p_d)
        arm = arm_d.cpu().numpy().astype(np.int64)
        p_gpu = p_d.cpu().numpy()
        a_ref, _, _ = ref.select(u)
        p_ref = ref.last_p
        # first order: dp_i = -eta p_i (dS_i - sum_j p_j dS_j), so |dp| <= 2 eta max|dS|
        eta = ref.learning_rate(t)
        S_gpu = lib.bs_bandit_read(state, lib.BS_EXP3, B, K)["S"]
        dS = np.abs(S_gpu - ref.S).max(axis=1)
        dp = np.abs(p_gpu - p_ref).max(axis=1)
        assert (dp <= 2.5 * eta * dS + 1e-14).all(), (t, float(dp.max()), float(dS.max()))
        worst_p = max(worst_p, float(dp.max()))
        c_gpu, c_ref = np.cumsum(p_gpu, axis=1), np.cumsum(p_ref, axis=1)
        for b in np.nonzero(arm != a_ref)[0]:
            differ += 1
            i = min(arm[b], a_ref[b])                            # the edge the two sides put on opposite sides of u
            assert abs(int(arm[b]) - int(a_ref[b])) == 1, (t, b)
            lo, hi = min(c_gpu[b, i], c_ref[b, i]), max(c_gpu[b, i], c_ref[b, i])
            assert lo - 1e-9 <= u[b] <= hi + 1e-9, (t, b, lo, float(u[b]), hi)
            between += 1
            ref.p_sel[b] = p_ref[b][arm[b]]                      # the oracle plays the device's arm with its own p
        phase = (t - 1) // 200
        alpha = rate[(arm + phase) % 4]
        passes = rng.random((B, L)) < alpha[:, None]
        run = np.where(passes.all(axis=1), L, np.argmin(passes, axis=1))
        y = (1 + np.minimum(run, np.asarray(arm_gamma)[arm])).astype(np.int32)
        lib.bs_bandit_update(state, lib.BS_EXP3, B, K, arm_d, torch.as_tensor(y, device=DEV))
        ref.update(arm, y)
    S_gpu = lib.bs_bandit_read(state, lib.BS_EXP3, B, K)["S"]
    drift = float((np.abs(S_gpu - ref.S) / np.maximum(np.abs(ref.S), 1e-12)).max())
    print(f"EXP3Spec, {rounds} rounds x {B} sequences without restart: {differ} of {rounds * B} arm choices differ, "
          f"all {between} with the uniform between the two CDF edges; largest |dp| {worst_p:.2e}, "
          f"final relative drift of S {drift:.2e}")
    assert differ == between and differ <= 40 and drift < 1e-4


def test_bandit_golden_tables_on_device(lib):
    from conftest import golden_lines
    rows = golden_lines("ucbspec_scripted.txt")
    state = lib.new_bandit(lib.BS_UCB, 1, (2, 4, 6), 0.5, DEV)
    arm_d = torch.empty(1, dtype=torch.int32, device=DEV); gam_d = torch.empty_like(arm_d)
    idx_d = torch.empty(1, 3, dtype=torch.float64, device=DEV)
    for f in rows:
        lib.bs_bandit_select(state, lib.BS_UCB, 1, 3, None, None, arm_d, gam_d, idx_d)
        assert int(arm_d[0]) == int(f[1])
        if f[3] != "rr":
            assert np.allclose(idx_d.cpu().numpy()[0], [float(x) for x in f[3:6]], atol=2e-6)
        lib.bs_bandit_update(state, lib.BS_UCB, 1, 3, arm_d, torch.tensor([int(f[2])], dtype=torch.int32, device=DEV))
    rows = golden_lines("exp3spec_scripted.txt")
    state = lib.new_bandit(lib.BS_EXP3, 1, (2, 4), 0.5, DEV)
    idx_d = torch.empty(1, 2, dtype=torch.float64, device=DEV)
    for f, u in zip(rows, [0.3, 0.9, 0.5, 0.2, 0.7]):
        lib.bs_bandit_select(state, lib.BS_EXP3, 1, 2, torch.tensor([u], dtype=torch.float32, device=DEV), None,
                             arm_d, gam_d, idx_d)
        assert int(arm_d[0]) == int(f[4])
        assert np.allclose(idx_d.cpu().numpy()[0], [float(f[2]), float(f[3])], atol=1e-6)
        lib.bs_bandit_update(state, lib.BS_EXP3, 1, 2, arm_d, torch.tensor([int(f[5])], dtype=torch.int32, device=DEV))
        S = lib.bs_bandit_read(state, lib.BS_EXP3, 1, 2)["S"][0]
        assert np.allclose(S, [float(f[7]), float(f[8])], atol=1e-6)


def test_bandit_checkpoint_and_active_mask(lib):
    B, arm_gamma = 5, (2, 4, 6)
    rng = np.random.default_rng(5)
    ys = rng.integers(1, 8, size=(64, B)).astype(np.int32)

    def run(state, lo, hi, arms):
        arm_d = torch.empty(B, dtype=torch.int32, device=DEV); gam_d = torch.empty_like(arm_d)
        for t in range(lo, hi):
            lib.bs_bandit_select(state, lib.BS_UCB, B, 3, None, None, arm_d, gam_d)
            arms.append(arm_d.cpu().numpy().copy())
            lib.bs_bandit_update(state, lib.BS_UCB, B, 3, arm_d, torch.as_tensor(ys[t], device=DEV))

    a1, a2 = [], []
    s1 = lib.new_bandit(lib.BS_UCB, B, arm_gamma, 0.5, DEV)
    run(s1, 0, 64, a1)
    s2 = lib.new_bandit(lib.BS_UCB, B, arm_gamma, 0.5, DEV)
    run(s2, 0, 32, a2)
    saved = s2.cpu()                                   # checkpoint = the bytes of the state
    s3 = saved.to(DEV)
    run(s3, 32, 64, a2)
    assert np.array_equal(np.stack(a1), np.stack(a2))
    # inactive sequences are frozen
    s4 = lib.new_bandit(lib.BS_UCB, B, arm_gamma, 0.5, DEV)
    act = torch.tensor([1, 0, 1, 0, 1], dtype=torch.uint8, device=DEV)
    arm_d = torch.empty(B, dtype=torch.int32, device=DEV); gam_d = torch.empty_like(arm_d)
    lib.bs_bandit_select(s4, lib.BS_UCB, B, 3, None, act, arm_d, gam_d)
    assert arm_d.cpu().tolist() == [0, -1, 0, -1, 0] and gam_d.cpu().tolist() == [2, 0, 2, 0, 2]
    lib.bs_bandit_update(s4, lib.BS_UCB, B, 3, arm_d, torch.full((B,), 2, dtype=torch.int32, device=DEV), act)
    assert lib.bs_bandit_read(s4, lib.BS_UCB, B, 3)["t"].tolist() == [1, 0, 1, 0, 1]


# ---- closed-loop rounds on the named workloads -----------------------------------------------

def test_closed_loop_tiny_ucb(lib):
    t = parity.closed_loop(lib, wl.WORKLOADS["tiny_ucb"], 64, DEV)
    assert t.sequences == 4 * 64 and t.flagged_accept + t.flagged_token <= 3


def test_closed_loop_tiny_ucb_greedy(lib):
    t = parity.closed_loop(lib, wl.WORKLOADS["tiny_ucb_greedy"], 64, DEV)
    assert t.flagged_accept == 0 and t.flagged_token == 0


def test_closed_loop_llama2_fixed(lib):
    w = wl.WORKLOADS["llama2_fixed"]
    t = parity.closed_loop(lib, w, 40, DEV)
    assert t.sequences == 32 * 40
    assert t.flagged_accept + t.flagged_token <= 0.01 * t.sequences + 2
    t2 = parity.closed_loop(lib, w, w.rounds - 40, DEV, sample=[0, 9, 18, 31], first_round=41)
    assert t2.sequences == 4 * (w.rounds - 40) and t2.flagged_accept + t2.flagged_token <= 0.01 * t2.sequences + 2


def test_closed_loop_llama3_ucb_full_size(lib):
    """Full-size ragged batch in the launch configuration the benchmark times; the oracle replays
    a sample of sequences each round, the bandits of all sequences are compared every round."""
    w = wl.WORKLOADS["llama3_ucb"]
    carry = {}
    t = parity.closed_loop(lib, w, 64, DEV, sample=[0, 1, 17, 40, 63], carry=carry)
    assert t.sequences == 5 * 64 and t.flagged_accept + t.flagged_token <= 5
    # the remaining rounds of the 500: every sequence's arm against the oracle bandit every round
    t2 = parity.closed_loop(lib, w, w.rounds - 64, DEV, sample=[], first_round=65, carry=carry)
    assert t2.flagged_arm <= 2


def test_closed_loop_qwen_exp3_full_size(lib):
    """The first 64 rounds with the oracle replaying three sequences per round, then the bandits alone
    (every sequence's arm compared every round, the oracle bandit fed the CUDA reward) up to the first
    change of the arms' draft quality at round 201, and rounds 190-260 across it with the oracle
    replaying again."""
    w = wl.WORKLOADS["qwen_exp3"]
    carry = {}
    t = parity.closed_loop(lib, w, 64, DEV, sample=[0, 100, 255], carry=carry)
    assert t.sequences == 3 * 64 and t.flagged_accept + t.flagged_token <= 5
    t2 = parity.closed_loop(lib, w, 125, DEV, sample=[], first_round=65, carry=carry)
    assert t2.sequences == 0 and t2.flagged_arm <= 2
    t3 = parity.closed_loop(lib, w, 71, DEV, sample=[7, 200], first_round=190, carry=carry)
    assert t3.sequences == 2 * 71 and t3.flagged_accept + t3.flagged_token <= 4
    # the rest of the 1000 rounds, bandits only: four more rotations of the arms' draft qualities
    flagged, worst = t2.flagged_arm, max(t.max_S_rel, t2.max_S_rel, t3.max_S_rel)
    for first in range(261, w.rounds + 1, 148):
        t4 = parity.closed_loop(lib, w, min(148, w.rounds + 1 - first), DEV, sample=[], first_round=first, carry=carry)
        flagged += t4.flagged_arm
        worst = max(worst, t4.max_S_rel)
    assert flagged <= 3
    print("largest relative difference of the cumulative loss estimates over a stretch:", worst)
    n = lib.bs_bandit_read(carry["state"], lib.BS_EXP3, w.B, w.K)["n"]
    assert (n.sum(axis=1) == w.rounds).all() and (n.sum(axis=0) > 0).all()


def test_full_size_invariants_all_sequences(lib):
    """Properties that hold for every sequence at full size: 1 <= y <= gamma + 1, accepted prefix
    equals the drafts, the emitted token is in range, identical models accept everything."""
    w = wl.WORKLOADS["llama3_ucb"]
    arm = np.arange(w.B) % w.K
    rnd = wl.make_round(w, 3, arm, device=DEV)
    rnd.draft[:8] = rnd.target[:8, :w.Gmax]
    rnd.tokens = wl.draw_draft_tokens(rnd.draft, w.temperature, rnd.uniforms.u_draft)
    out = parity.gpu_round(lib, rnd, w.temperature)
    y = out.out_len.cpu().numpy(); tau = out.accept_len.cpu().numpy(); ot = out.out_tokens.cpu().numpy()
    tk = rnd.tokens.cpu().numpy()
    assert ((y >= 1) & (y <= rnd.gamma + 1) & (y == tau + 1)).all()
    assert (tau[:8] == rnd.gamma[:8]).all()
    for b in range(w.B):
        assert (ot[b, :tau[b]] == tk[b, :tau[b]]).all() and 0 <= ot[b, tau[b]] < w.V and (ot[b, y[b]:] == -1).all()
    p = out.p_tok.cpu().numpy(); q = out.q_tok.cpu().numpy()
    assert np.allclose(p[:8], q[:8], atol=1e-7) and (p >= 0).all() and (p <= 1 + 1e-6).all()


@pytest.mark.parametrize("B,G,V,dtype", [(2, 1, 1 << 20, torch.float32), (2, 2, 1 << 20, torch.bfloat16),
                                         (4096, 1, 64, torch.float32)])
def test_largest_supported_sizes(lib, B, G, V, dtype):
    """The limits the header states: a vocabulary of 2^20 entries (128 / 64 segments per row, 4096
    residual pieces per sequence) and a batch of 4096 sequences."""
    assert lib.bs_workspace_bytes(B, G, V) > 0
    rng = np.random.default_rng(B + V)
    rnd = _random_round(rng, B, G, V, dtype, 1.0, sigma=0.5, std=2.0)
    out = parity.gpu_round(lib, rnd, 1.0)
    st = lib.bs_get_device_status(out.workspace, B, G, V)
    assert (st & ~lib.BS_DEV_RESIDUAL_FALLBACK == 0).all()
    tally = parity.Tally()
    seqs = range(B) if B <= 8 else list(range(0, B, 257))
    parity.check_round(out, rnd, 1.0, tally, seqs=seqs, where=f"max sizes B={B} V={V}")
    y = out.out_len.cpu().numpy(); tau = out.accept_len.cpu().numpy()
    assert ((y == tau + 1) & (tau >= 0) & (tau <= rnd.gamma)).all()
    # one more than the limits is refused on the host
    assert lib.bs_workspace_bytes(B, G, (1 << 20) + 8) == 0 and lib.bs_workspace_bytes(4097, G, V) == 0


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("V", [3000, 40000, 20011])
def test_masked_logits(lib, dtype, V):
    """Logits filtered the way a sampler's top-k does it: everything outside a model's k best entries is
    -inf, with a different set for the two models.  P or Q is exactly zero on most of the vocabulary; a
    drafted token the target has masked must be rejected, whole segments hold no mass at all.  Both the
    two-call path and the early-exit walk (aligned V only)."""
    rng = np.random.default_rng(V + 1)
    tally = parity.Tally()
    B, G, T = 6, 5, 0.9
    rnd = _random_round(rng, B, G, V, dtype, T, sigma=1.5)
    for x, k in ((rnd.target, 40), (rnd.draft, 25)):
        kth = x.float().topk(k, dim=-1).values[..., -1:]
        x.masked_fill_(x.float() < kth, float("-inf"))
    rnd.target[0, :, : V // 2] = float("-inf")                # the first half of the vocabulary carries nothing
    rnd.tokens = wl.draw_draft_tokens(rnd.draft, T, rnd.uniforms.u_draft).contiguous()
    rnd.gamma = np.array([G, G, G, 3, 1, 0], np.int32)
    out = parity.gpu_round(lib, rnd, T)
    st = lib.bs_get_device_status(out.workspace, B, G, V)
    assert (st & ~lib.BS_DEV_RESIDUAL_FALLBACK == 0).all(), st
    refs = parity.check_round(out, rnd, T, tally, where=f"masked V={V}")
    assert tally.sequences == B
    # a drafted token outside the target's kept set has p = 0: never accepted
    p = out.p_tok.cpu().numpy(); tau = out.accept_len.cpu().numpy()
    for b in range(B):
        for j in range(int(rnd.gamma[b])):
            if p[b, j] == 0.0:
                assert tau[b] <= j
    if V % 8 == 0:
        ow = lib.verify_round_walk(rnd.target, rnd.draft, rnd.tokens, torch.as_tensor(rnd.gamma, device=DEV),
                                   torch.as_tensor(rnd.uniforms.u_accept, device=DEV),
                                   torch.as_tensor(rnd.uniforms.u_resample, device=DEV), T)
        torch.cuda.synchronize()
        assert torch.equal(ow.accept_len, out.accept_len) and torch.equal(ow.out_tokens, out.out_tokens)
    # greedy on masked rows: the arg-max is a kept entry
    outg = parity.gpu_round(lib, rnd, 0.0)
    parity.check_round(outg, rnd, 0.0, tally, where=f"masked greedy V={V}")


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("T", [0.05, 0.1, 0.25, 2.0, 8.0])
def test_temperature_range(lib, dtype, T):
    """Sharp and flat distributions.  The exponent x*c - m*c (c = log2(e)/T) is formed in fp32 against the
    rounded product m*c; the kernels undo that rounding to first order (an FMA gives it exactly), so the
    error of a probability does not grow with |m| / T: without the correction it reached 1e-5 at T = 0.05."""
    rng = np.random.default_rng(int(T * 1000))
    tally = parity.Tally()
    for V in (3000, 40000):
        rnd = _random_round(rng, 6, 5, V, dtype, T)
        out = parity.gpu_round(lib, rnd, T)
        parity.check_round(out, rnd, T, tally, where=f"T={T} V={V}")
    assert tally.sequences == 12 and tally.max_p_err < 1e-6
