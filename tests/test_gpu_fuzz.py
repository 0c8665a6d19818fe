"""Seeded random shapes through every verification entry point (needs a B200): the two-call path,
the early-exit walk and the drafted variants must agree with one another on every shape (the
same decisions except at near-ties, the same invariants), and sampled sequences must match the
oracle.  The shapes cover batch sizes below and above the number of resident CTAs, vocabularies
below one segment and of many segments, ragged and zero speculation lengths, both dtypes."""
import numpy as np
import pytest
import torch

from paper_2505_15141_b200 import workloads as wl
import parity

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _shapes(n, seed):
    rng = np.random.default_rng(seed)
    out = []
    for _ in range(n):
        B = int(rng.choice([1, 2, 7, 33, 150, 297, 640]))
        G = int(rng.integers(0, 9))
        V = int(rng.choice([8, 520, 4096, 8200, 16384, 50008, 70000]))
        if B * (2 * G + 1) * V > 6e8:                      # keep a case below a few GB
            B = max(1, int(6e8 / ((2 * G + 1) * V)))
        out.append((B, G, V, bool(rng.integers(0, 2)), float(rng.choice([0.5, 1.0, 1.7]))))
    return out


@pytest.mark.parametrize("B,G,V,bf16,T", _shapes(24, 2024))
def test_entry_points_agree_on_random_shapes(lib, B, G, V, bf16, T):
    rng = np.random.default_rng(B * 131 + G * 17 + V)
    dtype = torch.bfloat16 if bf16 else torch.float32
    g = torch.Generator(device=DEV); g.manual_seed(B + V + G)
    t = torch.randn(B, G + 1, V, generator=g, device=DEV) * 3
    d = (t[:, :G] + 0.8 * torch.randn(B, G, V, generator=g, device=DEV)).to(dtype).contiguous()
    t = t.to(dtype).contiguous()
    gamma = rng.integers(0, G + 1, size=B).astype(np.int32)
    un = wl.round_uniforms(77, 1, B, G)
    gamma_d = torch.as_tensor(gamma, device=DEV)
    u_acc = torch.as_tensor(un.u_accept, device=DEV); u_res = torch.as_tensor(un.u_resample, device=DEV)
    u_dr = torch.as_tensor(un.u_draft, device=DEV)
    ws = lib.new_workspace(B, G, V, DEV)
    # drafting on the device supplies the tokens of this round
    tok = torch.zeros(B, G, dtype=torch.int32, device=DEV)
    for j in range(G):
        lib.bs_draft_sample(d, j, gamma_d, u_dr, T, tok, ws)
    rnd = wl.RoundInputs(target=t, draft=d, tokens=tok, gamma=gamma, uniforms=un)

    def run(kind):
        acc = torch.full((B,), -3, dtype=torch.int32, device=DEV)
        p = torch.zeros(B, G, device=DEV); q = torch.zeros(B, G, device=DEV)
        ot = torch.full((B, G + 1), -3, dtype=torch.int32, device=DEV); ol = torch.full((B,), -3, dtype=torch.int32, device=DEV)
        if kind in ("drafted", "walk_drafted"):              # the statistics are consumed by each use: draft again
            for j in range(G):
                lib.bs_draft_sample(d, j, gamma_d, u_dr, T, tok, ws)
        if kind == "plain":
            lib.bs_softmax_verify(t, d, tok, gamma_d, u_acc, T, acc, p, q, ws)
            lib.bs_residual_sample(t, d, tok, gamma_d, acc, u_res, T, ot, ol, ws)
        elif kind == "drafted":
            lib.bs_softmax_verify_drafted(t, d, tok, gamma_d, u_acc, T, acc, p, q, ws)
            lib.bs_residual_sample(t, d, tok, gamma_d, acc, u_res, T, ot, ol, ws)
        elif kind == "walk":
            lib.bs_verify_walk(t, d, tok, gamma_d, u_acc, u_res, T, acc, p, q, ot, ol, ws)
        else:
            lib.bs_verify_walk_drafted(t, d, tok, gamma_d, u_acc, u_res, T, acc, p, q, ot, ol, ws)
        torch.cuda.synchronize()
        st = lib.bs_get_device_status(ws, B, G, V)
        assert (st & ~lib.BS_DEV_RESIDUAL_FALLBACK == 0).all(), (kind, st)
        return lib.RoundOutput(acc, p, q, ot, ol, ws)

    outs = {k: run(k) for k in ("plain", "drafted", "walk", "walk_drafted")}
    ref = outs["plain"]
    tau = ref.accept_len.cpu().numpy()
    assert ((tau >= 0) & (tau <= gamma)).all() and (ref.out_len.cpu().numpy() == tau + 1).all()
    # Two paths may only differ on a sequence where the oracle sees a near-tie: every differing sequence
    # goes to the oracle on both sides, which accepts a deviation only if it is a flagged accept or
    # CDF-edge tie, and counts it.
    ties = parity.Tally()
    for k in ("drafted", "walk", "walk_drafted"):
        o = outs[k]
        assert torch.equal(o.out_len, o.accept_len + 1), k
        agree = (o.accept_len == ref.accept_len) & (o.out_tokens == ref.out_tokens).all(dim=1)
        differ = [int(b) for b in torch.nonzero(~agree).flatten().cpu().numpy()]
        if differ:
            before = ties.flagged_accept + ties.flagged_token + ties.flagged_fallback
            parity.check_round(ref, rnd, T, ties, seqs=differ, where=f"fuzz plain vs {k}")
            parity.check_round(o, rnd, T, ties, seqs=differ, where=f"fuzz {k} vs plain", walk=k.startswith("walk"))
            assert ties.flagged_accept + ties.flagged_token + ties.flagged_fallback > before, (k, differ)
    assert ties.flagged_accept + ties.flagged_token + ties.flagged_fallback <= max(4, B // 50), vars(ties)
    assert torch.equal(outs["drafted"].accept_len, ref.accept_len)              # same statistics kernels, same pieces
    # a few sequences of every path against the oracle
    seqs = sorted(set(int(x) for x in rng.integers(0, B, size=min(B, 3))))
    tally = parity.Tally()
    parity.check_round(ref, rnd, T, tally, seqs=seqs, where="fuzz plain")
    parity.check_round(outs["walk"], rnd, T, tally, seqs=seqs, where="fuzz walk", walk=True)
    parity.check_round(outs["walk_drafted"], rnd, T, tally, seqs=seqs, where="fuzz walk drafted", walk=True)
