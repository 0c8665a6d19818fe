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
