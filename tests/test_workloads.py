"""Input generators: Philox known answers, uniform mapping, shapes and determinism."""
import numpy as np
import pytest
import torch

from conftest import golden_lines
from paper_2505_15141_b200 import workloads as wl


def test_philox_known_answers():
    for f in golden_lines("philox4x32_10_kat.txt"):
        v = [int(x, 16) for x in f]
        out = wl.philox4x32_10(np.array(v[0:4], dtype=np.uint64), (v[4], v[5]))
        assert [int(x) for x in out] == v[6:10]


def test_philox_vectorised_matches_scalar():
    ctr = np.array([[1, 2, 3, 4], [5, 6, 7, 8], [0xFFFFFFFF, 0, 1, 2]], dtype=np.uint64)
    a = wl.philox4x32_10(ctr, (11, 22))
    for i in range(3):
        assert (wl.philox4x32_10(ctr[i], (11, 22)) == a[i]).all()


def test_uniform_mapping_is_open_interval_and_exact():
    w = np.array([0, 0x1FF, 0x200, 0xFFFFFFFF], dtype=np.uint32)
    u = wl.words_to_uniform(w)
    assert u.dtype == np.float32
    assert u[0] == np.float32(2.0 ** -24) and u[1] == u[0]
    assert u[2] == np.float32(3.0 * 2.0 ** -24)
    assert float(u[3]) == 1.0 - 2.0 ** -24 and u[3] < 1.0 and u[0] > 0.0


def test_round_uniforms_streams_are_distinct_and_reproducible():
    a = wl.round_uniforms(7, 3, B=5, Gmax=6)
    b = wl.round_uniforms(7, 3, B=5, Gmax=6)
    assert (a.u_accept == b.u_accept).all() and (a.u_resample == b.u_resample).all()
    assert a.u_accept.shape == (5, 6) and a.u_resample.shape == (5,) and a.u_arm.shape == (5,)
    assert not np.array_equal(a.u_accept, a.u_draft)
    c = wl.round_uniforms(7, 4, B=5, Gmax=6)
    assert not np.array_equal(a.u_accept, c.u_accept)
    # position j of a sequence does not depend on Gmax
    d = wl.round_uniforms(7, 3, B=5, Gmax=2)
    assert (d.u_accept == a.u_accept[:, :2]).all()
    big = wl.round_uniforms(1, 1, B=64, Gmax=8).u_accept
    assert 0.4 < big.mean() < 0.6


def test_make_round_shapes_and_determinism():
    w = wl.WORKLOADS["tiny_ucb"]
    arm = np.array([0, 1, 2, 1])
    r1 = wl.make_round(w, 5, arm)
    r2 = wl.make_round(w, 5, arm)
    assert r1.target.shape == (4, 7, 1024) and r1.draft.shape == (4, 6, 1024)
    assert r1.target.dtype == torch.float32
    assert torch.equal(r1.target, r2.target) and torch.equal(r1.draft, r2.draft)
    assert torch.equal(r1.tokens, r2.tokens)
    assert list(r1.gamma) == [2, 4, 6, 4]
    assert r1.tokens.dtype == torch.int32 and int(r1.tokens.min()) >= 0 and int(r1.tokens.max()) < 1024


def test_draft_tokens_follow_the_draft_distribution():
    # a 4-token row with known probabilities: the inverse CDF must land where the uniforms say
    logits = torch.log(torch.tensor([[[0.1, 0.2, 0.3, 0.4]]], dtype=torch.float64)).float()
    for u, want in [(0.05, 0), (0.15, 1), (0.29, 1), (0.31, 2), (0.61, 3), (0.99, 3)]:
        tok = wl.draw_draft_tokens(logits, 1.0, np.array([[u]], dtype=np.float32))
        assert int(tok[0, 0]) == want
    assert int(wl.draw_draft_tokens(logits, 0.0, np.array([[0.5]]))[0, 0]) == 3


def test_sigma_schedules():
    w = wl.WORKLOADS["qwen_exp3"]
    arm = np.array([0, 1, 2, 3] * 64)
    s1 = wl.round_sigma(w, 1, arm)
    s201 = wl.round_sigma(w, 201, arm)
    assert np.allclose(s1[:4], [0.3, 0.8, 1.5, 3.0]) and np.allclose(s201[:4], [0.8, 1.5, 3.0, 0.3])
    w3 = wl.WORKLOADS["llama3_ucb"]
    s = wl.round_sigma(w3, 1, None)
    assert s.shape == (64,) and s.min() >= 0.3 and s.max() <= 2.0
    assert (s == wl.round_sigma(w3, 99, None)).all()


def test_throughput_workloads_reward_range_and_step_duration():
    for name in ("llama3_tput", "tiny_tput"):
        w = wl.WORKLOADS[name]
        assert w.alg == "ucb_reward" and w.arm_gamma[0] == 0                 # canonical decoding is an arm
        # the stand-in for the measured step duration grows with the longest speculation length in the batch
        d = [wl.step_seconds(w, np.full(w.B, g)) for g in range(w.Gmax + 1)]
        assert d[0] == w.step_target_s and all(a < b for a, b in zip(d, d[1:]))
        mixed = np.zeros(w.B, dtype=np.int64); mixed[-1] = w.Gmax
        assert wl.step_seconds(w, mixed) == d[-1]
        # no round can earn more than the declared width: every sequence emits Gmax + 1 tokens in the shortest step
        best = (w.Gmax + 1) / d[0] * (w.B if w.whole_batch else 1)
        assert w.reward_width == pytest.approx(best) and w.reward_width > 0
        # gamma = 0 rounds have one target row per sequence and emit exactly one token
        rnd = wl.make_round(w, 1, np.zeros(w.B, dtype=np.int32), B=min(w.B, 3))
        assert (rnd.gamma == 0).all() and rnd.target.shape[1] == w.Gmax + 1


def test_tree_workload_inputs():
    from oracle import tree as ot
    w = wl.TREE_WORKLOADS["tiny_tree"]
    assert w.K == 3 and w.Nmax == 6 and w.depths == (3, 2, 1)
    a, b = wl.make_tree_inputs(w, 3), wl.make_tree_inputs(w, 3)
    assert torch.equal(a.target, b.target) and torch.equal(a.tokens, b.tokens)            # seeded
    assert a.target.shape == (w.B, w.Nmax + 1, w.V) and a.tokens.shape == (w.K, w.B, w.Nmax)
    assert a.shape_nodes.tolist() == [3, 6, 3] and a.shape_parent[1].tolist() == [0, 0, 1, 1, 2, 2]
    # parents come before children, and the shapes' depths are what the checker computes
    for k, s in enumerate(w.shapes):
        assert all(p < n + 1 for n, p in enumerate(s)) and max(ot.tree_depths(list(s), len(s))) == w.depths[k]
    # about p_right of the drafted nodes carry the target's arg-max at their parent
    big = wl.make_tree_inputs(wl.TREE_WORKLOADS["tiny_tree"].__class__("t", B=64, V=512, dtype="f32",
                              shapes=w.shapes, p_right=0.75, seed=1), 1)
    am = big.target.argmax(dim=-1)
    hits = tot = 0
    for k, s in enumerate(w.shapes):
        for n, p in enumerate(s):
            hits += int((big.tokens[k, :, n].long() == am[:, p]).sum()); tot += 64
    assert 0.68 < hits / tot < 0.83
