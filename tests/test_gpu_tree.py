"""Greedy verification of trees of drafted tokens on the GPU against the CPU checker (needs a B200),
through the C ABI: bs_tree_verify_greedy and bs_tree_expand_shapes, and tree shapes as the arms of
UCBSpec."""
import numpy as np
import pytest
import torch

from oracle import bandit as ob
from oracle import tree as ot
import parity

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _random_parents(rng, n, nmax, max_children=3):
    parent = []
    for node in range(1, n + 1):
        while True:
            p = int(rng.integers(0, node))
            if parent.count(p) < max_children:
                break
        parent.append(p)
    return parent + [0] * (nmax - n)


def _tokens_for(rng, rows_argmax, parent, n, V, p_right, nmax):
    """Drafted tokens: the target's arg-max at the parent with probability p_right (sometimes twice among siblings)."""
    tok = [int(rows_argmax[parent[k]]) if rng.random() < p_right else int(rng.integers(0, V)) for k in range(n)]
    return tok + [0] * (nmax - n)


def _run(lib, t, parent, tokens, n_nodes, ws=None):
    B, N1, V = t.shape
    N = N1 - 1
    ws = lib.new_workspace(B, N, V, DEV) if ws is None else ws
    acc = torch.full((B,), -5, dtype=torch.int32, device=DEV)
    on = torch.full((B, max(N, 1)), -5, dtype=torch.int32, device=DEV)[:, :N].contiguous()
    otk = torch.full((B, N + 1), -5, dtype=torch.int32, device=DEV)
    ol = torch.full((B,), -5, dtype=torch.int32, device=DEV)
    lib.bs_tree_verify_greedy(t, parent, tokens, n_nodes, acc, on if N else None, otk, ol, ws)
    torch.cuda.synchronize()
    return acc.cpu().numpy(), on.cpu().numpy(), otk.cpu().numpy(), ol.cpu().numpy(), ws


def _check(t, parent, tokens, n_nodes, out, seqs=None):
    acc, on, otk, ol, _ = out
    B, N1, _ = t.shape
    th = t.float().cpu().numpy()
    for b in (range(B) if seqs is None else seqs):
        n = int(n_nodes[b])
        ref = ot.verify_tree_greedy(th[b], parent[b], tokens[b], n)
        assert acc[b] == ref.tau and ol[b] == ref.y, (b, acc[b], ref.tau)
        assert list(otk[b, :ref.y]) == ref.out_tokens and (otk[b, ref.y:] == -1).all(), (b, otk[b], ref.out_tokens)
        if N1 > 1:
            assert list(on[b, :ref.tau]) == ref.nodes and (on[b, ref.tau:] == -1).all(), (b, on[b], ref.nodes)


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("N,V", [(0, 700), (1, 5), (7, 1000), (12, 1001), (31, 8192), (9, 40000), (5, 20011)])
def test_random_trees_match_the_oracle(lib, dtype, N, V):
    """Trees of every size up to the largest supported (31 nodes), vocabularies below and above one segment,
    rows that are and are not 16-byte aligned, coarse logits (many exact ties for the arg-max), drafts that are
    right 70 % of the time, and ragged node counts."""
    rng = np.random.default_rng(N * 1000 + V)
    B = 9
    t = torch.as_tensor(rng.integers(-4, 5, size=(B, N + 1, V)).astype(np.float32)).to(dtype).to(DEV)
    am = t.float().argmax(dim=-1).cpu().numpy()
    n_nodes = rng.integers(0, N + 1, size=B).astype(np.int32)
    n_nodes[0] = N
    parent = np.array([_random_parents(rng, int(n_nodes[b]), N) for b in range(B)], dtype=np.int32).reshape(B, N)
    tokens = np.array([_tokens_for(rng, am[b], parent[b], int(n_nodes[b]), V, 0.7, N) for b in range(B)],
                      dtype=np.int32).reshape(B, N)
    out = _run(lib, t, torch.as_tensor(parent, device=DEV), torch.as_tensor(tokens, device=DEV),
               torch.as_tensor(n_nodes, device=DEV))
    _check(t, parent, tokens, n_nodes, out)
    st = lib.bs_get_device_status(out[4], B, N, V)
    assert (st == 0).all()
    # the same call again on the same workspace: same answer (the counters were left clean)
    out2 = _run(lib, t, torch.as_tensor(parent, device=DEV), torch.as_tensor(tokens, device=DEV),
                torch.as_tensor(n_nodes, device=DEV), ws=out[4])
    for a, b_ in zip(out[:4], out2[:4]):
        assert np.array_equal(a, b_)


def test_chain_shaped_tree_equals_the_two_call_greedy_round(lib):
    rng = np.random.default_rng(3)
    B, G, V = 6, 5, 4096
    t = torch.as_tensor(rng.integers(-4, 5, size=(B, G + 1, V)).astype(np.float32)).to(DEV)
    gamma = rng.integers(0, G + 1, size=B).astype(np.int32)
    tok = t[:, :G].argmax(dim=-1).to(torch.int32)
    tok = torch.where(torch.as_tensor(rng.random((B, G)) < 0.3, device=DEV), (tok + 1) % V, tok).to(torch.int32).contiguous()
    parent = torch.arange(G, dtype=torch.int32, device=DEV).repeat(B, 1).contiguous()
    gam_d = torch.as_tensor(gamma, device=DEV)
    acc, on, otk, ol, ws = _run(lib, t, parent, tok, gam_d)
    ref = lib.verify_round(t, None, tok, gam_d, None, None, 0.0)
    assert np.array_equal(acc, ref.accept_len.cpu().numpy()) and np.array_equal(otk, ref.out_tokens.cpu().numpy())
    assert np.array_equal(ol, ref.out_len.cpu().numpy())


def test_bad_trees_are_reported_not_fatal(lib):
    rng = np.random.default_rng(4)
    B, N, V = 4, 6, 3000
    t = torch.as_tensor(rng.normal(0, 2, size=(B, N + 1, V)).astype(np.float32)).to(DEV)
    am = t.argmax(dim=-1).cpu().numpy()
    parent = np.array([[0, 1, 2, 3, 4, 5]] * B, dtype=np.int32)
    tokens = np.array([[am[b, k] for k in range(N)] for b in range(B)], dtype=np.int32)      # every draft right
    n_nodes = np.array([6, 6, 6, 9], dtype=np.int32)
    parent[1, 2] = 5                       # a parent that comes after its child
    tokens[2, 3] = V + 11                  # a token outside the vocabulary
    out = _run(lib, t, torch.as_tensor(parent, device=DEV), torch.as_tensor(tokens, device=DEV),
               torch.as_tensor(n_nodes, device=DEV))
    acc, on, otk, ol, ws = out
    st = lib.bs_get_device_status(ws, B, N, V)
    assert st[0] == 0 and acc[0] == 6 and list(otk[0]) == list(tokens[0]) + [am[0, 6]]
    assert st[1] & lib.BS_DEV_BAD_TREE and acc[1] == 2                  # nodes 1, 2 pass; node 3 is cut loose
    assert st[2] & lib.BS_DEV_BAD_TOKEN and acc[2] == 3
    assert st[3] & lib.BS_DEV_BAD_GAMMA and acc[3] == 0 and ol[3] == 1 and otk[3, 0] == am[3, 0]
    # host-side argument checks
    f = lib._lib.bs_tree_verify_greedy
    assert f(None, 0, None, None, None, 4, 2, 100, None, None, None, None, None, 0, None) == lib.BS_ERR_INVALID_ARG
    assert lib._lib.bs_tree_expand_shapes(None, None, None, 2, 4, 3, None, None, None) == lib.BS_ERR_INVALID_ARG


SHAPES = {                                   # parents of nodes 1..n; depth of the deepest node
    "chain5": ([0, 1, 2, 3, 4], 5),
    "binary3": ([0, 0, 1, 1, 2, 2, 3, 3, 4, 4, 5, 5, 6, 6], 3),
    "wide2": ([0, 0, 0, 1, 1, 1, 2, 2, 2, 3, 3, 3], 2),
}


def test_tree_shapes_as_arms_of_ucbspec_full_size(lib):
    """Section 3, example (2): the arms are tree shapes.  64 sequences, the LLaMA-3 vocabulary, bf16; each round
    UCBSpec picks a shape per sequence on the device, bs_tree_expand_shapes lays the trees out, the round is verified,
    and the accepted length y is the reward.  Arms against the oracle bandit every round, sampled sequences
    against the tree checker, invariants for all."""
    rng = np.random.default_rng(8)
    B, V = 64, 128256
    names = list(SHAPES)
    K = len(names)
    N = max(len(SHAPES[k][0]) for k in names)
    depth = [SHAPES[k][1] for k in names]
    shape_parent = np.zeros((K, N), dtype=np.int32)
    shape_nodes = np.zeros(K, dtype=np.int32)
    for i, k in enumerate(names):
        shape_parent[i, :len(SHAPES[k][0])] = SHAPES[k][0]
        shape_nodes[i] = len(SHAPES[k][0])
    sp_d, sn_d = torch.as_tensor(shape_parent, device=DEV), torch.as_tensor(shape_nodes, device=DEV)
    state = lib.new_bandit(lib.BS_UCB, B, depth, 0.5, DEV)           # the reward lies in [1, max depth + 1]
    ref_bandit = ob.UCBSpec(B, depth, 0.5)
    ws = lib.new_workspace(B, N, V, DEV)
    arm_d = torch.empty(B, dtype=torch.int32, device=DEV); gam_d = torch.empty_like(arm_d)
    parent_d = torch.empty(B, N, dtype=torch.int32, device=DEV); n_d = torch.empty(B, dtype=torch.int32, device=DEV)
    g = torch.Generator(device=DEV); g.manual_seed(11)
    for rnd in range(10):
        lib.bs_bandit_select(state, lib.BS_UCB, B, K, None, None, arm_d, gam_d)
        arm = arm_d.cpu().numpy().astype(np.int64)
        a_ref, _, flagged = ref_bandit.select()
        assert ((arm == a_ref) | flagged).all()
        lib.bs_tree_expand_shapes(sp_d, sn_d, arm_d, parent_d, n_d)
        parent = parent_d.cpu().numpy(); n_nodes = n_d.cpu().numpy()
        assert np.array_equal(parent, shape_parent[arm]) and np.array_equal(n_nodes, shape_nodes[arm])
        t = (torch.randn(B, N + 1, V, generator=g, device=DEV) * 3).to(torch.bfloat16)
        am = t.float().argmax(dim=-1).cpu().numpy()
        tokens = np.array([_tokens_for(rng, am[b], parent[b], int(n_nodes[b]), V, 0.75, N) for b in range(B)], dtype=np.int32)
        out = _run(lib, t, parent_d, torch.as_tensor(tokens, device=DEV), n_d, ws=ws)
        acc, on, otk, ol, _ = out
        assert (lib.bs_get_device_status(ws, B, N, V) == 0).all()
        _check(t, parent, tokens, n_nodes, out, seqs=[0, 9, 31, 63])
        assert ((ol == acc + 1) & (acc >= 0) & (acc <= np.asarray(depth)[arm])).all()
        y = torch.as_tensor(ol.astype(np.int32), device=DEV)
        lib.bs_bandit_update(state, lib.BS_UCB, B, K, arm_d, y)
        ref_bandit.update(arm, ol.astype(np.int64))
    stt = lib.bs_bandit_read(state, lib.BS_UCB, B, K)
    assert (stt["n"] == ref_bandit.n).all() and (stt["sumY"] == ref_bandit.sumY).all()
