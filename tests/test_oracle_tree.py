"""Pins of the tree checker (oracle/tree.py) against what the paper fixes for greedy decoding.

The paper gives no listing for trees; what it fixes is (a) Section 2: at temperature -> 0 the next
token is the arg-max of the logits, and (b) Proposition 1: whatever the speculative subroutine does,
its output must be what canonical decoding (Algorithm 1) would have produced.  Each test would fail for
a plausible mistake: testing a child against its own row instead of its parent's, taking the first
child instead of the matching one, stopping one level early or late, emitting a drafted token instead
of the arg-max at the stop, a wrong tie rule.
"""
import itertools

import numpy as np

from oracle import tree as ot
from oracle import verify as ov


def _random_tree(rng, n, max_children=3):
    parent = []
    for node in range(1, n + 1):
        while True:
            p = int(rng.integers(0, node))
            if parent.count(p) < max_children:
                break
        parent.append(p)
    return parent


def _toy_model(seed, V, coarse):
    """A 'language model': logits as a fixed function of the whole prefix."""
    def logits(prefix):
        h = hash((seed,) + tuple(int(t) for t in prefix)) & 0x7FFFFFFF
        r = np.random.default_rng(h)
        return r.integers(-3, 4, size=V).astype(np.float64) if coarse else r.normal(0, 2, size=V)
    return logits


def _rows_for_tree(model, prompt, parent, tokens):
    n = len(parent)
    paths = [list(prompt)]
    for node in range(1, n + 1):
        paths.append(paths[parent[node - 1]] + [int(tokens[node - 1])])
    return np.stack([model(p) for p in paths])


def test_output_is_canonical_greedy_decoding():
    """Proposition 1 at temperature -> 0: the emitted tokens are exactly the next y tokens of
    Algorithm 1 run with the arg-max as the sampler, for trees whose drafts are sometimes right."""
    rng = np.random.default_rng(5)
    lengths = []
    for trial in range(300):
        V = int(rng.integers(3, 9))
        coarse = bool(trial % 2)                       # integer logits: many exact ties
        model = _toy_model(trial, V, coarse)
        prompt = [int(t) for t in rng.integers(0, V, size=3)]
        n = int(rng.integers(0, 13))
        parent = _random_tree(rng, n)
        # draft tokens: the true continuation with probability 0.6, anything otherwise
        tokens, paths = [], [list(prompt)]
        for node in range(1, n + 1):
            pre = paths[parent[node - 1]]
            t = int(np.argmax(model(pre))) if rng.random() < 0.6 else int(rng.integers(0, V))
            tokens.append(t)
            paths.append(pre + [t])
        rows = _rows_for_tree(model, prompt, parent, tokens)
        res = ot.verify_tree_greedy(rows, parent, tokens, n)
        # Algorithm 1 with the arg-max sampler, y steps
        pre, want = list(prompt), []
        for _ in range(res.y):
            x = int(np.argmax(model(pre)))
            want.append(x)
            pre.append(x)
        assert res.out_tokens == want and res.y == res.tau + 1 == len(res.nodes) + 1
        # and no path could have gone further: every drafted continuation of the emitted tokens is used up
        prefixes = {tuple(prompt + want[:k]) for k in range(len(want) + 1)}
        assert not any(tuple(paths[c]) == tuple(prompt + want) for c in range(1, n + 1))
        assert all(tuple(paths[c]) in prefixes for c in res.nodes)
        lengths.append(res.y)
    assert max(lengths) >= 4 and min(lengths) == 1     # the cases do exercise deep and empty walks


def test_against_brute_force_over_all_paths():
    """The deepest node whose whole path passes (every node's token is the arg-max of its parent's row),
    the lowest-numbered node among equally deep ones, then the arg-max of that node's row."""
    rng = np.random.default_rng(6)
    for trial in range(300):
        V = int(rng.integers(2, 6))
        n = int(rng.integers(0, 11))
        parent = _random_tree(rng, n, max_children=4)
        rows = rng.integers(-2, 3, size=(n + 1, V)).astype(np.float64)
        tokens = [int(np.argmax(rows[parent[k]])) if rng.random() < 0.7 else int(rng.integers(0, V)) for k in range(n)]
        best = (0, [])                                   # (depth, path)
        for node in range(1, n + 1):
            path, c = [], node
            while c != 0:
                path.append(c)
                c = parent[c - 1]
            path.reverse()
            ok = all(tokens[c - 1] == int(np.argmax(rows[parent[c - 1]])) for c in path)
            if ok and len(path) > best[0]:                # nodes in index order: the first of the deepest stays
                best = (len(path), path)
        res = ot.verify_tree_greedy(rows, parent, tokens, n)
        last = best[1][-1] if best[1] else 0
        assert res.nodes == best[1] and res.tau == best[0]
        assert res.out_tokens == [tokens[c - 1] for c in best[1]] + [int(np.argmax(rows[last]))]


def test_chain_shaped_tree_is_the_chain_rule():
    """parent[n] = n - 1 is vanilla speculative decoding: the same result as the chain checker at T = 0."""
    rng = np.random.default_rng(7)
    for trial in range(100):
        g, V = int(rng.integers(0, 8)), int(rng.integers(2, 7))
        rows = rng.integers(-2, 3, size=(g + 1, V)).astype(np.float64)
        tokens = [int(np.argmax(rows[j])) if rng.random() < 0.75 else int(rng.integers(0, V)) for j in range(g)]
        res = ot.verify_tree_greedy(rows, list(range(g)), tokens, g)
        ref = ov.verify_sequence(rows, None, np.asarray(tokens, dtype=np.int64), g, np.zeros(g), 0.5, 0.0)
        assert res.tau == ref.tau and res.out_tokens == ref.out_tokens and res.nodes == list(range(1, ref.tau + 1))


def test_hand_worked_tree_with_ties_and_duplicates():
    # rows: 0 -> arg-max 2 (tie between 2 and 3: lowest index), row of node 3 -> arg-max 0, row of node 5 -> 1
    rows = np.array([[0., 1., 5., 5.],      # root
                     [9., 0., 0., 0.],      # node 1 (token 3: not the arg-max, never reached)
                     [0., 9., 0., 0.],      # node 2 (token 2, first match at the root)
                     [7., 7., 0., 0.],      # node 3 (token 2 again: a duplicate with nothing under it)
                     [0., 0., 0., 9.],      # node 4 (child of 2, token 0: wrong, row 2's arg-max is 1)
                     [0., 0., 4., 4.],      # node 5 (child of 2, token 1: right)
                     [1., 0., 0., 0.]])     # node 6 (child of 5, token 3: wrong, row 5's arg-max is 2)
    parent = [0, 0, 0, 2, 2, 5]
    tokens = [3, 2, 2, 0, 1, 3]
    res = ot.verify_tree_greedy(rows, parent, tokens, 6)
    assert res.nodes == [2, 5] and res.out_tokens == [2, 1, 2] and res.tau == 2 and res.y == 3
    assert ot.tree_depths(parent, 6) == [1, 1, 1, 2, 2, 3]
    # no nodes at all: canonical decoding, one token
    res = ot.verify_tree_greedy(rows, [], [], 0)
    assert res.nodes == [] and res.out_tokens == [2] and res.y == 1
    # only the first n_nodes nodes exist: node 5 cut off -> the path stops at node 2 and emits row 2's arg-max
    res = ot.verify_tree_greedy(rows, parent, tokens, 4)
    assert res.nodes == [2] and res.out_tokens == [2, 1]
    # a repeated sibling token: both copies pass, the deeper continuation hangs under the second copy
    rows2 = np.array([[0., 9.], [9., 0.], [9., 0.], [0., 9.]])
    res = ot.verify_tree_greedy(rows2, [0, 0, 2], [1, 1, 0], 3)
    assert res.nodes == [2, 3] and res.out_tokens == [1, 0, 1]
