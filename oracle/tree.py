"""CPU checker for greedy verification of a tree of drafted tokens.  TEST INFRASTRUCTURE.

Plain NumPy / Python.  It exists to check the CUDA path; nothing in the product path may import
it, and it imports nothing from the product.

What the paper fixes.  Section 3 names tree-shaped drafts as a second family of arms (example (2):
the hyperparameter S of the speculative-decoding subroutine is the tree structure) and gives no
verification rule for them; Section 2 fixes greedy decoding: at temperature -> 0 the next token is
the one with the highest logit, a degenerate distribution.  For a degenerate target the rule of
Algorithm 6 (accept iff r <= min{1, P/Q}) accepts a drafted token iff it IS the target's arg-max,
whatever the draft model says, and the correction / bonus token is the target's arg-max of the
position where the walk stops.  A tree only adds a choice of which drafted child to test at each
position, and at most one child can be the arg-max.  So the greedy rule is determined:

    node 0 is the prompt; node n >= 1 carries a drafted token tok[n] and hangs under parent[n] < n;
    row n of the target logits is the target's next-token distribution after the path to node n.
    A node PASSES iff its parent passes (the prompt does) and tok[n] is the arg-max of row parent[n]
    (lowest index among equal maxima).  Among distinct sibling tokens at most one can pass, so the
    passing nodes form one path -- unless the draft repeated a token among siblings, in which case
    every copy passes and the walk may continue under any of them.  The result is the DEEPEST passing
    node (the lowest-numbered one among equally deep ones): its path's tokens are accepted and the
    arg-max of its own row is emitted after them; y = depth + 1 counts that token, as the accepted
    length of Section 3 does.  Every passing path spells the same tokens -- those canonical greedy
    decoding would emit -- so taking the deepest one only decides how many of them a round yields.

Sampling-mode verification of a tree is NOT built: the paper prints no rule for it.

Pins (tests/test_oracle_tree.py): brute force over all root-to-node paths; equality with canonical
greedy decoding (Algorithm 1 at temperature -> 0) on models whose logits are a function of the
prefix, which is what Proposition 1 demands of any speculative subroutine; the chain-shaped tree
against the chain checker of oracle/verify.py; duplicate children and arg-max ties.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import List, Sequence

import numpy as np


@dataclass
class TreeResult:
    tau: int                 # accepted drafted tokens = depth of the node the walk stopped at
    y: int                   # tau + 1: the emitted tokens
    nodes: List[int]         # the accepted nodes, root excluded, in path order
    out_tokens: List[int]    # their tokens, then the arg-max of the last row


def argmax_lowest(row: np.ndarray) -> int:
    """Index of the largest logit, lowest index among equals (Section 2, greedy decoding)."""
    return int(np.argmax(np.asarray(row)))


def verify_tree_greedy(target_rows: np.ndarray, parent: Sequence[int], tokens: Sequence[int], n_nodes: int) -> TreeResult:
    """target_rows [>= n_nodes + 1, V]; parent[n - 1], tokens[n - 1] describe node n = 1..n_nodes."""
    n_nodes = int(n_nodes)
    passes = [True] + [False] * n_nodes
    depth = [0] * (n_nodes + 1)
    best = 0
    for n in range(1, n_nodes + 1):                       # parents come before their children
        par = int(parent[n - 1])
        depth[n] = depth[par] + 1
        passes[n] = passes[par] and int(tokens[n - 1]) == argmax_lowest(target_rows[par])
        if passes[n] and depth[n] > depth[best]:          # strictly deeper: the lowest index wins among equals
            best = n
    nodes: List[int] = []
    c = best
    while c != 0:
        nodes.append(c)
        c = int(parent[c - 1])
    nodes.reverse()
    out = [int(tokens[c - 1]) for c in nodes] + [argmax_lowest(target_rows[best])]
    return TreeResult(tau=len(nodes), y=len(nodes) + 1, nodes=nodes, out_tokens=out)


def tree_depths(parent: Sequence[int], n_nodes: int) -> List[int]:
    """Depth of every node 1..n_nodes (the root has depth 0)."""
    d = [0] * (n_nodes + 1)
    for n in range(1, n_nodes + 1):
        d[n] = d[int(parent[n - 1])] + 1
    return d[1:]
