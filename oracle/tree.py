"""CPU oracle: tree-based verification -- several draft candidates per position, one target call.

TEST INFRASTRUCTURE ONLY -- see oracle/llama.py.  Shares no code with the CUDA path.

The paper closes with "recent advancement in SPD algorithm to tree-based decoding can also be
used" (Sec. 5) and defines nothing further.  The reading taken here is the multi-candidate
rule of the tree-based systems it cites (SpecInfer's multi-step speculative sampling), which
keeps the guarantee of Sec. 2.1 -- the emitted tokens are distributed as the target's -- when
the candidates at a node are drawn independently (with replacement) from the draft's
distribution at that node.  Letters as everywhere here: p = target, q = draft.

Block layout.  Row 0 is the root: the last committed ("pending") token, not a draft token.
Rows 1..n are draft nodes; parent[i] < i is the row of node i's parent (parent[0] = -1), so
rows are in an order in which parents come first.  The target scores all rows in ONE call
(oracle/llama.py `forward_tree`); row i's output P[i] is the target's distribution for the token
after node i.  Q[i] is the draft's distribution at row i, from which the children of row i were
drawn.  Uniforms: u[i-1] is the accept test of node i (i = 1..n), u[n] the one final draw.

Rule, starting at node = root with cur = P[root]:
  for each child c of node, in row order:
      accept c with probability min(1, cur[x_c] / Q[node][x_c])        (u[c-1] < that value);
      on acceptance descend: node = c, cur = P[c], and start over with c's children;
      on rejection cur <- max(0, cur - Q[node]) / its sum, and the next child is tried;
  when node has no (more) children: the next token is drawn from cur with u[n].
A chain (one child per node) is exactly the rule of oracle/sampling.py: the draw after a
rejected last child is taken from the un-normalised max(0, cur - Q[node]) with the integer
inverse CDF, which is what `reject_sample` does, so the two agree bit for bit.  Between
siblings the residual has to be a probability row again; it is renormalised exactly like
oracle/warp.py renormalises (integer mass Z of the weights, S = fp32(Z) * 2^-32, w / S), so that
the result does not depend on summation order.  Greedy decoding: a child is accepted iff its
token is the arg-max of P[node]; otherwise the arg-max is emitted.

Pinned by tests/test_oracle_tree.py: the exact output law equals p by enumeration on tiny
vocabularies (two and three siblings, two levels), chain == reject_sample bit for bit, greedy
tree decoding == target-only greedy decoding, tree forward == per-path chain forward.
"""
from __future__ import annotations

import numpy as np

from . import sampling as S

F32 = np.float32
TWO32 = F32(4294967296.0)


def tree_layout(parent):
    """parent[0] = -1, parent[i] < i.  Returns (depth [n+1], sees [n+1] = ancestors-and-self as
    sorted row lists, children [n+1] = row lists in row order)."""
    n1 = len(parent)
    assert parent[0] == -1 and all(0 <= parent[i] < i for i in range(1, n1))
    depth = [0] * n1
    sees = [[0]] + [None] * (n1 - 1)
    children = [[] for _ in range(n1)]
    for i in range(1, n1):
        depth[i] = depth[parent[i]] + 1
        sees[i] = sees[parent[i]] + [i]
        children[parent[i]].append(i)
    return depth, sees, children


def level_tree(branching):
    """Parent array of the tree in which every node at depth d-1 has branching[d-1] children,
    rows ordered level by level (breadth first)."""
    parent, level = [-1], [0]
    for b in branching:
        nxt = []
        for node in level:
            for _ in range(int(b)):
                parent.append(node)
                nxt.append(len(parent) - 1)
        level = nxt
    return parent


def renormalised_residual(cur: np.ndarray, q: np.ndarray) -> np.ndarray:
    """max(0, cur - q) divided by its sum; the sum is taken over the integer masses
    trunc(w * 2^32) (order independent), converted once: S = fp32(Z) * 2^-32."""
    w = np.maximum(F32(0.0), cur.astype(F32) - q.astype(F32))
    Z = int(S.fixed_point(w).sum(dtype=np.uint64))
    if Z == 0:
        return w
    return w / (F32(np.uint64(Z)) * F32(2.0 ** -32))


def tree_reject_sample(P: np.ndarray, Q, parent, ids, u, greedy: bool = False):
    """P [n+1, V] target rows, Q [n+1, V] draft rows (rows of leaves unused; None when greedy),
    parent [n+1], ids [n] tokens of rows 1..n, u [n+1].  Returns (path, next_token): the rows of
    the accepted nodes from the root down (possibly empty) and the token emitted after them."""
    n = len(ids)
    assert P.shape[0] == n + 1 and len(parent) == n + 1
    _, _, children = tree_layout(list(parent))
    node, path = 0, []
    while True:
        cur = P[node].astype(F32)
        took = None
        kids = children[node]
        for k, c in enumerate(kids):
            x = int(ids[c - 1])
            if greedy:
                if S.argmax_lowest(P[node]) == x:
                    took = c
                    break
                continue
            if F32(u[c - 1]) < S.accept_prob(cur[x], Q[node][x]):
                took = c
                break
            if k + 1 < len(kids):
                cur = renormalised_residual(cur, Q[node])
            else:       # last child: the draw below takes the un-normalised residual, as in a chain
                cur = np.maximum(F32(0.0), cur - Q[node].astype(F32))
        if took is None:
            if greedy:
                return path, S.argmax_lowest(P[node])
            return path, S.sample_fixed_point(cur, u[n])
        path.append(took)
        node = took
