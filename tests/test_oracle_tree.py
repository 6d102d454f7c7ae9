"""Pins for the tree-based verification oracle (oracle/tree.py, Model.forward_tree, the tree
methods of SpdOracle).  CPU only.

What fixes it from outside: the method's guarantee (Sec. 2.1) that emitted tokens are distributed
as the target's -- checked as an exact identity on the rule's own acceptance probabilities and by
chi-squared on the sampler; a chain-shaped tree must be the plain rule bit for bit; greedy tree
decoding must equal the target's own greedy continuation (Sec. 4 "Decoding"); the tree-masked
forward must give every root-to-leaf path the numbers a plain chain gives it.
"""
import itertools

import numpy as np
import pytest
from scipy import stats

import synth
from oracle import llama, sampling as S, tree as T
from oracle.spd import SpdOracle

F32 = np.float32


def _rows(g, n, V, scale=1.0):
    return S.softmax_t((g.standard_normal((n, V)) * scale).astype(F32), 1.0)


def test_layouts():
    parent = T.level_tree([2, 1])
    assert parent == [-1, 0, 0, 1, 2]
    depth, sees, children = T.tree_layout(parent)
    assert depth == [0, 1, 1, 2, 2] and sees[3] == [0, 1, 3] and sees[4] == [0, 2, 4]
    assert children == [[1, 2], [3], [4], [], []]
    assert T.level_tree([1, 1, 1]) == [-1, 0, 1, 2] and T.level_tree([3]) == [-1, 0, 0, 0]


def _law_two_siblings(p, q):
    """Exact law of the emitted token for a root with two children drawn i.i.d. from q, written
    out from the rule's acceptance probabilities in fp64."""
    p, q = p.astype(np.float64), q.astype(np.float64)
    V = len(p)
    law = np.zeros(V)
    for x1, x2 in itertools.product(range(V), repeat=2):
        w = q[x1] * q[x2]
        a1 = min(1.0, p[x1] / q[x1])
        law[x1] += w * a1
        r1 = np.maximum(0.0, p - q)
        r1 = r1 / r1.sum() if r1.sum() > 0 else r1
        a2 = min(1.0, r1[x2] / q[x2])
        law[x2] += w * (1 - a1) * a2
        r2 = np.maximum(0.0, r1 - q)
        r2 = r2 / r2.sum() if r2.sum() > 0 else r1
        law += w * (1 - a1) * (1 - a2) * r2
    return law


@pytest.mark.parametrize("seed", [0, 1, 2])
def test_two_sibling_rule_has_the_targets_law_exactly(seed):
    g = np.random.default_rng(seed)
    p, q = _rows(g, 1, 4, 1.2)[0], _rows(g, 1, 4, 1.2)[0]
    assert np.allclose(_law_two_siblings(p, q), p.astype(np.float64), atol=1e-6)


def test_sampler_follows_the_law_two_and_three_siblings_chi_squared():
    g = np.random.default_rng(5)
    V, N = 5, 60000
    for k in (2, 3):
        p, q = _rows(g, 1, V, 1.3)[0], _rows(g, 1, V, 1.3)[0]
        parent = T.level_tree([k])
        P = np.stack([p] * (k + 1))
        Q = np.stack([q] * (k + 1))
        ud = synth.uniforms(70 + k, "tree.d", (N, k))
        uv = synth.uniforms(71 + k, "tree.v", (N, k + 1))
        counts = np.zeros(V)
        for t in range(N):
            ids = [S.sample_fixed_point(q, ud[t, j]) for j in range(k)]
            path, nxt = T.tree_reject_sample(P, Q, parent, ids, uv[t])
            counts[ids[path[0] - 1] if path else nxt] += 1
        e = p.astype(np.float64)
        _, pval = stats.chisquare(counts, e / e.sum() * N)
        assert pval > 1e-4, (k, pval)


def test_two_level_tree_joint_law_of_the_first_two_tokens():
    """Tree [2, 2]: the target's and the draft's rows at a depth-1 node depend on that node's
    token.  The pair (first, second) emitted token must follow p0(x) * p1[x](y)."""
    g = np.random.default_rng(9)
    V, N = 3, 80000
    p0, q0 = _rows(g, 1, V)[0], _rows(g, 1, V)[0]
    p1, q1 = _rows(g, V, V), _rows(g, V, V)          # conditional rows given the first token
    p2 = _rows(g, V * V, V).reshape(V, V, V)
    parent = T.level_tree([2, 2])
    depth, _, children = T.tree_layout(parent)
    ud = synth.uniforms(80, "tree2.d", (N, 6))
    uv = synth.uniforms(81, "tree2.v", (N, 7))
    counts = np.zeros((V, V))
    for t in range(N):
        ids = [0] * 6
        for c in children[0]:
            ids[c - 1] = S.sample_fixed_point(q0, ud[t, c - 1])
        for r in children[0]:
            for c in children[r]:
                ids[c - 1] = S.sample_fixed_point(q1[ids[r - 1]], ud[t, c - 1])
        P = np.zeros((7, V), F32)
        Q = np.zeros((7, V), F32)
        P[0], Q[0] = p0, q0
        for r in children[0]:
            P[r], Q[r] = p1[ids[r - 1]], q1[ids[r - 1]]
            for c in children[r]:
                P[c] = p2[ids[r - 1], ids[c - 1]]
        path, nxt = T.tree_reject_sample(P, Q, parent, ids, uv[t])
        toks = [ids[c - 1] for c in path] + [nxt]
        if len(toks) < 2:      # rejected at the root: the second token belongs to the next block; draw it from p1
            toks.append(S.sample_fixed_point(p1[toks[0]], ud[t, 5]))
        counts[toks[0], toks[1]] += 1
    want = (p0[:, None].astype(np.float64) * p1.astype(np.float64))
    _, pval = stats.chisquare(counts.ravel(), want.ravel() / want.sum() * N)
    assert pval > 1e-4, pval


def test_chain_shaped_tree_is_the_plain_rule_bit_for_bit():
    g = np.random.default_rng(3)
    V = 50
    for trial in range(400):
        gamma = 1 + trial % 5
        P, Q = _rows(g, gamma + 1, V, 2.0), _rows(g, gamma + 1, V, 2.0)
        if trial % 3 == 0:
            Q[:gamma] = P[:gamma]          # accept-everything branch
        ud = synth.uniforms(90, f"chain.{trial}", gamma)
        ids = [S.sample_fixed_point(Q[j], ud[j]) for j in range(gamma)]
        u = synth.uniforms(91, f"chain.v.{trial}", gamma + 1)
        parent = T.level_tree([1] * gamma)
        for greedy in (False, True):
            path, nxt = T.tree_reject_sample(P, Q, parent, ids, u, greedy)
            a, want = S.reject_sample(P, Q[:gamma], ids, u, greedy)
            assert path == list(range(1, a + 1)) and nxt == want


def _tiny(greedy, std=0.2):
    wl = synth.tiny_workload(4)
    tw = synth.Weights(wl.target, 1, "target", std=std)
    dw = synth.Weights(wl.draft, 1, "draft", std=std)
    mk = lambda: SpdOracle(llama.Model(wl.target, tw, 160), llama.Model(wl.draft, dw, 160), 1.0, greedy)
    return wl, tw, dw, mk


def test_tree_forward_chain_equals_forward_and_paths_equal_chains():
    wl, tw, dw, _ = _tiny(True)
    m = llama.Model(wl.target, tw, 64)
    g = np.random.default_rng(2)
    prefix = g.standard_normal((10, wl.target.d_model)).astype(F32)
    rows = g.standard_normal((5, wl.target.d_model)).astype(F32)
    c1, c2 = m.new_cache(), m.new_cache()
    m.forward(c1, prefix, 0)
    m.forward(c2, prefix, 0)
    a = m.forward(c1, rows, 10)
    b = m.forward_tree(c2, rows, 10, range(5), range(5), [list(range(i + 1)) for i in range(5)])
    assert np.array_equal(a, b) and np.array_equal(c1.k[:, :15], c2.k[:, :15])
    # branching tree: row order [root, a, b, a1, b1]; each path alone as a chain
    parent = T.level_tree([2, 1])
    depth, sees, _ = T.tree_layout(parent)
    c3 = m.new_cache()
    m.forward(c3, prefix, 0)
    tree_logits = m.forward_tree(c3, rows, 10, range(5), depth, sees)
    for leaf in (3, 4):
        path = sees[leaf]
        c4 = m.new_cache()
        m.forward(c4, prefix, 0)
        chain = m.forward(c4, rows[path], 10)
        assert np.abs(chain - tree_logits[path]).max() < 1e-5 * (1.0 + np.abs(chain).max())   # fp32 summation order
        for j, node in enumerate(path):
            assert np.abs(c4.k[:, 10 + j] - c3.k[:, 10 + node]).max() < 1e-5 * (1.0 + np.abs(c4.k[:, 10 + j]).max())


@pytest.mark.parametrize("branching", [[2, 2], [3, 1], [2, 1, 1], [7], [1, 1, 1]])
def test_greedy_tree_decoding_equals_target_only_greedy(branching):
    wl, tw, dw, mk = _tiny(True)
    img, ids = synth.image_embeds(wl), synth.prompt_ids(wl)
    a = mk()
    a.prefill(img, ids)
    want = a.generate_target_only(24)
    b = mk()
    b.prefill(img, ids)
    got, st = b.generate_tree(24, branching, None)
    assert np.array_equal(got, want)
    assert 1.0 <= st["tau"] <= len(branching) + 1


def test_tree_blocks_leave_exactly_the_emitted_tokens_in_both_caches():
    """After several sampled tree blocks (acceptance, rejection, compaction of accepted rows) the
    K/V rows below each cache's length must be those of a fresh model fed the emitted text."""
    wl, tw, dw, mk = _tiny(False, std=0.1)
    img, ids = synth.image_embeds(wl), synth.prompt_ids(wl)
    o = mk()
    o.prefill(img, ids, u0=0.3)
    u = synth.uniforms(21, "tree.loop", (12, 13))
    accepted = 0
    for b in range(10):
        parent, tids, Q = o.draft_tree([2, 2], u[b, :6])
        path, _ = o.verify_tree(parent, tids, Q, u[b, 6:])
        accepted += len(path)
    assert accepted > 0
    fresh_t, fresh_d = llama.Model(wl.target, tw, 160), llama.Model(wl.draft, dw, 160)
    ct, cd = fresh_t.new_cache(), fresh_d.new_cache()
    text = o.seq[:-1]
    fresh_t.forward(ct, np.concatenate([img, fresh_t.embed(text)]), 0)
    assert o.tc.length == ct.length
    assert np.abs(ct.k[:, :ct.length] - o.tc.k[:, :ct.length]).max() < 1e-4
    assert np.abs(ct.v[:, :ct.length] - o.tc.v[:, :ct.length]).max() < 1e-4
    fresh_d.forward(cd, fresh_d.embed(o.seq[:o.d_fed]), 0)
    assert o.dc.length == cd.length
    assert np.abs(cd.k[:, :cd.length] - o.dc.k[:, :cd.length]).max() < 1e-4
