"""Tree-based verification on the device (spd_draft_tree / spd_verify_tree) against the oracle
(oracle/tree.py, SpdOracle.draft_tree / verify_tree), block by block on the same seeded inputs:
draft nodes, the target's logits for every node (tree attention mask, shared positions), the
accepted path, the next token, and -- through the following blocks -- the K/V rows that the
compaction left behind.  Tolerances are those of the plain lock-step (tests/test_gpu_spd.py)."""
import numpy as np
import pytest

import synth
from oracle import sampling as S, tree as T

import harness as H
from test_gpu_spd import _lib

F32 = np.float32


def _walk_uniforms(su, P, Q, parent, ids):
    """Uniforms for one tree verification, chosen on the oracle's side along the walk the rule
    takes: every accept test keeps the stated distance from its threshold, the final draw keeps
    away from a CDF step; nodes the walk never tests get the next plain value."""
    n = len(ids)
    _, _, children = T.tree_layout(list(parent))
    u = np.array([su._next() for _ in range(n + 1)], dtype=F32)
    node = 0
    while True:
        cur = P[node].astype(F32)
        took = None
        kids = children[node]
        for k, c in enumerate(kids):
            x = int(ids[c - 1])
            u[c - 1] = su.for_accept(cur[x], Q[node][x])
            if u[c - 1] < S.accept_prob(cur[x], Q[node][x]):
                took = c
                break
            cur = T.renormalised_residual(cur, Q[node]) if k + 1 < len(kids) else np.maximum(F32(0), cur - Q[node])
        if took is None:
            u[n] = su.for_cdf(cur)
            return u
        node = took


def lockstep_tree(wl, greedy, shapes, n_blocks, logit_tol, std=0.02):
    spd = _lib()
    tw, dw = H.build_weights(wl, std)
    max_seq = wl.n_image + wl.n_prompt + 9 * (n_blocks + 2) + 16
    fp32 = wl.target.dtype == "fp32"
    orc = H.make_oracle(wl, tw, dw, max_seq, 1.0, greedy)
    gpu = H.make_gpu(wl, tw, dw, max_seq, 1.0, greedy)
    img, ids = synth.image_embeds(wl), synth.prompt_ids(wl)
    su = H.SafeUniforms(wl.seeds["uniforms"], f"tree.{wl.name}.{greedy}")
    rep = {"blocks": 0, "accepted": 0, "moved": 0, "tolerated": 0, "max_logit_err": 0.0, "max_draft_logit_err": 0.0}
    if greedy:
        x0 = orc.prefill(img, ids)
        g0 = gpu.prefill(img, ids)
    else:
        probe = H.make_oracle(wl, tw, dw, max_seq, 1.0, greedy)
        probe.prefill(img, ids, u0=0.5)
        u0 = su.for_cdf(S.softmax_t(probe.prefill_logits, 1.0))
        x0 = orc.prefill(img, ids, u0=u0)
        g0 = gpu.prefill(img, ids, u0=u0)
    if g0 != x0:
        gpu.rollback(len(ids), int(ids[-1]), x0)
        rep["tolerated"] += 1

    def resync():
        gpu.prefill(img, np.asarray(orc.seq[:-1], dtype=np.int32), u0=None if greedy else 0.5)
        gpu.rollback(len(orc.seq) - 1, orc.seq[-2], orc.seq[-1])
        rep["tolerated"] += 1

    for b in range(n_blocks):
        br = shapes[b % len(shapes)]
        parent, d_ids, Q = orc.draft_tree(br, None if greedy else (lambda i, prob: su.for_cdf(prob)))
        gparent, g_ids = gpu.draft_tree(br, None if greedy else orc.last_draft_u)
        assert list(gparent) == list(parent)
        n = len(d_ids)
        ids_same = np.array_equal(g_ids, d_ids)
        if not ids_same:
            # a differing node must be a near tie (greedy) / inside the CDF band (sampling) of its parent's row
            i = int(np.argmax(g_ids != d_ids))
            row = orc.last_draft_tree_logits[parent[i + 1]]
            if greedy:
                srt = np.sort(row)[::-1]
                assert np.min(np.abs(np.diff(srt[: max(br) + 1]))) < 1e-2, f"block {b}: node {i + 1} differs"
            else:
                assert H.token_within_cdf_band(Q[parent[i + 1]], orc.last_draft_u[i], int(g_ids[i]),
                                               H.cdf_band(fp32, 2e-5 if fp32 else 2e-3)), f"block {b}: node {i + 1}"
        path, nxt = orc.verify_tree(parent, d_ids, Q, None if greedy else
                                    (lambda P, Qr, par, tids: _walk_uniforms(su, P, Qr, par, tids)))
        if ids_same:
            gpath, gnxt = gpu.verify_tree(parent, None if greedy else orc.last_u)
        else:
            import torch
            gpath, gnxt = gpu.verify_tree(parent, None if greedy else orc.last_u, node_ids=d_ids,
                                          draft_probs=None if greedy else torch.from_numpy(Q).cuda())
        verr = float(np.abs(gpu.get_logits(n + 1) - orc.last_logits).max())
        rep["max_logit_err"] = max(rep["max_logit_err"], verr)
        assert verr < logit_tol, f"block {b}: tree logits differ by {verr}"
        rep["blocks"] += 1
        rep["accepted"] += len(path)
        rep["moved"] += sum(1 for j, node in enumerate(path, 1) if node != j)
        if (gpath, gnxt) == (path, nxt) and ids_same:
            assert gpu.get_state() == (len(orc.seq) - 1, orc.seq[-1])
            continue
        if (gpath, gnxt) != (path, nxt):
            if greedy:
                gaps = [H.top2_gap(orc.last_logits[r]) for r in [0] + path]
                assert min(gaps) < 1e-2, f"block {b}: {(gpath, gnxt)} vs oracle {(path, nxt)}"
            else:
                assert not fp32, f"block {b}: {(gpath, gnxt)} vs oracle {(path, nxt)} on an fp32 model"
                assert gpath == path, f"block {b}: path {gpath} vs oracle {path} (accept margins are 1e-4 wide)"
        resync()
    gpu.close()
    return rep


@pytest.mark.gpu
@pytest.mark.parametrize("greedy", [True, False])
def test_tiny_tree_lockstep(greedy):
    wl = synth.tiny_workload(4)
    r = lockstep_tree(wl, greedy, [[2, 2], [3, 1], [2, 1, 1], [7], [1, 1, 1], [1, 2, 1]], 18, 2e-4,
                      std=0.2 if greedy else 0.1)
    print("tiny tree", greedy, r)
    assert r["blocks"] == 18 and r["tolerated"] == 0
    if not greedy:
        assert r["accepted"] > 0 and r["moved"] > 0      # accepted nodes that had to change cache rows


@pytest.mark.gpu
def test_llava7b_shaped_two_layer_tree_lockstep():
    """Tree blocks at the LLaVA-7B / 115M layer shapes (bf16 weights and KV cache, tensor-core
    attention with the ancestor mask, 640 cached rows), 2 layers each."""
    wl = synth.llava7b_workload(gamma=5, n_layers=2, draft_layers=2)
    r = lockstep_tree(wl, False, [[2, 2], [3, 1], [2, 1, 1]], 4, 5e-2)
    print("two-layer tree", r)
    assert r["blocks"] == 4 and r["max_logit_err"] < 2e-2


@pytest.mark.gpu
def test_llava7b_full_size_tree_blocks_match_oracle():
    """Tree blocks at full depth (32 target layers, 12 draft layers, 576 image rows + 64 prompt ids),
    temperature 1: draft nodes, the target's logits for every node under the tree mask, accepted
    paths and next tokens against the oracle for the shapes [2, 2], [3, 1] and [2, 1, 1]."""
    wl = synth.llava7b_workload(gamma=5)
    r = lockstep_tree(wl, False, [[2, 2], [3, 1], [2, 1, 1]], 3, 5e-2)
    print("full-size tree", r)
    assert r["blocks"] == 3 and r["max_logit_err"] < 4e-2


@pytest.mark.gpu
def test_chain_shaped_tree_equals_the_plain_block_on_the_device():
    """branching [1, 1, 1, 1] is a plain block of gamma = 4: spd_draft_tree / spd_verify_tree must
    return the ids, the accepted count and the next token of spd_draft / spd_verify, block after
    block, for the same uniforms (sampling), and leave the same state."""
    wl = synth.tiny_workload(4)
    tw, dw = H.build_weights(wl, 0.1)
    img, ids = synth.image_embeds(wl), synth.prompt_ids(wl)
    a, b = H.make_gpu(wl, tw, dw, 160, 1.0, False), H.make_gpu(wl, tw, dw, 160, 1.0, False)
    assert a.prefill(img, ids, u0=0.3) == b.prefill(img, ids, u0=0.3)
    u = synth.uniforms(31, "chain.tree", (10, 9))
    accepted = 0
    for blk in range(10):
        d1 = a.draft(4, u[blk, :4])
        acc, nxt = a.verify(4, u[blk, 4:])
        parent, d2 = b.draft_tree([1, 1, 1, 1], u[blk, :4])
        path, nxt2 = b.verify_tree(parent, u[blk, 4:])
        assert np.array_equal(d1, d2) and path == list(range(1, acc + 1)) and nxt == nxt2
        assert a.get_state() == b.get_state()
        accepted += acc
    assert accepted > 0
    a.close()
    b.close()


@pytest.mark.gpu
@pytest.mark.parametrize("branching", [[2, 2], [3, 1], [7]])
def test_greedy_tree_decoding_equals_target_only_greedy_on_the_device(branching):
    """Sec. 4 "Decoding": greedy speculative output == the target's own greedy continuation, for
    any draft -- here a token tree of the draft's most probable continuations.  The draft is the
    target's own network reading the text without the image rows, so its candidates are right
    often enough (and not always as first child) for accepted paths and row moves to occur."""
    import paper_2404_08856_b200 as spd
    wl = synth.Workload("tree-greedy", synth.TINY_TARGET, synth.TINY_TARGET, 16, 16, 4, 32)
    tw = synth.Weights(wl.target, 1, "target", std=0.2)
    img, ids = synth.image_embeds(wl) * F32(0.3), synth.prompt_ids(wl)
    g = spd.Spd(wl.target, wl.target, tw.stored, tw.stored, 200, 7, 1.0, True)
    g.prefill(img, ids)
    want, _ = g.generate(40, 0)                        # the target alone
    first = g.prefill(img, ids)
    got, blocks, later_child = [first], 0, 0
    while len(got) < 40:
        parent, nodes = g.draft_tree(branching)
        path, nxt = g.verify_tree(parent)
        got += [int(nodes[c - 1]) for c in path] + [nxt]
        later_child += sum(1 for j, c in enumerate(path, 1) if c != j)
        blocks += 1
    print("greedy tree", branching, "blocks", blocks, "accepted nodes that were not first children", later_child)
    assert got[:40] == want.tolist()
    assert blocks < 39                                 # some candidates were accepted
    g.close()
