"""CPU oracle: the speculative-decoding block loop around a multimodal target.

TEST INFRASTRUCTURE ONLY -- see oracle/llama.py.  Shares no code with the CUDA path.

Follows Sec. 2.1 and Sec. 3 of the paper, step by step (letters: p = target, q = draft):

1. prefill: the target reads [V_1..V_m ; embed(X_1..X_n)] (Eq. 1) and its last row gives
   the first generated token; the draft reads embed(X_1..X_n) only (Sec. 3), or, for the
   draft with an image adapter (Sec. 4 "Draft Model Candidates", Appendix A.1), the rows
   [H W_a^T ; embed(X)] for a single linear adapter, or [rows ; embed(X)] when the caller
   hands in the output of the draft's own two-layer adapter (oracle/adapter.py);
2. draft: gamma tokens, auto-regressively, x_j ~ q_j(. | text so far) (Sec. 2.1);
3. verify: ONE target call on [pending, x_1..x_gamma] gives p_1..p_{gamma+1}; the
   rejection rule of oracle/sampling.py decides the accepted count a and the next token;
4. commit: x_1..x_a and the next token are emitted; both caches are cut back to the rows
   of emitted tokens (the paper is silent on caches; rows of rejected tokens are simply
   overwritten by the next block).

The last emitted token ("pending") has not been fed to either model yet.  `seq` holds the
prompt followed by every emitted token; position of pending in the target = m + len(seq)-1.

With top_k / top_p set (sampling only; the paper names them as future work, Sec. 4 "Decoding")
every probability row of both models is truncated and renormalised by oracle/warp.py before
it is used: the draft draws from its truncated rows and the rule runs on truncated rows.

Pinned by tests/test_oracle_spd.py: greedy speculative output == the target's own greedy
continuation (Sec. 4 "Decoding"), block efficiency <= gamma + 1, cache state after a
rejection == a fresh model fed only the emitted tokens, top_k = 1 sampling == greedy
decoding, emitted tokens inside the target's kept sets.
"""
from __future__ import annotations

import numpy as np

from .llama import Model, F32
from . import sampling as S
from . import warp as W
from . import tree as T


class SpdOracle:
    def __init__(self, target: Model, draft: Model, temperature: float = 1.0,
                 greedy: bool = False, adapter_w: np.ndarray | None = None,
                 top_k: int = 0, top_p: float = 1.0):
        self.t, self.d = target, draft
        self.temperature, self.greedy = float(temperature), bool(greedy)
        # top-k / top-p (oracle/warp.py): both models' rows are truncated and renormalised, the
        # draft draws from its truncated rows, the unchanged rule runs on the truncated rows
        self.top_k, self.top_p = int(top_k), float(top_p)
        self.truncate = (not self.greedy) and (self.top_k >= 1 or 0.0 < self.top_p < 1.0)
        self.adapter_w = adapter_w  # fp32 [d_draft, adapter_in] or None
        self.tc = self.dc = None
        self.last_logits = None
        self.last_draft_logits = None

    # ---- helpers
    def _probs(self, logits: np.ndarray) -> np.ndarray:
        """softmax(logits / T), truncated to top-k / top-p and renormalised when that is on."""
        prob = S.softmax_t(logits, self.temperature)
        return W.warp_rows(prob, self.top_k, self.top_p) if self.truncate else prob

    def _pick(self, logits_row: np.ndarray, u):
        if self.greedy:
            return S.argmax_lowest(logits_row), None
        prob = self._probs(logits_row)
        return S.sample_fixed_point(prob, u), prob

    @property
    def pending(self) -> int:
        return self.seq[-1]

    # ---- step 1
    def prefill(self, image_embeds, prompt_ids, u0=None, draft_image_feats=None):
        prompt_ids = [int(x) for x in prompt_ids]
        self.m = 0 if image_embeds is None else int(image_embeds.shape[0])
        self.tc, self.dc = self.t.new_cache(), self.d.new_cache()
        rows = self.t.embed(prompt_ids)
        if self.m:
            rows = np.concatenate([np.asarray(image_embeds, dtype=F32), rows], axis=0)
        logits = self.t.forward(self.tc, rows, 0)
        self.prefill_logits = logits[-1]
        x0, _ = self._pick(logits[-1], u0)

        drows = self.d.embed(prompt_ids)
        self.off = 0
        if self.adapter_w is not None or draft_image_feats is not None:
            adapted = np.asarray(draft_image_feats, dtype=F32)     # already in the draft's space ...
            if self.adapter_w is not None:
                adapted = adapted @ self.adapter_w.T                # ... or projected by W_a
            drows = np.concatenate([adapted, drows], axis=0)
            self.off = adapted.shape[0]
        self.d.forward(self.dc, drows, 0)
        self.seq = prompt_ids + [x0]
        self.d_fed = len(prompt_ids)      # tokens of seq whose rows the draft cache holds
        self.n_prompt = len(prompt_ids)
        return x0

    # ---- step 2
    def draft(self, gamma: int, u_draft):
        ids, probs, raw, used = [], [], [], []
        feed = self.seq[self.d_fed:]                    # pending, plus an unseen accepted token
        pos0 = self.off + self.d_fed
        for j in range(gamma):
            logits = self.d.forward(self.dc, self.d.embed(feed), pos0)
            raw.append(logits[-1])
            if self.greedy:
                uj = None
            elif callable(u_draft):      # the caller picks u after seeing q_j (test harness)
                uj = u_draft(j, self._probs(logits[-1]))
            else:
                uj = u_draft[j]
            x, prob = self._pick(logits[-1], uj)
            used.append(0.0 if uj is None else float(uj))
            ids.append(x)
            probs.append(prob)
            pos0 += len(feed)
            feed = [x]
        self.last_draft_logits = np.stack(raw) if raw else None
        self.last_draft_u = np.asarray(used, dtype=F32)
        q = None if (self.greedy or gamma == 0) else np.stack(probs).astype(F32)
        return np.asarray(ids, dtype=np.int32), q

    # ---- steps 3 and 4
    def verify(self, ids, q, u):
        ids = [int(x) for x in ids]
        gamma = len(ids)
        pos0 = self.m + len(self.seq) - 1
        logits = self.t.forward(self.tc, self.t.embed([self.pending] + ids), pos0)
        self.last_logits = logits
        if self.greedy:
            a, nxt = S.reject_sample(logits, None, ids, None, greedy=True)
        else:
            p = self._probs(logits)
            self.last_p = p
            if callable(u):              # the caller picks the uniforms after seeing p and q
                u = u(p, q, ids)
            self.last_u = np.asarray(u, dtype=F32)
            a, nxt = S.reject_sample(p, q, ids, u, greedy=False)
        old_len = len(self.seq)
        self.seq += ids[:a] + [nxt]
        self.tc.length = self.m + len(self.seq) - 1
        if gamma > 0:   # the draft holds rows for the old sequence and x_1..x_{gamma-1}
            self.d_fed = old_len + min(a, gamma - 1)
        self.dc.length = self.off + self.d_fed
        return a, nxt

    # ---- tree-based blocks (Sec. 5; rule and layout: oracle/tree.py)
    @staticmethod
    def _move_rows(cache, src: int, dst: int):
        if src != dst:
            cache.k[:, dst] = cache.k[:, src]
            cache.v[:, dst] = cache.v[:, src]

    def draft_tree(self, branching, u_draft):
        """A token tree below the pending token: every node at depth d-1 gets branching[d-1]
        children, drawn independently from the draft's distribution at that node (greedy: its
        branching[d-1] most probable tokens, lower index first among equals).  The draft is run
        level by level: first the rows it has not seen yet, ending with the root, then the nodes
        of each depth in one tree-masked call.  u_draft[i-1] (or u_draft(i-1, row)) draws node i.
        Returns (parent [n+1], ids [n], Q [n+1, V] or None when greedy)."""
        parent = T.level_tree(branching)
        n = len(parent) - 1
        depth, sees, children = T.tree_layout(parent)
        V = self.d.cfg.vocab
        ids = [0] * n
        Q = None if self.greedy else np.zeros((n + 1, V), dtype=F32)
        used = np.zeros(n, dtype=F32)
        feed = self.seq[self.d_fed:]                   # pending, plus an unseen accepted token
        pos0 = self.off + self.d_fed
        logits = self.d.forward(self.dc, self.d.embed(feed), pos0)
        origin = pos0 + len(feed) - 1                  # the root's position in the draft
        row_logits = {0: logits[-1]}
        level = [0]
        for lev in range(len(branching)):
            for r in level:
                kids = children[r]
                if self.greedy:
                    order = np.argsort(-row_logits[r].astype(np.float64), kind="stable")
                    for k, c in enumerate(kids):
                        ids[c - 1] = int(order[k])
                else:
                    prob = self._probs(row_logits[r])
                    Q[r] = prob
                    for c in kids:
                        uj = u_draft(c - 1, prob) if callable(u_draft) else u_draft[c - 1]
                        used[c - 1] = uj
                        ids[c - 1] = S.sample_fixed_point(prob, uj)
            nxt = [c for r in level for c in children[r]]
            if lev + 1 < len(branching) and nxt:
                lg = self.d.forward_tree(self.dc, self.d.embed([ids[c - 1] for c in nxt]), origin, nxt,
                                         [depth[c] for c in nxt], [sees[c] for c in nxt])
                for k, c in enumerate(nxt):
                    row_logits[c] = lg[k]
            level = nxt
        self.last_draft_u = used
        self.last_draft_tree_logits = row_logits
        self.tree_depth = len(branching)
        return parent, np.asarray(ids, dtype=np.int32), Q

    def verify_tree(self, parent, ids, Q, u):
        """ONE target call on [pending ; the n tree nodes] with the tree mask, the multi-candidate
        rule, then commit: the accepted path's tokens and the next token are emitted and the K/V
        rows of the accepted nodes are moved up to the positions they now hold (row of the node
        at depth j -> origin + j) in both caches.  Returns (path, next_token)."""
        ids = [int(x) for x in ids]
        parent = [int(x) for x in parent]
        n = len(ids)
        depth, sees, _ = T.tree_layout(parent)
        origin = self.m + len(self.seq) - 1
        logits = self.t.forward_tree(self.tc, self.t.embed([self.pending] + ids), origin, list(range(n + 1)),
                                     depth, sees)
        self.last_logits = logits
        if self.greedy:
            path, nxt = T.tree_reject_sample(logits, None, parent, ids, None, greedy=True)
        else:
            P = self._probs(logits)
            self.last_p = P
            if callable(u):
                u = u(P, Q, parent, ids)
            self.last_u = np.asarray(u, dtype=F32)
            path, nxt = T.tree_reject_sample(P, Q, parent, ids, u, greedy=False)
        old_len = len(self.seq)
        d_origin = self.off + old_len - 1
        fed_depth = self.tree_depth - 1                 # the draft was fed nodes down to this depth
        for j, node in enumerate(path, 1):
            self._move_rows(self.tc, origin + node, origin + j)
            if j <= fed_depth:
                self._move_rows(self.dc, d_origin + node, d_origin + j)
        self.seq += [ids[c - 1] for c in path] + [nxt]
        self.tc.length = self.m + len(self.seq) - 1
        self.d_fed = old_len + min(len(path), fed_depth)
        self.dc.length = self.off + self.d_fed
        return path, nxt

    def generate_tree(self, n_new: int, branching, uniforms):
        """Block loop with tree blocks.  uniforms [n_blocks_max, 2n+1]: n draws of the tree's
        nodes, then n accept tests and the final draw."""
        n = len(T.level_tree(branching)) - 1
        start = self.n_prompt
        blocks = accepted = 0
        while len(self.seq) - start < n_new:
            ub = None if uniforms is None else uniforms[blocks]
            parent, ids, Q = self.draft_tree(branching, None if ub is None else ub[:n])
            path, _ = self.verify_tree(parent, ids, Q, None if ub is None else ub[n:])
            blocks += 1
            accepted += len(path)
        emitted = len(self.seq) - start - 1
        return (np.asarray(self.seq[start:start + n_new], dtype=np.int32),
                {"blocks": blocks, "accepted": accepted, "tau": emitted / max(blocks, 1)})

    def target_decode(self, u=None) -> int:
        """Plain auto-regressive step of the target alone: a block with gamma = 0."""
        _, nxt = self.verify([], None, None if self.greedy else [u])
        return nxt

    # ---- loops
    def generate(self, n_new: int, gamma: int, uniforms):
        """Emit until n_new tokens after the prompt exist (the prefill's token counts as
        the first).  uniforms [n_blocks_max, 2*gamma+1]: gamma for the draft's draws, then
        gamma+1 for the verification.  Returns (tokens [n_new], stats)."""
        start = self.n_prompt
        blocks = accepted = 0
        while len(self.seq) - start < n_new:
            ub = None if uniforms is None else uniforms[blocks]
            ids, q = self.draft(gamma, None if ub is None else ub[:gamma])
            a, _ = self.verify(ids, q, None if ub is None else ub[gamma:])
            blocks += 1
            accepted += a
        emitted = len(self.seq) - start - 1   # tokens produced by the blocks themselves
        out = np.asarray(self.seq[start:start + n_new], dtype=np.int32)
        return out, {"blocks": blocks, "accepted": accepted,
                     "tau": emitted / max(blocks, 1)}

    def generate_target_only(self, n_new: int, uniforms=None):
        start = self.n_prompt
        step = 0
        while len(self.seq) - start < n_new:
            self.target_decode(None if uniforms is None else uniforms[step])
            step += 1
        return np.asarray(self.seq[start:start + n_new], dtype=np.int32)


def block_efficiency_closed_form(alpha: float, gamma: int) -> float:
    """Expected tokens per target call when each draft token is accepted independently
    with probability alpha: 1 + alpha + ... + alpha^gamma (bounded by gamma + 1, the
    maximum of block efficiency stated in Sec. 4 "Metrics")."""
    if abs(1.0 - alpha) < 1e-12:
        return float(gamma + 1)
    return (1.0 - alpha ** (gamma + 1)) / (1.0 - alpha)


def mbsu(tau: float, c: float, gamma: int) -> float:
    """Memory-bound speed-up (Sec. 4 "Metrics") with c = draft/target parameter ratio.
    The printed formula c*tau/(c*gamma+1) cannot produce the paper's 2.37x for c ~ 0.017;
    it is read as tau / (c*gamma + 1): a block costs gamma draft steps of relative cost c
    plus one target step, and yields tau tokens."""
    return tau / (c * gamma + 1.0)
