"""ORACLE (test infrastructure, not the product): Spec-VLA decoding, step by step.

Follows Algorithm 1 (Appendix B) with the draft model of Eq. 2 / Eq. 5 and the relaxed
acceptance rule of Eq. 4 (Section 4.3), as a tree (Section 4.1) rather than the chain the
pseudo-code prints. Readings taken where the paper is silent or inconsistent:

  * accept iff |bin(draft) - bin(target)| <= r (closed interval: r = 0 is strict matching,
    Section 5.2); an id outside the 256 action bins only matches itself;
  * an accepted position keeps the DRAFT token (Algorithm 1, "a_i <- a-hat_i");
  * with several accepted branches the deepest accepted node wins, ties to the lowest node
    index; the token appended after the accepted path is the target's greedy token there
    (the "resample" on reject and the "extra token" when all drafts pass are the same
    expression);
  * the feature handed to the draft model is the final-RMSNorm output; the draft input is
    [feature_i ; embedding_{i+1}] at draft position i (Eagle's one-step shift, Eq. 2);
  * the loop emits m + 1 tokens per iteration and the result is clipped to n_tokens.

Pins (tests/test_oracle_*.py): r = 0 reproduces greedy autoregressive decoding (SD is
lossless); r >= 255 accepts every action-token draft; path selection equals brute force
over all root-to-leaf paths; a one-node tree is one autoregressive step; the cache after
compaction equals a fresh prefill of prefix + emitted tokens. The draft model: every tree
row equals sequential causal draft decoding of its own path (masks, slots, positions of the
draft levels), and draft_forward equals a one-layer library Llama fed the fc output (Eq. 2's
composition and the [feature ; embedding] order). Parity unpinned: only the paper's acceptance
statistics, which need its data and trained weights.

Only tests, the smoke check and the benchmark's CPU-baseline leg may import this package.
"""
from __future__ import annotations

from dataclasses import dataclass, field, replace

import torch

from . import decoder as D


# ----------------------------------------------------------------------------- Eq. 4
def accepts(draft_tok: int, target_tok: int, r: int, action_base: int, n_bins: int) -> bool:
    """Relaxed acceptance test D(a, a-hat) <= r (Eq. 4). D is the absolute difference of
    bin ids when both tokens are action tokens, otherwise 0 if equal and infinite if not."""
    a_is = action_base <= draft_tok < action_base + n_bins
    t_is = action_base <= target_tok < action_base + n_bins
    if a_is and t_is:
        return abs((draft_tok - action_base) - (target_tok - action_base)) <= r
    return draft_tok == target_tok


def accept_and_select(tokens, parent, depth, g, r, action_base, n_bins):
    """Algorithm 1's accept loop on a tree.

    tokens/parent/depth: rows of the tree (row 0 = root, parent[0] = -1, parent[i] < i);
    g[i] = target's greedy token after row i. Node i is accepted when its own draft passes
    against g[parent[i]] and its parent is accepted. Returns (m, path, emitted):
    m = depth of the chosen node n*, path = rows root..n*, emitted = the m draft tokens on
    the path followed by g[n*].
    """
    n = len(tokens)
    acc = [False] * n
    acc[0] = True
    for i in range(1, n):
        acc[i] = acc[parent[i]] and accepts(tokens[i], g[parent[i]], r, action_base, n_bins)
    best = 0
    for i in range(1, n):
        if acc[i] and depth[i] > depth[best]:
            best = i
    path = []
    j = best
    while j != -1:
        path.append(j)
        j = parent[j]
    path.reverse()
    emitted = [tokens[j] for j in path[1:]] + [g[best]]
    return depth[best], path, emitted


# ----------------------------------------------------------------------------- state
def rerank_and_keep(tree, keep: int):
    """Dynamic draft tree (Section 4.1: the Eagle-2 strategy; Section 5.1: at most 50 nodes):
    after the last level every drafted node is ranked by its cumulative log-probability (ties to
    the lower node index) and only the `keep` best are verified. A node never outranks its
    parent (log-probabilities are <= 0 and a parent has the lower index), so the kept set is
    closed under ancestors; kept nodes keep their relative (creation) order."""
    n = len(tree.tokens)
    if n - 1 <= keep:
        return tree
    best = sorted(range(1, n), key=lambda i: (-tree.score[i], i))[:keep]
    kept = [0] + sorted(best)
    new_index = {old: new for new, old in enumerate(kept)}
    return Tree([tree.tokens[i] for i in kept],
                [-1 if tree.parent[i] < 0 else new_index[tree.parent[i]] for i in kept],
                [tree.depth[i] for i in kept],
                [tree.score[i] for i in kept])


@dataclass
class Episode:
    """Decoding state of one episode."""
    cache: D.KVCache                 # target KV, slots 0..P-1 committed
    dcache: D.KVCache                # draft KV, slots 0..Pd-1 committed
    P: int = 0                       # committed target positions
    Pd: int = 0                      # committed draft positions
    root: int = -1                   # last emitted token (not yet in the target cache)
    pending_feat: list = field(default_factory=list)   # draft rows waiting to run:
    pending_tok: list = field(default_factory=list)    # (feature_i, token_{i+1}) at position Pd + j
    emitted: list = field(default_factory=list)


@dataclass
class Tree:
    tokens: list
    parent: list
    depth: list
    score: list


class SpecVLAOracle:
    def __init__(self, desc, weights: dict, action_only: bool = True, max_seq: int = 512,
                 max_tree_rows: int = 128, dtype=torch.float64):
        self.desc = desc
        self.w = D.DecoderWeights(weights, dtype)
        self.action_only = bool(action_only)
        self.max_seq = max_seq
        self.max_tree_rows = max_tree_rows
        self.dtype = dtype

    # ------------------------------------------------------------------ helpers
    def _new_episode(self) -> Episode:
        d = self.desc
        slots = self.max_seq + self.max_tree_rows
        return Episode(D.KVCache(d.n_layers, slots, d.n_heads, d.head_dim, self.dtype),
                       D.KVCache(1, slots, d.n_heads, d.head_dim, self.dtype))

    def _embed(self, toks) -> torch.Tensor:
        return self.w("embed")[torch.tensor(list(toks), dtype=torch.long)]

    def _greedy(self, logits_row) -> int:
        return D.greedy_token(logits_row, self.desc, self.action_only)

    @staticmethod
    def _causal(n_before: int, T: int) -> torch.Tensor:
        """Row t (slot n_before + t) sees slots 0..n_before + t."""
        s = torch.arange(n_before + T)[None, :]
        return s <= (n_before + torch.arange(T))[:, None]

    @staticmethod
    def _tree_visible(n_before: int, parent, rows=None) -> torch.Tensor:
        """Row i (slot n_before + i) sees slots < n_before, its ancestors' slots and its own."""
        T = len(parent)
        vis = torch.zeros(T, n_before + T, dtype=torch.bool)
        vis[:, :n_before] = True
        for i in range(T):
            j = i
            while j != -1:
                vis[i, n_before + j] = True
                j = parent[j]
        return vis

    # ------------------------------------------------------------------ Section 4.1, prefill
    def _follow(self, logits_row, own: int, other, margin: float) -> int:
        """Re-synchronisation used by parity tests: where the top-2 margin of this row is at most
        `margin`, the two best tokens are equally valid at the compared precision, and decoding
        continues with the token `other` that the implementation under test chose, so that the
        rest of the chunk stays comparable. Everywhere else the oracle's own token stands."""
        if other is None or D.top2_margin(logits_row, self.desc, self.action_only) > margin:
            return own
        return int(other)

    def prefill(self, embeds, token_ids, want_logits: bool = False, follow=None):
        """Target forward over the P prefix rows (causal); first token a_1 = greedy token of
        the last row; draft forward over the P-1 shifted pairs (feature_i, input_{i+1}).
        follow = (token, margin): see _follow."""
        ep = self._new_episode()
        x = D.embed_rows(self.w, embeds, token_ids)
        P = x.shape[0]
        pos = torch.arange(P)
        feats = D.target_forward(self.w, self.desc, x, pos, pos, self._causal(0, P), ep.cache)
        logits_last = D.lm_head(self.w, feats[P - 1:P])[0]
        a1 = self._greedy(logits_last)
        if follow is not None:
            a1 = self._follow(logits_last, a1, follow[0], follow[1])
        if P > 1:
            dpos = torch.arange(P - 1)
            D.draft_forward(self.w, self.desc, feats[:P - 1], x[1:], dpos, dpos,
                            self._causal(0, P - 1), ep.dcache)
        ep.P, ep.Pd = P, P - 1
        ep.root = a1
        ep.emitted = [a1]
        ep.pending_feat = [feats[P - 1]]
        ep.pending_tok = [a1]
        if want_logits:
            return ep, logits_last, feats
        return ep

    # ------------------------------------------------------------------ Algorithm 1, draft loop
    def draft_tree(self, ep: Episode, shape, want_debug: bool = False) -> Tree:
        """Static-size Eagle-style tree: level l expands the shape.expand[l] best nodes of the
        previous level (by cumulative log-probability, ties to the lower node index), each
        into its shape.branch[l] most probable tokens."""
        desc = self.desc
        a0, nb = desc.action_base, desc.n_bins
        # catch-up: run the pending (feature, token) pairs, causal among themselves
        n_pend = len(ep.pending_tok)
        pos = torch.arange(ep.Pd, ep.Pd + n_pend)
        out = D.draft_forward(self.w, desc, torch.stack(ep.pending_feat),
                              self._embed(ep.pending_tok), pos, pos,
                              self._causal(ep.Pd, n_pend), ep.dcache)
        ep.Pd += n_pend
        ep.pending_feat, ep.pending_tok = [], []
        Pd = ep.Pd                                  # == ep.P: the root's draft row is slot Pd-1

        tokens, parent, depth, score = [ep.root], [-1], [0], [0.0]
        produced_by = {0: out[n_pend - 1]}          # node -> draft output that scores its children
        draft_row = {}                              # node -> tree row index in the draft cache
        row_parent = []                             # tree-row ancestry for the draft mask
        level = [0]
        debug = []
        for l in range(shape.depth):
            ranked = sorted(level, key=lambda n: (-score[n], n))[:shape.expand[l]]
            if l > 0:
                # one draft forward over the selected nodes of the previous level
                feat_in = torch.stack([produced_by[parent[n]] for n in ranked])
                emb_in = self._embed([tokens[n] for n in ranked])
                first = len(row_parent)
                for n in ranked:
                    draft_row[n] = len(row_parent)
                    row_parent.append(draft_row.get(parent[n], -1))
                T = len(ranked)
                vis = torch.zeros(T, Pd + len(row_parent), dtype=torch.bool)
                vis[:, :Pd] = True
                for t in range(T):
                    j = first + t
                    while j != -1:
                        vis[t, Pd + j] = True
                        j = row_parent[j]
                pos = torch.full((T,), Pd - 1 + l)
                slots = torch.arange(Pd + first, Pd + first + T)
                out = D.draft_forward(self.w, desc, feat_in, emb_in, pos, slots, vis, ep.dcache)
                for t, n in enumerate(ranked):
                    produced_by[n] = out[t]
            nxt = []
            for n in ranked:
                # the draft model scores with its own copy of the LM head when the target's is quantised
                head = "draft.lm_head" if "draft.lm_head" in self.w.raw else "lm_head"
                logits = D.lm_head(self.w, produced_by[n][None, :], head)[0]
                if self.action_only:
                    lp_all = torch.log_softmax(logits[a0:a0 + nb], dim=0)
                    base = a0
                else:
                    lp_all = torch.log_softmax(logits, dim=0)
                    base = 0
                order = sorted(range(lp_all.numel()), key=lambda v: (-float(lp_all[v]), v))
                if want_debug:
                    debug.append((n, lp_all.clone(), base, produced_by[n]))
                for v in order[:shape.branch[l]]:
                    nxt.append(len(tokens))
                    tokens.append(base + v)
                    parent.append(n)
                    depth.append(l + 1)
                    score.append(score[n] + float(lp_all[v]))
            level = nxt
        tree = Tree(tokens, parent, depth, score)
        if getattr(shape, "keep", 0) > 0:
            tree = rerank_and_keep(tree, shape.keep)
        if want_debug:
            return tree, debug
        return tree

    # ------------------------------------------------------------------ Algorithm 1, verify + accept
    def verify_forward(self, ep: Episode, tree: Tree):
        """One target forward over all tree rows (row i at position P + depth[i], slot P + i,
        attending the prefix, its ancestors and itself). Returns (logits [T, V], features)."""
        P = ep.P
        T = len(tree.tokens)
        x = self._embed(tree.tokens)
        pos = P + torch.tensor(tree.depth)
        slots = torch.arange(P, P + T)
        feats = D.target_forward(self.w, self.desc, x, pos, slots,
                                 self._tree_visible(P, tree.parent), ep.cache)
        return D.lm_head(self.w, feats), feats

    def verify_tree(self, ep: Episode, tree: Tree, r: int, want_debug: bool = False, follow=None):
        """Verify, accept (Eq. 4), select the longest accepted path, compact the cache and set
        up the next iteration. Returns (m, emitted tokens [m + 1]).
        follow = (tokens per row, margin): see _follow."""
        desc = self.desc
        logits, feats = self.verify_forward(ep, tree)
        g_own = [self._greedy(logits[i]) for i in range(len(tree.tokens))]
        g = g_own if follow is None else [self._follow(logits[i], g_own[i], follow[0][i], follow[1])
                                          for i in range(len(tree.tokens))]
        m, path, emitted = accept_and_select(tree.tokens, tree.parent, tree.depth, g, r,
                                             desc.action_base, desc.n_bins)
        # compaction: accepted rows move next to the root (ascending j: a destination slot
        # P + j is never the source of a later move because path[j'] >= j' > j)
        P = ep.P
        for l in range(desc.n_layers):
            for j in range(1, m + 1):
                ep.cache.k[l][P + j] = ep.cache.k[l][P + path[j]].clone()
                ep.cache.v[l][P + j] = ep.cache.v[l][P + path[j]].clone()
        ep.P = P + 1 + m
        ep.root = emitted[-1]
        ep.emitted += emitted
        ep.pending_feat = [feats[j] for j in path]
        ep.pending_tok = list(emitted)
        if want_debug:
            return m, emitted, dict(logits=logits, feats=feats, g=g, g_own=g_own, path=path)
        return m, emitted

    # ------------------------------------------------------------------ Algorithm 1, outer loop
    def generate_action(self, embeds, token_ids, shape, r: int, n_tokens: int = 7,
                        tree_fn=None, prune: bool = False):
        """Prefill, then draft -> verify -> accept until n_tokens are emitted; clip.
        tree_fn(ep, iteration) may supply the tree instead of the draft model (planted or
        random drafts). Returns (tokens [n_tokens], accept lengths per iteration).

        prune (not in Algorithm 1, which drafts to a fixed depth and clips the chunk at the end):
        an iteration that still misses k tokens drafts only k - 1 levels deep, since the
        verification adds one token of its own and everything beyond is clipped; with k = 1 it
        drafts nothing and verifies the root alone."""
        ep = self.prefill(embeds, token_ids)
        accept_lens = []
        it = 0
        while len(ep.emitted) < n_tokens:
            if tree_fn is not None:
                tree = tree_fn(ep, it)
            elif prune:
                k = min(shape.depth, n_tokens - len(ep.emitted) - 1)
                if k == 0:
                    tree = Tree([ep.root], [-1], [0], [0.0])
                else:
                    tree = self.draft_tree(ep, replace(shape, branch=tuple(shape.branch[:k]),
                                                       expand=tuple(shape.expand[:k])))
            else:
                tree = self.draft_tree(ep, shape)
            m, _ = self.verify_tree(ep, tree, r)
            accept_lens.append(m)
            it += 1
        return ep.emitted[:n_tokens], accept_lens

    # ------------------------------------------------------------------ Eq. 1
    def ar_generate(self, embeds, token_ids, n_tokens: int = 7, want_margins: bool = False, follow=None):
        """Plain greedy autoregressive decoding with the verification model alone.
        follow = (tokens, margin): see _follow; with it the returned list holds the oracle's own
        greedy token at every position, each conditioned on the tokens actually continued with."""
        d = self.desc
        cache = D.KVCache(d.n_layers, self.max_seq, d.n_heads, d.head_dim, self.dtype)
        x = D.embed_rows(self.w, embeds, token_ids)
        P = x.shape[0]
        pos = torch.arange(P)
        feats = D.target_forward(self.w, d, x, pos, pos, self._causal(0, P), cache)
        logits = D.lm_head(self.w, feats[P - 1:P])[0]
        toks = [self._greedy(logits)]
        margins = [D.top2_margin(logits, d, self.action_only)]
        while len(toks) < n_tokens:
            p = torch.tensor([P])
            last = toks[-1] if follow is None else self._follow(logits, toks[-1], follow[0][len(toks) - 1],
                                                                follow[1])
            feats = D.target_forward(self.w, d, self._embed([last]), p, p,
                                     self._causal(P, 1), cache)
            logits = D.lm_head(self.w, feats)[0]
            toks.append(self._greedy(logits))
            margins.append(D.top2_margin(logits, d, self.action_only))
            P += 1
        return (toks, margins) if want_margins else toks

    def detokenize(self, tokens):
        """Bin centre of each action token: 256 uniform bins over [-1, 1] (Section 4.3)."""
        a0, nb = self.desc.action_base, self.desc.n_bins
        return [(-1.0 + (2 * (t - a0) + 1) / nb) if a0 <= t < a0 + nb else float("nan")
                for t in tokens]
