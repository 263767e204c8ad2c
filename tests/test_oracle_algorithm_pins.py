"""Pins of the oracle's decoding algorithm against what the paper and the mathematics fix."""
import itertools
import os

import pytest
import torch

from oracle import decoder as D
from oracle.specvla import SpecVLAOracle, Tree, accept_and_select, accepts
from synth_inputs import configs as C, data

A0, NB = 768, 256
GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


# ------------------------------------------------------------------ Eq. 4: the distance test
def test_accept_window_counts_and_symmetry():
    """For target bin b exactly min(b+r,255) - max(b-r,0) + 1 draft bins pass; r = 0 is
    strict equality (Section 5.2); the rule is symmetric and monotone in r."""
    for r in (0, 1, 2, 5, 9, 16, 255, 300):
        for b in range(NB):
            ok = [a for a in range(NB) if accepts(A0 + a, A0 + b, r, A0, NB)]
            assert len(ok) == min(b + r, NB - 1) - max(b - r, 0) + 1
            assert ok == list(range(max(b - r, 0), min(b + r, NB - 1) + 1))
            if r == 0:
                assert ok == [b]
    for a, b in itertools.product(range(0, NB, 7), range(0, NB, 5)):
        for r in (0, 3, 9):
            assert accepts(A0 + a, A0 + b, r, A0, NB) == accepts(A0 + b, A0 + a, r, A0, NB)
            assert (not accepts(A0 + a, A0 + b, r, A0, NB)) or accepts(A0 + a, A0 + b, r + 1, A0, NB)


def test_non_action_tokens_need_exact_match():
    for r in (0, 9, 255):
        assert accepts(5, 5, r, A0, NB)
        assert not accepts(5, 6, r, A0, NB)
        assert not accepts(A0 - 1, A0, r, A0, NB)       # text id next to bin 0
        assert not accepts(A0, A0 - 1, r, A0, NB)
        assert not accepts(A0 + NB, A0 + NB - 1, r, A0, NB)


def test_case_study_sequences_consistent_with_closed_interval():
    """Fig. 5 / Section 6.3: with r = 9 the relaxed run keeps drafts 119 and 121 where the
    strict run's target tokens are 128 and 128 (9 and 7 bins away): accepted under
    |delta| <= r; an open interval (|delta| < r) would reject the first of them."""
    rows = {}
    for line in open(os.path.join(GOLDEN, "fig5_case_study.txt")):
        if line.startswith("#") or ":" not in line:
            continue
        k, v = line.split(":")
        rows[k.strip()] = [int(t) for t in v.split(",")]
    strict, relaxed = rows["action1_strict"], rows["action1_relaxed"]
    assert len(strict) == len(relaxed) == 7
    assert relaxed[1:4] == rows["action1_relaxed_first_iteration"]
    assert relaxed[4:] == rows["action1_relaxed_second_iteration"]
    # position 1: the context is identical in both runs, so the target token is 128
    assert accepts(A0 + relaxed[1] - 1, A0 + strict[1] - 1, 9, A0, NB)
    assert not accepts(A0 + relaxed[1] - 1, A0 + strict[1] - 1, 8, A0, NB)
    assert abs(relaxed[1] - strict[1]) == 9


# ------------------------------------------------------------------ path selection: brute force
def _all_parent_arrays(n):
    """Every rooted tree on n labelled rows with parent[i] < i."""
    for ps in itertools.product(*[range(i) for i in range(1, n)]):
        yield [-1] + list(ps)


def _brute_force(tokens, parent, depth, g, r):
    """Walk every root-to-leaf path, count its accepted prefix; first maximum wins, where
    "first" is the lowest index of the last accepted node."""
    n = len(tokens)
    children = [[] for _ in range(n)]
    for i in range(1, n):
        children[parent[i]].append(i)
    leaves = [i for i in range(n) if not children[i]]
    best = (0, 0)                                 # (accepted length, last accepted node)
    for leaf in leaves:
        path = []
        j = leaf
        while j != -1:
            path.append(j)
            j = parent[j]
        path.reverse()
        m, last = 0, 0
        for a, b in zip(path[:-1], path[1:]):
            if not accepts(tokens[b], g[a], r, A0, NB):
                break
            m, last = m + 1, b
        if m > best[0] or (m == best[0] and last < best[1]):
            best = (m, last)
    return best


@pytest.mark.parametrize("n", [1, 2, 3, 4, 5, 6])
def test_path_selection_equals_brute_force_all_topologies(n):
    gen = torch.Generator().manual_seed(100 + n)
    for parent in _all_parent_arrays(n):
        depth = [0] * n
        for i in range(1, n):
            depth[i] = depth[parent[i]] + 1
        for trial in range(3):
            # narrow token range so that accepted / rejected / tied branches all occur
            tokens = (A0 + 100 + torch.randint(0, 6, (n,), generator=gen)).tolist()
            g = (A0 + 100 + torch.randint(0, 6, (n,), generator=gen)).tolist()
            for r in (0, 1, 2):
                m, path, emitted = accept_and_select(tokens, parent, depth, g, r, A0, NB)
                bm, blast = _brute_force(tokens, parent, depth, g, r)
                assert (m, path[-1]) == (bm, blast)
                assert len(path) == m + 1 and path[0] == 0
                assert emitted == [tokens[j] for j in path[1:]] + [g[path[-1]]]
                for a, b in zip(path[:-1], path[1:]):
                    assert parent[b] == a


def test_path_selection_random_larger_trees():
    for seed in range(40):
        tok, par, dep = data.random_tree(12, C.TINY, seed=seed, max_depth=5)
        gen = torch.Generator().manual_seed(seed)
        tok = (A0 + 50 + torch.randint(0, 8, (12,), generator=gen)).tolist()
        g = (A0 + 50 + torch.randint(0, 8, (12,), generator=gen)).tolist()
        for r in (0, 1, 3, 255):
            m, path, _ = accept_and_select(tok, par, dep, g, r, A0, NB)
            assert (m, path[-1]) == _brute_force(tok, par, dep, g, r)


def test_large_threshold_accepts_every_action_draft():
    """r >= 255 covers the whole bin range: the first deepest node is chosen."""
    for seed in range(10):
        tok, par, dep = data.random_tree(30, C.TINY, seed=seed, max_depth=6)
        g = data.random_tree(30, C.TINY, seed=seed + 77)[0]
        m, path, emitted = accept_and_select(tok, par, dep, g, 255, A0, NB)
        deepest = max(dep)
        assert m == deepest and path[-1] == dep.index(deepest)
        assert emitted[:-1] == [tok[j] for j in path[1:]] and emitted[-1] == g[path[-1]]


# ------------------------------------------------------------------ model-level pins (tiny model)
@pytest.fixture(scope="module")
def ar_tokens(c0):
    orc = c0["make"]()
    return orc.ar_generate(c0["embeds"], c0["ids"], 7)


def test_strict_acceptance_is_lossless_with_draft_model(c0, ar_tokens):
    """r = 0: the chunk equals plain greedy decoding (Section 3.2: SD is lossless)."""
    orc = c0["make"]()
    toks, lens = orc.generate_action(c0["embeds"], c0["ids"], c0["wl"].tree, r=0)
    assert toks == ar_tokens
    assert len(lens) >= 1 and all(0 <= m <= 3 for m in lens)


def _random_scored_tree(seed, n, max_depth=5):
    import random
    rnd = random.Random(seed)
    parent, depth, score = [-1], [0], [0.0]
    for i in range(1, n):
        p = rnd.choice([j for j in range(i) if depth[j] < max_depth])
        parent.append(p)
        depth.append(depth[p] + 1)
        # cumulative log-probability: the parent's plus something <= 0 (sometimes exactly 0: a tie)
        score.append(score[p] - (0.0 if rnd.random() < 0.1 else rnd.expovariate(1.0)))
    return parent, depth, score


@pytest.mark.parametrize("seed", range(12))
def test_rerank_keeps_the_best_nodes_and_their_ancestors(seed):
    """Dynamic tree (Section 4.1 / 5.1): the kept nodes are the `keep` best by cumulative
    log-probability, the set is closed under ancestors, order and structure are preserved."""
    from oracle.specvla import Tree, rerank_and_keep
    n = 6 + 5 * seed
    parent, depth, score = _random_scored_tree(seed, n)
    tokens = [1000 + i for i in range(n)]                  # the token identifies the old node
    for keep in (1, 3, n // 2, n - 2, n - 1, n + 5):
        t = rerank_and_keep(Tree(tokens, parent, depth, score), keep)
        kept = [tok - 1000 for tok in t.tokens]
        assert kept[0] == 0 and kept == sorted(kept) and len(kept) == 1 + min(keep, n - 1)
        dropped = [i for i in range(1, n) if i not in kept]
        if dropped:
            assert min(score[i] for i in kept[1:]) >= max(score[i] for i in dropped)
            # among equal scores the lower index wins
            edge = min(score[i] for i in kept[1:])
            assert all(i > max(k for k in kept if score[k] == edge) for i in dropped if score[i] == edge)
        for new, old in enumerate(kept):
            if old:
                assert parent[old] in kept and t.parent[new] == kept.index(parent[old]) < new
            assert t.depth[new] == depth[old] and t.score[new] == score[old]


def test_dynamic_tree_of_the_draft_model_is_lossless_and_consistent(c0, ar_tokens):
    """Top-4 expansion to depth 3, best 10 nodes kept: a valid tree whose scores are sums of the
    draft model's log-probabilities along each path, and r = 0 still gives the greedy chunk."""
    from synth_inputs.configs import TreeShape
    shape = TreeShape((4, 4, 4), (1, 4, 4), keep=10)
    full = TreeShape((4, 4, 4), (1, 4, 4))
    orc = c0["make"]()
    ep = orc.prefill(c0["embeds"], c0["ids"])
    import copy
    t_full = orc.draft_tree(copy.deepcopy(ep), full)
    t = orc.draft_tree(ep, shape)
    assert len(t_full.tokens) == 1 + 4 + 16 + 16 and len(t.tokens) == 11
    for i in range(1, 11):
        assert 0 <= t.parent[i] < i and t.depth[i] == t.depth[t.parent[i]] + 1
        assert t.score[i] <= t.score[t.parent[i]]
    # every kept node is a node of the full tree with the same path of tokens
    def path(tr, i):
        out = []
        while i > 0:
            out.append(tr.tokens[i])
            i = tr.parent[i]
        return tuple(reversed(out))
    full_paths = {path(t_full, i): t_full.score[i] for i in range(1, len(t_full.tokens))}
    for i in range(1, 11):
        assert abs(full_paths[path(t, i)] - t.score[i]) < 1e-12
    assert sorted(full_paths.values(), reverse=True)[9] == min(t.score[1:])
    toks, lens = c0["make"]().generate_action(c0["embeds"], c0["ids"], shape, r=0)
    assert toks == ar_tokens


def test_depth_pruning_is_lossless_and_never_drafts_past_the_chunk(c0, ar_tokens, monkeypatch):
    """prune: an iteration drafts at most (missing tokens - 1) levels, nothing when one token is
    missing, and at r = 0 the chunk is still the greedy one."""
    orc = c0["make"]()
    depths, missing = [], []
    real = orc.draft_tree

    def spy(ep, shape, want_debug=False):
        depths.append(shape.depth)
        missing.append(7 - len(ep.emitted))
        return real(ep, shape, want_debug)

    monkeypatch.setattr(orc, "draft_tree", spy)
    toks, lens = orc.generate_action(c0["embeds"], c0["ids"], c0["wl"].tree, r=0, prune=True)
    assert toks == ar_tokens
    assert depths and all(d == min(c0["wl"].tree.depth, k - 1) and d >= 1 for d, k in zip(depths, missing))
    assert all(m <= d for m, d in zip(lens, depths + [0]))
    # the last iteration of a chunk that ends one token short verifies the root alone
    assert sum(m + 1 for m in lens) + 1 >= 7 and len(lens) >= len(depths)


@pytest.mark.parametrize("action_only", [True, False])
def test_strict_acceptance_is_lossless_with_arbitrary_trees(c0, action_only):
    orc = c0["make"](action_only=action_only)
    ref = orc.ar_generate(c0["embeds"], c0["ids"], 7)

    def tree_fn(ep, it):
        tok, par, dep = data.random_tree(9 + it, c0["desc"], seed=40 + it, max_depth=4,
                                         root_token=ep.root, stream_offset=it)
        return Tree(tok, par, dep, [0.0] * len(tok))

    toks, _ = orc.generate_action(c0["embeds"], c0["ids"], None, r=0, tree_fn=tree_fn)
    assert toks == ref


def test_strict_acceptance_is_lossless_with_perfect_drafts(c0, ar_tokens):
    """A chain that plants the greedy continuation is accepted in full at r = 0 and the
    chunk still equals greedy decoding; the number of iterations drops accordingly."""
    orc = c0["make"]()

    def tree_fn(ep, it):
        done = len(ep.emitted)
        chain = ar_tokens[done:done + 3]
        tok = [ep.root] + chain
        return Tree(tok, list(range(-1, len(chain))), list(range(len(chain) + 1)), [0.0] * len(tok))

    toks, lens = orc.generate_action(c0["embeds"], c0["ids"], None, r=0, tree_fn=tree_fn)
    assert toks == ar_tokens
    assert lens == [3, 2]            # 1 + (3+1) + (2+1) = 8 emitted, clipped to 7


def test_one_node_tree_is_one_autoregressive_step(c0, ar_tokens):
    orc = c0["make"]()
    ep = orc.prefill(c0["embeds"], c0["ids"])
    assert ep.root == ar_tokens[0]
    for k in range(1, 4):
        P = ep.P
        m, emitted = orc.verify_tree(ep, Tree([ep.root], [-1], [0], [0.0]), r=4)
        assert m == 0 and emitted == [ar_tokens[k]] and ep.P == P + 1


def test_tree_rows_equal_sequential_decoding_of_each_path(c0):
    """Logits of tree row i == last-row logits of a causal forward over prefix + its path."""
    desc = c0["desc"]
    orc = c0["make"]()
    ep = orc.prefill(c0["embeds"], c0["ids"])
    tok, par, dep = data.random_tree(11, desc, seed=9, max_depth=4, root_token=ep.root)
    logits, _ = orc.verify_forward(ep, Tree(tok, par, dep, [0.0] * 11))
    x0 = D.embed_rows(orc.w, c0["embeds"], c0["ids"])
    for i in range(11):
        path = []
        j = i
        while j != -1:
            path.append(tok[j])
            j = par[j]
        path.reverse()
        x = torch.cat([x0, orc._embed(path)], 0)
        n = x.shape[0]
        cache = D.KVCache(desc.n_layers, n, desc.n_heads, desc.head_dim)
        f = D.target_forward(orc.w, desc, x, torch.arange(n), torch.arange(n),
                             orc._causal(0, n), cache)
        seq = D.lm_head(orc.w, f[-1:])[0]
        assert (seq - logits[i]).abs().max() < 1e-10


def test_cache_after_compaction_equals_fresh_prefill(c0):
    """After accept + compaction the committed target cache equals the cache obtained by
    prefilling prefix + emitted tokens from scratch, and decoding continues identically."""
    desc = c0["desc"]
    orc = c0["make"]()
    ep = orc.prefill(c0["embeds"], c0["ids"])
    for it in range(3):
        tok, par, dep = data.random_tree(14, desc, seed=60 + it, max_depth=4,
                                         root_token=ep.root)
        orc.verify_tree(ep, Tree(tok, par, dep, [0.0] * 14), r=200)   # accepts deep paths
    assert ep.P > 64 + 3                                              # something was accepted
    toks = ep.emitted[:-1]                                            # the root is not cached yet
    emb = torch.cat([c0["embeds"], torch.zeros(len(toks), desc.d_model, dtype=torch.bfloat16)])
    ids = torch.cat([c0["ids"], torch.tensor(toks, dtype=torch.int32)])
    fresh = orc.prefill(emb, ids)
    assert fresh.P == ep.P
    for l in range(desc.n_layers):
        assert (fresh.cache.k[l][:ep.P] - ep.cache.k[l][:ep.P]).abs().max() < 1e-10
        assert (fresh.cache.v[l][:ep.P] - ep.cache.v[l][:ep.P]).abs().max() < 1e-10
    assert fresh.root == ep.root


def test_draft_state_after_commit_equals_fresh_prefill(c0):
    """The draft model's cache and pending rows after an iteration equal those of a fresh
    prefill over prefix + emitted tokens (same tree comes out)."""
    desc, shape = c0["desc"], c0["wl"].tree
    orc = c0["make"]()
    ep = orc.prefill(c0["embeds"], c0["ids"])
    for it in range(2):
        tree = orc.draft_tree(ep, shape)
        orc.verify_tree(ep, tree, r=40)
    nxt = orc.draft_tree(ep, shape)
    toks = ep.emitted[:-1]
    emb = torch.cat([c0["embeds"], torch.zeros(len(toks), desc.d_model, dtype=torch.bfloat16)])
    ids = torch.cat([c0["ids"], torch.tensor(toks, dtype=torch.int32)])
    fresh = orc.prefill(emb, ids)
    assert fresh.root == ep.root
    ref = orc.draft_tree(fresh, shape)
    assert ref.tokens == nxt.tokens and ref.parent == nxt.parent
    assert max(abs(a - b) for a, b in zip(ref.score, nxt.score)) < 1e-9


@pytest.mark.parametrize("shape", [C.TREE_C0, C.TreeShape((3, 2, 2, 1), (1, 2, 3, 2)),
                                   C.TreeShape((4, 4, 4), (1, 3, 4), keep=0)])
def test_draft_tree_rows_equal_sequential_draft_decoding(c0, shape):
    """Eq. 2 on a tree is Eq. 2 on each path: the predicted feature of every expanded node (the
    draft output that scores its children) equals the last row of one ordinary causal draft
    forward over the prefix pairs (f_i, e_{i+1}), the pair (f_{P-1}, e(a_1)) and the node's own
    path of (predicted feature of the parent, embedding of the node's token) pairs at positions
    0, 1, 2, ... - which fixes the draft-level masks, cache slots and positions."""
    desc = c0["desc"]
    orc = c0["make"]()
    ep, _, feats = orc.prefill(c0["embeds"], c0["ids"], want_logits=True)
    x0 = D.embed_rows(orc.w, c0["embeds"], c0["ids"])
    P = x0.shape[0]
    tree, dbg = orc.draft_tree(ep, shape, want_debug=True)
    out_of = {node: out for node, _, _, out in dbg}
    assert len(out_of) == 1 + sum(shape.expand[1:]) and max(tree.depth[n] for n in out_of) == shape.depth - 1
    for node, out in out_of.items():
        path = []
        j = node
        while j != -1:
            path.append(j)
            j = tree.parent[j]
        path.reverse()                                          # root .. node
        feat_in = [feats[i] for i in range(P)] + [out_of[tree.parent[j]] for j in path[1:]]
        emb_in = [x0[i] for i in range(1, P)] + [orc._embed([tree.tokens[j]])[0] for j in path]
        n = len(feat_in)
        assert n == len(emb_in) == P + len(path) - 1
        cache = D.KVCache(1, n, desc.n_heads, desc.head_dim)
        seq = D.draft_forward(orc.w, desc, torch.stack(feat_in), torch.stack(emb_in), torch.arange(n),
                              torch.arange(n), orc._causal(0, n), cache)
        assert (seq[-1] - out).abs().max() < 1e-10, (node, float((seq[-1] - out).abs().max()))


def test_draft_forward_matches_one_layer_hf_llama(c0):
    """Eq. 2 / Eq. 5 composition: fc over [feature ; embedding] followed by one decoder layer, the
    layer's output taken BEFORE any final norm. Library pin: a one-layer HuggingFace Llama fed
    inputs_embeds = feature @ Wfc[:, :d]^T + embedding @ Wfc[:, d:]^T, output read by a forward
    hook on its decoder layer."""
    from transformers import LlamaConfig, LlamaForCausalLM
    desc, w = c0["desc"], c0["weights"]
    d, hd, F = desc.d_model, desc.n_heads * desc.head_dim, desc.d_ffn
    cfg = LlamaConfig(vocab_size=desc.vocab, hidden_size=d, intermediate_size=F, num_hidden_layers=1,
                      num_attention_heads=desc.n_heads, num_key_value_heads=desc.n_heads,
                      head_dim=desc.head_dim, rms_norm_eps=desc.rms_eps, rope_theta=desc.rope_theta,
                      max_position_embeddings=1024, attention_bias=False, mlp_bias=False,
                      tie_word_embeddings=False)
    cfg._attn_implementation = "eager"
    m = LlamaForCausalLM(cfg).double().eval()
    q = "draft.layer."
    sd = {"model.layers.0.self_attn.q_proj.weight": w[q + "wqkv"][:hd],
          "model.layers.0.self_attn.k_proj.weight": w[q + "wqkv"][hd:2 * hd],
          "model.layers.0.self_attn.v_proj.weight": w[q + "wqkv"][2 * hd:],
          "model.layers.0.self_attn.o_proj.weight": w[q + "wo"],
          "model.layers.0.mlp.gate_proj.weight": w[q + "wgu"][:F],
          "model.layers.0.mlp.up_proj.weight": w[q + "wgu"][F:],
          "model.layers.0.mlp.down_proj.weight": w[q + "wd"],
          "model.layers.0.input_layernorm.weight": w[q + "norm1"],
          "model.layers.0.post_attention_layernorm.weight": w[q + "norm2"]}
    m.load_state_dict({k: v.double() for k, v in sd.items()}, strict=False)
    grabbed = []
    m.model.layers[0].register_forward_hook(
        lambda mod, args, out: grabbed.append(out[0] if isinstance(out, tuple) else out))
    orc = c0["make"]()
    n = 23
    g = torch.Generator().manual_seed(3)
    feat = torch.randn(n, d, generator=g, dtype=torch.float64)
    emb = torch.randn(n, d, generator=g, dtype=torch.float64)
    # a tree-ish mask and per-row positions, as the draft levels use them
    vis = orc._causal(0, n).clone()
    vis[15:, 10:15] = False
    pos = torch.cat([torch.arange(15), torch.tensor([15, 15, 16, 16, 16, 17, 17, 18])])
    cache = D.KVCache(1, n, desc.n_heads, desc.head_dim)
    mine = D.draft_forward(orc.w, desc, feat, emb, pos, torch.arange(n), vis, cache)
    Wfc = w["draft.fc"].double()
    z = feat @ Wfc[:, :d].T + emb @ Wfc[:, d:].T
    mask = torch.zeros(n, n, dtype=torch.float64)
    mask[~vis] = torch.finfo(torch.float64).min
    with torch.no_grad():
        m(inputs_embeds=z[None], attention_mask=mask[None, None], position_ids=pos[None])
    ref = grabbed[0].reshape(n, d)
    assert torch.allclose(mine, ref, atol=5e-6, rtol=0), float((mine - ref).abs().max())
    # [feature ; embedding] order: swapping the halves must be visible
    swapped = D.draft_forward(orc.w, desc, emb, feat, pos, torch.arange(n), vis,
                              D.KVCache(1, n, desc.n_heads, desc.head_dim))
    assert (swapped - ref).abs().max() > 1e-2


def test_draft_tree_invariants(c0):
    shape = c0["wl"].tree
    for action_only in (True, False):
        orc = c0["make"](action_only=action_only)
        ep = orc.prefill(c0["embeds"], c0["ids"])
        tree, dbg = orc.draft_tree(ep, shape, want_debug=True)
        n = len(tree.tokens)
        assert n == 1 + shape.n_nodes and tree.parent[0] == -1 and tree.tokens[0] == ep.root
        sizes = [tree.depth.count(l + 1) for l in range(shape.depth)]
        assert tuple(sizes) == shape.level_sizes
        for i in range(1, n):
            p = tree.parent[i]
            assert p < i and tree.depth[i] == tree.depth[p] + 1
            assert tree.score[i] <= tree.score[p] + 1e-12          # log-probs are <= 0
            if action_only:
                assert A0 <= tree.tokens[i] < A0 + NB
        for node, lp, base, _ in dbg:
            kids = [i for i in range(n) if tree.parent[i] == node]
            assert abs(float(torch.exp(lp).sum()) - 1.0) < 1e-9
            top = torch.topk(lp, len(kids))
            assert [tree.tokens[i] - base for i in kids] == top.indices.tolist()
            for i, v in zip(kids, top.values.tolist()):
                assert abs(tree.score[i] - tree.score[node] - v) < 1e-12
        # the expanded parents of each level are the best-scored nodes of that level
        for l in range(1, shape.depth):
            level = [i for i in range(n) if tree.depth[i] == l]
            expanded = sorted({tree.parent[i] for i in range(n) if tree.depth[i] == l + 1})
            want = sorted(sorted(level, key=lambda i: (-tree.score[i], i))[:shape.expand[l]])
            assert expanded == want


def test_relaxed_run_keeps_draft_tokens_and_large_r_takes_whole_path(c0):
    """r >= 255 with action-only decoding: every iteration accepts a full-depth path and the
    emitted tokens are the DRAFT tokens on it plus the target's token after its leaf."""
    orc = c0["make"]()
    ep = orc.prefill(c0["embeds"], c0["ids"])
    tree = orc.draft_tree(ep, c0["wl"].tree)
    m, emitted, dbg = orc.verify_tree(ep, tree, r=255, want_debug=True)
    assert m == 3
    first_leaf = tree.depth.index(3)
    assert dbg["path"][-1] == first_leaf
    assert emitted[:3] == [tree.tokens[j] for j in dbg["path"][1:]]
    assert emitted[3] == dbg["g"][first_leaf]


def test_detokenize_bin_centres(c0):
    orc = c0["make"]()
    v = orc.detokenize([A0, A0 + 255, A0 + 128])
    assert v == [-1 + 1 / 256, 1 - 1 / 256, 1 / 256]
