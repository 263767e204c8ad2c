"""Seeded synthetic weights, prefixes and draft trees.

Everything returned here is plain data (torch tensors / python lists) that is handed,
bit for bit, to both implementations under test. Matrices are N(0, 0.02) rounded once to
bfloat16; RMSNorm gains are 1 (a N(0, 0.02) gain would wipe out the signal).
"""
from __future__ import annotations

import math

import torch

from . import configs as C
from . import rng


def make_weights(desc: C.ModelDesc, seed: int, device="cpu", with_draft: bool = True) -> dict:
    """Weights of the target decoder and of the one-layer draft head.

    Layout (all matrices [out_features, in_features], bfloat16):
      embed, lm_head                        [V, d]
      layers.{l}.wqkv  = [Wq; Wk; Wv]       [3d, d]
      layers.{l}.wo                         [d, d]
      layers.{l}.wgu   = [Wgate; Wup]       [2F, d]
      layers.{l}.wd                         [d, F]
      layers.{l}.norm1 / norm2, final_norm  [d] float32, ones
      draft.fc                              [d, 2d]   input = [feature ; embedding]
      draft.layer.*                         as a target layer
    """
    d, F, V = desc.d_model, desc.d_ffn, desc.vocab
    hd = desc.n_heads * desc.head_dim
    w = {}

    def mat(stream, rows, cols):
        return rng.normal_bf16(seed, stream, (rows, cols), 0.02, device)

    def layer(prefix, base):
        w[prefix + "wqkv"] = torch.cat([mat(base + 0, hd, d), mat(base + 1, hd, d),
                                        mat(base + 2, hd, d)], 0)
        w[prefix + "wo"] = mat(base + 3, d, hd)
        w[prefix + "wgu"] = torch.cat([mat(base + 4, F, d), mat(base + 5, F, d)], 0)
        w[prefix + "wd"] = mat(base + 6, d, F)
        w[prefix + "norm1"] = torch.ones(d, dtype=torch.float32, device=device)
        w[prefix + "norm2"] = torch.ones(d, dtype=torch.float32, device=device)

    w["embed"] = mat(C.STREAM_EMBED, V, d)
    w["lm_head"] = mat(C.STREAM_LM_HEAD, V, d)
    w["final_norm"] = torch.ones(d, dtype=torch.float32, device=device)
    for l in range(desc.n_layers):
        layer(f"layers.{l}.", C.STREAM_LAYER0 + 10 * l)
    if with_draft:
        w["draft.fc"] = mat(C.STREAM_DRAFT_FC, d, 2 * d)
        layer("draft.layer.", C.STREAM_DRAFT_LAYER)
    return w


def make_prefix(wl: C.Workload, episode: int = 0, device="cpu", prefix_seed=None):
    """Prefix of one episode: visual rows given as embeddings, then text-token ids.

    Returns (embeds [P, d] bf16, token_ids [P] int32); token_ids[i] = -1 where the row is
    given by embeds[i], otherwise the row is the embedding of that id (embeds[i] is zero).
    """
    d = wl.model.d_model
    seed = wl.seed if prefix_seed is None else prefix_seed
    lo, hi = wl.n_text
    if hi > lo:
        n_text = int(rng.integers(seed, C.STREAM_TEXT_LEN, episode + 1, lo, hi + 1)[episode])
    else:
        n_text = lo
    P = wl.n_visual + n_text
    embeds = torch.zeros(P, d, dtype=torch.bfloat16, device=device)
    embeds[:wl.n_visual] = rng.normal_bf16(seed, C.STREAM_VISUAL + episode, (wl.n_visual, d),
                                           wl.visual_scale, device)
    ids = torch.full((P,), -1, dtype=torch.int32, device=device)
    if n_text:
        ids[wl.n_visual:] = rng.integers(seed, C.STREAM_TEXT_IDS + episode, n_text, 0,
                                         wl.model.action_base, device).to(torch.int32)
    return embeds, ids


def random_tree(n_rows: int, desc: C.ModelDesc, seed: int, max_depth: int = 8,
                root_token=None, stream_offset: int = 0):
    """Random tree topology with n_rows rows (row 0 = root) and random action-token drafts.

    parent[i] is uniform in [0, i); a draw that would exceed max_depth walks up to the first
    ancestor shallow enough. Returns python lists (tokens, parent, depth).
    """
    par = rng.integers(seed, C.STREAM_TREE_PARENT + stream_offset, n_rows, 0, 1 << 30).tolist()
    tok = rng.integers(seed, C.STREAM_TREE_TOKEN + stream_offset, n_rows, desc.action_base,
                       desc.action_base + desc.n_bins).tolist()
    parent, depth = [-1], [0]
    for i in range(1, n_rows):
        p = par[i] % i
        while depth[p] + 1 > max_depth:
            p = parent[p]
        parent.append(p)
        depth.append(depth[p] + 1)
    if root_token is not None:
        tok[0] = int(root_token)
    return tok, parent, depth


def static_topology(shape: C.TreeShape):
    """Parent/depth arrays of the fixed-shape tree used for planted drafts: at each level
    the first expand[l] nodes of the previous level are expanded, in order."""
    parent, depth = [-1], [0]
    prev = [0]
    for l in range(shape.depth):
        cur = []
        for p in prev[:shape.expand[l]]:
            for _ in range(shape.branch[l]):
                cur.append(len(parent))
                parent.append(p)
                depth.append(l + 1)
        prev = cur
    return parent, depth


def planted_offsets(seed: int, call: int, n: int):
    """n integer bin offsets: 0 with probability 0.5, otherwise +-k with k geometric(p=0.4)
    clipped to [1, 32] and a fair sign."""
    u = rng.uniform(seed, C.STREAM_PLANT + 3 * call, n).tolist()
    v = rng.uniform(seed, C.STREAM_PLANT + 3 * call + 1, n).tolist()
    s = rng.uniform(seed, C.STREAM_PLANT + 3 * call + 2, n).tolist()
    out = []
    for a, b, c in zip(u, v, s):
        if a < 0.5:
            out.append(0)
            continue
        k = 1 + int(math.floor(math.log(1.0 - b) / math.log(0.6)))
        k = max(1, min(32, k))
        out.append(k if c < 0.5 else -k)
    return out


def plant_children(greedy_bin: int, n_children: int, desc: C.ModelDesc, offsets):
    """Tokens of n_children sibling drafts around the target's greedy bin: child j takes the
    next offset from the iterator `offsets` whose clipped bin is not already used."""
    used, toks = set(), []
    while len(toks) < n_children:
        b = max(0, min(desc.n_bins - 1, greedy_bin + next(offsets)))
        if b in used:
            continue
        used.add(b)
        toks.append(desc.action_base + b)
    return toks


def plant_tree(shape: C.TreeShape, root_token: int, desc: C.ModelDesc, greedy_fn, seed: int, call: int):
    """Planted draft tree on the fixed topology of `shape`: the children of every expanded node
    are the target's greedy action bin after that node plus seeded offsets.

    greedy_fn(tokens, parent, depth) must return the target's greedy token after every row of
    the partial tree it is given (it is called once per level, root-only tree first).
    Returns (tokens, parent, depth)."""
    parent, depth = static_topology(shape)
    offs = iter(planted_offsets(seed, call, 4096))
    tokens = [int(root_token)]
    level_start = 1
    for l in range(shape.depth):
        g = greedy_fn(tokens, parent[:len(tokens)], depth[:len(tokens)])
        n_level = shape.level_sizes[l]
        parents_in_order = []
        for i in range(level_start, level_start + n_level):
            if parent[i] not in parents_in_order:
                parents_in_order.append(parent[i])
        for p in parents_in_order:
            gb = min(max(g[p] - desc.action_base, 0), desc.n_bins - 1)
            tokens += plant_children(gb, shape.branch[l], desc, offs)
        level_start += n_level
    return tokens, parent, depth
