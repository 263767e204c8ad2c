"""Shared helpers of the GPU parity tests (CUDA path through the C ABI vs the CPU oracle).

Policy of every comparison: logits within LOGIT_TOL; greedy tokens bit-exact wherever the oracle's
top-2 margin exceeds MARGIN, every position at or below it logged. Nothing is skipped after a
low-margin difference: the oracle continues with the GPU's token at exactly those positions
(SpecVLAOracle's `follow`), so accepted length, emitted tokens, path, cache and state are compared
on every call, and a Tally records how many comparisons of each kind were made."""
import torch

from oracle import decoder as D
from oracle.specvla import SpecVLAOracle, Tree
from synth_inputs import configs as C, data

MARGIN = 5e-2        # tokens must agree wherever the oracle's top-2 margin exceeds this
LOGIT_TOL = 2e-2     # max-abs logit difference, bf16 path vs float64 oracle
KV_TOL = 2e-3        # committed cache entries (fp32 on the GPU) vs the float64 oracle


class Tally:
    """What a parity test compared: rows whose token had to match, rows logged at a low margin,
    (m, emitted, path) comparisons, cache comparisons, iterations reached."""

    def __init__(self):
        self.rows_exact = self.rows_low = self.accepts = self.caches = self.iterations = 0
        self.max_logit_err = 0.0
        self.log = []

    def report(self, name):
        print(f"[{name}] rows compared bit-exactly {self.rows_exact}, low-margin rows logged {self.rows_low}, "
              f"(m, tokens, path) comparisons {self.accepts}, cache comparisons {self.caches}, "
              f"iterations {self.iterations}, max logit err {self.max_logit_err:.2e}")
        for line in self.log:
            print("   ", line)


def to_cuda(weights):
    return {k: v.cuda().contiguous() for k, v in weights.items()}


def make_gpu(desc, weights_cuda, **kw):
    from paper_2507_22424_b200.binding import SpecVLA
    return SpecVLA(desc, weights_cuda, **kw)


def tree_dict(t: Tree):
    return dict(tokens=list(t.tokens), parent=list(t.parent), depth=list(t.depth))


def margins(logits, desc, action_only):
    """Top-1 minus top-2 per row of an oracle logits matrix."""
    if action_only:
        logits = logits[:, desc.action_base:desc.action_base + desc.n_bins]
    top = torch.topk(logits, 2, dim=1).values
    return (top[:, 0] - top[:, 1])


def compare_tokens(gpu_tokens, oracle_tokens, margin_list, tally, where):
    """Bit-exact wherever the margin is large; every low-margin position is logged."""
    assert len(gpu_tokens) == len(oracle_tokens) == len(margin_list)
    for i, (a, b, mg) in enumerate(zip(gpu_tokens, oracle_tokens, margin_list)):
        if mg <= MARGIN:
            tally.rows_low += 1
            tally.log.append(f"{where}[{i}]: margin {mg:.4f} <= {MARGIN} (gpu {a}, oracle {b})")
        else:
            assert a == b, f"{where}[{i}]: gpu {a} != oracle {b} at margin {mg:.4f}"
            tally.rows_exact += 1


def prefill_both(orc, gpu, emb_cuda, ids, episode, tally, desc, action_only=True, where="a1"):
    """Prefill on both sides; logits and first token compared; the oracle's episode follows the
    GPU's first token if (and only if) that position is a logged low-margin one."""
    first, logits = gpu.prefill([episode], emb_cuda, ids.tolist(), [len(ids)], want_logits=True)
    ep, ref_logits, feats = orc.prefill(emb_cuda.cpu(), ids.cpu(), want_logits=True, follow=(first[0], MARGIN))
    err = float((logits[0].cpu().double() - ref_logits).abs().max())
    tally.max_logit_err = max(tally.max_logit_err, err)
    assert err < LOGIT_TOL, err
    own = D.greedy_token(ref_logits, desc, action_only)
    compare_tokens(first, [own], [D.top2_margin(ref_logits, desc, action_only)], tally, where)
    assert first[0] == ep.root
    return ep, ref_logits, feats


def check_verify_outputs(gpu, tally, desc, g_gpu_rows, m, emitted, ref, ep_after, P_before, index=0,
                         episode=0, kv=True, n_ep=1):
    """(m, emitted, path) of call slot `index`, then cache and state of `episode`, against the oracle's
    result `ref` = (m_ref, emitted_ref, dbg) obtained with `follow`."""
    m_ref, emitted_ref, dbg = ref
    assert g_gpu_rows == dbg["g"]            # holds by construction of `follow` once tokens compared
    assert (m[index], emitted[index]) == (m_ref, emitted_ref), (m[index], emitted[index], m_ref, emitted_ref)
    path = gpu.read_buffer(4, 9 * n_ep, torch.int32).tolist()[9 * index:9 * index + m_ref + 1]
    assert path == dbg["path"], (path, dbg["path"])
    tally.accepts += 1
    st = gpu.read_buffer(5, 4 * (episode + 1), torch.int32).tolist()[4 * episode:4 * episode + 4]
    assert (st[0], st[2], st[3]) == (ep_after.P, ep_after.root, m_ref + 1), (st, ep_after.P, ep_after.root)
    assert P_before + 1 + m_ref == ep_after.P
    if kv:
        worst = 0.0
        for l in range(desc.n_layers):
            for which, refc in ((0, ep_after.cache.k[l]), (1, ep_after.cache.v[l])):
                got = gpu.read_kv(episode, l, which, 0, ep_after.P).double()
                want = refc[:ep_after.P].reshape(ep_after.P, -1)
                worst = max(worst, float((got - want).abs().max()))
        assert worst < KV_TOL, worst
        tally.caches += 1


def verify_both(orc, gpu, ep, tree, r, tally, desc, action_only=True, episode=0, kv=True, where="g"):
    """One verification of `tree` for one episode on both sides, everything compared."""
    n = len(tree.tokens)
    P = ep.P
    m, emitted, logits = gpu.verify_tree([episode], [tree_dict(tree)], r, want_logits=True)
    g_gpu = gpu.read_buffer(1, n, torch.int32).tolist()
    ref = orc.verify_tree(ep, tree, r, want_debug=True, follow=(g_gpu, MARGIN))
    dbg = ref[2]
    err = float((logits.cpu().double() - dbg["logits"]).abs().max())
    tally.max_logit_err = max(tally.max_logit_err, err)
    assert err < LOGIT_TOL, err
    compare_tokens(g_gpu, dbg["g_own"], margins(dbg["logits"], desc, action_only).tolist(), tally, where)
    check_verify_outputs(gpu, tally, desc, g_gpu, m, emitted, ref, ep, P, episode=episode, kv=kv,
                         n_ep=1)
    tally.iterations += 1
    return ref


def compare_draft_trees(got, ref, dbg, shape, tally):
    """GPU draft tree `got` (dict) against the oracle's `ref` (Tree) with the oracle's per-parent
    log-probabilities `dbg` = [(node, lp over the ranked ids, id of column 0)] in expansion order.
    Nodes are compared in creation order. The first node that differs must be explained by a
    ranking decision of the oracle taken at a gap below MARGIN: a sibling order (same parent, the
    two tokens' log-probabilities closer than MARGIN) or an expansion choice (different parent, the
    two candidate parents' scores closer than MARGIN). Later nodes are checked for structure only.
    Returns the number of leading nodes that are identical."""
    n = len(ref.tokens)
    assert len(got["tokens"]) == n and got["parent"][0] == -1 and got["tokens"][0] == ref.tokens[0]
    for i in range(1, n):
        assert 0 <= got["parent"][i] < i and got["depth"][i] == got["depth"][got["parent"][i]] + 1
    lp_of = {node: (lp, base) for node, lp, base, _ in dbg}
    same = 1
    for i in range(1, n):
        if got["parent"][i] == ref.parent[i] and got["tokens"][i] == ref.tokens[i]:
            assert abs(got["score"][i] - ref.score[i]) < 5e-2, (i, got["score"][i], ref.score[i])
            same += 1
            continue
        if got["parent"][i] == ref.parent[i]:
            lp, base = lp_of[ref.parent[i]]
            gap = float(lp[ref.tokens[i] - base] - lp[got["tokens"][i] - base])
            what = f"sibling order under node {ref.parent[i]}"
        else:
            gap = abs(ref.score[ref.parent[i]] - ref.score[got["parent"][i]])
            what = f"expansion choice between nodes {ref.parent[i]} and {got['parent'][i]}"
        assert 0 <= gap < MARGIN, (i, what, gap)
        tally.log.append(f"draft tree: node {i} differs ({what}, oracle gap {gap:.4f}); {same} of {n} nodes identical")
        break
    return same
