"""CUDA path vs the CPU oracle on the OpenVLA-7B-shaped workloads C1-C4 (full sizes).

The oracle runs live on the host cores (float64); the weights are generated once on the GPU
and the same bits are copied to the host for it. Logits must agree within 2e-2 max-abs;
greedy tokens, accepted lengths and emitted tokens bit-exactly wherever the oracle's top-2
margin exceeds 5e-2 (positions below that are printed)."""
import pytest
import torch

from oracle.specvla import SpecVLAOracle, Tree, accept_and_select
from synth_inputs import configs as C, data

import gpu_helpers as G

pytestmark = pytest.mark.gpu
DESC = C.OPENVLA_7B


@pytest.fixture(scope="module")
def env():
    from paper_2507_22424_b200.binding import make_shape
    torch.set_grad_enabled(False)
    wc = data.make_weights(DESC, C.C1.seed, device="cuda")
    wh = {k: v.cpu() for k, v in wc.items()}
    orc = SpecVLAOracle(DESC, wh, action_only=True, max_seq=448, max_tree_rows=128)
    gpu = G.make_gpu(DESC, wc, max_seq=512, max_episodes=16, max_rows=16 * 320, action_only=True)
    emb, ids = data.make_prefix(C.C1, device="cuda")
    yield dict(orc=orc, gpu=gpu, emb=emb, ids=ids, shape=make_shape(C.TREE_26.branch, C.TREE_26.expand))
    gpu.close()


def _prefill_both(env, emb, ids, episode=0):
    ep, ref_logits, _ = env["orc"].prefill(emb.cpu(), ids.cpu(), want_logits=True)
    first, logits = env["gpu"].prefill([episode], emb, ids.tolist(), [len(ids)], want_logits=True)
    return ep, ref_logits, first[0], logits[0]


def _check_verify(env, ep, tree, r, episode=0, log=None, dbg_ref=None):
    """Verifies `tree` on both sides; returns True when the states stay comparable."""
    log = [] if log is None else log
    if dbg_ref is None:
        m_ref, emitted_ref, dbg = env["orc"].verify_tree(ep, tree, r, want_debug=True)
    else:
        m_ref, emitted_ref, dbg = dbg_ref
    n = len(tree.tokens)
    m, emitted, logits = env["gpu"].verify_tree([episode], [G.tree_dict(tree)], r, want_logits=True)
    err = float((logits.cpu().double() - dbg["logits"][:n]).abs().max())
    assert err < G.LOGIT_TOL, err
    g_gpu = env["gpu"].read_buffer(1, n, torch.int32).tolist()
    G.compare_tokens(g_gpu, dbg["g"][:n], G.margins(dbg["logits"][:n], DESC, True).tolist(), log, "g")
    if g_gpu != dbg["g"][:n]:
        return False, err
    assert (m[0], emitted[0]) == (m_ref, emitted_ref)
    return True, err


def test_c1_prefill_draft_verify_lockstep(env):
    orc, gpu = env["orc"], env["gpu"]
    ep, ref_logits, first, logits = _prefill_both(env, env["emb"], env["ids"])
    err = float((logits.cpu().double() - ref_logits).abs().max())
    print("C1 prefill logits max-abs err", err)
    assert err < G.LOGIT_TOL
    from oracle import decoder as D
    log = []
    G.compare_tokens([first], [ep.root], [D.top2_margin(ref_logits, DESC, True)], log, "a1")
    if first != ep.root:
        pytest.skip("first token at a low margin")
    for it in range(6):
        ref_tree, dbg = orc.draft_tree(ep, C.TREE_26, want_debug=True)
        got = gpu.draft_tree([0], env["shape"])[0]
        assert len(got["tokens"]) == 27 and got["tokens"][0] == ep.root
        if got["tokens"] == ref_tree.tokens:
            assert got["parent"] == ref_tree.parent and got["depth"] == ref_tree.depth
            assert max(abs(a - b) for a, b in zip(got["score"], ref_tree.score)) < 5e-2
        else:
            gap = min(float(torch.sort(lp, descending=True).values[:5].diff().abs().min()) for _, lp, _ in dbg)
            log.append(f"it{it}: draft tree differs; smallest ranking gap {gap:.4f}")
            assert gap < G.MARGIN
        ok, err = _check_verify(env, ep, ref_tree, 0, log=log)
        print(f"it{it}: verify logits err {err:.4f}")
        if not ok or len(ep.emitted) >= 7:
            break
    print("\n".join(log))


def test_c1_generate_action_strict_equals_greedy(env):
    orc, gpu = env["orc"], env["gpu"]
    from paper_2507_22424_b200.binding import make_shape
    ref, mg = orc.ar_generate(env["emb"].cpu(), env["ids"].cpu(), 7, want_margins=True)
    toks, acts, stats = gpu.generate_action([0], env["emb"], env["ids"].tolist(), [len(env["ids"])],
                                            env["shape"], 0, 7)
    ar, _, _ = gpu.generate_action([0], env["emb"], env["ids"].tolist(), [len(env["ids"])],
                                   make_shape((), ()), 0, 7)
    assert toks == ar
    pruned, _, st3 = gpu.generate_action([0], env["emb"], env["ids"].tolist(), [len(env["ids"])],
                                         make_shape(C.TREE_26.branch, C.TREE_26.expand, prune=True), 0, 7)
    assert pruned == toks and st3.ms_draft < stats.ms_draft
    # the paper's own tree (Section 5.1 / Table 4): top-8, depth 5, the best 50 of 264 drafted nodes
    dyn, _, st4 = gpu.generate_action([0], env["emb"], env["ids"].tolist(), [len(env["ids"])],
                                      make_shape((8,) * 5, (1, 8, 8, 8, 8), keep=50), 0, 7)
    assert dyn == toks
    for i in range(7):
        if mg[i] <= G.MARGIN:
            print(f"position {i}: margin {mg[i]:.4f}; comparison stops here")
            break
        assert toks[0][i] == ref[i]
    print("chunk", toks[0], "oracle", ref, "margins", [round(x, 3) for x in mg])


def test_c3_verify_sweep_tree_sizes(env):
    """Rows {1, 8, 26, 27, 60, 128}: every size is a prefix of the same 128-row random tree, and a
    row's logits depend only on its ancestors, so one oracle pass over 128 rows gives the
    expected logits of all of them."""
    orc, gpu = env["orc"], env["gpu"]
    emb, ids = data.make_prefix(C.C3, device="cuda")
    assert 290 <= len(ids) <= 297
    ep = orc.prefill(emb.cpu(), ids.cpu())
    tok, par, dep = data.random_tree(128, DESC, seed=C.C3.extra["tree_seed"], max_depth=8, root_token=ep.root)
    logits, _ = orc.verify_forward(ep, Tree(tok, par, dep, [0.0] * 128))
    g = [orc._greedy(logits[i]) for i in range(128)]
    r = 16
    for n in C.C3.extra["rows"] + (27,):
        first = gpu.prefill([0], emb, ids.tolist(), [len(ids)])
        if first[0] != ep.root:
            pytest.skip("first token at a low margin")
        sub = Tree(tok[:n], par[:n], dep[:n], [0.0] * n)
        m_ref, path, emitted_ref = accept_and_select(sub.tokens, sub.parent, sub.depth, g[:n], r,
                                                     DESC.action_base, DESC.n_bins)
        log = []
        ok, err = _check_verify(env, None, sub, r, log=log,
                                dbg_ref=(m_ref, emitted_ref, dict(logits=logits, g=g)))
        print(f"T={n}: logits err {err:.4f}, m={m_ref}, comparable={ok}; " + "; ".join(log))


def _oracle_planted(orc, ep, seed, call):
    def greedy_fn(tokens, parent, depth):
        lg, _ = orc.verify_forward(ep, Tree(tokens, parent, depth, [0.0] * len(tokens)))
        return [orc._greedy(lg[i]) for i in range(len(tokens))]
    tok, par, dep = data.plant_tree(C.TREE_26, ep.root, DESC, greedy_fn, seed, call)
    return Tree(tok, par, dep, [0.0] * len(tok))


def test_c2_planted_drafts_threshold_sweep(env):
    """Three oracle-planted trees of the first iteration, each verified at every threshold."""
    orc, gpu = env["orc"], env["gpu"]
    ep = orc.prefill(env["emb"].cpu(), env["ids"].cpu())
    for call in (0, 1, 2):
        tree = _oracle_planted(orc, ep, C.C2.seed, call)
        logits, _ = orc.verify_forward(ep, tree)
        g = [orc._greedy(logits[i]) for i in range(27)]
        ms = []
        for r in C.C2.extra["r"]:
            first = gpu.prefill([0], env["emb"], env["ids"].tolist(), [len(env["ids"])])
            if first[0] != ep.root:
                pytest.skip("first token at a low margin")
            m_ref, path, emitted_ref = accept_and_select(tree.tokens, tree.parent, tree.depth, g, r,
                                                         DESC.action_base, DESC.n_bins)
            ok, err = _check_verify(env, None, tree, r, dbg_ref=(m_ref, emitted_ref, dict(logits=logits, g=g)))
            ms.append((r, m_ref, ok))
        print(f"C2 planted tree {call}, (r, accepted length, comparable):", ms)
        assert [m for _, m, _ in ms] == sorted(m for _, m, _ in ms)  # accepted length grows with r


def test_c2_planted_chunk_lockstep_r4(env):
    """A whole chunk with oracle-planted trees at r = 4, iteration by iteration."""
    orc, gpu = env["orc"], env["gpu"]
    ep, _, first, _ = _prefill_both(env, env["emb"], env["ids"])
    if first != ep.root:
        pytest.skip("first token at a low margin")
    log, lens = [], []
    for it in range(6):
        tree = _oracle_planted(orc, ep, C.C2.seed, 10 + it)
        gpu.draft_tree([0], env["shape"], want_trees=False)       # keeps the draft state in step
        n_before = len(ep.emitted)
        ok, err = _check_verify(env, ep, tree, 4, log=log)
        lens.append(len(ep.emitted) - n_before - 1)
        if not ok or len(ep.emitted) >= 7:
            break
    print("accepted lengths", lens, "emitted", ep.emitted[:7], "\n".join(log))


def test_c4_sixteen_ragged_episodes(env):
    """16 episodes prefilled and verified in one call each; episodes 0 and 15 are checked
    against the oracle (planted trees, r = 4), the others carry random trees."""
    orc, gpu = env["orc"], env["gpu"]
    n_ep, r = C.C4.extra["episodes"], C.C4.extra["r"]
    pre = [data.make_prefix(C.C4, episode=e, device="cuda", prefix_seed=C.C4.extra["prefix_seed"])
           for e in range(n_ep)]
    lens = [len(i) for _, i in pre]
    assert min(lens) >= 276 and max(lens) <= 316 and len(set(lens)) > 4
    emb = torch.cat([e for e, _ in pre])
    ids = torch.cat([i for _, i in pre]).tolist()
    first, logits = gpu.prefill(list(range(n_ep)), emb, ids, lens, want_logits=True)
    trees, refs = [], {}
    for e in range(n_ep):
        if e in (0, 15):
            ep, ref_logits, _ = orc.prefill(pre[e][0].cpu(), pre[e][1].cpu(), want_logits=True)
            assert float((logits[e].cpu().double() - ref_logits).abs().max()) < G.LOGIT_TOL
            t = _oracle_planted(orc, ep, C.C4.extra["prefix_seed"], 100 + e)
            refs[e] = (ep, t, orc.verify_tree(ep, t, r, want_debug=True))
            trees.append(G.tree_dict(t))
        else:
            tok, par, dep = data.random_tree(27, DESC, seed=50 + e, max_depth=5, root_token=first[e])
            trees.append(dict(tokens=tok, parent=par, depth=dep))
    if any(first[e] != refs[e][0].emitted[0] for e in refs):
        pytest.skip("first token at a low margin")
    m, emitted, vlogits = gpu.verify_tree(list(range(n_ep)), trees, r, want_logits=True)
    g_all = gpu.read_buffer(1, 27 * n_ep, torch.int32).tolist()
    for e, (ep, t, (m_ref, emitted_ref, dbg)) in refs.items():
        rows = slice(27 * e, 27 * e + 27)
        err = float((vlogits[rows].cpu().double() - dbg["logits"]).abs().max())
        assert err < G.LOGIT_TOL, err
        log = []
        G.compare_tokens(g_all[rows], dbg["g"], G.margins(dbg["logits"], DESC, True).tolist(), log, f"ep{e}.g")
        if g_all[rows] == dbg["g"]:
            assert (m[e], emitted[e]) == (m_ref, emitted_ref)
        print(f"episode {e}: P={lens[e]}, logits err {err:.4f}, m={m_ref}; " + "; ".join(log))
    st = gpu.read_buffer(5, 4 * n_ep, torch.int32).reshape(n_ep, 4).tolist()
    for e in range(n_ep):
        assert st[e][0] == lens[e] + 1 + m[e] and st[e][3] == m[e] + 1


@pytest.mark.parametrize("T,N,K", [(27, 22016, 4096), (27, 4096, 11008), (128, 12288, 4096),
                                   (27, 32064, 4096), (290, 4096, 4096)])
def test_gemm_full_size_sampled_outputs(T, N, K):
    """7B-shaped GEMMs: 256 sampled outputs recomputed one by one in float64."""
    from paper_2507_22424_b200.binding import gemm
    from synth_inputs import rng
    x = rng.normal(21, 1, (T, K), 1.0, "cuda", dtype=torch.float32)
    w = rng.normal_bf16(21, 2, (N, K), 0.02, "cuda")
    y = gemm(x, w).cpu()
    ts = rng.integers(21, 3, 256, 0, T).tolist()
    ns = rng.integers(21, 4, 256, 0, N).tolist()
    ns[:4] = [0, N - 1, N - 64, 127]
    xc, wc = x.cpu().double(), w.cpu()
    for t, n in zip(ts, ns):
        ref = float(xc[t] @ wc[n].double())
        assert abs(float(y[t, n]) - ref) < 1e-4 * 0.02 * (K ** 0.5) + 1e-6
