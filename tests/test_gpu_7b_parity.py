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


KV_LAYERS = (0, 13, 31)      # layers whose committed cache is read back and compared


def _check_state_and_cache(gpu, tally, cache, P_before, m_ref, path, root, episode):
    """State of `episode` after a commit and its cache slots [0, P + 1 + m): prefix rows as they
    were, then the rows of `path` (oracle cache still holds the tree rows at slots P + row)."""
    st = gpu.read_buffer(5, 4 * (episode + 1), torch.int32).tolist()[4 * episode:4 * episode + 4]
    assert (st[0], st[2], st[3]) == (P_before + 1 + m_ref, root, m_ref + 1), st
    src = list(range(P_before)) + [P_before + j for j in path]
    worst = 0.0
    for l in KV_LAYERS:
        for which, refc in ((0, cache.k[l]), (1, cache.v[l])):
            got = gpu.read_kv(episode, l, which, 0, len(src)).double()
            want = refc[src].reshape(len(src), -1)
            worst = max(worst, float((got - want).abs().max()))
    assert worst < G.KV_TOL, worst
    tally.caches += 1


def _verify_against_logits(env, tree, r, logits, cache, P, tally, where, episode=0, index=0, n_ep=1,
                           call=None):
    """Verification of `tree` on the GPU against oracle logits of (a superset of) its rows computed
    beforehand: logits, greedy tokens, then acceptance, path and tokens through the oracle's
    accept_and_select on the greedy vector with the GPU's token at logged low-margin rows."""
    gpu = env["gpu"]
    n = len(tree.tokens)
    if call is None:
        m, emitted, glog = gpu.verify_tree([episode], [G.tree_dict(tree)], r, want_logits=True)
        g_gpu = gpu.read_buffer(1, n, torch.int32).tolist()
    else:
        m, emitted, glog, g_gpu = call
    err = float((glog.cpu().double() - logits[:n]).abs().max())
    tally.max_logit_err = max(tally.max_logit_err, err)
    assert err < G.LOGIT_TOL, err
    mg = G.margins(logits[:n], DESC, True).tolist()
    g_own = [env["orc"]._greedy(logits[i]) for i in range(n)]
    G.compare_tokens(g_gpu, g_own, mg, tally, where)
    g = [g_gpu[i] if mg[i] <= G.MARGIN else g_own[i] for i in range(n)]
    m_ref, path, emitted_ref = accept_and_select(tree.tokens, tree.parent, tree.depth, g, r,
                                                 DESC.action_base, DESC.n_bins)
    assert (m[index], emitted[index]) == (m_ref, emitted_ref), (m[index], emitted[index], m_ref, emitted_ref)
    got_path = gpu.read_buffer(4, 9 * n_ep, torch.int32).tolist()[9 * index:9 * index + m_ref + 1]
    assert got_path == path
    tally.accepts += 1
    tally.iterations += 1
    _check_state_and_cache(gpu, tally, cache, P, m_ref, path, emitted_ref[-1], episode)
    return m_ref, err


def test_c1_prefill_draft_verify_lockstep(env):
    """C1 iteration by iteration until the chunk is complete: draft tree against the oracle's, then
    the oracle's tree verified on both sides with everything compared (all 32 layers of the cache)."""
    orc, gpu = env["orc"], env["gpu"]
    tally = G.Tally()
    ep, _, _ = G.prefill_both(orc, gpu, env["emb"], env["ids"], 0, tally, DESC)
    print("C1 prefill logits max-abs err", tally.max_logit_err)
    same = []
    while len(ep.emitted) < 7:
        ref_tree, dbg = orc.draft_tree(ep, C.TREE_26, want_debug=True)
        got = gpu.draft_tree([0], env["shape"])[0]
        same.append(G.compare_draft_trees(got, ref_tree, dbg, C.TREE_26, tally))
        G.verify_both(orc, gpu, ep, ref_tree, 0, tally, DESC, where=f"it{tally.iterations}.g")
    tally.report("C1 lockstep")
    print("identical leading draft-tree nodes per iteration:", same)
    assert tally.iterations >= 3 and tally.accepts == tally.caches == tally.iterations
    assert tally.rows_exact >= 2 * tally.rows_low            # sigma_logit = 1.3: most rows are decided
    assert max(same) == 27                                    # some iteration's tree is identical throughout


def test_c1_generate_action_strict_equals_greedy(env):
    orc, gpu = env["orc"], env["gpu"]
    from paper_2507_22424_b200.binding import make_shape
    toks, acts, stats = gpu.generate_action([0], env["emb"], env["ids"].tolist(), [len(env["ids"])],
                                            env["shape"], 0, 7)
    ar, _, _ = gpu.generate_action([0], env["emb"], env["ids"].tolist(), [len(env["ids"])],
                                   make_shape((), ()), 0, 7)
    assert toks == ar and stats.device_loop == 1
    # the same loop driven from the host (one read-back per iteration): same chunk, same statistics
    from paper_2507_22424_b200 import binding as B
    gpu.set_option(B.OPT_DEVICE_LOOP, 0)
    host, _, sth = gpu.generate_action([0], env["emb"], env["ids"].tolist(), [len(env["ids"])], env["shape"], 0, 7)
    gpu.set_option(B.OPT_DEVICE_LOOP, 1)
    assert host == toks and sth.device_loop == 0 and sth.iterations == stats.iterations
    assert list(sth.accept_len) == list(stats.accept_len) and list(sth.pos_accept_sum) == list(stats.pos_accept_sum)
    print(f"loop on the device {stats.ms_loop:.2f} ms, on the host {sth.ms_loop:.2f} ms ({stats.iterations} iterations)")
    pruned, _, st3 = gpu.generate_action([0], env["emb"], env["ids"].tolist(), [len(env["ids"])],
                                         make_shape(C.TREE_26.branch, C.TREE_26.expand, prune=True), 0, 7)
    assert pruned == toks and st3.ms_draft < sth.ms_draft
    # the paper's own tree (Section 5.1 / Table 4): top-8, depth 5, the best 50 of 264 drafted nodes
    dyn, _, st4 = gpu.generate_action([0], env["emb"], env["ids"].tolist(), [len(env["ids"])],
                                      make_shape((8,) * 5, (1, 8, 8, 8, 8), keep=50), 0, 7)
    assert dyn == toks
    ref, mg = orc.ar_generate(env["emb"].cpu(), env["ids"].cpu(), 7, want_margins=True,
                              follow=(toks[0], G.MARGIN))
    tally = G.Tally()
    G.compare_tokens(toks[0], ref, mg, tally, "chunk")
    tally.report("C1 generate r=0")
    assert tally.rows_exact + tally.rows_low == 7 and tally.rows_exact >= 4
    print("chunk", toks[0], "oracle", ref, "margins", [round(x, 3) for x in mg])


def test_c3_verify_sweep_tree_sizes(env):
    """Rows {1, 8, 26, 27, 60, 128}: every size is a prefix of the same 128-row random tree, and a
    row's logits depend only on its ancestors, so one oracle pass over 128 rows gives the
    expected logits and cache rows of all of them."""
    orc, gpu = env["orc"], env["gpu"]
    emb, ids = data.make_prefix(C.C3, device="cuda")
    assert 290 <= len(ids) <= 297
    tally = G.Tally()
    ep, _, _ = G.prefill_both(orc, gpu, emb, ids, 0, tally, DESC)
    P = ep.P
    tok, par, dep = data.random_tree(128, DESC, seed=C.C3.extra["tree_seed"], max_depth=8, root_token=ep.root)
    logits, _ = orc.verify_forward(ep, Tree(tok, par, dep, [0.0] * 128))
    r = 16
    for n in C.C3.extra["rows"] + (27,):
        first = gpu.prefill([0], emb, ids.tolist(), [len(ids)])
        assert first[0] == ep.root                       # same call as above: deterministic
        sub = Tree(tok[:n], par[:n], dep[:n], [0.0] * n)
        m_ref, err = _verify_against_logits(env, sub, r, logits, ep.cache, P, tally, f"g(T={n})")
        print(f"T={n}: logits err {err:.4f}, m={m_ref}")
    tally.report("C3 sweep")
    assert tally.accepts == tally.caches == 6 and tally.rows_exact >= 150


def _oracle_planted(orc, ep, seed, call):
    def greedy_fn(tokens, parent, depth):
        lg, _ = orc.verify_forward(ep, Tree(tokens, parent, depth, [0.0] * len(tokens)))
        return [orc._greedy(lg[i]) for i in range(len(tokens))]
    tok, par, dep = data.plant_tree(C.TREE_26, ep.root, DESC, greedy_fn, seed, call)
    return Tree(tok, par, dep, [0.0] * len(tok))


def test_c2_planted_drafts_threshold_sweep(env):
    """Three oracle-planted trees of the first iteration, each verified at every threshold."""
    orc, gpu = env["orc"], env["gpu"]
    tally = G.Tally()
    ep, _, _ = G.prefill_both(orc, gpu, env["emb"], env["ids"], 0, tally, DESC)
    P = ep.P
    for call in (0, 1, 2):
        tree = _oracle_planted(orc, ep, C.C2.seed, call)
        logits, _ = orc.verify_forward(ep, tree)
        ms = []
        for r in C.C2.extra["r"]:
            first = gpu.prefill([0], env["emb"], env["ids"].tolist(), [len(env["ids"])])
            assert first[0] == ep.root
            m_ref, err = _verify_against_logits(env, tree, r, logits, ep.cache, P, tally, f"tree{call}.r{r}.g")
            ms.append((r, m_ref))
        print(f"C2 planted tree {call}, (r, accepted length):", ms)
        assert [m for _, m in ms] == sorted(m for _, m in ms)  # accepted length grows with r
    tally.report("C2 threshold sweep")
    assert tally.accepts == tally.caches == 18


def test_c2_planted_chunk_lockstep_r4(env):
    """A whole chunk with oracle-planted trees at r = 4, iteration by iteration."""
    orc, gpu = env["orc"], env["gpu"]
    tally = G.Tally()
    ep, _, _ = G.prefill_both(orc, gpu, env["emb"], env["ids"], 0, tally, DESC)
    lens = []
    while len(ep.emitted) < 7:
        tree = _oracle_planted(orc, ep, C.C2.seed, 10 + tally.iterations)
        gpu.draft_tree([0], env["shape"], want_trees=False)       # keeps the draft state in step
        ref = G.verify_both(orc, gpu, ep, tree, 4, tally, DESC, where=f"it{tally.iterations}.g")
        lens.append(ref[0])
    tally.report("C2 chunk r=4")
    print("accepted lengths", lens, "emitted", ep.emitted[:7])
    assert tally.accepts == tally.caches == tally.iterations == len(lens) and sum(lens) >= 1


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
    tally = G.Tally()
    trees, refs = [], {}
    from oracle import decoder as D
    for e in range(n_ep):
        if e in (0, 15):
            ep, ref_logits, _ = orc.prefill(pre[e][0].cpu(), pre[e][1].cpu(), want_logits=True,
                                            follow=(first[e], G.MARGIN))
            assert float((logits[e].cpu().double() - ref_logits).abs().max()) < G.LOGIT_TOL
            G.compare_tokens([first[e]], [D.greedy_token(ref_logits, DESC, True)],
                             [D.top2_margin(ref_logits, DESC, True)], tally, f"ep{e}.a1")
            t = _oracle_planted(orc, ep, C.C4.extra["prefix_seed"], 100 + e)
            refs[e] = (ep, t, orc.verify_forward(ep, t)[0])
            trees.append(G.tree_dict(t))
        else:
            tok, par, dep = data.random_tree(27, DESC, seed=50 + e, max_depth=5, root_token=first[e])
            trees.append(dict(tokens=tok, parent=par, depth=dep))
    m, emitted, vlogits = gpu.verify_tree(list(range(n_ep)), trees, r, want_logits=True)
    g_all = gpu.read_buffer(1, 27 * n_ep, torch.int32).tolist()
    for e, (ep, t, ref_logits) in refs.items():
        rows = slice(27 * e, 27 * e + 27)
        m_ref, err = _verify_against_logits(env, t, r, ref_logits, ep.cache, lens[e], tally, f"ep{e}.g",
                                            episode=e, index=e, n_ep=n_ep,
                                            call=(m, emitted, vlogits[rows], g_all[rows]))
        print(f"episode {e}: P={lens[e]}, logits err {err:.4f}, m={m_ref}")
    st = gpu.read_buffer(5, 4 * n_ep, torch.int32).reshape(n_ep, 4).tolist()
    for e in range(n_ep):
        assert st[e][0] == lens[e] + 1 + m[e] and st[e][3] == m[e] + 1
    tally.report("C4 batch")
    assert tally.accepts == tally.caches == 2


@pytest.mark.parametrize("T,N,K,packed", [(27, 22016, 4096, False), (27, 4096, 11008, False),
                                          (128, 12288, 4096, False), (27, 32064, 4096, False),
                                          (290, 4096, 4096, False), (27, 22016, 4096, True),
                                          (27, 4096, 11008, True), (27, 32064, 4096, True),
                                          (290, 12288, 4096, True)])
def test_gemm_full_size_sampled_outputs(T, N, K, packed):
    """7B-shaped GEMMs: 256 sampled outputs recomputed one by one in float64. `packed`: through
    the repacked weights and plain bulk copies, the path the decoder itself uses; else through the
    strided tensor-map boxes over the caller's row-major matrix."""
    from paper_2507_22424_b200.binding import gemm, gemm_prepacked, pack_weights
    from synth_inputs import rng
    x = rng.normal(21, 1, (T, K), 1.0, "cuda", dtype=torch.float32)
    w = rng.normal_bf16(21, 2, (N, K), 0.02, "cuda")
    y = (gemm_prepacked(x, pack_weights(w), N) if packed else gemm(x, w)).cpu()
    ts = rng.integers(21, 3, 256, 0, T).tolist()
    ns = rng.integers(21, 4, 256, 0, N).tolist()
    ns[:4] = [0, N - 1, N - 64, 127]
    xc, wc = x.cpu().double(), w.cpu()
    for t, n in zip(ts, ns):
        ref = float(xc[t] @ wc[n].double())
        assert abs(float(y[t, n]) - ref) < 1e-4 * 0.02 * (K ** 0.5) + 1e-6


def test_c1_persistent_forward_kernel_matches_oracle(env):
    """The same verification step through the single cooperative forward kernel (opt-in): one
    iteration of C1 with the oracle's draft tree, everything compared."""
    from paper_2507_22424_b200.binding import OPT_PERSISTENT_FORWARD
    orc, gpu = env["orc"], env["gpu"]
    gpu.set_option(OPT_PERSISTENT_FORWARD, 1)
    try:
        tally = G.Tally()
        ep, _, _ = G.prefill_both(orc, gpu, env["emb"], env["ids"], 0, tally, DESC)
        tree = orc.draft_tree(ep, C.TREE_26)
        gpu.draft_tree([0], env["shape"], want_trees=False)
        G.verify_both(orc, gpu, ep, tree, 0, tally, DESC, where="pk.g")
        tally.report("C1 persistent forward")
        assert tally.accepts == tally.caches == 1 and tally.rows_exact >= 18
    finally:
        gpu.set_option(OPT_PERSISTENT_FORWARD, 0)


def test_c1_quantised_target_matches_quantised_oracle(env):
    """Appendix C on the 7B-shaped model: int8 target (this repository's per-row scheme), bf16 draft
    model. Prefill and one verification of the oracle's draft tree, everything compared."""
    from oracle import quant as Q
    from oracle.specvla import SpecVLAOracle
    wc = env["gpu"].w
    wh = env["orc"].w.raw
    orc = SpecVLAOracle(DESC, Q.quantize_target(wh), action_only=True, max_seq=448, max_tree_rows=128)
    gpu = G.make_gpu(DESC, wc, max_seq=512, max_episodes=1, max_rows=512, action_only=True, weight_bits=8)
    try:
        tally = G.Tally()
        ep, _, _ = G.prefill_both(orc, gpu, env["emb"], env["ids"], 0, tally, DESC)
        tree = orc.draft_tree(ep, C.TREE_26)
        gpu.draft_tree([0], env["shape"], want_trees=False)
        G.verify_both(orc, gpu, ep, tree, 0, tally, DESC, where="q8.g")
        tally.report("C1 int8 target")
        assert tally.accepts == tally.caches == 1 and tally.rows_exact >= 18
    finally:
        gpu.close()
