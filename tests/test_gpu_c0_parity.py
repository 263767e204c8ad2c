"""CUDA path (through the C ABI) vs the CPU oracle on the tiny workload C0, plus the GEMM
kernel alone on shapes that span several tiles, split-K ranges and ragged tails."""
import pytest
import torch

from oracle import decoder as D
from oracle.specvla import SpecVLAOracle, Tree
from synth_inputs import configs as C, data, rng

import gpu_helpers as G

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def wcuda(c0):
    return G.to_cuda(c0["weights"])


def _gpu(c0, wcuda, persistent=False, **kw):
    args = dict(max_seq=256, max_episodes=2, max_rows=256, action_only=True)
    args.update(kw)
    gpu = G.make_gpu(c0["desc"], wcuda, **args)
    if persistent:
        from paper_2507_22424_b200.binding import OPT_PERSISTENT_FORWARD
        gpu.set_option(OPT_PERSISTENT_FORWARD, 1)
    return gpu


@pytest.mark.parametrize("T,N,K", [(1, 256, 256), (15, 1376, 256), (15, 256, 688), (27, 4096, 4096),
                                   (33, 1000, 1024), (64, 136, 72), (128, 512, 2048), (130, 384, 520),
                                   (290, 768, 512), (27, 8448, 1024), (9, 16384, 768)])
def test_gemm_matches_float64_matmul(T, N, K):
    from paper_2507_22424_b200.binding import gemm
    x = rng.normal(11, 1, (T, K), 1.0, dtype=torch.float32)
    w = rng.normal_bf16(11, 2, (N, K), 0.02)
    ref = x.double() @ w.double().T
    y = gemm(x.cuda(), w.cuda()).cpu().double()
    # two-limb activations (2^-18 relative) and fp32 accumulation; outputs ~0.02 * sqrt(K)
    tol = 1e-4 * 0.02 * (K ** 0.5) + 1e-6
    assert (y - ref).abs().max() < tol, float((y - ref).abs().max())


@pytest.mark.parametrize("T,N,K", [(1, 256, 256), (15, 1376, 256), (33, 1000, 1024), (130, 384, 520), (9, 16384, 768)])
def test_prepacked_gemm_matches_float64_matmul(T, N, K):
    """The same product through the library's repacked weights (the decoder's own path)."""
    from paper_2507_22424_b200.binding import gemm_prepacked, pack_weights
    x = rng.normal(12, 1, (T, K), 1.0, dtype=torch.float32)
    w = rng.normal_bf16(12, 2, (N, K), 0.02)
    ref = x.double() @ w.double().T
    y = gemm_prepacked(x.cuda(), pack_weights(w.cuda()), N).cpu().double()
    tol = 1e-4 * 0.02 * (K ** 0.5) + 1e-6
    assert (y - ref).abs().max() < tol, float((y - ref).abs().max())


def test_device_side_wait_runs_out_and_the_context_survives():
    """Failure detection without a fault: the producer of the next GEMM withholds one K block and
    the wait limit is 2 ms; the kernel must record the failure and RETURN (status word ->
    SPECVLA_ERR_TIMEOUT), and the very next ordinary call on the same context must be correct."""
    import ctypes as C
    from paper_2507_22424_b200 import binding as B
    T, N, K = 16, 256, 512
    x = rng.normal(13, 1, (T, K), 1.0, dtype=torch.float32).cuda()
    w = rng.normal_bf16(13, 2, (N, K), 0.02).cuda()
    ref = x.cpu().double() @ w.cpu().double().T
    y = torch.zeros(T, N, dtype=torch.float32, device="cuda")
    nb = B.lib.specvla_gemm_scratch_bytes(T, N, K)
    scratch = torch.empty(nb + 1024, dtype=torch.uint8, device="cuda")
    sp = (scratch.data_ptr() + 1023) // 1024 * 1024
    assert B.lib.specvla_gemm_fault_test(2_000_000, 1) == 0          # 2 ms, K block 1 of every CTA's range
    t0 = torch.cuda.Event(enable_timing=True)
    t1 = torch.cuda.Event(enable_timing=True)
    t0.record()
    rc = B.lib.specvla_gemm(C.c_void_p(x.data_ptr()), C.c_void_p(w.data_ptr()), C.c_void_p(y.data_ptr()), T, N, K,
                            C.c_void_p(sp), nb, B._stream())
    t1.record()
    assert rc == 0
    assert B.lib.specvla_gemm_status(C.c_void_p(sp), B._stream()) == -6   # SPECVLA_ERR_TIMEOUT
    assert 2.0 <= t0.elapsed_time(t1) < 200.0                          # it waited the limit out, and returned
    # the hook held for that one call: the next call on the same scratch is an ordinary, correct GEMM
    got = B.gemm(x, w).cpu().double()
    assert (got - ref).abs().max() < 1e-4 * 0.02 * (K ** 0.5) + 1e-6
    rc = B.lib.specvla_gemm(C.c_void_p(x.data_ptr()), C.c_void_p(w.data_ptr()), C.c_void_p(y.data_ptr()), T, N, K,
                            C.c_void_p(sp), nb, B._stream())
    assert rc == 0 and B.lib.specvla_gemm_status(C.c_void_p(sp), B._stream()) == 0
    assert (y.cpu().double() - ref).abs().max() < 1e-4 * 0.02 * (K ** 0.5) + 1e-6


@pytest.mark.parametrize("action_only", [True, False])
def test_prefill_logits_and_first_token(c0, wcuda, action_only):
    orc = c0["make"](action_only=action_only)
    gpu = _gpu(c0, wcuda, action_only=action_only)
    tally = G.Tally()
    ep, ref_logits, feats = G.prefill_both(orc, gpu, c0["embeds"].cuda(), c0["ids"], 0, tally, c0["desc"],
                                           action_only)
    f = gpu.read_buffer(3, 64 * 256, torch.float32).reshape(64, 256).double()
    assert (f - feats).abs().max() < 2e-2
    tally.report(f"C0 prefill action_only={action_only}")
    assert tally.rows_exact + tally.rows_low == 1
    gpu.close()


@pytest.mark.parametrize("n_rows,seed,persistent", [(1, 0, False), (15, 1, False), (27, 2, False), (60, 3, False),
                                                    (128, 4, False), (1, 0, True), (15, 1, True), (27, 2, True),
                                                    (32, 5, True)])
def test_verify_tree_matches_oracle(c0, wcuda, n_rows, seed, persistent):
    """Logits, greedy tokens, accepted length, emitted tokens, path, compacted cache and state of
    one verification, for every tree size: all compared on every run (see gpu_helpers). With
    `persistent` the forward runs as the single cooperative kernel (up to 32 rows)."""
    desc = c0["desc"]
    orc = c0["make"]()
    gpu = _gpu(c0, wcuda, persistent=persistent)
    tally = G.Tally()
    ep, _, _ = G.prefill_both(orc, gpu, c0["embeds"].cuda(), c0["ids"], 0, tally, desc)
    tok, par, dep = data.random_tree(n_rows, desc, seed=seed, max_depth=8, root_token=ep.root)
    G.verify_both(orc, gpu, ep, Tree(tok, par, dep, [0.0] * n_rows), 40, tally, desc, where=f"g(T={n_rows})")
    tally.report(f"C0 verify T={n_rows}")
    assert tally.accepts == 1 and tally.caches == 1 and tally.rows_exact + tally.rows_low == n_rows + 1
    # the tiny model's logits are close together (sigma 0.3): still, most rows must be compared
    assert tally.rows_exact >= (n_rows + 1) // 3
    gpu.close()


def test_relaxed_threshold_sweep_on_fixed_tree(c0, wcuda):
    """Same tree, r in {0, 1, 4, 16, 255}: accepted length and tokens equal the oracle's."""
    desc = c0["desc"]
    tally = G.Tally()
    ms = []
    for r in (0, 1, 4, 16, 255):
        orc = c0["make"]()
        gpu = _gpu(c0, wcuda)
        ep, _, _ = G.prefill_both(orc, gpu, c0["embeds"].cuda(), c0["ids"], 0, tally, desc)
        tok, par, dep = data.random_tree(40, desc, seed=21, max_depth=6, root_token=ep.root)
        ref = G.verify_both(orc, gpu, ep, Tree(tok, par, dep, [0.0] * 40), r, tally, desc, where=f"g(r={r})")
        ms.append(ref[0])
        gpu.close()
    tally.report("C0 threshold sweep")
    assert tally.accepts == 5 and tally.caches == 5
    assert ms == sorted(ms) and ms[-1] == max(dep)       # r = 255 accepts the whole deepest path


def test_draft_tree_matches_oracle(c0, wcuda):
    """The draft model's tree (Eq. 2, Section 4.1): node by node against the oracle's up to the first
    ranking decision that the oracle itself takes at a gap below the margin; then the GPU's tree,
    whatever it is, is verified on both sides."""
    desc, shape = c0["desc"], c0["wl"].tree
    from paper_2507_22424_b200.binding import make_shape
    orc = c0["make"]()
    gpu = _gpu(c0, wcuda)
    tally = G.Tally()
    ep, _, _ = G.prefill_both(orc, gpu, c0["embeds"].cuda(), c0["ids"], 0, tally, desc)
    ref, dbg = orc.draft_tree(ep, shape, want_debug=True)
    got = gpu.draft_tree([0], make_shape(shape.branch, shape.expand))[0]
    same = G.compare_draft_trees(got, ref, dbg, shape, tally)
    assert same >= 3                                    # at least the root and its two children
    G.verify_both(orc, gpu, ep, Tree(got["tokens"], got["parent"], got["depth"], got["score"]), 4, tally, desc)
    tally.report("C0 draft tree")
    gpu.close()


@pytest.mark.parametrize("branch,expand,keep", [((4, 4, 4), (1, 4, 4), 10), ((8, 8, 8), (1, 8, 8), 50),
                                                ((8, 8), (1, 8), 100)])
def test_dynamic_draft_tree_matches_oracle(c0, wcuda, branch, expand, keep):
    """Dynamic tree: wide levels (up to 64 nodes), the best `keep` nodes by cumulative
    log-probability stay. Structure always valid; tokens, parents and scores equal the oracle's
    unless two candidates' scores are closer than the comparison margin. The GPU's tree is then
    verified on both sides (strict acceptance) with everything compared."""
    from paper_2507_22424_b200.binding import make_shape
    from synth_inputs.configs import TreeShape
    import copy
    desc = c0["desc"]
    shape = TreeShape(branch, expand, keep=keep)
    orc = c0["make"]()
    gpu = _gpu(c0, wcuda)
    tally = G.Tally()
    ep, _, _ = G.prefill_both(orc, gpu, c0["embeds"].cuda(), c0["ids"], 0, tally, desc)
    full = orc.draft_tree(copy.deepcopy(ep), TreeShape(branch, expand))
    ref = orc.draft_tree(ep, shape)
    got = gpu.draft_tree([0], make_shape(branch, expand, keep=keep))[0]
    n = 1 + min(keep, shape.n_nodes)
    assert len(got["tokens"]) == n == len(ref.tokens)
    assert got["parent"][0] == -1 and got["tokens"][0] == ep.root
    for i in range(1, n):
        assert 0 <= got["parent"][i] < i and got["depth"][i] == got["depth"][got["parent"][i]] + 1
        assert got["score"][i] <= got["score"][got["parent"][i]] + 1e-6
    if got["tokens"] == ref.tokens and got["parent"] == ref.parent:
        assert max(abs(a - b) for a, b in zip(got["score"], ref.score)) < 5e-2
        tally.log.append("dynamic tree identical to the oracle's")
    else:
        ranked = sorted(full.score[1:], reverse=True)
        gap = min(a - b for a, b in zip(ranked, ranked[1:]))
        assert gap < G.MARGIN, (got["tokens"], ref.tokens)
        tally.log.append(f"dynamic tree differs where two candidates are {gap} apart")
    G.verify_both(orc, gpu, ep, Tree(got["tokens"], got["parent"], got["depth"], got["score"]), 0, tally, desc)
    tally.report(f"C0 dynamic tree keep={keep}")
    gpu.close()


def test_dynamic_tree_two_ragged_episodes_in_one_call(c0, wcuda):
    """Two episodes of different prefix lengths drafted, re-ranked and verified together equal
    the same episodes run alone."""
    from paper_2507_22424_b200.binding import make_shape
    desc = c0["desc"]
    emb2 = rng.normal_bf16(5, 1, (40, desc.d_model), 1.0)
    ids2 = torch.full((40,), -1, dtype=torch.int32)
    ids2[30:] = rng.integers(5, 2, 10, 0, desc.action_base).to(torch.int32)
    shape = make_shape((8, 8, 8), (1, 8, 8), keep=30)
    gpu = _gpu(c0, wcuda)
    alone = []
    for emb, ids, n in ((c0["embeds"], c0["ids"], 64), (emb2, ids2, 40)):
        gpu.prefill([0], emb.cuda(), ids.tolist(), [n])
        tree = gpu.draft_tree([0], shape)[0]
        alone.append((tree, gpu.verify_tree([0], None, 4)))
    emb = torch.cat([c0["embeds"], emb2]).cuda()
    gpu.prefill([1, 0], emb, c0["ids"].tolist() + ids2.tolist(), [64, 40])
    trees = gpu.draft_tree([1, 0], shape)
    m, emitted = gpu.verify_tree([1, 0], None, 4)
    for k in range(2):
        assert len(trees[k]["tokens"]) == 31
        assert trees[k]["tokens"] == alone[k][0]["tokens"] and trees[k]["parent"] == alone[k][0]["parent"]
        assert (m[k], emitted[k]) == (alone[k][1][0][0], alone[k][1][1][0])
    gpu.close()


def test_generate_action_with_dynamic_tree_is_lossless(c0, wcuda):
    from paper_2507_22424_b200.binding import make_shape
    gpu = _gpu(c0, wcuda)
    args = ([0], c0["embeds"].cuda(), c0["ids"].tolist(), [64])
    ar, _, _ = gpu.generate_action(*args, make_shape((), ()), 0, 7)
    dyn, _, st = gpu.generate_action(*args, make_shape((8, 8, 8), (1, 8, 8), keep=50), 0, 7)
    both, _, _ = gpu.generate_action(*args, make_shape((8, 8, 8), (1, 8, 8), keep=50, prune=True), 0, 7)
    assert dyn[0] == ar[0] and both[0] == ar[0] and st.iterations <= 6
    gpu.close()


@pytest.mark.parametrize("r,action_only,persistent", [(0, True, False), (4, True, False), (0, False, False),
                                                      (4, False, False), (4, True, True), (0, False, True)])
def test_generate_action_lockstep_with_oracle(c0, wcuda, r, action_only, persistent):
    """Iteration by iteration until the chunk is complete: the oracle's draft tree is verified on
    both sides; accepted length, emitted tokens, path, cache and state agree in every iteration."""
    desc, shape = c0["desc"], c0["wl"].tree
    orc = c0["make"](action_only=action_only)
    gpu = _gpu(c0, wcuda, action_only=action_only, persistent=persistent)
    tally = G.Tally()
    ep, _, _ = G.prefill_both(orc, gpu, c0["embeds"].cuda(), c0["ids"], 0, tally, desc, action_only)
    from paper_2507_22424_b200.binding import make_shape
    cshape = make_shape(shape.branch, shape.expand)
    while len(ep.emitted) < 7:
        tree = orc.draft_tree(ep, shape)
        gpu.draft_tree([0], cshape, want_trees=False)         # advances the GPU's draft state
        G.verify_both(orc, gpu, ep, tree, r, tally, desc, action_only, where=f"it{tally.iterations}.g")
    tally.report(f"C0 lockstep r={r} action_only={action_only}")
    assert tally.iterations >= 2 and tally.accepts == tally.iterations == tally.caches
    gpu.close()


def test_generate_action_strict_equals_greedy_decoding(c0, wcuda):
    """r = 0 through the library's own loop equals the oracle's autoregressive tokens at all seven
    positions (exactly where the margin allows, logged elsewhere, the oracle continuing with the
    GPU's token there), and depth-0 decoding gives the same chunk."""
    from paper_2507_22424_b200.binding import make_shape
    desc, shape = c0["desc"], c0["wl"].tree
    orc = c0["make"]()
    gpu = _gpu(c0, wcuda)
    toks, acts, stats = gpu.generate_action([0], c0["embeds"].cuda(), c0["ids"].tolist(), [64],
                                            make_shape(shape.branch, shape.expand), 0, 7)
    ar, _, st2 = gpu.generate_action([0], c0["embeds"].cuda(), c0["ids"].tolist(), [64],
                                     make_shape((), ()), 0, 7)
    assert st2.iterations == 6
    assert toks[0] == ar[0]          # lossless inside the CUDA path itself, whatever the margins
    # depth pruning (an iteration drafts no deeper than the tokens still missing): same chunk
    pr, _, st3 = gpu.generate_action([0], c0["embeds"].cuda(), c0["ids"].tolist(), [64],
                                     make_shape(shape.branch, shape.expand, prune=True), 0, 7)
    assert pr[0] == toks[0] and st3.iterations >= stats.iterations
    ref, mg = orc.ar_generate(c0["embeds"], c0["ids"], 7, want_margins=True, follow=(toks[0], G.MARGIN))
    tally = G.Tally()
    G.compare_tokens(toks[0], ref, mg, tally, "chunk")
    tally.report("C0 generate r=0")
    assert tally.rows_exact + tally.rows_low == 7
    want = orc.detokenize(toks[0])
    assert all(abs(a - b) < 1e-6 for a, b in zip(acts[0], want))
    gpu.close()


@pytest.mark.parametrize("branch,expand,keep,r,n_tokens", [
    ((4, 2, 2, 1, 1), (1, 2, 2, 2, 2), 0, 0, 7), ((4, 2, 2, 1, 1), (1, 2, 2, 2, 2), 0, 4, 7),
    ((8, 8, 8), (1, 8, 8), 50, 2, 7), ((), (), 0, 0, 7), ((3, 2), (1, 3), 0, 9, 12), ((2,), (1,), 0, 0, 1)])
def test_chunk_loop_on_the_device_equals_the_loop_on_the_host(c0, wcuda, branch, expand, keep, r, n_tokens):
    """Algorithm 1's loop as one graph launch (a while node around draft, verification and the
    appending of the emitted tokens) against the same loop driven from the host with a read-back
    per iteration: tokens, actions, iteration count, accepted lengths, per-position statistics,
    episode state, both caches, the launch count, and what a further draft + verification gives."""
    from paper_2507_22424_b200 import binding as B
    shape = B.make_shape(branch, expand, keep=keep)
    emb2 = rng.normal_bf16(5, 1, (40, c0["desc"].d_model), 1.0)
    ids2 = torch.full((40,), -1, dtype=torch.int32)
    emb = torch.cat([c0["embeds"], emb2]).cuda()
    ids = c0["ids"].tolist() + ids2.tolist()
    out = []
    for device_loop in (1, 0):
        gpu = _gpu(c0, wcuda)
        gpu.set_option(B.OPT_DEVICE_LOOP, device_loop)
        before = gpu.kernel_launches()
        toks, acts, st = gpu.generate_action([1, 0], emb, ids, [64, 40], shape, r, n_tokens)
        launches = gpu.kernel_launches() - before
        again, _, st_again = gpu.generate_action([1, 0], emb, ids, [64, 40], shape, r, n_tokens)   # kept graph
        assert again == toks and st_again.iterations == st.iterations
        assert st.device_loop == device_loop
        state = gpu.read_buffer(5, 8, torch.int32).tolist()
        P = [state[4], state[0]]
        kv = [gpu.read_kv(e, l, w, 0, P[i]) for i, e in enumerate((1, 0)) for l in range(c0["desc"].n_layers)
              for w in (0, 1)]
        kvd = [gpu.read_kv(e, 0, w, 0, state[4 * e + 1], draft=True) for e in (1, 0) for w in (0, 1)]
        follow = None
        if branch:
            trees = gpu.draft_tree([1, 0], shape)
            follow = (trees, gpu.verify_tree([1, 0], None, r))
        out.append(dict(toks=toks, acts=acts, it=st.iterations, emitted=st.tokens_emitted,
                        m=list(st.accept_len), pi=list(st.pos_iterations), ps=list(st.pos_accept_sum),
                        state=state, kv=kv, kvd=kvd, follow=follow, launches=launches))
        gpu.close()
    dev, host = out
    for key in ("toks", "acts", "it", "emitted", "m", "pi", "ps", "state", "follow"):
        assert dev[key] == host[key], key
    for a, b in zip(dev["kv"] + dev["kvd"], host["kv"] + host["kvd"]):
        assert torch.equal(a, b)
    assert len(dev["toks"][0]) == n_tokens and dev["it"] >= (1 if n_tokens > 1 else 0)
    # the device loop adds: the kernel that starts the chunk, the one that arms the loop, one append per iteration
    assert dev["launches"] == host["launches"] + 2 + dev["it"]


def test_weight_matrices_may_be_released_after_creation(c0, wcuda):
    """The library keeps its own repacked copy of every weight matrix: once the context exists the
    caller's matrices can go (here: overwritten with zeros); embedding and norm gains stay. Logits
    (whole LM head), draft trees and the chunk are unchanged."""
    from paper_2507_22424_b200.binding import make_shape
    mine = {k: v.clone() for k, v in wcuda.items()}
    gpu = _gpu(c0, mine)
    shape = make_shape(c0["wl"].tree.branch, c0["wl"].tree.expand)
    args = ([0], c0["embeds"].cuda(), c0["ids"].tolist(), [64])

    def run():
        first, logits = gpu.prefill(*args, want_logits=True)
        tree = gpu.draft_tree([0], shape)[0]
        given = dict(tokens=tree["tokens"], parent=tree["parent"], depth=tree["depth"])
        m, emitted, vlogits = gpu.verify_tree([0], [given], 2, want_logits=True)
        toks, _, _ = gpu.generate_action(*args, shape, 2, 7)
        return first, logits.clone(), tree["tokens"], m, emitted, vlogits.clone(), toks

    before = run()
    kept = 0
    for k, v in mine.items():
        if v.dim() == 2 and "embed" not in k:
            v.zero_()
        else:
            kept += 1
    torch.cuda.synchronize()
    after = run()
    assert kept >= 2 and before[0] == after[0] and before[2:5] == after[2:5] and before[6] == after[6]
    assert torch.equal(before[1], after[1]) and torch.equal(before[5], after[5])
    gpu.close()


def test_two_episodes_ragged_prefixes(c0, wcuda):
    """Two episodes with different prefix lengths (one of them with text ids, i.e. rows gathered
    from the embedding) in one prefill call and one verification call equal two separate oracle
    runs: first tokens, logits, greedy tokens, accepted lengths, tokens, paths, caches, states."""
    desc = c0["desc"]
    emb2 = rng.normal_bf16(5, 1, (40, desc.d_model), 1.0)
    ids2 = torch.full((40,), -1, dtype=torch.int32)
    ids2[30:] = rng.integers(5, 2, 10, 0, desc.action_base).to(torch.int32)
    orc = c0["make"]()
    gpu = _gpu(c0, wcuda)
    tally = G.Tally()
    emb = torch.cat([c0["embeds"], emb2]).cuda()
    ids = c0["ids"].tolist() + ids2.tolist()
    episodes = [1, 0]                                     # call slot 0 is episode 1 and vice versa
    first, plogits = gpu.prefill(episodes, emb, ids, [64, 40], want_logits=True)
    eps = []
    for k, (e, i) in enumerate(((c0["embeds"], c0["ids"]), (emb2, ids2))):
        ep, ref_logits, _ = orc.prefill(e, i, want_logits=True, follow=(first[k], G.MARGIN))
        assert float((plogits[k].cpu().double() - ref_logits).abs().max()) < G.LOGIT_TOL
        G.compare_tokens([first[k]], [D.greedy_token(ref_logits, desc, True)],
                         [D.top2_margin(ref_logits, desc, True)], tally, f"a1(slot {k})")
        eps.append(ep)
    assert tally.rows_exact >= 1          # the 40-row prefix's first token has a margin of 6.6e-2
    trees = []
    for ep, seed in zip(eps, (31, 32)):
        tok, par, dep = data.random_tree(15 + seed % 4, desc, seed=seed, max_depth=5, root_token=ep.root)
        trees.append(Tree(tok, par, dep, [0.0] * len(tok)))
    P0 = [ep.P for ep in eps]
    m, emitted, logits = gpu.verify_tree(episodes, [G.tree_dict(t) for t in trees], 30, want_logits=True)
    n0 = len(trees[0].tokens)
    g_gpu = gpu.read_buffer(1, n0 + len(trees[1].tokens), torch.int32).tolist()
    rows = [g_gpu[:n0], g_gpu[n0:]]
    lg = [logits[:n0], logits[n0:]]
    for k in range(2):
        ref = orc.verify_tree(eps[k], trees[k], 30, want_debug=True, follow=(rows[k], G.MARGIN))
        dbg = ref[2]
        err = float((lg[k].cpu().double() - dbg["logits"]).abs().max())
        assert err < G.LOGIT_TOL, err
        G.compare_tokens(rows[k], dbg["g_own"], G.margins(dbg["logits"], desc, True).tolist(), tally, f"g(slot {k})")
        G.check_verify_outputs(gpu, tally, desc, rows[k], m, emitted, ref, eps[k], P0[k], index=k,
                               episode=episodes[k], n_ep=2)
    tally.report("C0 two ragged episodes")
    assert tally.accepts == 2 and tally.caches == 2
    gpu.close()


def test_bad_arguments_are_rejected_before_any_launch(c0, wcuda):
    from paper_2507_22424_b200.binding import SpecVLAError
    gpu = _gpu(c0, wcuda, max_seq=96)
    with pytest.raises(SpecVLAError) as e:
        gpu.verify_tree([0], [dict(tokens=[800], parent=[-1], depth=[0])], 0)
    assert e.value.code == -4                                     # not prefilled
    gpu.prefill([0], c0["embeds"].cuda(), c0["ids"].tolist(), [64])
    n0 = gpu.kernel_launches()
    bad = [dict(tokens=[800, 801], parent=[-1, 1], depth=[0, 1]),          # parent >= index
           dict(tokens=[800, 801], parent=[-1, 0], depth=[0, 2]),          # wrong depth
           dict(tokens=[800, 801], parent=[0, 0], depth=[0, 1]),           # root has a parent
           dict(tokens=[800, 5000], parent=[-1, 0], depth=[0, 1])]         # token out of range
    for t in bad:
        with pytest.raises(SpecVLAError) as e:
            gpu.verify_tree([0], [t], 0)
        assert e.value.code == -3
    tok, par, dep = data.random_tree(40, c0["desc"], seed=1)
    with pytest.raises(SpecVLAError) as e:                        # 64 + 40 > max_seq
        gpu.verify_tree([0], [dict(tokens=tok, parent=par, depth=dep)], 0)
    assert e.value.code == -2
    with pytest.raises(SpecVLAError):
        gpu.verify_tree([3], [bad[0]], 0)
    # tree shapes: a level wider than 16 nodes needs the dynamic tree (keep > 0); at most 127 kept
    # nodes and 319 drafted ones; level 0 expands the root alone; capacity of the caches
    from paper_2507_22424_b200.binding import make_shape
    for sh, code in [(make_shape((8, 8), (1, 8)), -1), (make_shape((8, 8), (1, 8), keep=128), -1),
                     (make_shape((8,) * 7, (1,) + (8,) * 6, keep=50), -1), (make_shape((4, 4), (2, 4)), -1),
                     (make_shape((4, 4), (1, 5)), -1), (make_shape((9,), (1,)), -1),
                     (make_shape((8, 8), (1, 8), keep=40), -2)]:          # 64 + 41 rows > max_seq
        with pytest.raises(SpecVLAError) as e:
            gpu.draft_tree([0], sh, want_trees=False)
        assert e.value.code == code, (e.value.code, code)
    assert gpu.kernel_launches() == n0
    gpu.close()
