"""Quantised target (Appendix C; this repository's int8 specification, oracle/quant.py): the CUDA
path with weight_bits = 8 against the oracle run on the dequantised weights W' = scale * code.
Codes are defined in float32 (IEEE division, round-half-even), so both sides hold the same W'
bit for bit and the comparison is as tight as for the bf16 model."""
import pytest
import torch

from oracle import quant as Q
from oracle.specvla import SpecVLAOracle, Tree
from synth_inputs import configs as C, data

import gpu_helpers as G

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def q0(c0):
    wq = Q.quantize_target(c0["weights"])
    return dict(wq=wq, wcuda=G.to_cuda(c0["weights"]), make=lambda **kw: SpecVLAOracle(C.TINY, wq, **kw))


def _gpu(c0, q0, **kw):
    args = dict(max_seq=256, max_episodes=2, max_rows=256, action_only=True, weight_bits=8)
    args.update(kw)
    return G.make_gpu(c0["desc"], q0["wcuda"], **args)


@pytest.mark.parametrize("n_rows,seed", [(1, 0), (15, 1), (27, 2), (60, 3), (128, 4)])
def test_quantised_verify_matches_quantised_oracle(c0, q0, n_rows, seed):
    desc = c0["desc"]
    orc = q0["make"]()
    gpu = _gpu(c0, q0)
    tally = G.Tally()
    ep, _, _ = G.prefill_both(orc, gpu, c0["embeds"].cuda(), c0["ids"], 0, tally, desc)
    tok, par, dep = data.random_tree(n_rows, desc, seed=seed, max_depth=8, root_token=ep.root)
    G.verify_both(orc, gpu, ep, Tree(tok, par, dep, [0.0] * n_rows), 40, tally, desc, where=f"q8.g(T={n_rows})")
    tally.report(f"C0 int8 verify T={n_rows}")
    assert tally.accepts == 1 and tally.caches == 1
    # one wrong code would move a logit by about 1e-3; identical codes leave fp32 rounding only
    assert tally.max_logit_err < 2e-4, tally.max_logit_err
    gpu.close()


def test_quantised_model_differs_from_the_bf16_model_and_follows_its_own_oracle(c0, q0):
    """Guard for the test above: the quantised GPU model is NOT the bf16 model (so agreeing with the
    quantised oracle means the codes and scales are really in use)."""
    gpu = _gpu(c0, q0)
    ref = G.make_gpu(c0["desc"], q0["wcuda"], max_seq=256, max_episodes=1, max_rows=256, action_only=True)
    _, lq = gpu.prefill([0], c0["embeds"].cuda(), c0["ids"].tolist(), [64], want_logits=True)
    _, lb = ref.prefill([0], c0["embeds"].cuda(), c0["ids"].tolist(), [64], want_logits=True)
    d = float((lq - lb).abs().max())
    assert 1e-4 < d < 0.2, d
    gpu.close()
    ref.close()


@pytest.mark.parametrize("r", [0, 4])
def test_quantised_chunk_lockstep(c0, q0, r):
    """Whole chunk, iteration by iteration, draft model (bf16, original LM-head rows) + quantised
    target: the oracle's draft tree verified on both sides."""
    from paper_2507_22424_b200.binding import make_shape
    desc, shape = c0["desc"], c0["wl"].tree
    orc = q0["make"]()
    gpu = _gpu(c0, q0)
    tally = G.Tally()
    ep, _, _ = G.prefill_both(orc, gpu, c0["embeds"].cuda(), c0["ids"], 0, tally, desc)
    cshape = make_shape(shape.branch, shape.expand)
    first_tree = None
    while len(ep.emitted) < 7:
        tree, dbg = orc.draft_tree(ep, shape, want_debug=True)
        got = gpu.draft_tree([0], cshape)[0]
        if first_tree is None:
            first_tree = G.compare_draft_trees(got, tree, dbg, shape, tally)
        G.verify_both(orc, gpu, ep, tree, r, tally, desc, where=f"q8.it{tally.iterations}.g")
    tally.report(f"C0 int8 lockstep r={r}")
    assert tally.iterations >= 2 and tally.accepts == tally.caches == tally.iterations and first_tree >= 3
    # strict decoding through the library's own loop is lossless for the quantised model too
    toks, _, _ = gpu.generate_action([0], c0["embeds"].cuda(), c0["ids"].tolist(), [64], cshape, 0, 7)
    ar, _, _ = gpu.generate_action([0], c0["embeds"].cuda(), c0["ids"].tolist(), [64], make_shape((), ()), 0, 7)
    assert toks == ar
    gpu.close()
