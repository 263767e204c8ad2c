"""Pins of the oracle's int8 weight quantiser (oracle/quant.py) against what its specification and
the arithmetic fix: error bound, extreme codes, idempotence, zero rows, ties, brute force."""
import math

import torch

from oracle import quant as Q
from synth_inputs import rng


def _w(seed, n, k, scale=0.02):
    return rng.normal_bf16(seed, 7, (n, k), scale)


def test_error_bound_and_extreme_codes():
    w = _w(3, 96, 320)
    q, s = Q.quantize_rows_int8(w)
    assert q.dtype == torch.int8 and s.dtype == torch.float32 and q.shape == w.shape and s.shape == (96,)
    wd = Q.dequantize(q, s)
    err = (w.double() - wd).abs()
    # half a step, plus the float32 rounding of the quotient (2^-24 relative of at most 127 steps)
    assert bool((err <= s.double()[:, None] * (0.5 + 127 * 2.0 ** -23)).all())
    assert int(q.abs().max()) == 127 and bool((q.abs().amax(dim=1) == 127).all())
    # the element of largest magnitude of every row carries code +-127 with its own sign
    idx = w.float().abs().argmax(dim=1)
    rows = torch.arange(96)
    assert bool((q[rows, idx].float() == 127 * torch.sign(w.float()[rows, idx])).all())


def test_requantising_the_dequantised_matrix_reproduces_the_codes():
    w = _w(4, 64, 256)
    q, s = Q.quantize_rows_int8(w)
    wd32 = (q.float() * s[:, None])                      # float32 dequantisation
    q2, s2 = Q.quantize_rows_int8(wd32)
    assert torch.equal(q, q2)
    assert bool(((s2 - s).abs() <= s * 2.0 ** -22).all())


def test_zero_row_and_constant_row():
    w = torch.zeros(3, 16, dtype=torch.bfloat16)
    w[1] = 0.5
    w[2, 3] = -0.25
    q, s = Q.quantize_rows_int8(w)
    assert torch.equal(q[0], torch.zeros(16, dtype=torch.int8)) and float(s[0]) == 1.0
    assert torch.equal(q[1], torch.full((16,), 127, dtype=torch.int8)) and float(s[1]) == float(torch.tensor(0.5) / torch.tensor(127.0))
    assert int(q[2, 3]) == -127 and int(q[2].abs().sum()) == 127


def test_ties_round_to_even_and_codes_equal_brute_force():
    # a row whose scale is exactly 2^-7 * 127 / 127: amax = 127 * 2^-7 makes scale = 2^-7, so that
    # multiples of 2^-8 fall exactly between two codes
    row = torch.tensor([127 / 128, 0.5 / 128, 1.5 / 128, 2.5 / 128, -0.5 / 128, -1.5 / 128, 3 / 128, 0.0],
                       dtype=torch.float32).to(torch.bfloat16)
    q, s = Q.quantize_rows_int8(row[None])
    assert float(s[0]) == 2.0 ** -7
    assert q[0].tolist() == [127, 0, 2, 2, 0, -2, 3, 0]
    # brute force, element by element, in python floats restricted to float32 operations
    w = _w(5, 7, 40, scale=0.3)
    q, s = Q.quantize_rows_int8(w)
    import numpy as np
    for n in range(7):
        amax = np.float32(max(abs(float(v)) for v in w[n].float()))
        sc = np.float32(amax) / np.float32(127.0)
        assert np.float32(s[n].item()) == sc
        for k in range(40):
            t = np.float32(w[n, k].float().item()) / sc
            code = int(np.clip(np.rint(t), -127, 127))
            assert int(q[n, k]) == code, (n, k)


def test_quantised_model_is_the_same_decoder_on_dequantised_weights(c0):
    """The quantised oracle is the ordinary oracle on W' = scale * code: layer matrices and the LM
    head change, the embedding and the draft model (with its own LM head copy) do not."""
    from oracle import decoder as D
    w = c0["weights"]
    wq = Q.quantize_target(w)
    assert isinstance(wq["layers.0.wqkv"], tuple) and isinstance(wq["lm_head"], tuple)
    assert wq["embed"] is w["embed"] and wq["draft.fc"] is w["draft.fc"] and wq["draft.lm_head"] is w["lm_head"]
    dw = D.DecoderWeights(wq)
    for name in ("layers.1.wgu", "lm_head"):
        q, s = wq[name]
        assert torch.equal(dw(name), Q.dequantize(q, s))
        rel = (dw(name) - w[name].double()).abs().max() / w[name].double().abs().max()
        assert 0 < float(rel) < 1.0 / 127
    from oracle.specvla import SpecVLAOracle
    a = SpecVLAOracle(c0["desc"], wq)
    b = SpecVLAOracle(c0["desc"], w)
    _, la, _ = a.prefill(c0["embeds"], c0["ids"], want_logits=True)
    _, lb, _ = b.prefill(c0["embeds"], c0["ids"], want_logits=True)
    d = float((la - lb).abs().max())
    assert 1e-5 < d < 0.2                     # quantisation moves the logits, a little
