"""ORACLE (test infrastructure, not the product): weight-only int8 quantisation of the target.

The paper runs Spec-VLA on quantised verification models (Appendix C, Tables 5-6: int8 and int4
targets) but does not say how the weights are quantised (it names no scheme, group size or
rounding). This repository's own specification, chosen to be the plainest one that halves the
weight stream, is:

  * per OUTPUT ROW n of a weight matrix W [N, K] (bf16 values): amax_n = max_k |W[n, k]|,
    scale_n = amax_n / 127 (1 if the row is all zero);
  * code q[n, k] = round-half-to-even(W[n, k] / scale_n), clipped to [-127, 127] (int8);
  * the quantised model uses W'[n, k] = scale_n * q[n, k] wherever the original used W[n, k];
  * quantised: the four matrices of every target layer and the LM head the target scores with.
    Embedding, RMSNorm gains and the whole draft model (which also keeps the original bf16 LM head
    rows) stay as they are;
  * scale and quotient are taken in IEEE float32 (division and round-to-nearest-even are exactly
    specified there), so every implementation derives the same codes bit for bit; the quantised
    model itself is then evaluated here in float64 like the unquantised one.

Everything else (decoder math, Algorithm 1) is oracle/decoder.py and oracle/specvla.py run on W'.

Pins (tests/test_oracle_quant_pins.py): |W - W'| <= scale / 2 elementwise; the row maximum maps to
+-127; re-quantising W' reproduces the codes; an all-zero row gives codes 0 and scale 1; codes
equal a brute-force per-element python evaluation; halves and ties round to even.
Parity unpinned: the paper's int8/int4 speed ratios and success rates (its scheme is not given).

Only tests, the smoke check and the benchmark's CPU-baseline leg may import this package.
"""
from __future__ import annotations

import torch

QUANTISED_SUFFIXES = ("wqkv", "wo", "wgu", "wd")


def quantize_rows_int8(w: torch.Tensor):
    """w [N, K] (any float dtype holding bf16-representable values). Returns (q int8 [N, K],
    scale float32 [N])."""
    w32 = w.detach().to(device="cpu", dtype=torch.float32)
    amax = w32.abs().amax(dim=1)
    scale = torch.where(amax > 0, amax / torch.tensor(127.0, dtype=torch.float32), torch.ones_like(amax))
    t = w32 / scale[:, None]                          # float32 division
    q = torch.clamp(torch.round(t), -127, 127)        # torch.round: half to even
    return q.to(torch.int8), scale


def dequantize(q: torch.Tensor, scale: torch.Tensor, dtype=torch.float64) -> torch.Tensor:
    return q.to(dtype) * scale.to(dtype)[:, None]


def quantize_target(weights: dict) -> dict:
    """The weight dict of the quantised model: target layer matrices and the LM head become
    (codes, scales) pairs, which oracle.decoder.DecoderWeights expands to scale * code on use;
    the draft model keeps scoring with the original LM head, kept under 'draft.lm_head'."""
    out = {}
    for name, w in weights.items():
        is_layer = name.startswith("layers.") and name.rsplit(".", 1)[-1] in QUANTISED_SUFFIXES
        if is_layer or name == "lm_head":
            out[name] = quantize_rows_int8(w)
        else:
            out[name] = w
    out["draft.lm_head"] = weights["lm_head"]
    return out
