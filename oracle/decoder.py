"""ORACLE (test infrastructure, not the product): Llama-style decoder math on the CPU.

Plain, slow, float64 PyTorch-CPU statement of what one forward pass of the verification
model M_V (and of the one-layer draft model M_D) computes. The paper only names the
architecture ("a Llama decoder layer", Section 4.1; OpenVLA's Llama-2-7B verifier,
Section 5.1); the formulas below are the textbook Llama ones:

  * pre-norm residual blocks; RMSNorm  y = x * rsqrt(mean(x^2) + eps) * g
  * multi-head attention, scores scaled by 1/sqrt(head_dim), softmax over visible keys
  * rotary position embedding, "rotate-half" pairing (dim i with dim i + head_dim/2),
    frequency theta^(-2i/head_dim), applied to q and k before k is cached
  * SwiGLU MLP  W_d( silu(W_g x) * (W_u x) ),  silu(z) = z / (1 + exp(-z))
  * no biases, untied embedding and LM head, final RMSNorm before the LM head

Weights arrive as bfloat16 values and are used exactly (upcast); every activation,
cache entry and accumulation is float64 (or float32 when dtype=torch.float32 is asked
for). No blocking, fusion or reordering: one matmul per projection, one softmax per head.

Only tests, the smoke check and the benchmark's CPU-baseline leg may import this package.
Pins (tests/test_oracle_*.py): logits against the HuggingFace Llama implementation under a
causal mask and under a tree mask; tree rows against sequential decoding of each path;
draft_forward against a one-layer library Llama fed the fc output, read before any final norm.
"""
from __future__ import annotations

import math

import torch


class DecoderWeights:
    """Read-only view of a weight dict (see synth_inputs.data.make_weights for names)."""

    def __init__(self, weights: dict, dtype=torch.float64):
        self.raw = weights
        self.dtype = dtype

    def __call__(self, name: str) -> torch.Tensor:
        raw = self.raw[name]
        if isinstance(raw, tuple):
            # a quantised matrix (oracle/quant.py): int8 codes and one float32 scale per output row
            q, scale = raw
            return q.to(device="cpu", dtype=self.dtype) * scale.to(device="cpu", dtype=self.dtype)[:, None]
        return raw.to(device="cpu", dtype=self.dtype)


def rmsnorm(x: torch.Tensor, gain: torch.Tensor, eps: float) -> torch.Tensor:
    ms = (x * x).sum(dim=-1, keepdim=True) / x.shape[-1]
    return x / torch.sqrt(ms + eps) * gain


def rope(x: torch.Tensor, pos: torch.Tensor, theta: float) -> torch.Tensor:
    """x [T, H, dh]; pos [T] integer positions. Rotate-half convention."""
    T, H, dh = x.shape
    half = dh // 2
    i = torch.arange(half, dtype=x.dtype)
    inv_freq = theta ** (-2.0 * i / dh)                        # [half]
    ang = pos.to(x.dtype)[:, None] * inv_freq[None, :]         # [T, half]
    c, s = torch.cos(ang)[:, None, :], torch.sin(ang)[:, None, :]
    lo, hi = x[..., :half], x[..., half:]
    return torch.cat([lo * c - hi * s, hi * c + lo * s], dim=-1)


def silu(z: torch.Tensor) -> torch.Tensor:
    return z / (1.0 + torch.exp(-z))


class KVCache:
    """Per-layer key/value rows indexed by slot, [n_layers][max_slots, H, dh]."""

    def __init__(self, n_layers, max_slots, n_heads, head_dim, dtype=torch.float64):
        self.k = [torch.zeros(max_slots, n_heads, head_dim, dtype=dtype) for _ in range(n_layers)]
        self.v = [torch.zeros(max_slots, n_heads, head_dim, dtype=dtype) for _ in range(n_layers)]

    def clone(self):
        c = KVCache.__new__(KVCache)
        c.k = [t.clone() for t in self.k]
        c.v = [t.clone() for t in self.v]
        return c


def decoder_layer(w: DecoderWeights, prefix: str, desc, x, pos, slots, visible, cache: KVCache,
                  layer_index: int):
    """One pre-norm decoder layer over T rows.

    x [T, d]; pos [T] RoPE positions; slots [T] cache slots the rows' k, v are written to;
    visible [T, S] boolean: row t may attend cache slot s (evaluated after the write).
    """
    T, d = x.shape
    H, dh = desc.n_heads, desc.head_dim
    S = visible.shape[1]
    xn = rmsnorm(x, w(prefix + "norm1"), desc.rms_eps)
    qkv = xn @ w(prefix + "wqkv").T
    q = rope(qkv[:, :H * dh].reshape(T, H, dh), pos, desc.rope_theta)
    k = rope(qkv[:, H * dh:2 * H * dh].reshape(T, H, dh), pos, desc.rope_theta)
    v = qkv[:, 2 * H * dh:].reshape(T, H, dh)
    K, V = cache.k[layer_index], cache.v[layer_index]
    K[slots] = k
    V[slots] = v
    o = torch.zeros(T, H, dh, dtype=x.dtype)
    for h in range(H):
        scores = (q[:, h, :] @ K[:S, h, :].T) / math.sqrt(dh)          # [T, S]
        scores = scores.masked_fill(~visible, float("-inf"))
        p = torch.exp(scores - scores.max(dim=1, keepdim=True).values)
        p = p / p.sum(dim=1, keepdim=True)
        o[:, h, :] = p @ V[:S, h, :]
    x = x + o.reshape(T, H * dh) @ w(prefix + "wo").T
    xn = rmsnorm(x, w(prefix + "norm2"), desc.rms_eps)
    gu = xn @ w(prefix + "wgu").T
    F = desc.d_ffn
    x = x + (silu(gu[:, :F]) * gu[:, F:]) @ w(prefix + "wd").T
    return x


def target_forward(w: DecoderWeights, desc, x, pos, slots, visible, cache: KVCache):
    """All target layers + final RMSNorm. Returns the features [T, d] (LM-head inputs)."""
    for l in range(desc.n_layers):
        x = decoder_layer(w, f"layers.{l}.", desc, x, pos, slots, visible, cache, l)
    return rmsnorm(x, w("final_norm"), desc.rms_eps)


def lm_head(w: DecoderWeights, features: torch.Tensor, name: str = "lm_head") -> torch.Tensor:
    return features @ w(name).T


def draft_forward(w: DecoderWeights, desc, feat_in, emb_in, pos, slots, visible, cache: KVCache):
    """Draft model M_D (Eq. 2): fc over [feature ; embedding], then one decoder layer.
    The layer output is the predicted next feature and feeds the shared LM head directly."""
    z = torch.cat([feat_in, emb_in], dim=1) @ w("draft.fc").T
    return decoder_layer(w, "draft.layer.", desc, z, pos, slots, visible, cache, 0)


def embed_rows(w: DecoderWeights, embeds: torch.Tensor, token_ids: torch.Tensor) -> torch.Tensor:
    """Input rows: embeds[i] where token_ids[i] < 0, else row token_ids[i] of the embedding."""
    x = embeds.to(device="cpu", dtype=w.dtype).clone()
    E = w("embed")
    ids = token_ids.to("cpu").long()
    sel = ids >= 0
    x[sel] = E[ids[sel]]
    return x


def greedy_token(logits_row: torch.Tensor, desc, action_only: bool) -> int:
    """argmax with ties to the lowest id (Eq. 1), optionally over the action ids only."""
    if action_only:
        a0 = desc.action_base
        return a0 + int(torch.argmax(logits_row[a0:a0 + desc.n_bins]))
    return int(torch.argmax(logits_row))


def top2_margin(logits_row: torch.Tensor, desc, action_only: bool) -> float:
    if action_only:
        logits_row = logits_row[desc.action_base:desc.action_base + desc.n_bins]
    t = torch.topk(logits_row, 2).values
    return float(t[0] - t[1])
