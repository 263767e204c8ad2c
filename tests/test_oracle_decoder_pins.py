"""Pins of the oracle's decoder math against an independent library implementation.

The HuggingFace Llama model (eager attention, float64) is loaded with the same weights and
evaluated (a) under a causal mask and (b) under the draft-tree mask with per-row position
ids, without any KV cache. The oracle must reproduce its logits, which fixes RMSNorm,
rotate-half RoPE, the 1/sqrt(dh) softmax attention, SwiGLU, the LM head, the tree mask,
the tree positions and the cache append in one comparison.

Tolerance 5e-6: the library evaluates the rotary cos/sin tables in float32 whatever the
model dtype (observed difference 1.2e-7); a wrong convention anywhere moves logits by
1e-2 or more.
"""
import pytest
import torch

from oracle import decoder as D
from oracle.specvla import SpecVLAOracle, Tree
from synth_inputs import configs as C, data


def _hf_model(desc, w):
    from transformers import LlamaConfig, LlamaForCausalLM
    cfg = LlamaConfig(vocab_size=desc.vocab, hidden_size=desc.d_model,
                      intermediate_size=desc.d_ffn, num_hidden_layers=desc.n_layers,
                      num_attention_heads=desc.n_heads, num_key_value_heads=desc.n_heads,
                      head_dim=desc.head_dim, rms_norm_eps=desc.rms_eps,
                      rope_theta=desc.rope_theta, max_position_embeddings=1024,
                      attention_bias=False, mlp_bias=False, tie_word_embeddings=False)
    cfg._attn_implementation = "eager"
    m = LlamaForCausalLM(cfg).double().eval()
    hd, F = desc.n_heads * desc.head_dim, desc.d_ffn
    sd = {"model.embed_tokens.weight": w["embed"], "lm_head.weight": w["lm_head"],
          "model.norm.weight": w["final_norm"]}
    for l in range(desc.n_layers):
        p, q = f"model.layers.{l}.", f"layers.{l}."
        sd[p + "self_attn.q_proj.weight"] = w[q + "wqkv"][:hd]
        sd[p + "self_attn.k_proj.weight"] = w[q + "wqkv"][hd:2 * hd]
        sd[p + "self_attn.v_proj.weight"] = w[q + "wqkv"][2 * hd:]
        sd[p + "self_attn.o_proj.weight"] = w[q + "wo"]
        sd[p + "mlp.gate_proj.weight"] = w[q + "wgu"][:F]
        sd[p + "mlp.up_proj.weight"] = w[q + "wgu"][F:]
        sd[p + "mlp.down_proj.weight"] = w[q + "wd"]
        sd[p + "input_layernorm.weight"] = w[q + "norm1"]
        sd[p + "post_attention_layernorm.weight"] = w[q + "norm2"]
    missing = m.load_state_dict({k: v.double() for k, v in sd.items()}, strict=False)
    assert not [k for k in missing.missing_keys if "rotary" not in k], missing
    return m


def _additive(visible):
    mask = torch.zeros(visible.shape, dtype=torch.float64)
    mask[~visible] = torch.finfo(torch.float64).min
    return mask[None, None]


@pytest.fixture(scope="module")
def hf(c0):
    return _hf_model(c0["desc"], c0["weights"])


def test_causal_logits_match_hf_llama(c0, hf):
    orc = c0["make"](action_only=False)
    x = D.embed_rows(orc.w, c0["embeds"], c0["ids"])
    P = x.shape[0]
    ep, logits_last, feats = orc.prefill(c0["embeds"], c0["ids"], want_logits=True)
    with torch.no_grad():
        out = hf(inputs_embeds=x[None], attention_mask=_additive(orc._causal(0, P)),
                 position_ids=torch.arange(P)[None]).logits[0]
    mine = D.lm_head(orc.w, feats)
    assert torch.allclose(mine, out, atol=5e-6, rtol=0)
    assert int(torch.argmax(out[-1])) == ep.root


def test_mask_is_honoured_by_hf(c0, hf):
    """Guard for the pin itself: the library run must depend on the mask we pass."""
    orc = c0["make"]()
    x = D.embed_rows(orc.w, c0["embeds"], c0["ids"])[:8]
    with torch.no_grad():
        a = hf(inputs_embeds=x[None], attention_mask=_additive(orc._causal(0, 8)),
               position_ids=torch.arange(8)[None]).logits[0]
        full = torch.ones(8, 8, dtype=torch.bool)
        b = hf(inputs_embeds=x[None], attention_mask=_additive(full),
               position_ids=torch.arange(8)[None]).logits[0]
    assert (a[0] - b[0]).abs().max() > 1e-3


def test_tree_verify_logits_match_hf_llama(c0, hf):
    desc = c0["desc"]
    orc = c0["make"]()
    ep = orc.prefill(c0["embeds"], c0["ids"])
    P = ep.P
    tok, par, dep = data.random_tree(19, desc, seed=5, max_depth=6, root_token=ep.root)
    tree = Tree(tok, par, dep, [0.0] * len(tok))
    logits, _ = orc.verify_forward(ep, tree)
    T = len(tok)
    x = torch.cat([D.embed_rows(orc.w, c0["embeds"], c0["ids"]), orc._embed(tok)], 0)
    vis = torch.zeros(P + T, P + T, dtype=torch.bool)
    vis[:P, :P] = orc._causal(0, P)
    vis[P:, :] = orc._tree_visible(P, par)
    pos = torch.cat([torch.arange(P), P + torch.tensor(dep)])
    with torch.no_grad():
        out = hf(inputs_embeds=x[None], attention_mask=_additive(vis),
                 position_ids=pos[None]).logits[0]
    assert torch.allclose(logits, out[P:], atol=5e-6, rtol=0)


def test_float32_mode_agrees_with_float64(c0):
    a = c0["make"]()
    b = c0["make"](dtype=torch.float32)
    _, la, _ = a.prefill(c0["embeds"], c0["ids"], want_logits=True)
    _, lb, _ = b.prefill(c0["embeds"], c0["ids"], want_logits=True)
    assert (la - lb.double()).abs().max() < 1e-4
