"""Pins for the oracle's decoder forward: independent library implementations and closed forms."""
import math

import pytest
import torch

import synth
from oracle import swift_oracle as so


def _oracle(cfg, weights, dtype=torch.float64, max_positions=128):
    return so.Oracle(so.Shape.of(cfg), weights, dtype=dtype, max_positions=max_positions)


def test_forward_matches_huggingface_llama(small_cfg, small_weights):
    """The paper ran Huggingface's LLaMA (Appendix B.2); the oracle's one-shot forward must equal it.
    Catches a wrong RoPE pairing, eps placement, GQA head mapping, SwiGLU order or a transposed weight."""
    pytest.importorskip("transformers")
    from transformers import LlamaConfig, LlamaForCausalLM
    c = small_cfg
    hf_cfg = LlamaConfig(vocab_size=c.vocab, hidden_size=c.d_model, intermediate_size=c.ffn,
                         num_hidden_layers=c.n_blocks, num_attention_heads=c.n_heads,
                         num_key_value_heads=c.n_kv_heads, head_dim=c.head_dim, rms_norm_eps=c.rms_eps,
                         rope_theta=c.rope_theta, max_position_embeddings=256, attention_bias=False,
                         mlp_bias=False, tie_word_embeddings=False, attn_implementation="eager")
    model = LlamaForCausalLM(hf_cfg).to(torch.float64).eval()
    sd = {"model.embed_tokens.weight": small_weights["embed"], "lm_head.weight": small_weights["lm_head"],
          "model.norm.weight": small_weights["final_norm"]}
    names = {"wq": "self_attn.q_proj", "wk": "self_attn.k_proj", "wv": "self_attn.v_proj",
             "wo": "self_attn.o_proj", "wgate": "mlp.gate_proj", "wup": "mlp.up_proj", "wdown": "mlp.down_proj",
             "attn_norm": "input_layernorm", "mlp_norm": "post_attention_layernorm"}
    for b, wb in enumerate(small_weights["blocks"]):
        for k, v in wb.items():
            sd[f"model.layers.{b}.{names[k]}.weight"] = v
    missing, unexpected = model.load_state_dict({k: v.to(torch.float64) for k, v in sd.items()}, strict=False)
    assert not unexpected and all("rotary" in m or "inv_freq" in m for m in missing), (missing, unexpected)
    toks = synth.prompt(c, 23)
    with torch.no_grad():
        ref = model(torch.tensor([toks])).logits[0]
    got = _oracle(c, small_weights).forward_rows(toks, 0)
    # the library builds its rotary frequency table in fp32, so agreement stops near 1e-6; any
    # structural mistake shows up at the scale of the logits themselves (order 1)
    assert torch.allclose(got, ref, atol=5e-5, rtol=0), float((got - ref).abs().max())


def test_attention_matches_torch_sdpa():
    torch.manual_seed(0)
    M, n, H, Hkv, dh = 5, 19, 6, 2, 8
    q = torch.randn(M, H, dh, dtype=torch.float64)
    K = torch.randn(n, Hkv, dh, dtype=torch.float64)
    V = torch.randn(n, Hkv, dh, dtype=torch.float64)
    allowed = torch.rand(M, n) > 0.3
    allowed[:, 0] = True
    got = so.attention(q, K, V, allowed)
    Kx = K.repeat_interleave(H // Hkv, dim=1)
    Vx = V.repeat_interleave(H // Hkv, dim=1)
    ref = torch.nn.functional.scaled_dot_product_attention(
        q.transpose(0, 1)[None], Kx.transpose(0, 1)[None], Vx.transpose(0, 1)[None], attn_mask=allowed[None, None])
    assert torch.allclose(got, ref[0].transpose(0, 1), atol=1e-12)


def test_attention_single_key_returns_value():
    q = torch.randn(3, 2, 4, dtype=torch.float64)
    K = torch.randn(1, 2, 4, dtype=torch.float64)
    V = torch.randn(1, 2, 4, dtype=torch.float64)
    out = so.attention(q, K, V, torch.ones(3, 1, dtype=torch.bool))
    assert torch.allclose(out, V.expand(3, 2, 4))


def test_rope_depends_on_relative_position_only():
    torch.manual_seed(1)
    q = torch.randn(1, 1, 16, dtype=torch.float64)
    k = torch.randn(1, 1, 16, dtype=torch.float64)

    def score(pq, pk):
        return float((so.rope(q, torch.tensor([pq]), 1e4) * so.rope(k, torch.tensor([pk]), 1e4)).sum())
    assert abs(score(7, 3) - score(104, 100)) < 1e-9
    assert abs(score(7, 3) - score(8, 3)) > 1e-6          # and does depend on the difference
    assert torch.equal(so.rope(q, torch.tensor([0]), 1e4), q)    # position 0 is the identity
    assert abs(float(so.rope(q, torch.tensor([55]), 1e4).norm() - q.norm())) < 1e-12


def test_rope_first_pair_rotates_by_position_radians():
    """theta^0 = 1: dims (0, d_h/2) rotate by exactly `position` radians."""
    x = torch.zeros(1, 1, 8, dtype=torch.float64)
    x[0, 0, 0] = 1.0
    y = so.rope(x, torch.tensor([2]), 1e4)
    assert abs(float(y[0, 0, 0]) - math.cos(2.0)) < 1e-12 and abs(float(y[0, 0, 4]) - math.sin(2.0)) < 1e-12


def test_rmsnorm_closed_form():
    g = torch.tensor([1.0, 2.0, 0.5, 1.0], dtype=torch.float64)
    x = torch.full((1, 4), 3.0, dtype=torch.float64)
    y = so.rmsnorm(x, g, 1e-5)
    assert torch.allclose(y, g * 3.0 / math.sqrt(9.0 + 1e-5))
    x = torch.tensor([[3.0, 4.0, 0.0, 0.0]], dtype=torch.float64)   # mean square = 25/4
    assert torch.allclose(so.rmsnorm(x, torch.ones(4), 0.0), x / 2.5)


def test_swiglu_closed_form():
    g = torch.tensor([0.0, 1.0, -2.0], dtype=torch.float64)
    u = torch.tensor([5.0, 2.0, 3.0], dtype=torch.float64)
    ref = torch.tensor([0.0, 2.0 / (1 + math.exp(-1.0)), -6.0 / (1 + math.exp(2.0))], dtype=torch.float64)
    assert torch.allclose(so.swiglu(g, u), ref)


def test_incremental_rows_equal_one_shot(small_cfg, small_weights):
    """Cached forward, a few rows at a time, equals one causal pass over the whole sequence."""
    toks = synth.prompt(small_cfg, 20)
    ref = _oracle(small_cfg, small_weights).forward_rows(toks, 0)
    o = _oracle(small_cfg, small_weights)
    parts, pos = [], 0
    for m in (7, 1, 4, 1, 1, 6):
        parts.append(o.forward_rows(toks[pos:pos + m], pos))
        pos += m
    assert torch.allclose(torch.cat(parts), ref, atol=1e-10)


def test_skipping_everything_leaves_embedding_to_head(small_cfg, small_weights):
    toks = synth.prompt(small_cfg, 5)
    o = _oracle(small_cfg, small_weights)
    got = o.forward_rows(toks, 0, z=[1] * (2 * small_cfg.n_blocks))
    h = small_weights["embed"][torch.tensor(toks)].double()
    ref = so.rmsnorm(h, small_weights["final_norm"], small_cfg.rms_eps) @ small_weights["lm_head"].double().T
    assert torch.allclose(got, ref, atol=1e-12)


def test_skipped_attention_writes_no_kv(small_cfg, small_weights):
    o = _oracle(small_cfg, small_weights)
    z = [0] * (2 * small_cfg.n_blocks)
    z[2] = 1                                   # attention sub-layer of block 1
    o.forward_rows(synth.prompt(small_cfg, 6), 0, z=z)
    assert float(o.K[1].abs().sum()) == 0.0 and float(o.K[0].abs().sum()) > 0.0


def test_fp32_oracle_close_to_fp64(small_cfg, small_weights):
    toks = synth.prompt(small_cfg, 12)
    a = _oracle(small_cfg, small_weights, torch.float64).forward_rows(toks, 0)
    b = _oracle(small_cfg, small_weights, torch.float32).forward_rows(toks, 0)
    assert float((a - b.double()).abs().max()) < 1e-4 * float(a.std())
