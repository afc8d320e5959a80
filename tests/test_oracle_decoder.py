"""Pins for oracle/decoder.py: closed forms, invariants, and library routines
that implement the same published architecture independently."""
import math

import pytest
import torch

from oracle.decoder import Decoder, KVCache, attention, rms_norm, rope, silu
from workloads import ModelShape, make_weights

SMALL = ModelShape(2, 32, 4, 2, 8, 48, 64)


def small_model(dtype=torch.float64, seed=3, jitter=0.1, std=0.3):
    w = make_weights(SMALL, seed, False, std=std, norm_gain_jitter=jitter)
    return Decoder(SMALL, w, dtype), w


# ---- RoPE ---------------------------------------------------------------
def test_rope_closed_form_angle():
    # hd = 2: one pair rotated by pos * theta^0 = pos radians; (1,0) -> (cos p, sin p)
    x = torch.tensor([[[1.0, 0.0]], [[0.0, 1.0]]], dtype=torch.float64)
    y = rope(x, torch.tensor([2, 3]), 1e4)
    assert torch.allclose(y[0, 0], torch.tensor([math.cos(2.0), math.sin(2.0)], dtype=torch.float64))
    assert torch.allclose(y[1, 0], torch.tensor([-math.sin(3.0), math.cos(3.0)], dtype=torch.float64))


def test_rope_pairing_and_frequencies():
    # hd = 4, theta = 100: pairs (0,2) and (1,3); second pair turns at 100^(-2/4) = 0.1 rad per position
    x = torch.zeros(1, 1, 4, dtype=torch.float64)
    x[0, 0, 1] = 1.0
    y = rope(x, torch.tensor([5]), 100.0)
    assert torch.allclose(y[0, 0], torch.tensor([0.0, math.cos(0.5), 0.0, math.sin(0.5)], dtype=torch.float64))


def test_rope_identity_at_zero_norm_and_relative_property():
    g = torch.Generator().manual_seed(0)
    q = torch.randn(1, 3, 16, generator=g, dtype=torch.float64)
    k = torch.randn(1, 3, 16, generator=g, dtype=torch.float64)
    assert torch.equal(rope(q, torch.tensor([0]), 1e4), q)
    for p in (1, 17, 4095):
        assert torch.allclose(rope(q, torch.tensor([p]), 1e4).norm(dim=-1), q.norm(dim=-1))
    # <R_m q, R_n k> depends on m - n only
    def dot(m, n):
        return (rope(q, torch.tensor([m]), 1e4) * rope(k, torch.tensor([n]), 1e4)).sum(-1)
    assert torch.allclose(dot(9, 4), dot(105, 100), atol=1e-10)
    assert not torch.allclose(dot(9, 4), dot(9, 5), atol=1e-3)


# ---- RMSNorm, SiLU -----------------------------------------------------
def test_rmsnorm_constant_vector_and_scale_invariance():
    g = torch.linspace(0.5, 1.5, 8, dtype=torch.float64)
    for c in (3.0, -0.25):
        y = rms_norm(torch.full((1, 8), c, dtype=torch.float64), g, 0.0)
        assert torch.allclose(y[0], math.copysign(1.0, c) * g)
    x = torch.randn(4, 8, dtype=torch.float64)
    assert torch.allclose(rms_norm(7.0 * x, g, 0.0), rms_norm(x, g, 0.0))
    # eps enters under the root: x = (2,0,0,0), mean square 1, eps 3 -> 2 / sqrt(4) = 1
    y = rms_norm(torch.tensor([[2.0, 0, 0, 0]], dtype=torch.float64), torch.ones(4, dtype=torch.float64), 3.0)
    assert torch.allclose(y, torch.tensor([[1.0, 0, 0, 0]], dtype=torch.float64))


def test_silu_identities():
    x = torch.linspace(-6, 6, 25, dtype=torch.float64)
    assert torch.allclose(silu(x) - silu(-x), x)            # x*s(x) + x*s(-x) = x
    assert float(silu(torch.tensor(0.0))) == 0.0
    assert abs(float(silu(torch.tensor(1.0, dtype=torch.float64))) - 1.0 / (1.0 + math.exp(-1.0))) < 1e-15
    assert torch.allclose(silu(x), torch.nn.functional.silu(x))


# ---- attention -----------------------------------------------------------
def test_attention_single_key_and_uniform_scores():
    v = torch.randn(5, 1, 4, dtype=torch.float64)
    k = torch.zeros(5, 1, 4, dtype=torch.float64)            # all scores 0 -> uniform weights
    q = torch.randn(5, 2, 4, dtype=torch.float64)
    out = attention(q, k, v, torch.arange(5))
    for r in range(5):
        want = v[:r + 1, 0].mean(dim=0)
        assert torch.allclose(out[r, 0], want) and torch.allclose(out[r, 1], want)


def test_attention_matches_library_sdpa_with_gqa_and_offset():
    g = torch.Generator().manual_seed(1)
    Tk, Tq, Hq, Hkv, hd = 11, 3, 4, 2, 8
    q = torch.randn(Tq, Hq, hd, generator=g, dtype=torch.float64)
    k = torch.randn(Tk, Hkv, hd, generator=g, dtype=torch.float64)
    v = torch.randn(Tk, Hkv, hd, generator=g, dtype=torch.float64)
    pos = torch.arange(Tk - Tq, Tk)
    mine = attention(q, k, v, pos)
    mask = torch.arange(Tk)[None, :] <= pos[:, None]
    kk = k.repeat_interleave(Hq // Hkv, dim=1)
    vv = v.repeat_interleave(Hq // Hkv, dim=1)
    lib = torch.nn.functional.scaled_dot_product_attention(
        q.transpose(0, 1)[None], kk.transpose(0, 1)[None], vv.transpose(0, 1)[None], attn_mask=mask[None, None])
    assert torch.allclose(mine, lib[0].transpose(0, 1), atol=1e-12)


# ---- whole forward ---------------------------------------------------------
def test_cached_incremental_equals_full_recompute_and_widths():
    dec, _ = small_model()
    toks = [5, 9, 9, 1, 33, 7, 2, 60, 5, 9]
    full = dec.forward(toks, dec.new_cache())
    c = dec.new_cache()
    parts = [dec.forward(toks[:4], c), dec.forward(toks[4:5], c), dec.forward(toks[5:], c)]
    assert c.length == len(toks)
    assert torch.allclose(torch.cat(parts), full, atol=1e-10)
    # truncate then recompute = never having consumed the dropped tokens
    c.truncate(6)
    again = dec.forward(toks[6:], c)
    assert torch.allclose(again, full[6:], atol=1e-10)


def test_causality():
    dec, _ = small_model()
    a = dec.forward([3, 4, 5, 6], dec.new_cache())
    b = dec.forward([3, 4, 50, 60], dec.new_cache())
    assert torch.allclose(a[:2], b[:2], atol=1e-12) and not torch.allclose(a[2:], b[2:], atol=1e-3)


def test_zero_output_projections_reduce_to_embedding_readout():
    dec, w = small_model(jitter=0.0)
    for l in range(SMALL.n_layers):
        w[f"l{l}.wo"].zero_()
        w[f"l{l}.w_down"].zero_()
    toks = [1, 2, 3]
    logits = dec.forward(toks, dec.new_cache())
    e = w["embed"][toks].double()
    h = e / torch.sqrt((e * e).mean(-1, keepdim=True) + SMALL.rms_eps)
    assert torch.allclose(logits, h @ w["lm_head"].double().T, atol=1e-12)


def test_whole_forward_matches_library_llama():
    tr = pytest.importorskip("transformers")
    cfg = tr.LlamaConfig(vocab_size=SMALL.vocab, hidden_size=SMALL.d_model, intermediate_size=SMALL.d_ffn,
                         num_hidden_layers=SMALL.n_layers, num_attention_heads=SMALL.n_q_heads,
                         num_key_value_heads=SMALL.n_kv_heads, head_dim=SMALL.head_dim,
                         rms_norm_eps=SMALL.rms_eps, rope_theta=SMALL.rope_theta, tie_word_embeddings=False,
                         attention_bias=False, mlp_bias=False, max_position_embeddings=128)
    cfg._attn_implementation = "eager"
    lib = tr.LlamaForCausalLM(cfg).double().eval()
    dec, w = small_model()
    names = {"embed": "model.embed_tokens.weight", "final_norm": "model.norm.weight", "lm_head": "lm_head.weight"}
    per_layer = {"attn_norm": "input_layernorm", "wq": "self_attn.q_proj", "wk": "self_attn.k_proj",
                 "wv": "self_attn.v_proj", "wo": "self_attn.o_proj", "ffn_norm": "post_attention_layernorm",
                 "w_gate": "mlp.gate_proj", "w_up": "mlp.up_proj", "w_down": "mlp.down_proj"}
    sd = {v: w[k].double() for k, v in names.items()}
    for l in range(SMALL.n_layers):
        for k, v in per_layer.items():
            sd[f"model.layers.{l}.{v}.weight"] = w[f"l{l}.{k}"].double()
    missing = lib.load_state_dict(sd, strict=False)
    assert not [m for m in missing.missing_keys if "rotary" not in m]
    toks = [5, 9, 9, 1, 33, 7, 2, 60, 5, 9, 0, 63]
    with torch.no_grad():
        want = lib(torch.tensor([toks])).logits[0]
    got = dec.forward(toks, dec.new_cache())
    # the library keeps its rotary cos/sin tables in fp32, hence 1e-5 and not 1e-12;
    # any structural mistake (pairing, transposed weight, missing norm) shows as O(0.1-1)
    assert torch.allclose(got, want, atol=1e-5), float((got - want).abs().max())


def test_float32_mode_close_to_float64():
    d64, w = small_model()
    d32 = Decoder(SMALL, w, torch.float32)
    toks = [5, 9, 9, 1, 33, 7, 2, 60]
    a, b = d64.forward(toks, d64.new_cache()), d32.forward(toks, d32.new_cache())
    assert b.dtype == torch.float32 and float((a - b.double()).abs().max()) < 1e-4


# ---- bf16 storage of the KV cache (fixed by the workloads, not by the paper) ----
def _is_bf16_valued(t: torch.Tensor) -> bool:
    return bool(torch.equal(t.to(torch.float32).to(torch.bfloat16).to(t.dtype), t))


def test_bf16_cache_option_stores_bf16_values_and_changes_nothing_else():
    dec, w = small_model()
    dec16 = Decoder(SMALL, w, torch.float64, kv_dtype=torch.bfloat16)
    toks = [3, 17, 5, 40, 9, 22]
    c0, c1 = dec.new_cache(), dec16.new_cache()
    l0, l1 = dec.forward(toks, c0), dec16.forward(toks, c1)
    for l in range(SMALL.n_layers):
        assert _is_bf16_valued(c1.k[l]) and _is_bf16_valued(c1.v[l])
        assert not _is_bf16_valued(c0.k[l])                       # the plain cache keeps full precision
    # layer 0 sees the same inputs in both runs: its stored keys are the plain keys, rounded
    assert torch.equal(c1.k[0], c0.k[0].to(torch.float32).to(torch.bfloat16).to(torch.float64))
    assert torch.equal(c1.v[0], c0.v[0].to(torch.float32).to(torch.bfloat16).to(torch.float64))
    # a perturbation of relative size 2^-9 per cached element: small but not zero
    d = float((l0 - l1).abs().max())
    assert 0.0 < d < 0.05 * float(l0.abs().max())
    # switched off it is the plain forward
    assert torch.equal(Decoder(SMALL, w, torch.float64, kv_dtype=None).forward(toks, dec.new_cache()), l0)


def test_bf16_cache_incremental_equals_full():
    _, w = small_model()
    dec16 = Decoder(SMALL, w, torch.float64, kv_dtype=torch.bfloat16)
    toks = [1, 2, 3, 4, 5, 6, 7]
    full = dec16.forward(toks, dec16.new_cache())
    c = dec16.new_cache()
    a = dec16.forward(toks[:4], c)
    b = dec16.forward(toks[4:], c)
    assert torch.allclose(torch.cat([a, b]), full, atol=1e-12, rtol=0)


def test_keep_cast_changes_no_value():
    # casting each weight once and keeping the copy is the same arithmetic on the same values
    w = make_weights(SMALL, 5, True, std=0.3)                       # bf16 matrices: a real cast happens
    toks = [3, 9, 27, 5, 1]
    for dtype in (torch.float32, torch.float64):
        a, b = Decoder(SMALL, w, dtype), Decoder(SMALL, w, dtype, keep_cast=True)
        ca, cb = a.new_cache(), b.new_cache()
        for chunk in (toks[:3], toks[3:]):                          # second call uses the kept copies
            assert torch.equal(a.forward(chunk, ca), b.forward(chunk, cb))
