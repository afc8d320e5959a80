"""ORACLE (test infrastructure, not the product): LLaMA-style decoder forward.

The "LLM" of Algorithm 1: LLM(prompt) (prefill) and LLM(drafts) (one forward
over the K+1 tokens of a step against the KV cache, Section 3.1 "Verification").
The paper names only the model family; the internals below are the published
LLaMA architecture (RMSNorm with eps under the root, rotary
embedding with rotate-half pairing, no biases, SwiGLU, untied LM head).

Plain torch CPU ops in a chosen dtype (float64 by default; float32 on request),
no blocking or fusion: one matmul per projection, a softmax per head.  Weights
are inputs; they are used at the values given (an fp32 or bf16 tensor is cast,
exactly, to the compute dtype).  Only tests, the smoke check and the
benchmark's CPU baseline may import this file; it shares no code with the CUDA
library.

Pinned by tests/test_oracle_decoder.py: closed forms (RoPE angle, RMSNorm of a
constant vector, SiLU identity), invariants (cached == uncached, causality,
relative-position property), library routines (scaled_dot_product_attention,
and the whole forward against an independent library LLaMA implementation);
the bf16 cache option by its defining properties (no effect on values that bf16
holds exactly, a bounded effect otherwise, the plain result when switched off).
"""
from __future__ import annotations

import math

import torch


class KVCache:
    """Per layer, the keys and values of the positions consumed so far."""

    def __init__(self, n_layers: int):
        self.k: list[torch.Tensor | None] = [None] * n_layers   # [T, Hkv, hd]
        self.v: list[torch.Tensor | None] = [None] * n_layers
        self.length = 0

    def truncate(self, length: int) -> None:
        """Discard the entries of rejected positions (Section 3.1: tokens that fail
        validation are dropped together with everything after them)."""
        assert 0 <= length <= self.length
        for l in range(len(self.k)):
            if self.k[l] is not None:
                self.k[l] = self.k[l][:length]
                self.v[l] = self.v[l][:length]
        self.length = length


def rms_norm(x: torch.Tensor, gain: torch.Tensor, eps: float) -> torch.Tensor:
    return x * torch.rsqrt(x.pow(2).mean(dim=-1, keepdim=True) + eps) * gain


def rope(x: torch.Tensor, positions: torch.Tensor, theta: float) -> torch.Tensor:
    """Rotary embedding of x [T, H, hd] at absolute `positions` [T].

    Pair (i, i + hd/2) is rotated by the angle pos * theta^(-2i/hd).
    """
    hd = x.shape[-1]
    half = hd // 2
    i = torch.arange(half, dtype=torch.float64)
    inv_freq = theta ** (-2.0 * i / hd)
    ang = positions.to(torch.float64)[:, None] * inv_freq[None, :]      # [T, half]
    cos = torch.cos(ang).to(x.dtype)[:, None, :]
    sin = torch.sin(ang).to(x.dtype)[:, None, :]
    x1, x2 = x[..., :half], x[..., half:]
    return torch.cat([x1 * cos - x2 * sin, x2 * cos + x1 * sin], dim=-1)


def silu(x: torch.Tensor) -> torch.Tensor:
    return x / (1.0 + torch.exp(-x))


def attention(q: torch.Tensor, k: torch.Tensor, v: torch.Tensor, q_positions: torch.Tensor) -> torch.Tensor:
    """q [Tq, Hq, hd]; k, v [Tk, Hkv, hd] for positions 0..Tk-1; query r sees keys <= q_positions[r].

    Grouped-query: query head h reads kv head h // (Hq / Hkv).  Returns [Tq, Hq, hd].
    """
    Tq, Hq, hd = q.shape
    Tk, Hkv, _ = k.shape
    group = Hq // Hkv
    out = torch.empty_like(q)
    key_pos = torch.arange(Tk)
    visible = key_pos[None, :] <= q_positions[:, None]                    # [Tq, Tk]
    for h in range(Hq):
        kh, vh = k[:, h // group, :], v[:, h // group, :]
        s = (q[:, h, :] @ kh.T) / math.sqrt(hd)
        s = s.masked_fill(~visible, float("-inf"))
        p = torch.softmax(s, dim=-1)
        out[:, h, :] = p @ vh
    return out


class Decoder:
    def __init__(self, shape, weights: dict, dtype=torch.float64, kv_dtype=None, keep_cast: bool = False):
        """`shape`: any object with n_layers, d_model, n_q_heads, n_kv_heads, head_dim,
        d_ffn, vocab, rope_theta, rms_eps.  `weights`: name -> tensor, matrices
        stored [out, in].

        `kv_dtype`: storage type of the KV cache.  None keeps keys and values at the compute
        dtype (the plain definition).  The paper does not say how the cache is stored; the
        workloads fix a bf16 cache, and with kv_dtype=torch.bfloat16 every key (after the rotary
        embedding) and value is rounded to bf16 (round to nearest even, from fp32) at the moment
        it enters the cache, the rows of the current call included; everything else is unchanged.

        `keep_cast`: keep each weight's copy in the compute dtype after its first use instead of
        casting it again in every forward (same values, more memory: used when the oracle is timed)."""
        self.s = shape
        self.w = weights
        self.dtype = dtype
        self.kv_dtype = kv_dtype
        self._cast: dict[str, torch.Tensor] | None = {} if keep_cast else None

    def _stored(self, t: torch.Tensor) -> torch.Tensor:
        if self.kv_dtype is None:
            return t
        return t.to(torch.float32).to(self.kv_dtype).to(self.dtype)

    def _w(self, name: str) -> torch.Tensor:
        if self._cast is None:
            return self.w[name].to(self.dtype)
        if name not in self._cast:
            self._cast[name] = self.w[name].to(self.dtype)
        return self._cast[name]

    def new_cache(self) -> KVCache:
        return KVCache(self.s.n_layers)

    def forward(self, tokens, cache: KVCache) -> torch.Tensor:
        """Consume `tokens` at positions cache.length.., append their K/V, return logits [T, V]."""
        s = self.s
        tok = torch.as_tensor(tokens, dtype=torch.long).reshape(-1)
        T = tok.numel()
        pos = torch.arange(cache.length, cache.length + T)
        x = self.w["embed"][tok].to(self.dtype)                            # [T, d]
        for l in range(s.n_layers):
            h = rms_norm(x, self._w(f"l{l}.attn_norm"), s.rms_eps)
            q = (h @ self._w(f"l{l}.wq").T).view(T, s.n_q_heads, s.head_dim)
            k = (h @ self._w(f"l{l}.wk").T).view(T, s.n_kv_heads, s.head_dim)
            v = (h @ self._w(f"l{l}.wv").T).view(T, s.n_kv_heads, s.head_dim)
            q = rope(q, pos, s.rope_theta)
            k = self._stored(rope(k, pos, s.rope_theta))
            v = self._stored(v)
            cache.k[l] = k if cache.k[l] is None else torch.cat([cache.k[l], k], dim=0)
            cache.v[l] = v if cache.v[l] is None else torch.cat([cache.v[l], v], dim=0)
            a = attention(q, cache.k[l], cache.v[l], pos).reshape(T, -1)
            x = x + a @ self._w(f"l{l}.wo").T
            h = rms_norm(x, self._w(f"l{l}.ffn_norm"), s.rms_eps)
            g = silu(h @ self._w(f"l{l}.w_gate").T) * (h @ self._w(f"l{l}.w_up").T)
            x = x + g @ self._w(f"l{l}.w_down").T
        cache.length += T
        h = rms_norm(x, self._w("final_norm"), s.rms_eps)
        return h @ self._w("lm_head").T
