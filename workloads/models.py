"""Model shapes, workload configurations and seeded random-init weights.

The weights are inputs: they are generated once here and the same values are
given to the CPU oracle and to the CUDA library.  Matrices are stored
[out_features, in_features] row-major (y = x @ W^T); the tensor names and their
order are the ones `include/anpd.h` documents for anpd_model_create.
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np
import torch

from .rng import normal_tensor
from .prompts import markov_prompt


@dataclass(frozen=True)
class ModelShape:
    n_layers: int
    d_model: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    d_ffn: int
    vocab: int
    rope_theta: float = 1.0e4
    rms_eps: float = 1.0e-5

    @property
    def streamed_params(self) -> int:
        """Parameters read once per decode step (the embedding table is only gathered)."""
        qkv = (self.n_q_heads + 2 * self.n_kv_heads) * self.head_dim * self.d_model
        o = self.d_model * self.n_q_heads * self.head_dim
        ffn = 3 * self.d_model * self.d_ffn
        return self.n_layers * (qkv + o + ffn) + self.vocab * self.d_model

    @property
    def kv_bytes_per_token(self) -> int:
        return 2 * self.n_layers * self.n_kv_heads * self.head_dim * 2  # bf16 K and V


@dataclass(frozen=True)
class Workload:
    name: str
    shape: ModelShape
    weights_bf16: bool
    weight_seed: int
    prompt_len: int
    markov_order: int
    copy_spans: bool
    max_new: int
    n_max: int
    K: int
    batch: int = 1
    prompt_seed: int = 1000
    n_min: int = 2
    # orbit workloads (workloads/orbit.py): a model whose greedy continuation is known, and a prompt that makes the
    # n-gram drafts right part of the time; orbit_S = 0 means the ordinary random-init model and Markov prompt
    orbit_S: int = 0
    corrupt: float = 0.0


TINY = ModelShape(2, 256, 4, 4, 64, 688, 4096)
S1B = ModelShape(22, 2048, 32, 4, 64, 5632, 32000)
S7B = ModelShape(32, 4096, 32, 32, 128, 11008, 32000)
S13B = ModelShape(40, 5120, 40, 40, 128, 13824, 32000)

WORKLOADS = {
    "C1": Workload("C1", TINY, False, 0, 128, 2, False, 64, 3, 4, 1, 1000),
    "C2": Workload("C2", S1B, True, 1, 512, 3, True, 256, 5, 5, 1, 1001),
    "C3": Workload("C3", S7B, True, 2, 1536, 3, True, 256, 5, 5, 1, 1002),
    # C4 (verify-step microbenchmark) reuses the C3 model; see bench.py
    "C5": Workload("C5", S13B, True, 3, 2048, 3, True, 512, 7, 6, 8, 1004),
    # The 7B shape with a controlled answer (orbit model, same byte traffic as C3): prompts whose n-gram drafts hit about
    # 20 % / 60 % of the time (the paper's case study reports a hit ratio of 20.59 %, Section 4.4).
    "C3-A20": Workload("C3-A20", S7B, True, 2, 1536, 3, False, 256, 5, 5, 1, 1012, orbit_S=4096, corrupt=0.39),
    "C3-A60": Workload("C3-A60", S7B, True, 2, 1536, 3, False, 256, 5, 5, 1, 1013, orbit_S=4096, corrupt=0.15),
    # the same construction at the 1.1B shape and at a size the oracle's full decoder runs in seconds
    "C2-A40": Workload("C2-A40", S1B, True, 1, 512, 3, False, 256, 5, 5, 1, 1014, orbit_S=2048, corrupt=0.25),
    "C1-A50": Workload("C1-A50", TINY, False, 0, 128, 2, False, 64, 3, 4, 1, 1015, orbit_S=256, corrupt=0.2),
    # two layers of the 7B shape: the per-layer kernels of C3 at a size a profiler capture can hold
    "C3-2L": Workload("C3-2L", ModelShape(2, 4096, 32, 32, 128, 11008, 32000), True, 2, 1536, 3, True, 256, 5, 5, 1, 1002),
}

LAYER_TENSORS = ("attn_norm", "wq", "wk", "wv", "wo", "ffn_norm", "w_gate", "w_up", "w_down")


def tensor_shapes(s: ModelShape) -> list[tuple[str, tuple[int, ...]]]:
    """(name, shape) in the order anpd_model_create takes them."""
    out: list[tuple[str, tuple[int, ...]]] = [("embed", (s.vocab, s.d_model))]
    dq, dkv = s.n_q_heads * s.head_dim, s.n_kv_heads * s.head_dim
    for l in range(s.n_layers):
        out += [
            (f"l{l}.attn_norm", (s.d_model,)),
            (f"l{l}.wq", (dq, s.d_model)),
            (f"l{l}.wk", (dkv, s.d_model)),
            (f"l{l}.wv", (dkv, s.d_model)),
            (f"l{l}.wo", (s.d_model, dq)),
            (f"l{l}.ffn_norm", (s.d_model,)),
            (f"l{l}.w_gate", (s.d_ffn, s.d_model)),
            (f"l{l}.w_up", (s.d_ffn, s.d_model)),
            (f"l{l}.w_down", (s.d_model, s.d_ffn)),
        ]
    out += [("final_norm", (s.d_model,)), ("lm_head", (s.vocab, s.d_model))]
    return out


def make_weights(s: ModelShape, seed: int, bf16: bool, device="cpu", std: float = 0.02,
                 norm_gain_jitter: float = 0.0) -> dict[str, torch.Tensor]:
    """Random-init weights: matrices and the embedding ~ N(0, std^2), norm gains 1.

    `bf16=True` rounds the matrices to bf16 (round-to-nearest-even) and returns
    bf16 tensors; norm gains stay fp32.  `norm_gain_jitter` > 0 draws the gains
    from 1 + N(0, jitter^2) instead, for tests that must see the gain applied.
    """
    w: dict[str, torch.Tensor] = {}
    for stream, (name, shape) in enumerate(tensor_shapes(s)):
        n = int(np.prod(shape))
        if len(shape) == 1:
            if norm_gain_jitter > 0.0:
                t = 1.0 + normal_tensor(seed, stream, n, norm_gain_jitter, device)
            else:
                t = torch.ones(n, dtype=torch.float32, device=device)
        else:
            t = normal_tensor(seed, stream, n, std, device).view(shape)
            if bf16:
                t = t.to(torch.bfloat16)
        w[name] = t
    return w


def make_prompts(wl: Workload) -> list[np.ndarray]:
    """One int32 prompt per sequence of the workload's batch."""
    return [markov_prompt(wl.prompt_len, wl.shape.vocab, wl.markov_order,
                          wl.prompt_seed + 7919 * b, copy_spans=wl.copy_spans)
            for b in range(wl.batch)]
