"""Shared set-up for the GPU parity tests (no arithmetic of the method here)."""
from __future__ import annotations

import numpy as np
import torch

from workloads import tensor_shapes


def require_gpu():
    import pytest
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    from paper_2404_08698_b200 import build
    build.build()


def gpu_model(A, shape, weights, stream: int = 0) -> int:
    return A.anpd_model_create(shape, [weights[n] for n, _ in tensor_shapes(shape)], stream)


def as_bf16_values(weights: dict) -> dict:
    """The weights at the values the library computes with: matrices rounded to bf16."""
    return {k: (v.to(torch.bfloat16).to(torch.float32) if v.dim() == 2 else v.to(torch.float32)).cpu()
            for k, v in weights.items()}


def top2_margin(logits_row: torch.Tensor) -> float:
    t = torch.topk(logits_row, 2).values
    return float(t[0] - t[1])


def oracle_greedy_with_margins(dec, prompt, max_new):
    """Oracle greedy tokens and, per generated token, the top-2 logit margin that decided it."""
    from oracle.anpd import argmax_lowest
    cache = dec.new_cache()
    logits = dec.forward(list(prompt), cache)
    toks, margins = [argmax_lowest(logits[-1])], [top2_margin(logits[-1])]
    while len(toks) < max_new:
        logits = dec.forward([toks[-1]], cache)
        toks.append(argmax_lowest(logits[-1]))
        margins.append(top2_margin(logits[-1]))
    return toks, margins


def agree_until_low_margin(got, want, margins, min_margin=5e-2) -> int:
    """Asserts got[i] == want[i] up to the first position whose deciding margin is below
    min_margin (beyond it a rounding difference may legitimately change the stream).
    Returns the number of positions checked."""
    n = 0
    for g, w, mg in zip(got, want, margins):
        if mg <= min_margin:
            break
        assert int(g) == int(w), f"token {n}: got {g}, oracle {w}, margin {mg}"
        n += 1
    return n
