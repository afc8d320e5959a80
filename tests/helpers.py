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


_streams = []


def new_stream() -> int:
    """A non-default CUDA stream handle (steps on such a stream run as replayed CUDA graphs)."""
    st = torch.cuda.Stream()
    _streams.append(st)
    return st.cuda_stream


def gpu_model(A, shape, weights, stream: int = 0) -> int:
    return A.anpd_model_create(shape, [weights[n] for n, _ in tensor_shapes(shape)], stream)


def as_bf16_values(weights: dict) -> dict:
    """The weights at the values the library computes with: matrices rounded to bf16."""
    return {k: (v.to(torch.bfloat16).to(torch.float32) if v.dim() == 2 else v.to(torch.float32)).cpu()
            for k, v in weights.items()}


def top2_margin(logits_row: torch.Tensor) -> float:
    t = torch.topk(logits_row, 2).values
    return float(t[0] - t[1])


def check_stream_against_oracle(dec, prompt, got, min_margin=5e-2) -> int:
    """Teacher-forced comparison of a generated token stream with the oracle: the oracle
    consumes the prompt and then the stream itself, and at every position whose top-2 logit
    margin exceeds min_margin its argmax must be the stream's token (below the margin a
    rounding difference may legitimately pick the other candidate).  Returns the number of
    positions that were decided by a large enough margin."""
    from oracle.anpd import argmax_lowest
    cache = dec.new_cache()
    logits = dec.forward(list(prompt), cache)
    checked = 0
    for i, tok in enumerate(got):
        if top2_margin(logits[-1]) > min_margin:
            want = argmax_lowest(logits[-1])
            assert int(tok) == want, f"token {i}: got {int(tok)}, oracle {want}, margin {top2_margin(logits[-1])}"
            checked += 1
        logits = dec.forward([int(tok)], cache)
    return checked
