"""Seeded synthetic prompts: an order-m Markov source with Zipf successors, and
the same source with verbatim copies of earlier spans mixed in.

These stand in for the summarisation / code prompts the paper measures on
(long context, Zipfian token use, repeated names and phrases that an n-gram
module can pick up).  The recipe, not any dataset item, is what is reproduced.
"""
from __future__ import annotations

import bisect
from functools import lru_cache

import numpy as np

from .rng import hash_at, mix64, uniform_at, randint_at, MASK64

_S_FIRST, _S_RANK, _S_COPY, _S_LEN, _S_SRC = 1, 2, 3, 4, 5


@lru_cache(maxsize=8)
def _zipf_cdf(vocab: int, exponent: float) -> np.ndarray:
    w = np.arange(1, vocab + 1, dtype=np.float64) ** (-exponent)
    c = np.cumsum(w)
    return c / c[-1]


def _successor(seed: int, state: tuple, rank: int, vocab: int) -> int:
    """Token that holds rank `rank` among the successors of `state`.

    Each state has its own fixed ranking: the token is a hash of
    (seed, state, rank), so low ranks (the likely ones under Zipf) always map
    to the same few tokens for a given state.
    """
    z = mix64(seed ^ 0xA5A5A5A55A5A5A5A)
    for s in state:
        z = mix64((z + s + 1) & MASK64)
    return mix64((z + rank * 0x9E3779B97F4A7C15) & MASK64) % vocab


def markov_prompt(length: int, vocab: int, order: int, seed: int,
                  zipf_exponent: float = 1.1, copy_spans: bool = False,
                  copy_start: int = 64, copy_prob: float = 1.0 / 61.0,
                  copy_min: int = 8, copy_max: int = 32) -> np.ndarray:
    """int32[length] token ids.

    Without `copy_spans`: the first `order` tokens are uniform, each later
    token is the rank-r successor of the previous `order` tokens with
    P(r) ~ r^-zipf_exponent over r in [1, vocab].

    With `copy_spans`: at every position t >= copy_start a copy of l ~ U{copy_min
    ..copy_max} tokens starting at a uniform earlier offset begins with
    probability copy_prob (E[l] = 20 and copy_prob = 1/61 give an expected
    copied fraction of 25 %); otherwise one Markov token is emitted.
    """
    cdf = _zipf_cdf(vocab, zipf_exponent)
    out: list[int] = []
    draw = 0
    while len(out) < length:
        t = len(out)
        if t < order:
            out.append(randint_at(seed, _S_FIRST, t, 0, vocab - 1))
            continue
        if copy_spans and t >= copy_start:
            u = uniform_at(seed, _S_COPY, draw)
            if u < copy_prob:
                span = randint_at(seed, _S_LEN, draw, copy_min, copy_max)
                src = randint_at(seed, _S_SRC, draw, 0, t - span)
                draw += 1
                # token-by-token so a span may overlap its own output, as a
                # repeated phrase would
                for i in range(span):
                    if len(out) < length:
                        out.append(out[src + i])
                continue
        u = uniform_at(seed, _S_RANK, draw)
        draw += 1
        rank = bisect.bisect_right(cdf, u) + 1
        rank = min(rank, vocab)
        out.append(_successor(seed, tuple(out[t - order:t]), rank, vocab))
    return np.asarray(out[:length], dtype=np.int32)


def periodic_prompt(length: int, period: int, vocab: int, seed: int) -> np.ndarray:
    """`period` distinct tokens repeated: every n-gram query has one answer."""
    assert period <= vocab
    base: list[int] = []
    i = 0
    while len(base) < period:
        tok = hash_at(seed, _S_FIRST, i) % vocab
        i += 1
        if tok not in base:
            base.append(tok)
    return np.asarray([base[t % period] for t in range(length)], dtype=np.int32)
