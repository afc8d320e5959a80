"""GPU MLN tables and drafts against the oracle: bit-exact."""
import random

import numpy as np
import pytest

from helpers import require_gpu
from oracle.mln import MLN
from workloads import WORKLOADS, make_prompts, markov_prompt, periodic_prompt

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def A():
    require_gpu()
    from paper_2404_08698_b200 import binding
    return binding


def compare_all(A, ctx, mln, n_min, n_max):
    for n in range(n_min, n_max + 1):
        assert A.anpd_ngram_dump(ctx, n) == mln.dump(n), f"level {n} records"
        got = [(k, s) for k, s, _, _ in A.anpd_ngram_dump_best(ctx, n)]
        assert got == mln.dump_best(n), f"level {n} best successors"
    for K in range(0, 8):
        assert A.anpd_ngram_draft(ctx, K) == mln.draft(K), f"draft K={K}"


@pytest.mark.parametrize("policy", [0, 1])
@pytest.mark.parametrize("seed", range(4))
def test_random_sequences_bulk_and_incremental(A, seed, policy):
    rng = random.Random(seed)
    V = rng.choice([2, 3, 7, 50])
    n_max = rng.randint(2, 8)
    T = rng.randint(1, 300)
    toks = [rng.randrange(V) for _ in range(T)]
    ctx = A.anpd_ngram_create(2, n_max, 512, policy)
    mln = MLN(2, n_max, policy)
    try:
        cut = rng.randint(0, T)
        if cut:
            A.anpd_ngram_update(ctx, toks[:cut])      # Initialize: one parallel fold
        mln.initialize(toks[:cut])
        if cut:
            compare_all(A, ctx, mln, 2, n_max)
        i = cut
        while i < T:                                   # Update: a few tokens at a time
            step = min(rng.randint(1, 8), T - i)
            A.anpd_ngram_update(ctx, toks[i:i + step])
            for t in toks[i:i + step]:
                mln.update(t)
            i += step
        assert A.anpd_ngram_len(ctx) == T
        compare_all(A, ctx, mln, 2, n_max)
        A.anpd_ngram_reset(ctx)
        assert A.anpd_ngram_len(ctx) == 0 and A.anpd_ngram_dump(ctx, 2) == []
    finally:
        A.anpd_ngram_destroy(ctx)


@pytest.mark.parametrize("name", ["C1", "C2", "C5"])
def test_workload_prompts(A, name):
    wl = WORKLOADS[name]
    prompt = make_prompts(wl)[0].tolist()
    ctx = A.anpd_ngram_create(wl.n_min, wl.n_max, wl.prompt_len + wl.max_new + 8)
    mln = MLN(wl.n_min, wl.n_max)
    try:
        A.anpd_ngram_update(ctx, prompt)
        mln.initialize(prompt)
        compare_all(A, ctx, mln, wl.n_min, wl.n_max)
    finally:
        A.anpd_ngram_destroy(ctx)


def test_periodic_and_distinct_closed_forms(A):
    p = periodic_prompt(40, 5, 1000, 3).tolist()
    ctx = A.anpd_ngram_create(2, 4, 64)
    try:
        A.anpd_ngram_update(ctx, p)
        assert A.anpd_ngram_draft(ctx, 7) == [p[(40 + i) % 5] for i in range(7)]
        A.anpd_ngram_reset(ctx)
        A.anpd_ngram_update(ctx, list(range(100, 140)))
        assert A.anpd_ngram_draft(ctx, 7) == []
    finally:
        A.anpd_ngram_destroy(ctx)


def test_n_min_above_two_is_a_single_level(A):
    toks = markov_prompt(200, 16, 2, 5).tolist()
    ctx = A.anpd_ngram_create(3, 3, 256)
    mln = MLN(3, 3)
    try:
        A.anpd_ngram_update(ctx, toks)
        mln.initialize(toks)
        compare_all(A, ctx, mln, 3, 3)
    finally:
        A.anpd_ngram_destroy(ctx)


def test_error_paths(A):
    ctx = A.anpd_ngram_create(2, 3, 16)
    try:
        with pytest.raises(A.AnpdError) as e:
            A.anpd_ngram_draft(ctx, 3)                  # nothing committed yet
        assert e.value.status == A.ERR_STATE
        A.anpd_ngram_update(ctx, list(range(10)))
        with pytest.raises(A.AnpdError) as e:
            A.anpd_ngram_update(ctx, list(range(7)))    # 17 > max_ctx
        assert e.value.status == A.ERR_CAPACITY
        assert A.anpd_ngram_len(ctx) == 10              # nothing changed
        with pytest.raises(A.AnpdError) as e:
            A.anpd_ngram_update(ctx, [-1])
        assert e.value.status == A.ERR_RANGE
        with pytest.raises(A.AnpdError) as e:
            A.anpd_ngram_draft(ctx, 8)
        assert e.value.status == A.ERR_RANGE
        A.anpd_ngram_update(ctx, list(range(10, 16)))   # exactly full
        assert A.anpd_ngram_len(ctx) == 16
    finally:
        A.anpd_ngram_destroy(ctx)
