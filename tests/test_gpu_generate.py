"""Algorithm 1 on the GPU: the ANPD token stream is bit-identical to the same library's greedy
stream (losslessness), agrees with the oracle's greedy stream wherever the oracle's deciding
margin is large enough, and its per-step drafts / accepted lengths follow the oracle's."""
import numpy as np
import pytest
import torch

from helpers import as_bf16_values, check_stream_against_oracle, gpu_model, new_stream, require_gpu, top2_margin
from oracle.anpd import argmax_lowest, verify as oracle_verify
from oracle.decoder import Decoder
from oracle.mln import MLN
from workloads import WORKLOADS, ModelShape, make_prompts, make_weights, markov_prompt, periodic_prompt

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def A():
    require_gpu()
    from paper_2404_08698_b200 import binding
    return binding


@pytest.fixture(scope="module")
def c1(A):
    wl = WORKLOADS["C1"]
    w = make_weights(wl.shape, wl.weight_seed, wl.weights_bf16)
    st = new_stream()                                   # a real stream: the loop replays CUDA graphs
    m = gpu_model(A, wl.shape, w, st)
    kv = A.anpd_kv_create(m, 512)
    yield wl, w, m, kv, st
    A.anpd_kv_destroy(kv)
    A.anpd_model_destroy(m)


def test_c1_anpd_equals_greedy_equals_oracle(A, c1):
    wl, w, m, kv, st = c1
    prompt = make_prompts(wl)[0]
    ctx = A.anpd_ngram_create(wl.n_min, wl.n_max, 512, 0, st)
    try:
        out, st = A.anpd_generate(m, kv, ctx, prompt, wl.max_new, wl.K)
        ref, st0 = A.anpd_generate(m, kv, ctx, prompt, wl.max_new, 0)
        assert np.array_equal(out, ref)                                 # losslessness, bit for bit
        assert st0["steps"] == wl.max_new and st0["drafted"] == 0
        # progress: each step commits 1..K+1 tokens; generated = steps + accepted
        assert st["generated"] == st["steps"] + st["accepted"] and st["generated"] >= wl.max_new
        assert sum(st["hist_accepted"]) == st["steps"] and sum(st["hist_accepted"][wl.K + 1:]) == 0
        assert st["accepted"] == sum(i * h for i, h in enumerate(st["hist_accepted"]))
        dec = Decoder(wl.shape, as_bf16_values(w), torch.float64)
        n = check_stream_against_oracle(dec, prompt.tolist(), ref.tolist())
        assert n >= wl.max_new // 5, n
    finally:
        A.anpd_ngram_destroy(ctx)


def test_algorithm1_step_by_step_from_the_boundary_calls(A, c1):
    """Algorithm 1 driven from the host through anpd_ngram_update -> anpd_ngram_draft -> anpd_verify, compared
    with the oracle at EVERY step: the draft bit for bit, the accepted length and the next token wherever every
    logit row that decides them has a top-2 margin above 5e-2 in the oracle.  Where a decision falls under the
    margin and the two sides differ, the oracle is put on the library's path (its cache rolled back or extended
    to the library's accepted length), so that all later steps are compared too."""
    wl, w, m, kv, st = c1
    prompt = make_prompts(wl)[0].tolist()
    K, M, MARGIN = wl.K, wl.max_new, 5e-2
    dec = Decoder(wl.shape, as_bf16_values(w), torch.float64)
    ctx = A.anpd_ngram_create(wl.n_min, wl.n_max, 512, 0, st)
    try:
        A.anpd_kv_truncate(kv, 0, 0)
        mln = MLN(wl.n_min, wl.n_max)
        mln.initialize(prompt)
        A.anpd_ngram_update(ctx, prompt)
        cache = dec.new_cache()
        logits = dec.forward(prompt, cache)
        confirmed = A.anpd_prefill(m, kv, prompt)
        if top2_margin(logits[-1]) > MARGIN:
            assert confirmed == argmax_lowest(logits[-1])
        out, steps, decided, accepted_total = [], 0, 0, 0
        while len(out) < M:
            out.append(confirmed)
            mln.update(confirmed)
            A.anpd_ngram_update(ctx, [confirmed])
            want_draft = mln.draft(K)
            draft = A.anpd_ngram_draft(ctx, K)
            assert draft == want_draft, (steps, draft, want_draft)                  # bit-exact, every step
            P = cache.length
            a_o, nxt_o, preds, lg = oracle_verify(dec, cache, confirmed, draft)
            a, nxt = A.anpd_verify(m, kv, confirmed, draft)
            assert A.anpd_kv_len(kv) == P + a + 1
            # rows 0..min(a, a_o) decide the accepted length; row a decides the next token
            rows = range(min(a, a_o) + 1)
            clear = all(top2_margin(lg[r]) > MARGIN for r in rows)
            if clear:
                assert a == a_o and nxt == nxt_o, (steps, a, a_o, nxt, nxt_o)
                decided += 1
            if a != a_o:                                                           # only possible under the margin
                if a > a_o:
                    dec.forward(draft[a_o:a], cache)
                else:
                    cache.truncate(P + a + 1)
            assert cache.length == P + a + 1
            for t in draft[:a]:
                out.append(t)
                mln.update(t)
            if a:
                A.anpd_ngram_update(ctx, draft[:a])
            accepted_total += a
            confirmed = nxt
            steps += 1
        assert decided >= 8, (decided, steps)          # steps whose every deciding row cleared the margin
        assert accepted_total > 0
        # the library's own loop takes the same steps
        got, gst = A.anpd_generate(m, kv, ctx, prompt, M, K)
        assert got.tolist() == out[:M]
        assert gst["steps"] == steps and gst["accepted"] == accepted_total
    finally:
        A.anpd_ngram_destroy(ctx)


def test_tables_after_generate_match_oracle_on_the_generated_stream(A, c1):
    wl, w, m, kv, st = c1
    prompt = make_prompts(wl)[0]
    ctx = A.anpd_ngram_create(2, 4, 512, 0, st)
    try:
        ref, _ = A.anpd_generate(m, kv, ctx, prompt, 48, 0)             # greedy, a little longer
        out, st = A.anpd_generate(m, kv, ctx, prompt, 40, 5)
        assert np.array_equal(out, ref[:40])
        n_ctx = A.anpd_ngram_len(ctx)
        # the context also holds the token confirmed by the last step, which Algorithm 1 would
        # only move to the output at the top of its next iteration
        assert n_ctx == len(prompt) + st["generated"] + 1 and 40 <= st["generated"] <= 45
        assert A.anpd_kv_len(kv) == n_ctx - 1                           # the last token is not in the cache yet
        # the loop may overshoot max_new; by losslessness the context holds the greedy stream
        committed = prompt.tolist() + ref[:st["generated"] + 1].tolist()
        assert A.anpd_ngram_draft(ctx, 0) == []                         # folds the last step's tokens
        mln = MLN(2, 4)
        mln.initialize(committed)
        for n in (2, 3, 4):
            assert A.anpd_ngram_dump(ctx, n) == mln.dump(n)
        assert A.anpd_ngram_draft(ctx, 5) == mln.draft(5)
    finally:
        A.anpd_ngram_destroy(ctx)


@pytest.mark.parametrize("K,N,policy", [(1, 2, 0), (3, 2, 1), (5, 5, 0), (7, 8, 0), (7, 3, 1), (2, 6, 0)])
def test_losslessness_over_K_N_policy(A, K, N, policy):
    shape = ModelShape(2, 128, 4, 2, 64, 200, 300)
    w = make_weights(shape, 21, False, std=0.08)
    m = gpu_model(A, shape, w)
    kv = A.anpd_kv_create(m, 256)
    ctx = A.anpd_ngram_create(2, N, 256, policy)
    try:
        base = periodic_prompt(30, 6, shape.vocab, 4)
        prompt = np.concatenate([base, markov_prompt(30, shape.vocab, 2, 8), base[:13]])
        ref, _ = A.anpd_generate(m, kv, ctx, prompt, 48, 0)
        out, st = A.anpd_generate(m, kv, ctx, prompt, 48, K)
        assert np.array_equal(out, ref)
        assert st["generated"] == st["steps"] + st["accepted"]
        assert st["drafted"] <= K * st["steps"]
    finally:
        A.anpd_ngram_destroy(ctx)
        A.anpd_kv_destroy(kv)
        A.anpd_model_destroy(m)


def test_cyclic_copy_model_accepts_every_draft(A):
    """A decoder whose attention and FFN outputs are zero and whose LM head reads the embedding of
    the successor in a fixed cycle: greedy output is that cycle (closed form), and once a period has
    been seen every draft is accepted."""
    V, d = 16, 64
    shape = ModelShape(1, d, 1, 1, 64, 64, V)
    w = make_weights(shape, 3, False, std=0.05)
    w["l0.wo"].zero_()
    w["l0.w_down"].zero_()
    e = torch.zeros(V, d)
    for t in range(V):
        e[t, t] = 1.0
    w["embed"] = e
    perm = [(t + 1) % 5 if t < 5 else 0 for t in range(V)]               # cycle 0 1 2 3 4
    lm = torch.zeros(V, d)
    for t in range(V):
        lm[perm[t], t] = 1.0                                             # logits[perm[t]] = h[t]
    w["lm_head"] = lm
    m = gpu_model(A, shape, w)
    kv = A.anpd_kv_create(m, 256)
    ctx = A.anpd_ngram_create(2, 3, 256)
    try:
        prompt = [t % 5 for t in range(12)]
        K, M = 4, 40
        out, st = A.anpd_generate(m, kv, ctx, prompt, M, K)
        assert out.tolist() == [(12 + i) % 5 for i in range(M)]
        assert st["hist_accepted"][K] == st["steps"] and st["steps"] == -(-M // (K + 1))
    finally:
        A.anpd_ngram_destroy(ctx)
        A.anpd_kv_destroy(kv)
        A.anpd_model_destroy(m)


def test_batch_equals_independent_runs(A):
    shape = ModelShape(2, 128, 4, 4, 64, 200, 300)
    w = make_weights(shape, 9, False, std=0.08)
    st = new_stream()
    m = gpu_model(A, shape, w, st)
    B, plen, M, K = 3, 70, 30, 4
    prompts = np.stack([np.concatenate([markov_prompt(35, shape.vocab, 2, 50 + b)] * 2) for b in range(B)])
    kv1 = A.anpd_kv_create(m, 256, 1)
    kvb = A.anpd_kv_create(m, 256, B, True)
    ctxs = [A.anpd_ngram_create(2, 4, 256, 0, st) for _ in range(B)]
    try:
        singles = [A.anpd_generate(m, kv1, ctxs[0], prompts[b], M, K) for b in range(B)]
        outs, stats = A.anpd_generate_batch(m, kvb, ctxs, prompts, M, K)
        for b in range(B):
            assert np.array_equal(outs[b], singles[b][0]), b
            for k in ("steps", "drafted", "accepted", "generated", "hist_accepted"):
                assert stats[b][k] == singles[b][1][k], (b, k)
        greedy, _ = A.anpd_generate_batch(m, kvb, ctxs, prompts, M, 0)
        assert np.array_equal(greedy, outs)
    finally:
        for c in ctxs:
            A.anpd_ngram_destroy(c)
        A.anpd_kv_destroy(kv1)
        A.anpd_kv_destroy(kvb)
        A.anpd_model_destroy(m)


def test_generate_error_paths(A, c1):
    wl, w, m, kv, st = c1
    ctx = A.anpd_ngram_create(2, 3, 128, 0, st)
    try:
        with pytest.raises(A.AnpdError) as e:
            A.anpd_generate(m, kv, ctx, list(range(100)), 64, 4)         # context too small
        assert e.value.status == A.ERR_CAPACITY
        with pytest.raises(A.AnpdError) as e:
            A.anpd_generate(m, kv, ctx, [1, 2, 3], 8, 8)                 # K > 7
        assert e.value.status == A.ERR_RANGE
        with pytest.raises(A.AnpdError) as e:
            A.anpd_generate(m, kv, ctx, [1, 2, 5000], 8, 2)              # token out of vocab
        assert e.value.status == A.ERR_RANGE
    finally:
        A.anpd_ngram_destroy(ctx)


def test_device_resident_loop_equals_host_stepped_loop(A, monkeypatch):
    """The decoding loop as one graph launch (a WHILE node around the step, no host round trip per step) against the
    same loop stepped from the host (ANPD_HOST_LOOP=1): same tokens, same statistics, for ANPD and for greedy, on a
    model that accepts drafts (orbit workload) and on the random tiny model; the device loop launches the same kernels
    per step plus the one that decides whether to go on."""
    from workloads import workload_inputs
    results = {}
    for host_loop in (False, True):
        if host_loop:
            monkeypatch.setenv("ANPD_HOST_LOOP", "1")
        for name in ("C1-A50", "C1"):
            wl = WORKLOADS[name]
            w, prompts, _ = workload_inputs(wl)
            st = new_stream()
            m = gpu_model(A, wl.shape, w, st)
            kv = A.anpd_kv_create(m, 512)
            ctx = A.anpd_ngram_create(wl.n_min, wl.n_max, 512, 0, st)
            try:
                A.anpd_generate(m, kv, ctx, prompts[0], 8, wl.K)                  # first run of a handle: eager first step
                A.anpd_launch_count(True)
                out, stats = A.anpd_generate(m, kv, ctx, prompts[0], wl.max_new, wl.K)
                launches = A.anpd_launch_count(True)
                greedy, gstats = A.anpd_generate(m, kv, ctx, prompts[0], wl.max_new, 0)
            finally:
                A.anpd_ngram_destroy(ctx)
                A.anpd_kv_destroy(kv)
                A.anpd_model_destroy(m)
            keep = {k: stats[k] for k in ("steps", "drafted", "accepted", "generated", "hist_accepted")}
            results[(name, host_loop)] = (out.tolist(), greedy.tolist(), keep, gstats["steps"], launches)
    for name in ("C1-A50", "C1"):
        dev, host = results[(name, False)], results[(name, True)]
        assert dev[:4] == host[:4], name
        assert dev[0] == dev[1]                                                  # losslessness in the device loop
        steps = dev[2]["steps"]
        assert dev[4] - host[4] == steps, (dev[4], host[4], steps)               # one more kernel per step, nothing else
    assert results[("C1-A50", False)][2]["accepted"] > 0
