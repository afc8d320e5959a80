"""Two candidates verified per step (the Conclusion's outlook on verifying several candidates in parallel).

  - the forward of a two-candidate step, row by row against the decoder oracle: the second candidate's rows are computed
    as if the first candidate were not there (positions, mask, cache slots), across a page boundary, on both attention
    kernels and with grouped query heads;
  - the commit: whichever candidate wins, the cache afterwards holds its rows at their positions (the next step's logits
    equal the oracle's on the committed sequence);
  - the decoding loop with two candidates: the stream is the library's greedy stream bit for bit; on orbit workloads
    whose prompts make the long n-gram contexts misleading it equals the closed form and the loop statistics (steps,
    drafted, accepted, histogram, steps won by the second candidate) equal the oracle's two-candidate Algorithm 1.
"""
import numpy as np
import pytest
import torch

from helpers import as_bf16_values, gpu_model, new_stream, require_gpu
from oracle.anpd import anpd_generate_two_candidates as oracle_two
from oracle.decoder import Decoder
from workloads import (WORKLOADS, ModelShape, ScriptedOrbitModel, make_orbit_weights, make_weights, markov_prompt,
                       orbit_continuation, orbit_fork_prompt, periodic_prompt)

pytestmark = pytest.mark.gpu

LOGIT_TOL = 5e-3      # max-abs against the oracle on the bf16-rounded weights (activation / KV rounding only), relative to
                      # the largest logit where that exceeds 1


def close(got, want):
    err = float((got - want).abs().max())
    return err <= LOGIT_TOL * max(1.0, float(want.abs().max()))


@pytest.fixture(scope="module")
def A():
    require_gpu()
    from paper_2404_08698_b200 import binding
    return binding


def oracle_rows(dec, cache, P, rows):
    """Logits of `rows` fed after the first P cached positions; the cache is rolled back to P afterwards."""
    cache.truncate(P)
    out = dec.forward(rows, cache)
    cache.truncate(P)
    return out


# (layers, d_model, q heads, kv heads, head_dim, d_ffn, vocab): mma.sync attention (head_dim 64) and the tensor-core
# kernel (head_dim 128) with 1, 2 and 4 query heads per kv head
SHAPES = [ModelShape(2, 128, 2, 2, 64, 192, 160), ModelShape(2, 128, 4, 2, 64, 192, 160),
          ModelShape(2, 256, 2, 2, 128, 320, 200), ModelShape(2, 256, 4, 2, 128, 320, 200), ModelShape(2, 512, 4, 1, 128, 320, 200)]


@pytest.mark.parametrize("shape", SHAPES, ids=lambda s: f"hd{s.head_dim}_g{s.n_q_heads // s.n_kv_heads}")
@pytest.mark.parametrize("plen", [125, 40])
def test_two_candidate_step_rows_and_commit(A, shape, plen):
    w = make_weights(shape, 31, False, std=0.02)
    m = gpu_model(A, shape, w)
    kv = A.anpd_kv_create(m, 384, 1, 1)                        # shuffled pages
    dec = Decoder(shape, as_bf16_values(w), torch.float64)
    try:
        prompt = markov_prompt(plen, shape.vocab, 5, 3).tolist()
        V = shape.vocab
        # the library's own greedy continuation g0 g1 ... (decisions are the library's; values are checked against the oracle)
        ctx = A.anpd_ngram_create(2, 3, 384)
        g, _ = A.anpd_generate(m, kv, ctx, prompt, 12, 0)
        A.anpd_ngram_destroy(ctx)
        g = g.tolist()
        cache = dec.new_cache()
        dec.forward(prompt, cache)

        def restart():
            A.anpd_kv_truncate(kv, 0, 0)
            assert A.anpd_prefill(m, kv, prompt) == g[0]
            cache.truncate(plen)

        # 1) the second candidate is the greedy continuation, the first is wrong from its first token: B wins with 3
        restart()
        a = [(g[1] + 1) % V, 5, 6, 7]
        b = g[1:4]
        chosen, acc, nxt, lg = A.anpd_verify_two_candidates(m, kv, g[0], a, b, V)
        want_a = oracle_rows(dec, cache, plen, [g[0]] + a)
        want_b = oracle_rows(dec, cache, plen, [g[0]] + b)
        got = torch.from_numpy(lg).double()
        assert close(got[:5], want_a)
        assert close(got[5:], want_b[1:])        # as if the first candidate were not there
        assert (chosen, acc, nxt) == (1, 3, g[4])
        assert A.anpd_kv_len(kv) == plen + 4
        # the cache now holds g0 g1 g2 g3 behind the prompt: the next step's rows against the oracle
        dec.forward(g[0:4], cache)
        got2 = torch.from_numpy(A.anpd_verify_logits(m, kv, g[4], g[5:8], V)).double()
        want2 = oracle_rows(dec, cache, plen + 4, g[4:8])
        assert close(got2, want2)
        acc2, nxt2 = A.anpd_verify(m, kv, g[4], g[5:8])
        assert (acc2, nxt2) == (3, g[8])

        # 2) the first candidate is right for two tokens, the second for one (its first token only): A wins, nothing moves
        restart()
        a = [g[1], g[2], (g[3] + 1) % V, 9]
        b = [g[1], (g[2] + 1) % V]
        chosen, acc, nxt, lg = A.anpd_verify_two_candidates(m, kv, g[0], a, b, V)
        got = torch.from_numpy(lg).double()
        assert close(got[:5], oracle_rows(dec, cache, plen, [g[0]] + a))
        assert close(got[5:], oracle_rows(dec, cache, plen, [g[0]] + b)[1:])
        assert (chosen, acc, nxt) == (0, 2, g[3])
        assert A.anpd_kv_len(kv) == plen + 3
        dec.forward(g[0:3], cache)
        got2 = torch.from_numpy(A.anpd_verify_logits(m, kv, g[3], g[4:6], V)).double()
        assert close(got2, oracle_rows(dec, cache, plen + 3, g[3:6]))

        # 3) a tie (both right for one token) goes to the first candidate; B longer than A and overlapping on the move
        restart()
        chosen, acc, nxt, _ = A.anpd_verify_two_candidates(m, kv, g[0], [g[1], (g[2] + 1) % V], [g[1], (g[2] + 2) % V])
        assert (chosen, acc, nxt) == (0, 1, g[2])
        restart()
        chosen, acc, nxt, _ = A.anpd_verify_two_candidates(m, kv, g[0], [(g[1] + 1) % V], g[1:7])
        assert (chosen, acc, nxt) == (1, 6, g[7])                  # rows move down by one slot only: ranges overlap
        dec.forward(g[0:7], cache)
        moved = A.anpd_verify_logits(m, kv, g[7], g[8:10], V)
        assert close(torch.from_numpy(moved).double(), oracle_rows(dec, cache, plen + 7, g[7:10]))
        # the same tokens committed by an ordinary step: the cache must hold the same rows (up to the order of the sums
        # inside the attention of the step that wrote them)
        restart()
        assert A.anpd_verify(m, kv, g[0], g[1:7]) == (6, g[7])
        plain = A.anpd_verify_logits(m, kv, g[7], g[8:10], V)
        assert float(np.abs(moved - plain).max()) <= 1e-4
    finally:
        A.anpd_kv_destroy(kv)
        A.anpd_model_destroy(m)


@pytest.mark.parametrize("K,N,policy", [(1, 2, 0), (3, 2, 1), (5, 5, 0), (7, 8, 0), (7, 3, 1), (2, 6, 0)])
def test_two_candidate_loop_is_lossless_on_a_random_decoder(A, K, N, policy):
    shape = ModelShape(2, 128, 4, 2, 64, 200, 300)
    w = make_weights(shape, 21, False, std=0.08)
    st = new_stream()
    m = gpu_model(A, shape, w, st)
    kv = A.anpd_kv_create(m, 256)
    ctx = A.anpd_ngram_create(2, N, 256, policy, st)
    try:
        base = periodic_prompt(30, 6, shape.vocab, 4)
        prompt = np.concatenate([base, markov_prompt(30, shape.vocab, 2, 8), base[:13]])
        ref, _ = A.anpd_generate(m, kv, ctx, prompt, 48, 0)
        A.anpd_kv_set_candidates(kv, 2)
        out, s2 = A.anpd_generate(m, kv, ctx, prompt, 48, K)
        A.anpd_kv_set_candidates(kv, 1)
        out1, s1 = A.anpd_generate(m, kv, ctx, prompt, 48, K)
        assert np.array_equal(out, ref) and np.array_equal(out1, ref)
        assert s2["generated"] == s2["steps"] + s2["accepted"]
        assert s2["drafted"] <= (min(K, 4) + min(K, 3)) * s2["steps"]
        assert sum(s2["hist_accepted"][min(K, 4) + 1:]) == 0 and s1["alt_wins"] == 0
        with pytest.raises(Exception):
            A.anpd_kv_set_candidates(kv, 3)
    finally:
        A.anpd_ngram_destroy(ctx)
        A.anpd_kv_destroy(kv)
        A.anpd_model_destroy(m)


def run_fork_workload(A, name, oracle_model_factory, K, policy=0):
    """An orbit model of workload `name`'s shape on a forked prompt (workloads.orbit_fork_prompt)."""
    wl = WORKLOADS[name]
    dev = "cuda" if wl.shape.streamed_params > 1e8 else "cpu"
    w, pi = make_orbit_weights(wl.shape, wl.weight_seed, wl.orbit_S, device=dev, bf16=wl.weights_bf16)
    prompt = orbit_fork_prompt(pi, wl.prompt_len, wl.prompt_seed)
    st = new_stream()
    m = gpu_model(A, wl.shape, w, st)
    max_len = wl.prompt_len + wl.max_new + 64
    kv = A.anpd_kv_create(m, max_len)
    ctx = A.anpd_ngram_create(wl.n_min, wl.n_max, max_len, policy, st)
    try:
        A.anpd_kv_set_candidates(kv, 2)
        out, stats = A.anpd_generate(m, kv, ctx, prompt, wl.max_new, K)
        A.anpd_kv_set_candidates(kv, 1)
        one, stats1 = A.anpd_generate(m, kv, ctx, prompt, wl.max_new, min(K, 4))
    finally:
        A.anpd_ngram_destroy(ctx)
        A.anpd_kv_destroy(kv)
        A.anpd_model_destroy(m)
    want = orbit_continuation(pi, prompt[-1], wl.max_new).tolist()
    assert out.tolist() == want and one.tolist() == want                          # the closed form, both ways
    got, ost, _ = oracle_two(oracle_model_factory(wl, w, pi), prompt.tolist(), wl.max_new, K, n_max=wl.n_max, n_min=wl.n_min,
                             policy=policy)
    assert got == want
    assert (stats["steps"], stats["drafted"], stats["accepted"], stats["alt_wins"]) == (ost.steps, ost.drafted, ost.accepted, ost.alt_wins)
    assert stats["hist_accepted"] == ost.hist_accepted
    assert stats["alt_wins"] > 0 and stats["steps"] < stats1["steps"]             # the second candidate saves steps here
    return stats, stats1


@pytest.mark.parametrize("K,policy", [(4, 0), (7, 1), (2, 0)])
def test_two_candidate_loop_on_tiny_forked_orbit_against_the_decoder_oracle(A, K, policy):
    run_fork_workload(A, "C1-A50", lambda wl, w, pi: Decoder(wl.shape, w, torch.float64), K, policy)


@pytest.mark.parametrize("name", ["C2-A40", "C3-A20"])
def test_two_candidate_loop_at_full_size(A, name):
    wl = WORKLOADS[name]
    s2, s1 = run_fork_workload(A, name, lambda wl, w, pi: ScriptedOrbitModel(pi, wl.shape.vocab), wl.K)
    print(f"{name}: two candidates {s2['steps']} steps ({s2['alt_wins']} won by the second), one candidate {s1['steps']} steps")


def test_two_candidate_host_stepped_loop_equals_device_loop(A, monkeypatch):
    wl = WORKLOADS["C1-A50"]
    f = lambda wl, w, pi: ScriptedOrbitModel(pi, wl.shape.vocab)
    s_dev, _ = run_fork_workload(A, "C1-A50", f, 5)
    monkeypatch.setenv("ANPD_HOST_LOOP", "1")
    s_host, _ = run_fork_workload(A, "C1-A50", f, 5)
    for k in ("steps", "drafted", "accepted", "alt_wins", "hist_accepted", "generated"):
        assert s_dev[k] == s_host[k]


def test_two_candidate_batch_equals_independent_runs(A):
    """Three sequences in one kv handle (shuffled pages), each with its own forked prompt: the batched two-candidate
    loop gives every sequence the stream and statistics of its own single-sequence run and of the oracle."""
    wl = WORKLOADS["C1-A50"]
    w, pi = make_orbit_weights(wl.shape, wl.weight_seed, wl.orbit_S, bf16=wl.weights_bf16)
    st = new_stream()
    m = gpu_model(A, wl.shape, w, st)
    B, M, K = 3, 48, 5
    prompts = np.stack([orbit_fork_prompt(pi, wl.prompt_len, 300 + b, every=7 + b) for b in range(B)])
    max_len = wl.prompt_len + M + 64
    kv1 = A.anpd_kv_create(m, max_len, 1)
    kvb = A.anpd_kv_create(m, max_len, B, True)
    ctxs = [A.anpd_ngram_create(wl.n_min, wl.n_max, max_len, 0, st) for _ in range(B)]
    try:
        A.anpd_kv_set_candidates(kv1, 2)
        A.anpd_kv_set_candidates(kvb, 2)
        singles = [A.anpd_generate(m, kv1, ctxs[0], prompts[b], M, K) for b in range(B)]
        outs, stats = A.anpd_generate_batch(m, kvb, ctxs, prompts, M, K)
        wins = 0
        for b in range(B):
            assert outs[b].tolist() == orbit_continuation(pi, prompts[b][-1], M).tolist()
            assert np.array_equal(outs[b], singles[b][0]), b
            _, ost, _ = oracle_two(ScriptedOrbitModel(pi, wl.shape.vocab), prompts[b].tolist(), M, K, n_max=wl.n_max, n_min=wl.n_min)
            for k in ("steps", "drafted", "accepted", "generated", "hist_accepted", "alt_wins"):
                assert stats[b][k] == singles[b][1][k], (b, k)
            assert (stats[b]["steps"], stats[b]["drafted"], stats[b]["accepted"], stats[b]["alt_wins"]) == \
                   (ost.steps, ost.drafted, ost.accepted, ost.alt_wins)
            wins += stats[b]["alt_wins"]
        assert wins > 0
    finally:
        for c in ctxs:
            A.anpd_ngram_destroy(c)
        A.anpd_kv_destroy(kv1)
        A.anpd_kv_destroy(kvb)
        A.anpd_model_destroy(m)


def test_two_candidate_error_paths(A):
    shape = ModelShape(1, 128, 2, 2, 64, 192, 160)
    w = make_weights(shape, 5, False, std=0.02)
    m = gpu_model(A, shape, w)
    kv = A.anpd_kv_create(m, 256)
    kvb = A.anpd_kv_create(m, 256, 2)
    try:
        first = A.anpd_prefill(m, kv, [1, 2, 3, 4, 5])
        for a, b in [([], [1]), ([1], []), ([1, 2, 3, 4], [1, 2, 3, 4]), ([1], [shape.vocab]), ([-1], [1])]:
            with pytest.raises(Exception):
                A.anpd_verify_two_candidates(m, kv, first, a, b)
        assert A.anpd_kv_len(kv) == 5                                 # nothing was committed by the rejected calls
        with pytest.raises(Exception):
            A.anpd_verify_two_candidates(m, kvb, 1, [1], [2])        # batch 1 only
        for bad in (0, 3, -1):
            with pytest.raises(Exception):
                A.anpd_kv_set_candidates(kv, bad)
        chosen, acc, nxt, _ = A.anpd_verify_two_candidates(m, kv, first, [1], [2])
        assert chosen in (0, 1) and 0 <= acc <= 1 and A.anpd_kv_len(kv) == 6 + acc
    finally:
        A.anpd_kv_destroy(kv)
        A.anpd_kv_destroy(kvb)
        A.anpd_model_destroy(m)
