"""Pins for oracle/anpd.py: losslessness (ANPD == greedy), the progress
invariant, the definitional accepted length, closed forms on scripted models,
and the case-study bound printed in the paper."""
import os
import random

import pytest
import torch

from oracle.anpd import (accept_length, anpd_generate, anpd_generate_two_candidates, argmax_lowest, greedy, speedup_bound,
                         two_candidate_lengths, verify)
from oracle.decoder import Decoder
from oracle.mln import POLICY_LAST_SEEN, POLICY_MAX_COUNT
from workloads import ModelShape, WORKLOADS, make_prompts, make_weights, periodic_prompt

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


class _Hist:
    def __init__(self):
        self.toks = []

    @property
    def length(self):
        return len(self.toks)

    def truncate(self, n):
        assert n <= len(self.toks)
        del self.toks[n:]


class ScriptedModel:
    """next token = f(all tokens consumed so far); logits are one-hot on it."""

    def __init__(self, vocab, fn):
        self.vocab, self.fn, self.forwards, self.rows = vocab, fn, 0, 0

    def new_cache(self):
        return _Hist()

    def forward(self, tokens, cache):
        self.forwards += 1
        self.rows += len(tokens)
        out = torch.zeros(len(tokens), self.vocab, dtype=torch.float64)
        for r, t in enumerate(tokens):
            cache.toks.append(int(t))
            out[r, self.fn(cache.toks)] = 1.0
        return out


def test_argmax_ties_go_to_lowest_index():
    assert argmax_lowest(torch.tensor([0.0, 2.0, 2.0, 1.0])) == 1
    assert argmax_lowest(torch.tensor([5.0, 5.0])) == 0


def test_accept_length_definition_cases():
    assert accept_length([], [7]) == 0
    assert accept_length([1, 2, 3], [1, 2, 3, 9]) == 3            # all match -> bonus token
    assert accept_length([1, 2, 3], [1, 2, 4, 9]) == 2            # mismatch at the last draft
    assert accept_length([1, 2, 3], [5, 2, 3, 9]) == 0            # later matches do not count
    # brute force over all short cases: longest prefix with draft[i] == preds[i]
    rng = random.Random(0)
    for _ in range(200):
        k = rng.randint(0, 6)
        d = [rng.randrange(3) for _ in range(k)]
        p = [rng.randrange(3) for _ in range(k + 1)]
        want = max(a for a in range(k + 1) if all(d[i] == p[i] for i in range(a)))
        assert accept_length(d, p) == want


def test_verify_next_token_is_prediction_after_last_accepted():
    # model: next = (last + 1) mod 10.  confirmed 3, draft 4 5 9 1 -> accepts 4 5, then model says 6
    m = ScriptedModel(10, lambda h: (h[-1] + 1) % 10)
    c = m.new_cache()
    m.forward([1, 2], c)
    a, nxt, preds, _ = verify(m, c, 3, [4, 5, 9, 1])
    assert (a, nxt) == (2, 6) and preds[:3] == [4, 5, 6]
    assert c.toks == [1, 2, 3, 4, 5]                               # rejected rows rolled back
    # every draft right, including the last: the bonus token follows the last draft
    a, nxt, _, _ = verify(m, c, 6, [7, 8])
    assert (a, nxt) == (2, 9) and c.length == 8
    # last draft wrong: next token is the model's token at that position, not one after it
    a, nxt, _, _ = verify(m, c, 9, [0, 5])
    assert (a, nxt) == (1, 1)


def test_cyclic_model_closed_form():
    """next = perm(last) with one cycle of length p.  Greedy output is the cycle; once the
    tables have seen one full period every draft is accepted, so each step yields K+1 tokens."""
    p, K, M = 5, 4, 60
    cyc = [3, 8, 1, 6, 4]
    nxt = {cyc[i]: cyc[(i + 1) % p] for i in range(p)}
    model = ScriptedModel(10, lambda h: nxt.get(h[-1], cyc[0]))
    prompt = [cyc[i % p] for i in range(2 * p + 3)]
    want = [cyc[(len(prompt) + i) % p] for i in range(M)]
    assert greedy(model, prompt, M) == want
    out, st, _ = anpd_generate(model, prompt, M, K, n_max=3)
    assert out == want
    assert st.accepted_lens == [K] * st.steps and st.steps == -(-M // (K + 1))
    assert st.hit_ratio == 1.0 and speedup_bound(st.hit_ratio, K) == K + 1


def test_never_accept_model_degenerates_to_greedy_steps():
    # a counter model never repeats, so no context is ever seen twice: no drafts, one token per step
    model = ScriptedModel(1000, lambda h: len(h) % 1000)
    prompt = list(range(500, 510))
    out, st, _ = anpd_generate(model, prompt, 20, 5, n_max=4)
    assert out == greedy(model, prompt, 20)
    assert st.steps == 20 and st.drafted == 0 and st.accepted == 0


@pytest.mark.parametrize("policy", [POLICY_MAX_COUNT, POLICY_LAST_SEEN])
def test_losslessness_on_scripted_pseudo_random_model(policy):
    # deterministic "LM" with short memory and a small vocabulary: plenty of partial acceptances
    def fn(h):
        return (h[-1] * 7 + (h[-2] if len(h) > 1 else 0) * 3 + (len(h) % 5 == 0)) % 6
    model = ScriptedModel(6, fn)
    prompt = [1, 4, 2, 2, 5, 0, 3, 1, 4, 2]
    want = greedy(model, prompt, 80)
    seen_partial = False
    for K in range(0, 8):
        for N in range(2, 8):
            out, st, _ = anpd_generate(model, prompt, 80, K, n_max=N, policy=policy)
            assert out == want, (K, N)
            # progress: every step commits between 1 and K+1 tokens; generated = steps + accepted
            assert all(0 <= a <= K for a in st.accepted_lens)
            assert st.generated == st.steps + st.accepted and st.generated >= 80
            assert all(len(d) <= K for d in st.drafts)
            seen_partial |= any(0 < a < len(d) for a, d in zip(st.accepted_lens, st.drafts))
    assert seen_partial


def test_losslessness_on_tiny_decoder_all_K_N():
    wl = WORKLOADS["C1"]
    shape = ModelShape(2, 64, 4, 2, 16, 96, 128)
    dec = Decoder(shape, make_weights(shape, 5, False, std=0.2), torch.float64)
    prompt = periodic_prompt(24, 6, shape.vocab, 9).tolist()
    want = greedy(dec, prompt, 24)
    for K, N in [(0, 2), (1, 2), (4, 3), (7, 5), (5, 7)]:
        out, st, _ = anpd_generate(dec, prompt, 24, K, n_max=N)
        assert out == want
        assert st.generated == st.steps + st.accepted


def test_c1_workload_oracle_runs_and_is_lossless():
    wl = WORKLOADS["C1"]
    dec = Decoder(wl.shape, make_weights(wl.shape, wl.weight_seed, wl.weights_bf16), torch.float64)
    prompt = make_prompts(wl)[0].tolist()
    want = greedy(dec, prompt, wl.max_new)
    out, st, _ = anpd_generate(dec, prompt, wl.max_new, wl.K, n_max=wl.n_max)
    assert out == want and len(out) == wl.max_new


def test_case_study_bound_from_the_paper():
    vals = {}
    with open(os.path.join(GOLDEN, "speedup_bound_case_study.txt")) as f:
        for line in f:
            if line.strip() and not line.startswith("#"):
                k, v = line.split()
                vals[k] = float(v)
    assert round(speedup_bound(vals["alpha"], int(vals["K"])), 2) == vals["bound"]


def test_full_drafts_mean_tokens_per_step_is_one_plus_alpha_K():
    p, K = 4, 3
    cyc = [2, 7, 5, 9]
    nxt = {cyc[i]: cyc[(i + 1) % p] for i in range(p)}
    # a model that leaves the cycle every 6th position -> some rejections, drafts still full length
    def fn(h):
        return 0 if len(h) % 6 == 0 else nxt.get(h[-1], cyc[0])
    model = ScriptedModel(10, fn)
    prompt = [cyc[i % p] for i in range(13)] + [0] + [cyc[i % p] for i in range(8)]
    out, st, _ = anpd_generate(model, prompt, 90, K, n_max=2)
    assert out == greedy(model, prompt, 90)
    if all(len(d) == K for d in st.drafts):
        assert abs(st.generated / st.steps - speedup_bound(st.hit_ratio, K)) < 1e-12


@pytest.mark.parametrize("policy", [POLICY_MAX_COUNT, POLICY_LAST_SEEN])
def test_two_candidates_are_lossless_and_never_slower_per_step(policy):
    """Two candidates per step: the output is still the greedy output for every K and N; each step commits at least
    what the first candidate alone would have committed from the same state (so never more steps than with the first
    candidate's length alone), the alternative wins somewhere, and drafted counts both candidates."""
    def fn(h):
        return (h[-1] * 7 + (h[-2] if len(h) > 1 else 0) * 3 + (len(h) % 5 == 0)) % 6
    model = ScriptedModel(6, fn)
    prompt = [1, 4, 2, 2, 5, 0, 3, 1, 4, 2]
    want = greedy(model, prompt, 80)
    wins = 0
    for K in range(0, 8):
        ka, kb = two_candidate_lengths(K)
        assert ka <= 4 and kb <= 3 and ka + kb <= 7 and ka <= K and kb <= K
        for N in range(2, 8):
            out, st, _ = anpd_generate_two_candidates(model, prompt, 80, K, n_max=N, policy=policy)
            assert out == want, (K, N)
            assert st.generated == st.steps + st.accepted and st.generated >= 80
            assert all(len(a) <= ka and len(b) <= kb for a, b in st.drafts)
            assert all(not b or (a and b[0] != a[0]) for a, b in st.drafts)
            assert st.drafted == sum(len(a) + len(b) for a, b in st.drafts)
            one, st1, _ = anpd_generate(model, prompt, 80, ka, n_max=N, policy=policy)
            assert one == want and st.steps <= st1.steps, (K, N, st.steps, st1.steps)
            wins += st.alt_wins
    assert wins > 0


def test_two_candidates_on_tiny_decoder():
    wl = WORKLOADS["C1"]
    w = make_weights(wl.shape, wl.weight_seed, wl.weights_bf16)
    dec = Decoder(wl.shape, w, torch.float64)
    prompt = make_prompts(wl)[0].tolist()
    want = greedy(dec, prompt, 24)
    out, st, _ = anpd_generate_two_candidates(dec, prompt, 24, 4, n_max=3)
    assert out == want and st.generated == st.steps + st.accepted
