"""ORACLE (test infrastructure, not the product): greedy decoding, the
verification stage and the ANPD loop (Algorithm 1).

ANPD is lossless (Section 3.1): its output is, token for token, the model's own
greedy autoregressive output.  So the result has a plain definition, `greedy`,
and `anpd_generate` follows Algorithm 1 step by step so that drafts, accepted
lengths and table states can be compared too.  `model` is anything with
`new_cache()` and `forward(tokens, cache) -> logits [len(tokens), V]` whose
cache has `.length` and `.truncate(n)`: the decoder oracle, or a scripted
stand-in in tests.  Only tests, the smoke check and the benchmark's CPU
baseline may import this file.

Readings taken where Algorithm 1 is ambiguous:
  * drafts[1] of a step is the already confirmed token; the model's prediction
    after consuming drafts[1..i] is compared with drafts[i+1].
  * after `a` accepted drafts the next confirmed token is the prediction that
    follows the last accepted one, whether the loop ended by a mismatch or by
    running out of drafts (the only reading under which the output is
    lossless).
  * a NULL answer from the N-gram module ends drafting early; a step with no
    drafts is a plain greedy step.
  * the loop runs while fewer than M tokens are out and the result is cut to M.
"""
from __future__ import annotations

from dataclasses import dataclass, field

import torch

from .mln import MLN, POLICY_MAX_COUNT


def argmax_lowest(row: torch.Tensor) -> int:
    """Index of the maximum; ties go to the lowest index."""
    m = row.max()
    return int(torch.nonzero(row == m)[0, 0])


def greedy(model, prompt, max_new: int) -> list[int]:
    """The plain definition: one token per forward, each the argmax of the last logits."""
    cache = model.new_cache()
    logits = model.forward(list(prompt), cache)
    out = [argmax_lowest(logits[-1])]
    while len(out) < max_new:
        logits = model.forward([out[-1]], cache)
        out.append(argmax_lowest(logits[-1]))
    return out[:max_new]


def accept_length(draft, preds) -> int:
    """Longest prefix of `draft` with draft[i] == preds[i] (preds[i] = the model's
    token after consuming the confirmed token and draft[0..i-1])."""
    a = 0
    while a < len(draft) and int(draft[a]) == int(preds[a]):
        a += 1
    return a


def verify(model, cache, last_tok: int, draft) -> tuple[int, int, list[int], torch.Tensor]:
    """One verification forward over [last_tok, draft...] at positions cache.length...

    Returns (accepted_len, next_tok, preds, logits); the cache keeps the entries of
    last_tok and of the accepted drafts only.
    """
    P = cache.length
    rows = [int(last_tok)] + [int(t) for t in draft]
    logits = model.forward(rows, cache)
    preds = [argmax_lowest(logits[r]) for r in range(len(rows))]
    a = accept_length(draft, preds)
    cache.truncate(P + a + 1)
    return a, preds[a], preds, logits


@dataclass
class Stats:
    steps: int = 0
    drafted: int = 0
    accepted: int = 0
    generated: int = 0
    hist_accepted: list = field(default_factory=lambda: [0] * 8)
    drafts: list = field(default_factory=list)          # per step, the draft
    accepted_lens: list = field(default_factory=list)   # per step, accepted_len

    @property
    def hit_ratio(self) -> float:
        """alpha of Section 4.4: accepted drafts over proposed drafts."""
        return self.accepted / self.drafted if self.drafted else 0.0


def speedup_bound(alpha: float, K: int) -> float:
    """Section 4.4: theoretical upper bound of the acceleration, alpha * K + 1."""
    return alpha * K + 1.0


def two_candidate_lengths(K: int) -> tuple[int, int]:
    """Draft lengths of the two candidates of a step when a step has room for 7 draft rows: the first
    candidate keeps up to 4 tokens, the alternative up to 3 (both at most K)."""
    return min(K, 4), min(K, 3)


def anpd_generate_two_candidates(model, prompt, max_new: int, K: int, n_max: int = 5, n_min: int = 2,
                                 policy: int = POLICY_MAX_COUNT):
    """Algorithm 1 with two candidates per step (the conclusion's future-work item: several candidates verified
    at once).  Each step drafts the usual candidate A and an alternative B (MLN.draft_alternative), verifies
    both against the same cache state - written here as two forwards from the same state; one forward with a tree
    mask computes the same rows - and keeps the one with the longer accepted prefix (A on a tie).  The output is
    still the model's greedy output.  Returns (tokens[:max_new], Stats, mln); Stats.drafted counts the tokens of
    both candidates, Stats.drafts holds (A, B) per step and Stats.alt_wins the steps B won."""
    mln = MLN(n_min, n_max, policy)
    mln.initialize(prompt)
    st = Stats()
    st.alt_wins = 0
    ka, kb = two_candidate_lengths(K)
    cache = model.new_cache()
    logits = model.forward(list(prompt), cache)
    confirmed = argmax_lowest(logits[-1])
    out: list[int] = []
    while len(out) < max_new:
        out.append(confirmed)
        mln.update(confirmed)
        da = mln.draft(ka)
        db = mln.draft_alternative(da[0] if da else None, kb)
        P = cache.length
        a_a, nxt_a, _, _ = verify(model, cache, confirmed, da)
        a_b, nxt_b = 0, None
        if db:
            cache.truncate(P)
            a_b, nxt_b, _, _ = verify(model, cache, confirmed, db)
        if a_b > a_a:
            chosen, a, nxt = db, a_b, nxt_b
            st.alt_wins += 1
        else:
            chosen, a, nxt = da, a_a, nxt_a
            if db:                                       # the cache holds B's rows: put A's accepted rows back
                cache.truncate(P)
                verify(model, cache, confirmed, da[:a_a])
        for tok in chosen[:a]:
            out.append(tok)
            mln.update(tok)
        st.steps += 1
        st.drafted += len(da) + len(db)
        st.accepted += a
        st.hist_accepted[a] += 1
        st.drafts.append((list(da), list(db)))
        st.accepted_lens.append(a)
        confirmed = nxt
    st.generated = len(out)
    return out[:max_new], st, mln


def anpd_generate(model, prompt, max_new: int, K: int, n_max: int = 5, n_min: int = 2,
                  policy: int = POLICY_MAX_COUNT, mln: MLN | None = None):
    """Algorithm 1.  Returns (tokens[:max_new], Stats, mln)."""
    if mln is None:
        mln = MLN(n_min, n_max, policy)
    mln.initialize(prompt)                                   # Memory <- Initialize(token_ids)
    st = Stats()
    cache = model.new_cache()
    logits = model.forward(list(prompt), cache)              # pred <- LLM(prompt)
    confirmed = argmax_lowest(logits[-1])
    out: list[int] = []
    while len(out) < max_new:
        out.append(confirmed)
        mln.update(confirmed)
        draft = mln.draft(K) if K > 0 else []
        a, nxt, _, _ = verify(model, cache, confirmed, draft)
        for tok in draft[:a]:
            out.append(tok)
            mln.update(tok)
        st.steps += 1
        st.drafted += len(draft)
        st.accepted += a
        st.hist_accepted[a] += 1
        st.drafts.append(list(draft))
        st.accepted_lens.append(a)
        confirmed = nxt
    st.generated = len(out)
    return out[:max_new], st, mln
