"""Pins for oracle/mln.py: brute-force recounts and string search on tiny
contexts, closed forms, and a hand-worked example (tests/golden)."""
import os
import random

import pytest

from oracle.mln import MLN, POLICY_MAX_COUNT, POLICY_LAST_SEEN

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def brute_counts(tokens, n):
    """Every n-gram of the sequence recounted by a double loop over positions."""
    out = {}
    T = len(tokens)
    for t in range(n - 1, T):
        g = tuple(tokens[t - n + 1:t + 1])
        if g in out:
            continue
        cnt, last = 0, -1
        for u in range(n - 1, T):
            if all(tokens[u - n + 1 + i] == g[i] for i in range(n)):
                cnt += 1
                last = u
        out[g] = (cnt, last)
    return out


def brute_query(tokens, ctx, n_min, n_max, policy):
    """Back-off by string search: the longest suffix of ctx (length <= n_max-1) that
    occurs in `tokens` followed by a token decides; its best successor is returned."""
    for n in range(n_max, n_min - 1, -1):
        if len(ctx) < n - 1:
            continue
        key = list(ctx[len(ctx) - (n - 1):])
        cands = {}
        for t in range(n - 1, len(tokens)):
            if tokens[t - n + 1:t] == key:
                c, _ = cands.get(tokens[t], (0, -1))
                cands[tokens[t]] = (c + 1, t)
        if cands:
            if policy == POLICY_MAX_COUNT:
                return max(cands, key=lambda s: cands[s])
            return max(cands, key=lambda s: cands[s][1])
    return None


@pytest.mark.parametrize("seed", range(6))
def test_tables_equal_bruteforce_recount(seed):
    rng = random.Random(seed)
    V, T = rng.choice([2, 3, 5, 8]), rng.randint(1, 32)
    toks = [rng.randrange(V) for _ in range(T)]
    m = MLN(2, 5)
    m.initialize(toks)
    for n in range(2, 6):
        want = brute_counts(toks, n)
        got = {ctx + (s,): (c, last) for ctx, s, c, last in m.dump(n)}
        assert got == want
        # number of records = number of distinct n-grams
        assert len(got) == len({tuple(toks[t - n + 1:t + 1]) for t in range(n - 1, T)})
        # counts of a context's successors add up to its occurrences followed by anything
        for ctx, cands in m.succ[n].items():
            occ = sum(1 for t in range(n - 1, T) if tuple(toks[t - n + 1:t]) == ctx)
            assert sum(c for c, _ in cands.values()) == occ


@pytest.mark.parametrize("policy", [POLICY_MAX_COUNT, POLICY_LAST_SEEN])
@pytest.mark.parametrize("seed", range(8))
def test_draft_equals_bruteforce_longest_suffix_search(seed, policy):
    rng = random.Random(100 + seed)
    V, T, N = rng.choice([2, 3, 4, 6]), rng.randint(2, 40), rng.randint(2, 6)
    toks = [rng.randrange(V) for _ in range(T)]
    m = MLN(2, N, policy)
    m.initialize(toks)
    K = 6
    want, ctx = [], list(toks)
    for _ in range(K):
        s = brute_query(toks, ctx, 2, N, policy)
        if s is None:
            break
        want.append(s)
        ctx.append(s)
    assert m.draft(K) == want
    assert m.tokens == toks            # drafting leaves the committed state alone


def test_incremental_update_equals_initialize():
    rng = random.Random(7)
    toks = [rng.randrange(4) for _ in range(50)]
    a, b = MLN(2, 4), MLN(2, 4)
    a.initialize(toks)
    b.initialize(toks[:20])
    for t in toks[20:]:
        b.update(t)
    for n in (2, 3, 4):
        assert a.dump(n) == b.dump(n)
        assert a.dump_best(n) == b.dump_best(n)


@pytest.mark.parametrize("p,N,K", [(3, 2, 4), (5, 5, 7), (7, 3, 5), (1, 2, 3)])
def test_periodic_sequence_closed_form(p, N, K):
    """Period p of distinct symbols: every context has one successor, so
    draft_i = x[(T+i-1) mod p] and the draft is always full."""
    base = [10 + 3 * i for i in range(p)]
    T = 2 * p + N + 1
    toks = [base[t % p] for t in range(T)]
    m = MLN(2, N)
    m.initialize(toks)
    assert m.draft(K) == [base[(T + i) % p] for i in range(K)]


def test_all_distinct_tokens_draft_nothing():
    m = MLN(2, 5)
    m.initialize(list(range(30)))
    assert m.draft(5) == []
    assert m.query([29]) is None


def test_level_skipped_while_context_too_short():
    m = MLN(2, 5)
    m.initialize([4])
    assert m.draft(3) == []
    m.update(4)                       # 4 4 : level 2 knows (4)->4, higher levels nothing yet
    assert m.dump(2) == [((4,), 4, 1, 1)] and m.dump(3) == []
    assert m.draft(3) == [4, 4, 4]


def test_backoff_prefers_longest_level():
    # ... 1 2 9 ... 7 2 8 ... 1 2 : level 3 context (1,2) says 9, level 2 context (2) has 9 and 8 (8 more recent)
    toks = [1, 2, 9, 7, 2, 8, 1, 2]
    m3 = MLN(2, 3)
    m3.initialize(toks)
    assert m3.draft(1) == [9]
    m2 = MLN(2, 2)
    m2.initialize(toks)
    assert m2.draft(1) == [8]


def _read_golden(name):
    d = {}
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            line = line.strip()
            if line and not line.startswith("#"):
                k, *v = line.split()
                d[k] = [float(x) if "." in x else int(x) for x in v]
    return d


def test_hand_worked_example():
    g = _read_golden("mln_hand_example.txt")
    m = MLN(2, g["n_max"][0])
    m.initialize(g["tokens"])
    assert m.draft(4) == g["draft_K4"]
    m.update(g["after_update"][0])
    assert m.draft(4) == g["draft_K4_after"]
    a = MLN(2, 3, POLICY_MAX_COUNT)
    a.initialize(g["tokens2"])
    b = MLN(2, 3, POLICY_LAST_SEEN)
    b.initialize(g["tokens2"])
    assert a.draft(1) == g["first_draft_max_count"]
    assert b.draft(1) == g["first_draft_last_seen"]


def brute_level_answer(tokens, ctx, n, policy):
    """Answer of level n alone, by string search: best successor of the last n-1 tokens of ctx in `tokens`."""
    if len(ctx) < n - 1:
        return None
    key = list(ctx[len(ctx) - (n - 1):])
    cands = {}
    for t in range(n - 1, len(tokens)):
        if tokens[t - n + 1:t] == key:
            c, _ = cands.get(tokens[t], (0, -1))
            cands[tokens[t]] = (c + 1, t)
    if not cands:
        return None
    if policy == POLICY_MAX_COUNT:
        return max(cands, key=lambda s: cands[s])
    return max(cands, key=lambda s: cands[s][1])


@pytest.mark.parametrize("policy", [POLICY_MAX_COUNT, POLICY_LAST_SEEN])
@pytest.mark.parametrize("seed", range(12))
def test_alternative_draft_equals_bruteforce(seed, policy):
    """The second candidate of a step: its first token is what the longest level that DISAGREES with the first
    candidate's first token proposes (string search per level); it continues by ordinary back-off queries."""
    rng = random.Random(500 + seed)
    V, T, N = rng.choice([2, 3, 4]), rng.randint(4, 48), rng.randint(2, 6)
    toks = [rng.randrange(V) for _ in range(T)]
    m = MLN(2, N, policy)
    m.initialize(toks)
    first = m.draft(1)
    assert m.draft_alternative(first[0] if first else None, 0) == []
    assert m.draft_alternative(None, 3) == []
    got = m.draft_alternative(first[0] if first else None, 3)
    want = []
    if first:
        alt = None
        for n in range(N, 1, -1):
            a = brute_level_answer(toks, toks, n, policy)
            if a is not None and a != first[0]:
                alt = a
                break
        if alt is not None:
            want, ctx = [alt], list(toks) + [alt]
            while len(want) < 3:
                s = brute_query(toks, ctx, 2, N, policy)
                if s is None:
                    break
                want.append(s)
                ctx.append(s)
    assert got == want
    assert not got or got[0] != first[0]
    assert m.tokens == toks


def test_alternative_draft_hand_case():
    # after "... 7": the trigram context (5, 7) was followed by 1; the bigram context (7) by 1 once and by 2 twice
    toks = [5, 7, 1, 9, 7, 2, 8, 7, 2, 5, 7]
    m = MLN(2, 3)
    m.initialize(toks)
    assert m.draft(1) == [1]                      # longest level wins
    assert m.draft_alternative(1, 1) == [2]       # the bigram level disagrees
    assert m.draft_alternative(2, 1) == [1]       # had 2 been drafted, the trigram level would be the one that differs
