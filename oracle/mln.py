"""ORACLE (test infrastructure, not the product): the Multi-Level N-gram module.

A plain, slow, exact CPU statement of the paper's N-gram module (Section 3.1,
"Token Level N-gram Module": Initialize / Update / Query) and of its
multi-level back-off (Section 3.2 and Algorithm 2), written with Python dicts
over token-id tuples.  Only tests, the smoke check and the benchmark's CPU
baseline may import this file; it shares no code with the CUDA library.

Readings taken where the paper is silent:
  * Query returns the most probable successor under the frequency counts of
    Eq. 1, i.e. the successor with the largest count; equal counts are broken
    in favour of the successor seen most recently ("max-count" policy).  A
    second policy, "last-seen", returns the successor of the context's most
    recent occurrence.
  * Memory is persistent: built once from the prompt and updated token by
    token; Algorithm 2's per-query Initialize is not taken literally.
  * Level n is keyed on the previous n-1 tokens; a level is skipped while the
    context is shorter than that.
Pinned by tests/test_oracle_mln.py (brute-force recounts, a periodic sequence's
closed form, an all-distinct sequence, a hand-worked example).
"""
from __future__ import annotations

POLICY_MAX_COUNT = 0
POLICY_LAST_SEEN = 1


class MLN:
    """N-1 n-gram modules, n in [n_min, n_max] (Section 3.2: n in [2, N])."""

    def __init__(self, n_min: int = 2, n_max: int = 5, policy: int = POLICY_MAX_COUNT):
        if not (2 <= n_min <= n_max):
            raise ValueError("need 2 <= n_min <= n_max")
        if policy not in (POLICY_MAX_COUNT, POLICY_LAST_SEEN):
            raise ValueError("unknown policy")
        self.n_min, self.n_max, self.policy = n_min, n_max, policy
        self.tokens: list[int] = []
        # succ[n][context (n-1 tokens)][successor] = [count, last position of the successor]
        self.succ: dict[int, dict[tuple, dict[int, list[int]]]] = {
            n: {} for n in range(n_min, n_max + 1)}

    # -- Initialize / Update (Section 3.1) -----------------------------------
    def update(self, tok: int) -> None:
        """Commit one token: at every level n it is paired with its previous n-1 tokens."""
        self.tokens.append(int(tok))
        t = len(self.tokens) - 1
        for n in range(self.n_min, self.n_max + 1):
            if t < n - 1:
                continue
            ctx = tuple(self.tokens[t - n + 1:t])
            rec = self.succ[n].setdefault(ctx, {}).setdefault(int(tok), [0, -1])
            rec[0] += 1
            rec[1] = t

    def initialize(self, token_ids) -> None:
        """Initialize = the statistics of the whole prompt = Update for each id in order."""
        for tok in token_ids:
            self.update(tok)

    # -- Query (Section 3.1) and MLN back-off (Algorithm 2) -------------------
    def query_level(self, n: int, ctx) -> int | None:
        """Most probable next token after the last n-1 tokens of `ctx`, or None."""
        if len(ctx) < n - 1:
            return None
        key = tuple(int(x) for x in ctx[len(ctx) - (n - 1):])
        cands = self.succ[n].get(key)
        if not cands:
            return None
        if self.policy == POLICY_MAX_COUNT:
            return max(cands.items(), key=lambda kv: (kv[1][0], kv[1][1]))[0]
        return max(cands.items(), key=lambda kv: kv[1][1])[0]

    def query(self, ctx) -> int | None:
        """Multi-level back-off (Section 3.2, Algorithm 2): the answer of the highest level
        n in [n_min, n_max] whose table knows the last n-1 tokens of `ctx`; None if no level does."""
        answers = (self.query_level(n, ctx) for n in range(self.n_max, self.n_min - 1, -1))
        return next((a for a in answers if a is not None), None)

    def draft(self, K: int) -> list[int]:
        """Drafting stage (Section 3.1, Algorithm 1's inner loop): K chained queries,
        each answer appended to a temporary context; stops at the first miss on
        every level.  The tables are not modified."""
        ctx = list(self.tokens[-(self.n_max - 1):]) if self.n_max > 1 else []
        out: list[int] = []
        for _ in range(K):
            s = self.query(ctx)
            if s is None:
                break
            out.append(s)
            ctx.append(s)
        return out

    def draft_alternative(self, first: int | None, K: int) -> list[int]:
        """A second candidate for the same step (the paper's conclusion names verifying several candidates at
        once as future work; this is the reading taken here).  Its first token is the answer of the highest
        level whose answer DIFFERS from `first` (the first token of `draft`): where the longest matching context
        and a shorter one disagree about the next token, the shorter one's answer is the alternative.  The
        candidate then continues like `draft`, by chained back-off queries on its own temporary context, up to
        K tokens in all.  Empty if K is 0, if `first` is None (nothing was drafted) or if no level disagrees."""
        if K <= 0 or first is None:
            return []
        ctx = list(self.tokens[-(self.n_max - 1):]) if self.n_max > 1 else []
        answers = (self.query_level(n, ctx) for n in range(self.n_max, self.n_min - 1, -1))
        alt = next((a for a in answers if a is not None and a != int(first)), None)
        if alt is None:
            return []
        out = [alt]
        ctx.append(alt)
        while len(out) < K:
            s = self.query(ctx)
            if s is None:
                break
            out.append(s)
            ctx.append(s)
        return out

    # -- canonical dumps, for comparing with another implementation ----------
    def dump(self, n: int) -> list[tuple[tuple, int, int, int]]:
        """Every level-n record as (context, successor, count, last_pos), sorted."""
        rows = []
        for ctx, cands in self.succ[n].items():
            for s, (c, last) in cands.items():
                rows.append((ctx, s, c, last))
        rows.sort()
        return rows

    def dump_best(self, n: int) -> list[tuple[tuple, int]]:
        """(context, answer of query_level) for every context of level n, sorted."""
        return sorted((ctx, self.query_level(n, list(ctx))) for ctx in self.succ[n])
