"""A decoder whose greedy continuation is known in closed form, and prompts that make an n-gram module right a
chosen fraction of the time.

Random-init weights never continue their prompt, so on the random workloads every draft is rejected.  To measure the
method at work on a full-size shape, this module builds inputs of the SAME shape and byte traffic with a controlled
answer:

  - the model ("orbit model"): the output projections of attention and FFN (wo, w_down) are zero, so the residual
    stream stays the embedding; tokens 0..S-1 (S <= d_model) embed as unit vectors and the LM head holds a
    permutation pi of them, so the model's argmax after token t is pi(t), whatever the context.  pi is one cycle
    through all S tokens.  Every other matrix is random as usual: a step streams and multiplies the same bytes as the
    random model's.
  - the prompt: the orbit y, pi(y), pi^2(y), ... with each token independently replaced by a random one with
    probability `corrupt`, closed by an early orbit token, so that the continuation re-walks a stretch the prompt has
    already shown.  Where the prompt is intact an n-gram draft is right; at a replaced token it is wrong, and the token
    after it has no precedent (no draft) - so `corrupt` sets the hit ratio.

Nothing here is part of the decoding method; these are inputs, handed to the CPU oracle and the CUDA library alike.
"""
from __future__ import annotations

import numpy as np
import torch

from .models import ModelShape, make_weights
from .rng import hash_at, uniform_at, randint_at

_S_PERM, _S_CORRUPT, _S_NOISE = 11, 12, 13


def orbit_permutation(S: int, seed: int) -> np.ndarray:
    """pi as an array (pi[t] = successor of t): one cycle through 0..S-1 in a seeded random order."""
    keys = np.array([hash_at(seed, _S_PERM, i) for i in range(S)], dtype=np.uint64)
    order = np.argsort(keys, kind="stable")                    # the cycle visits order[0], order[1], ...
    pi = np.empty(S, dtype=np.int64)
    pi[order] = np.roll(order, -1)
    return pi


def make_orbit_weights(s: ModelShape, seed: int, S: int, device="cpu", bf16: bool = True) -> tuple[dict[str, torch.Tensor], np.ndarray]:
    """(weights, pi).  Matrices as in the random workloads (bf16 for the full-size shapes); wo and w_down zero;
    embed / lm_head as above."""
    assert S <= s.d_model and S <= s.vocab
    w = make_weights(s, seed, bf16, device=device)
    for l in range(s.n_layers):
        w[f"l{l}.wo"].zero_()
        w[f"l{l}.w_down"].zero_()
    pi = orbit_permutation(S, seed)
    idx = torch.arange(S, device=device)
    w["embed"][:S].zero_()
    w["embed"][idx, idx] = 1.0                                 # token t -> unit vector e_t
    w["lm_head"].zero_()
    w["lm_head"][torch.from_numpy(pi).to(device), idx] = 1.0   # logit of pi(t) reads dimension t
    return w, pi


def orbit_prompt(pi: np.ndarray, length: int, corrupt: float, seed: int, replay_from: int = 8) -> np.ndarray:
    """int32[length]: the orbit from a seeded start with corrupted tokens, closed by its own token `replay_from`."""
    S = len(pi)
    t = randint_at(seed, _S_NOISE, 0, 0, S - 1)
    clean = []
    for _ in range(length - 1):
        clean.append(t)
        t = int(pi[t])
    out = list(clean)
    for i in range(replay_from + 1, length - 1):               # the replay's first token stays intact
        if uniform_at(seed, _S_CORRUPT, i) < corrupt:
            out[i] = randint_at(seed, _S_NOISE, i + 1, 0, S - 1)
    out.append(clean[replay_from])
    return np.asarray(out, dtype=np.int32)


def orbit_fork_prompt(pi: np.ndarray, length: int, seed: int, every: int = 9) -> np.ndarray:
    """int32[length]: a stretch of the orbit shown three times, closed by the stretch's first token, built so that at
    every `every`-th token d of the stretch (predecessor c, successor e) a decoding step STARTS at d with n-gram
    tables whose long contexts are misleading and whose one-token context is right:
      - the first showing replaces e by a random token x: the only time d stood behind c it was followed by x;
      - the other two showings insert a token z between c and d: c is followed by z twice (so the draft made at c is
        wrong and the next step starts at d), and d, now behind z, is followed by e twice.
    A module that verifies one candidate drafts x after d; one that also verifies the answer of a shorter level drafts e
    as well.  Leading tokens, if any, are random filler."""
    S = len(pi)
    L = 8
    while 3 * (L + 1) + 2 * len(range(4, L + 1 - 2, every)) + 1 <= length:
        L += 1
    forks = list(range(4, L - 2, every))
    t = randint_at(seed, _S_NOISE, 0, 0, S - 1)
    stretch = []
    for _ in range(L):
        stretch.append(t)
        t = int(pi[t])
    def other(k, avoid):
        r = randint_at(seed, _S_NOISE, 1 + k, 0, S - 1)
        return r if r != avoid else (r + 1) % S
    body = []
    for rep in range(3):
        for i, tok in enumerate(stretch):
            if rep > 0 and i in forks:
                body.append(other(2 * i, stretch[i]))                   # z: the same in both showings
            body.append(other(2 * i + 1, tok) if (rep == 0 and i - 1 in forks) else tok)
    body.append(stretch[0])
    fill = [randint_at(seed, _S_NOISE, 1 + 2 * L + k, 0, S - 1) for k in range(length - len(body))]
    return np.asarray(fill + body, dtype=np.int32)


def orbit_continuation(pi: np.ndarray, last_tok: int, n: int) -> np.ndarray:
    """The model's greedy output after a prompt ending in last_tok: pi(last), pi^2(last), ..."""
    out, t = [], int(last_tok)
    for _ in range(n):
        t = int(pi[t])
        out.append(t)
    return np.asarray(out, dtype=np.int32)


class ScriptedOrbitModel:
    """The orbit model as a stand-in for oracle.anpd's `model` argument: logits put 1 on pi(token), 0 elsewhere."""

    class _Cache:
        def __init__(self):
            self.length = 0

        def truncate(self, n):
            assert 0 <= n <= self.length
            self.length = n

    def __init__(self, pi: np.ndarray, vocab: int):
        self.pi, self.vocab = pi, vocab

    def new_cache(self):
        return self._Cache()

    def forward(self, tokens, cache):
        toks = [int(t) for t in tokens]
        logits = torch.zeros(len(toks), self.vocab, dtype=torch.float64)
        for r, t in enumerate(toks):
            logits[r, int(self.pi[t])] = 1.0
        cache.length += len(toks)
        return logits


def workload_inputs(wl, device="cpu"):
    """(weights, prompts, expected): the inputs of workload `wl`; `expected` is the closed-form greedy continuation
    (one int32 array per sequence) for an orbit workload, None for a random-init one."""
    from .models import make_prompts
    if wl.orbit_S == 0:
        return make_weights(wl.shape, wl.weight_seed, wl.weights_bf16, device=device), make_prompts(wl), None
    w, pi = make_orbit_weights(wl.shape, wl.weight_seed, wl.orbit_S, device=device, bf16=wl.weights_bf16)
    prompts = [orbit_prompt(pi, wl.prompt_len, wl.corrupt, wl.prompt_seed + 7919 * b) for b in range(wl.batch)]
    expected = [orbit_continuation(pi, p[-1], wl.max_new + 8) for p in prompts]
    return w, prompts, expected
