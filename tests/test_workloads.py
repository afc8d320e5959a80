"""The seeded input generators: determinism, agreement of the two hash
implementations, and the statistical shape the recipe promises."""
import numpy as np
import torch

from workloads import (TINY, S7B, WORKLOADS, make_weights, markov_prompt, periodic_prompt,
                       tensor_shapes)
from workloads.rng import hash_at, hash_tensor, normal_tensor, MASK64


def test_hash_python_and_torch_agree():
    for seed, stream, start in [(0, 0, 0), (5, 3, 10), (2**40 + 7, 99, 12345)]:
        h = hash_tensor(seed, stream, start, 64)
        assert [x & MASK64 for x in h.tolist()] == [hash_at(seed, stream, start + i) for i in range(64)]


def test_normal_moments_and_determinism():
    a = normal_tensor(11, 4, 200_000, 0.02)
    b = normal_tensor(11, 4, 200_000, 0.02, chunk=4096)
    assert torch.equal(a, b)
    assert abs(float(a.mean())) < 3e-4
    assert abs(float(a.std()) - 0.02) < 3e-4
    # tails exist (not a bounded approximation of a normal)
    assert float(a.abs().max()) > 0.02 * 3.5
    assert not torch.equal(a, normal_tensor(12, 4, 200_000, 0.02))


def test_weight_set_names_and_streamed_bytes():
    names = [n for n, _ in tensor_shapes(TINY)]
    assert names[0] == "embed" and names[-1] == "lm_head" and len(names) == 1 + 9 * 2 + 2
    w = make_weights(TINY, 0, False)
    assert w["l1.w_down"].shape == (256, 688) and w["l0.attn_norm"].eq(1).all()
    # bytes per verify step of the 7B shape quoted in the scope table: 13.214 GB + 524288 B/token
    assert abs(S7B.streamed_params * 2 / 1e9 - 13.214) < 1e-3
    assert S7B.kv_bytes_per_token == 524288
    wb = make_weights(TINY, 0, True)
    assert wb["l0.wq"].dtype == torch.bfloat16
    assert torch.equal(wb["l0.wq"], w["l0.wq"].to(torch.bfloat16))


def test_markov_prompt_shape():
    wl = WORKLOADS["C3"]
    p = markov_prompt(wl.prompt_len, wl.shape.vocab, 3, wl.prompt_seed, copy_spans=True)
    q = markov_prompt(wl.prompt_len, wl.shape.vocab, 3, wl.prompt_seed, copy_spans=True)
    assert p.dtype == np.int32 and p.shape == (1536,) and np.array_equal(p, q)
    assert p.min() >= 0 and p.max() < wl.shape.vocab
    # copied spans: a fair share of positions end an 8-gram already seen before
    seen, rep = set(), 0
    for i in range(8, len(p)):
        g = tuple(p[i - 8:i])
        rep += g in seen
        seen.add(g)
    assert 0.04 < rep / len(p) < 0.35
    plain = markov_prompt(1536, wl.shape.vocab, 3, wl.prompt_seed, copy_spans=False)
    seen, rep = set(), 0
    for i in range(8, len(plain)):
        g = tuple(plain[i - 8:i])
        rep += g in seen
        seen.add(g)
    assert rep / len(plain) < 0.02


def test_periodic_prompt():
    p = periodic_prompt(40, 7, 100, 3)
    assert len(set(p[:7].tolist())) == 7
    assert all(p[i] == p[i % 7] for i in range(40))


# ---- orbit workloads: a model with a closed-form continuation -------------------------------------
def test_orbit_permutation_is_one_cycle_and_prompt_replays_it():
    from workloads import orbit_continuation, orbit_permutation, orbit_prompt
    pi = orbit_permutation(97, 5)
    assert sorted(pi.tolist()) == list(range(97))
    t, n = 0, 0
    while True:
        t, n = int(pi[t]), n + 1
        if t == 0:
            break
    assert n == 97                                              # a single cycle through every token
    p = orbit_prompt(pi, 60, 0.0, 3)
    assert all(int(pi[p[i]]) == p[i + 1] for i in range(58))    # uncorrupted: the orbit itself
    assert p[-1] == p[8]                                        # closed by its own ninth token
    assert orbit_continuation(pi, p[-1], 20).tolist() == p[9:29].tolist()
    q = orbit_prompt(pi, 60, 0.5, 3)
    assert 10 < int((q[:-1] != p[:-1]).sum()) < 45 and q[:9].tolist() == p[:9].tolist()


def test_orbit_model_continues_its_orbit_under_the_oracle_decoder():
    """The real decoder on the orbit weights decodes exactly the closed-form continuation, and the scripted stand-in
    takes the same ANPD steps (it is what the full-size GPU tests compare their statistics with)."""
    import torch
    from oracle.anpd import anpd_generate, greedy
    from oracle.decoder import Decoder
    from workloads import WORKLOADS, ScriptedOrbitModel, orbit_permutation, workload_inputs
    wl = WORKLOADS["C1-A50"]
    w, prompts, expected = workload_inputs(wl)
    dec = Decoder(wl.shape, w, torch.float64)
    prompt = prompts[0].tolist()
    assert greedy(dec, prompt, 24) == expected[0][:24].tolist()
    out, st, _ = anpd_generate(dec, prompt, wl.max_new, wl.K, n_max=wl.n_max)
    pi = orbit_permutation(wl.orbit_S, wl.weight_seed)
    out2, st2, _ = anpd_generate(ScriptedOrbitModel(pi, wl.shape.vocab), prompt, wl.max_new, wl.K, n_max=wl.n_max)
    assert out == out2 == expected[0][:wl.max_new].tolist()
    assert (st.steps, st.drafted, st.accepted, st.hist_accepted, st.drafts, st.accepted_lens) == \
           (st2.steps, st2.drafted, st2.accepted, st2.hist_accepted, st2.drafts, st2.accepted_lens)
    assert 0.3 < st.hit_ratio < 0.8


def test_forked_orbit_prompt_makes_the_second_candidate_win():
    """orbit_fork_prompt: the stretch appears three times with the promised edits (a wrong successor once, an inserted
    token twice) and ends on the stretch's first token; under the oracle the one-candidate loop drafts the wrong token
    at every fork while the two-candidate loop's alternative is accepted there, so it takes fewer steps; the scripted
    stand-in and the real decoder on the orbit weights take the same steps."""
    from oracle.anpd import anpd_generate, anpd_generate_two_candidates
    from oracle.decoder import Decoder
    from workloads import ScriptedOrbitModel, make_orbit_weights, orbit_continuation, orbit_fork_prompt, orbit_permutation
    pi = orbit_permutation(211, 9)
    p = orbit_fork_prompt(pi, 150, 4, every=7).tolist()
    assert len(p) == 150 and p == orbit_fork_prompt(pi, 150, 4, every=7).tolist()
    # the last token opens the stretch; the stretch's second token follows it somewhere in the prompt
    first = p[-1]
    assert sum(1 for i in range(149) if p[i] == first and p[i + 1] == int(pi[first])) == 3
    # transitions that follow the orbit dominate; the edits are a minority
    on_orbit = sum(1 for i in range(149) if int(pi[p[i]]) == p[i + 1])
    assert 0.6 * 149 < on_orbit < 149
    mdl = ScriptedOrbitModel(pi, 256)
    want = orbit_continuation(pi, p[-1], 40).tolist()
    for policy in (0, 1):
        o1, s1, _ = anpd_generate(mdl, p, 40, 4, n_max=4, policy=policy)
        o2, s2, _ = anpd_generate_two_candidates(mdl, p, 40, 4, n_max=4, policy=policy)
        assert o1 == want and o2 == want
        assert s2.alt_wins >= 3 and s2.steps < s1.steps
    wl = WORKLOADS["C1-A50"]
    w, pi2 = make_orbit_weights(wl.shape, wl.weight_seed, wl.orbit_S, bf16=wl.weights_bf16)
    q = orbit_fork_prompt(pi2, wl.prompt_len, wl.prompt_seed).tolist()
    a, sa, _ = anpd_generate_two_candidates(Decoder(wl.shape, w, torch.float64), q, 32, 4, n_max=wl.n_max)
    b, sb, _ = anpd_generate_two_candidates(ScriptedOrbitModel(pi2, wl.shape.vocab), q, 32, 4, n_max=wl.n_max)
    assert a == b == orbit_continuation(pi2, q[-1], 32).tolist()
    assert (sa.steps, sa.drafts, sa.accepted_lens, sa.alt_wins) == (sb.steps, sb.drafts, sb.accepted_lens, sb.alt_wins) and sa.alt_wins > 0
