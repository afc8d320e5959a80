"""ANPD with non-zero acceptance at every model size: orbit workloads (workloads/orbit.py).

A random-init decoder never continues its prompt, so on the random workloads every draft is rejected and the
accepted-prefix commit is never exercised at full width.  The orbit model has the shape and byte traffic of the
random model and a greedy continuation known in closed form; its prompts make the n-gram drafts right a chosen
fraction of the time.  The library's stream must equal the closed form, equal its own greedy stream, and its loop
statistics (steps, drafts proposed and accepted, histogram of accepted lengths) must equal those of the oracle's
Algorithm 1 run on the same prompt - with the full decoder oracle where it is small, with the scripted stand-in of
the orbit model (pinned against the decoder oracle in tests/test_workloads.py) at the 1.1B and 7B shapes."""
import numpy as np
import pytest
import torch

from helpers import gpu_model, new_stream, require_gpu
from oracle.anpd import anpd_generate as oracle_anpd
from oracle.decoder import Decoder
from workloads import WORKLOADS, ScriptedOrbitModel, orbit_permutation, workload_inputs

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def A():
    require_gpu()
    from paper_2404_08698_b200 import binding
    return binding


def run_orbit_workload(A, name, oracle_model_factory):
    wl = WORKLOADS[name]
    dev = "cuda" if wl.shape.streamed_params > 1e8 else "cpu"
    w, prompts, expected = workload_inputs(wl, device=dev)
    st = new_stream()
    m = gpu_model(A, wl.shape, w, st)
    max_len = wl.prompt_len + wl.max_new + 64
    kv = A.anpd_kv_create(m, max_len)
    ctx = A.anpd_ngram_create(wl.n_min, wl.n_max, max_len, 0, st)
    try:
        out, stats = A.anpd_generate(m, kv, ctx, prompts[0], wl.max_new, wl.K)
        greedy, gstats = A.anpd_generate(m, kv, ctx, prompts[0], wl.max_new, 0)
    finally:
        A.anpd_ngram_destroy(ctx)
        A.anpd_kv_destroy(kv)
        A.anpd_model_destroy(m)
    assert np.array_equal(out, greedy)                                           # losslessness, bit for bit
    assert out.tolist() == expected[0][:wl.max_new].tolist()                     # the closed-form continuation
    want, ost, _ = oracle_anpd(oracle_model_factory(wl, w), prompts[0].tolist(), wl.max_new, wl.K, n_max=wl.n_max, n_min=wl.n_min)
    assert want == out.tolist()
    assert (stats["steps"], stats["drafted"], stats["accepted"]) == (ost.steps, ost.drafted, ost.accepted)
    assert stats["hist_accepted"] == ost.hist_accepted
    assert stats["accepted"] > 0 and stats["steps"] < gstats["steps"] == wl.max_new
    return stats["accepted"] / stats["drafted"], wl.max_new / stats["steps"]


def scripted(wl, w):
    return ScriptedOrbitModel(orbit_permutation(wl.orbit_S, wl.weight_seed), wl.shape.vocab)


def test_tiny_orbit_workload_against_the_decoder_oracle(A):
    alpha, per_step = run_orbit_workload(A, "C1-A50", lambda wl, w: Decoder(wl.shape, w, torch.float64))
    assert 0.3 < alpha < 0.8 and per_step > 1.5


@pytest.mark.parametrize("name,lo,hi", [("C2-A40", 0.2, 0.5), ("C3-A20", 0.15, 0.27), ("C3-A60", 0.5, 0.7)])
def test_full_size_orbit_workloads(A, name, lo, hi):
    """Drafts accepted at the 1.1B and 7B shapes: commits of 1..K+1 rows per step at full width, statistics equal to the
    oracle's step by step (same histogram), hit ratio where the workload puts it."""
    alpha, per_step = run_orbit_workload(A, name, scripted)
    print(f"{name}: hit ratio {alpha:.3f}, {per_step:.2f} tokens per verify step")
    assert lo < alpha < hi, alpha


def test_row_range_projections_give_the_same_stream(A, monkeypatch):
    """The optional row-range projection kernels (ANPD_RR=1: fused epilogues, single-sequence steps) on the 1.1B orbit
    workload: same closed-form stream and statistics, i.e. the same decisions as the default path."""
    monkeypatch.setenv("ANPD_RR", "1")
    alpha, _ = run_orbit_workload(A, "C2-A40", scripted)
    assert 0.2 < alpha < 0.5
