"""The optional persistent step kernel (ANPD_STEP_KERNEL=1: one kernel per decode step, csrc/step_kernel.cu) against the
oracle and against the closed-form orbit continuation.  It computes the same forward as the default chain of kernels with
another summation order (RMSNorm applied after the projection, pages merged by other threads), so it is held to the same
bars against the oracle rather than to bit equality with the default path."""
import numpy as np
import pytest
import torch

from helpers import gpu_model, new_stream, require_gpu
from oracle.decoder import Decoder
from test_gpu_orbit import run_orbit_workload, scripted
from workloads import ModelShape, make_weights, markov_prompt

pytestmark = pytest.mark.gpu

LOGIT_TOL = 2e-2
MARGIN = 5e-2


@pytest.fixture(scope="module")
def A():
    require_gpu()
    from paper_2404_08698_b200 import binding
    return binding


@pytest.mark.parametrize("shape,plen", [
    (ModelShape(1, 4096, 32, 32, 128, 11008, 32000), 2048),      # 7B width: 148 CTAs, three or four pages per CTA
    (ModelShape(2, 5120, 40, 40, 128, 13824, 32000), 700),       # 13B width, two layers: other splits, pages of a second layer
], ids=["d4096", "d5120"])
def test_step_kernel_logits_against_the_oracle(A, shape, plen, monkeypatch):
    monkeypatch.setenv("ANPD_STEP_KERNEL", "1")
    w = make_weights(shape, 11, True, device="cuda")
    torch.cuda.synchronize()
    m = gpu_model(A, shape, w, new_stream())
    w_cpu = {k: v.cpu() for k, v in w.items()}
    del w
    prompt = markov_prompt(plen, shape.vocab, 3, 4242 + plen, copy_spans=True).tolist()
    draft = [int(t) for t in markov_prompt(7, shape.vocab, 3, 99)]
    kv = A.anpd_kv_create(m, plen + 64)
    try:
        first = A.anpd_prefill(m, kv, prompt)
        before = A.anpd_launch_count(True)
        got = A.anpd_verify_logits(m, kv, first, draft, shape.vocab)
        launches = A.anpd_launch_count(True)
    finally:
        A.anpd_kv_destroy(kv)
        A.anpd_model_destroy(m)
    assert launches <= 4, launches                                # plan, step kernel, accept: the path under test really ran
    dec = Decoder(shape, w_cpu, torch.float64, kv_dtype=torch.bfloat16)
    cache = dec.new_cache()
    dec.forward(prompt, cache)
    want = dec.forward([first] + draft, cache)
    err = float((torch.from_numpy(got).double() - want).abs().max())
    print(f"d{shape.d_model}: step kernel vs bf16-cache oracle max-abs {err:.2e}")
    assert err <= LOGIT_TOL, err
    for r in range(want.shape[0]):
        t2 = torch.topk(want[r], 2).values
        if float(t2[0] - t2[1]) > MARGIN:
            assert int(np.argmax(got[r])) == int(torch.argmax(want[r])), r


def test_step_kernel_orbit_stream_at_the_7b_shape(A, monkeypatch):
    """Accepted prefixes of every length, KV commit and rollback through the step kernel: closed-form stream, ANPD == greedy
    bit for bit, loop statistics equal to the oracle's."""
    monkeypatch.setenv("ANPD_STEP_KERNEL", "1")
    alpha, _ = run_orbit_workload(A, "C3-A60", scripted)
    assert 0.5 < alpha < 0.7
