"""The CUDA verify forward against the oracle decoder: logits within 2e-2 (bf16 operands and
bf16 KV cache on the GPU, fp64 on the CPU), decisions equal wherever the oracle's top-2 margin
exceeds 5e-2, and bit-identical results regardless of row count or page order."""
import numpy as np
import pytest
import torch

from helpers import as_bf16_values, gpu_model, new_stream, require_gpu, top2_margin
from oracle.anpd import accept_length, argmax_lowest
from oracle.decoder import Decoder
from workloads import WORKLOADS, ModelShape, make_prompts, make_weights, markov_prompt

pytestmark = pytest.mark.gpu

LOGIT_TOL = 2e-2      # max-abs, GPU bf16 path vs CPU oracle
MARGIN = 5e-2         # decisions are compared only where the oracle's top-2 margin exceeds this


@pytest.fixture(scope="module")
def A():
    require_gpu()
    from paper_2404_08698_b200 import binding
    return binding


class Rig:
    def __init__(self, A, shape, seed=0, std=0.02, jitter=0.0, max_len=512, shuffle=False, bf16=False):
        self.A, self.shape = A, shape
        self.w = make_weights(shape, seed, bf16, std=std, norm_gain_jitter=jitter)
        self.m = gpu_model(A, shape, self.w)
        self.kv = A.anpd_kv_create(self.m, max_len, 1, shuffle)
        self.dec = Decoder(shape, {k: v.float() if v.dim() == 2 else v for k, v in self.w.items()}, torch.float64)
        self.dec_bf16 = Decoder(shape, as_bf16_values(self.w), torch.float64)

    def close(self):
        self.A.anpd_kv_destroy(self.kv)
        self.A.anpd_model_destroy(self.m)


@pytest.fixture(scope="module")
def c1(A):
    r = Rig(A, WORKLOADS["C1"].shape)
    yield r
    r.close()


def test_c1_logits_parity_after_prefill(A, c1):
    wl = WORKLOADS["C1"]
    prompt = make_prompts(wl)[0].tolist()
    A.anpd_kv_truncate(c1.kv, 0, 0)
    first = A.anpd_prefill(c1.m, c1.kv, prompt)
    assert A.anpd_kv_len(c1.kv) == len(prompt)
    cache = c1.dec.new_cache()
    lp = c1.dec.forward(prompt, cache)
    if top2_margin(lp[-1]) > MARGIN:
        assert first == argmax_lowest(lp[-1])
    # a verify step with a 7-token draft: all 8 rows against the oracle's logits
    draft = [int(t) for t in prompt[3:10]]
    got = A.anpd_verify_logits(c1.m, c1.kv, first, draft, wl.shape.vocab)
    assert A.anpd_kv_len(c1.kv) == len(prompt)                     # the hook commits nothing
    want = c1.dec.forward([first] + draft, cache)
    err = float((torch.from_numpy(got).double() - want).abs().max())
    assert err <= LOGIT_TOL, err
    # against the oracle on the bf16-rounded weight values only activation/KV rounding is left
    cb = c1.dec_bf16.new_cache()
    c1.dec_bf16.forward(prompt, cb)
    want_b = c1.dec_bf16.forward([first] + draft, cb)
    err_b = float((torch.from_numpy(got).double() - want_b).abs().max())
    assert err_b <= 5e-3, err_b


def test_verify_decisions_match_oracle(A, c1):
    wl = WORKLOADS["C1"]
    prompt = make_prompts(wl)[0].tolist()
    A.anpd_kv_truncate(c1.kv, 0, 0)
    last = A.anpd_prefill(c1.m, c1.kv, prompt)
    cache = c1.dec_bf16.new_cache()
    c1.dec_bf16.forward(prompt, cache)
    rng = np.random.default_rng(0)
    checked = 0
    for step in range(40):
        # a draft that follows the oracle's own predictions for `good` tokens, then departs
        P = cache.length
        k = int(rng.integers(0, 8))
        good = int(rng.integers(0, k + 1))
        draft, rows = [], [last]
        for i in range(k):
            lg = c1.dec_bf16.forward([rows[-1]], cache)
            t = argmax_lowest(lg[-1])
            if i >= good:
                t = (t + 1 + int(rng.integers(0, 5))) % wl.shape.vocab
            draft.append(t)
            rows.append(t)
        cache.truncate(P)
        logits = c1.dec_bf16.forward([last] + draft, cache)
        preds = [argmax_lowest(logits[r]) for r in range(k + 1)]
        a_want = accept_length(draft, preds)
        safe = all(top2_margin(logits[r]) > MARGIN for r in range(a_want + 1))
        a, nxt = A.anpd_verify(c1.m, c1.kv, last, draft)
        assert 0 <= a <= k and A.anpd_kv_len(c1.kv) == P + a + 1
        if safe:
            assert (a, nxt) == (a_want, preds[a_want]), (step, draft, preds)
            checked += 1
        # follow the library's decision so both sides stay on one stream
        cache.truncate(P + a + 1)
        last = nxt
    assert checked >= 5, checked


def test_rows_are_independent_of_row_count_and_drafts(A, c1):
    wl = WORKLOADS["C1"]
    prompt = make_prompts(wl)[0].tolist()[:100]
    A.anpd_kv_truncate(c1.kv, 0, 0)
    first = A.anpd_prefill(c1.m, c1.kv, prompt)
    draft = prompt[10:17]
    full = A.anpd_verify_logits(c1.m, c1.kv, first, draft, wl.shape.vocab)          # 8 real rows
    one = A.anpd_verify_logits(c1.m, c1.kv, first, [], wl.shape.vocab)              # 1 real row
    assert np.array_equal(full[0], one[0])
    part = A.anpd_verify_logits(c1.m, c1.kv, first, draft[:3], wl.shape.vocab)
    assert np.array_equal(full[:4], part)
    # row r of the wide step == row 0 of a one-row step taken after committing r tokens
    seq = [first] + draft
    for r in range(1, 6):
        # commit exactly one more token: a step whose (empty) draft accepts nothing
        A.anpd_verify(c1.m, c1.kv, seq[r - 1], [])
        assert A.anpd_kv_len(c1.kv) == len(prompt) + r
        single = A.anpd_verify_logits(c1.m, c1.kv, seq[r], [], wl.shape.vocab)
        assert np.array_equal(single[0], full[r]), r
    # roll back and redo: same bits again
    A.anpd_kv_truncate(c1.kv, 0, len(prompt))
    again = A.anpd_verify_logits(c1.m, c1.kv, first, draft, wl.shape.vocab)
    assert np.array_equal(again, full)


def test_page_order_does_not_matter(A):
    shape = WORKLOADS["C1"].shape
    prompt = markov_prompt(300, shape.vocab, 2, 77).tolist()          # three pages, ragged tail
    outs = []
    for shuffle in (False, True):
        r = Rig(A, shape, max_len=512, shuffle=shuffle)
        try:
            first = A.anpd_prefill(r.m, r.kv, prompt)
            outs.append((first, A.anpd_verify_logits(r.m, r.kv, first, prompt[5:12], shape.vocab)))
        finally:
            r.close()
    assert outs[0][0] == outs[1][0] and np.array_equal(outs[0][1], outs[1][1])


@pytest.mark.parametrize("shape,plen", [
    (ModelShape(2, 128, 8, 2, 64, 200, 512), 150),      # grouped-query, 4 q heads per kv head, hd 64
    (ModelShape(1, 256, 2, 2, 128, 264, 300), 131),     # hd 128, ragged vocab / ffn
    (ModelShape(2, 128, 8, 1, 64, 136, 1030), 9),       # 8 q heads on one kv head, prompt shorter than a pass
    (ModelShape(2, 256, 4, 2, 128, 264, 300), 200),     # hd 128 (tensor-memory attention), 2 q heads per kv head, two key pages
    (ModelShape(1, 256, 4, 1, 128, 136, 300), 140),     # hd 128, 4 q heads on one kv head
    (ModelShape(1, 256, 8, 1, 128, 136, 300), 130),     # hd 128, 8 q heads on one kv head
])
def test_other_shapes_logits_parity(A, shape, plen):
    r = Rig(A, shape, seed=11, std=0.05, jitter=0.1, max_len=256)
    try:
        prompt = markov_prompt(plen, shape.vocab, 2, 5).tolist()
        first = A.anpd_prefill(r.m, r.kv, prompt)
        cache = r.dec_bf16.new_cache()
        lp = r.dec_bf16.forward(prompt, cache)
        if top2_margin(lp[-1]) > MARGIN:
            assert first == argmax_lowest(lp[-1])
        draft = prompt[1:6]
        got = A.anpd_verify_logits(r.m, r.kv, first, draft, shape.vocab)
        want = r.dec_bf16.forward([first] + draft, cache)
        err = float((torch.from_numpy(got).double() - want).abs().max())
        assert err <= LOGIT_TOL, err
    finally:
        r.close()


def test_bf16_weight_input_equals_fp32_input_rounded(A):
    shape = ModelShape(1, 64, 1, 1, 64, 64, 128)
    w32 = make_weights(shape, 4, False, std=0.1)
    w16 = {k: (v.to(torch.bfloat16) if v.dim() == 2 else v) for k, v in w32.items()}
    outs = []
    for w in (w32, w16, {k: v.cuda() for k, v in w16.items()}):
        m = gpu_model(A, shape, w)
        kv = A.anpd_kv_create(m, 64)
        try:
            first = A.anpd_prefill(m, kv, [1, 2, 3, 4, 5])
            outs.append(A.anpd_verify_logits(m, kv, first, [7, 8], shape.vocab))
        finally:
            A.anpd_kv_destroy(kv)
            A.anpd_model_destroy(m)
    assert np.array_equal(outs[0], outs[1]) and np.array_equal(outs[1], outs[2])


def test_verify_error_paths(A, c1):
    A.anpd_kv_truncate(c1.kv, 0, 0)
    with pytest.raises(A.AnpdError) as e:
        A.anpd_verify(c1.m, c1.kv, 4096, [])                           # token id == vocab
    assert e.value.status == A.ERR_RANGE
    with pytest.raises(A.AnpdError) as e:
        A.anpd_verify(c1.m, c1.kv, 1, list(range(8)))                  # K > 7
    assert e.value.status == A.ERR_RANGE
    A.anpd_prefill(c1.m, c1.kv, [1, 2, 3])
    with pytest.raises(A.AnpdError) as e:
        A.anpd_prefill(c1.m, c1.kv, [1, 2, 3])                         # cache not empty
    assert e.value.status == A.ERR_STATE
    # a second committing step may not be enqueued before the outcome of the first is known to the host
    A.anpd_verify_stage(c1.m, c1.kv, [5], [[6, 7]])
    A.anpd_verify_enqueue(c1.m, c1.kv)
    with pytest.raises(A.AnpdError) as e:
        A.anpd_verify_enqueue(c1.m, c1.kv)
    assert e.value.status == A.ERR_STATE
    A.anpd_kv_truncate(c1.kv, 0, 3)                                    # tells the library the length again
    A.anpd_verify_enqueue(c1.m, c1.kv)
    acc, nxt = A.anpd_verify_result(c1.m, c1.kv)
    assert 0 <= acc[0] <= 2
    A.anpd_verify_enqueue(c1.m, c1.kv)                                 # allowed again after the result was read
    A.anpd_verify_result(c1.m, c1.kv)
    with pytest.raises(A.AnpdError) as e:
        A.anpd_kv_truncate(c1.kv, 0, 10)                               # cannot grow
    assert e.value.status == A.ERR_RANGE
    with pytest.raises(A.AnpdError) as e:
        A.anpd_prefill(c1.m, c1.kv, list(range(600)))                  # longer than the cache
    assert e.value.status in (A.ERR_STATE, A.ERR_CAPACITY)


def test_tensor_memory_attention_agrees_with_mma_sync_attention(A, monkeypatch):
    """Head dimension 128 has two attention kernels (tcgen05 with tensor-memory accumulators, and the
    mma.sync one that head dimension 64 always uses).  They add the keys of a page in different orders,
    so the logits agree closely but not bit for bit; three key pages, grouped-query heads."""
    shape = ModelShape(2, 256, 4, 2, 128, 264, 300)
    prompt = markov_prompt(300, shape.vocab, 2, 9).tolist()
    w = make_weights(shape, 21, False, std=0.05, norm_gain_jitter=0.1)
    outs = []
    for legacy in (False, True):
        if legacy:
            monkeypatch.setenv("ANPD_ATTN_MMA_SYNC", "1")
        else:
            monkeypatch.delenv("ANPD_ATTN_MMA_SYNC", raising=False)
        m = gpu_model(A, shape, w)
        kv = A.anpd_kv_create(m, 512)
        try:
            first = A.anpd_prefill(m, kv, prompt)
            outs.append((first, A.anpd_verify_logits(m, kv, first, prompt[2:9], shape.vocab)))
        finally:
            A.anpd_kv_destroy(kv)
            A.anpd_model_destroy(m)
    assert outs[0][0] == outs[1][0]
    # two summation orders of the same fp32 sums, seen through two layers and the LM head (measured: 1.0e-4)
    assert float(np.abs(outs[0][1] - outs[1][1]).max()) <= 3e-4


def test_long_context_attention_slots_take_several_pages(A, monkeypatch):
    """93 key pages x 8 kv heads = 744 work items for the persistent tensor-memory attention kernel, more than
    its 148 x 4 slots on a B200: some slots walk through two pages and reuse their buffers and barriers.  Also
    the page combine beyond 32 pages.  Checked against the oracle (prompt fed in chunks to bound its memory)
    and against the mma.sync attention kernel."""
    shape = ModelShape(1, 256, 8, 8, 128, 264, 300)
    plen = 92 * 128 + 57
    prompt = markov_prompt(plen, shape.vocab, 2, 13).tolist()
    w = make_weights(shape, 23, False, std=0.05, norm_gain_jitter=0.1)
    draft = prompt[5:12]
    outs = []
    for legacy in (False, True):
        if legacy:
            monkeypatch.setenv("ANPD_ATTN_MMA_SYNC", "1")
        else:
            monkeypatch.delenv("ANPD_ATTN_MMA_SYNC", raising=False)
        m = gpu_model(A, shape, w)
        kv = A.anpd_kv_create(m, 96 * 128)
        try:
            first = A.anpd_prefill(m, kv, prompt)
            outs.append((first, A.anpd_verify_logits(m, kv, first, draft, shape.vocab)))
        finally:
            A.anpd_kv_destroy(kv)
            A.anpd_model_destroy(m)
    assert outs[0][0] == outs[1][0]
    assert float(np.abs(outs[0][1] - outs[1][1]).max()) <= 1e-4
    dec = Decoder(shape, as_bf16_values(w), torch.float64)
    cache = dec.new_cache()
    lp = None
    for s in range(0, plen, 1024):
        lp = dec.forward(prompt[s:s + 1024], cache)
    if top2_margin(lp[-1]) > MARGIN:
        assert outs[0][0] == argmax_lowest(lp[-1])
    want = dec.forward([outs[0][0]] + draft, cache)
    err = float((torch.from_numpy(outs[0][1]).double() - want).abs().max())
    assert err <= LOGIT_TOL, err


@pytest.mark.parametrize("shape,plen", [(ModelShape(2, 256, 4, 4, 64, 688, 4096), 140),      # the tiny workload's shape
                                        (ModelShape(2, 512, 4, 2, 128, 1000, 3001), 300),    # hd 128, grouped heads, odd vocabulary, ragged K
                                        (ModelShape(1, 1024, 8, 1, 128, 2816, 5000), 90)])   # 8 query heads per kv head
def test_row_range_projections_logits_parity(A, monkeypatch, shape, plen):
    """The optional single-sequence path (ANPD_RR=1: projections with rotary/append, residual + deferred RMSNorm, SwiGLU
    and the vocabulary argmax fused into their epilogues) against the oracle, same bars as the default path."""
    monkeypatch.setenv("ANPD_RR", "1")
    r = Rig(A, shape, seed=31, jitter=0.1)
    try:
        prompt = markov_prompt(plen, shape.vocab, 2, 77).tolist()
        first = A.anpd_prefill(r.m, r.kv, prompt)
        draft = [int(t) for t in prompt[5:12]]
        got = A.anpd_verify_logits(r.m, r.kv, first, draft, shape.vocab)
        cache = r.dec.new_cache()
        r.dec.forward(prompt, cache)
        want = r.dec.forward([first] + draft, cache)
        err = float((torch.from_numpy(got).double() - want).abs().max())
        assert err <= LOGIT_TOL, err
        # and the committing step takes the decisions the logits imply
        acc, nxt = A.anpd_verify(r.m, r.kv, first, draft)
        preds = [int(np.argmax(got[i])) for i in range(8)]
        assert acc == accept_length(draft, preds) and nxt == preds[acc]
        assert A.anpd_kv_len(r.kv) == plen + acc + 1
    finally:
        r.close()


@pytest.mark.parametrize("shape,plen", [
    (ModelShape(2, 256, 2, 2, 128, 688, 4096), 2050),      # head dimension 128, one query head per kv head: the prompt kernels
    (ModelShape(2, 256, 4, 2, 64, 688, 4096), 2101),       # head dimension 64, grouped heads: page partials and their merge
], ids=["hd128", "hd64"])
def test_prompt_longer_than_one_pass(A, shape, plen):
    """A prompt of more than 2048 tokens takes two prompt passes; the second is short (2 and 53 tokens: 8 and 56 rows) and
    attends to the pages the first one wrote.  First token and the logits of a verify step after it against the oracle."""
    w = make_weights(shape, 5, False, std=0.05)
    prompt = markov_prompt(plen, shape.vocab, 2, 77).tolist()
    draft = [int(t) for t in markov_prompt(7, shape.vocab, 2, 78)]
    m = gpu_model(A, shape, w, new_stream())
    kv = A.anpd_kv_create(m, plen + 64)
    try:
        first = A.anpd_prefill(m, kv, prompt)
        got = A.anpd_verify_logits(m, kv, first, draft, shape.vocab)
    finally:
        A.anpd_kv_destroy(kv)
        A.anpd_model_destroy(m)
    dec = Decoder(shape, as_bf16_values(w), torch.float64, kv_dtype=torch.bfloat16)
    cache = dec.new_cache()
    lp = dec.forward(prompt, cache)
    if top2_margin(lp[-1]) > 5e-2:
        assert first == argmax_lowest(lp[-1])
    want = dec.forward([first] + draft, cache)
    err = float((torch.from_numpy(got).double() - want).abs().max())
    print(f"{plen} tokens, hd {shape.head_dim}: max-abs {err:.2e}")
    assert err <= 5e-3, err


@pytest.mark.parametrize("heads", [(2, 2), (4, 2), (4, 1)], ids=lambda h: f"g{h[0] // h[1]}")
@pytest.mark.parametrize("std", [0.05, 0.4])
def test_prompt_attention_with_128_row_tiles(A, monkeypatch, std, heads):
    """The prompt-pass attention with the query rows on the tensor-memory lanes (head dimension 128; 1, 2 and 4 query heads
    per kv head): prompts that end inside a row tile, on a page boundary and several tiles in, against the oracle and against
    the kernels it replaces (16 rows per slot; page partials + merge where query heads share a kv head).  At the larger
    weight scale the softmax is close to an argmax and the model amplifies any rounding: there the bar against the oracle
    is the oracle's own sensitivity to the cache's bf16 rounding (its distance to itself with a full-precision cache), as
    in the deep-model tests, and the comparison with the replaced kernels (same cache, same roundings elsewhere) is the
    sharp one.  The larger weight scale spreads the scores over many powers of two, so that the
    lazily moved reference maximum has to move (and the output accumulator be rescaled) inside a prompt."""
    shape = ModelShape(2, 256, heads[0], heads[1], 128, 320, 200)
    w = make_weights(shape, 17, False, std=std, norm_gain_jitter=0.1)
    dec = Decoder(shape, as_bf16_values(w), torch.float64, kv_dtype=torch.bfloat16)
    dec_plain = Decoder(shape, as_bf16_values(w), torch.float64)
    draft = [int(t) for t in markov_prompt(7, shape.vocab, 2, 5)]
    for plen in (5, 127, 128, 129, 300, 1000):
        prompt = markov_prompt(plen, shape.vocab, 2, 100 + plen).tolist()
        got = {}
        for old in (False, True):
            if old:
                monkeypatch.setenv("ANPD_ATTN_PROMPT_TILE16", "1")
            else:
                monkeypatch.delenv("ANPD_ATTN_PROMPT_TILE16", raising=False)
            m = gpu_model(A, shape, w)
            kv = A.anpd_kv_create(m, plen + 64, 1, True)
            try:
                first = A.anpd_prefill(m, kv, prompt)
                got[old] = (first, A.anpd_verify_logits(m, kv, first, draft, shape.vocab))
            finally:
                A.anpd_kv_destroy(kv)
                A.anpd_model_destroy(m)
        monkeypatch.delenv("ANPD_ATTN_PROMPT_TILE16", raising=False)
        cache = dec.new_cache()
        lp = dec.forward(prompt, cache)
        first = got[False][0]
        if top2_margin(lp[-1]) > 5e-2 * max(1.0, float(lp[-1].abs().max())):
            assert first == argmax_lowest(lp[-1])
        want = dec.forward([first] + draft, cache)
        scale = max(1.0, float(want.abs().max()))
        err = float((torch.from_numpy(got[False][1]).double() - want).abs().max())
        cp = dec_plain.new_cache()
        dec_plain.forward(prompt, cp)
        cache_effect = float((dec_plain.forward([first] + draft, cp) - want).abs().max())
        assert err <= max(5e-3 * scale, cache_effect), (plen, err, scale, cache_effect)
        if got[True][0] == first:                          # the two kernels sum in different orders: equal up to rounding
            cross = float(np.abs(got[False][1] - got[True][1]).max())
            assert cross <= 1e-3 * scale, (plen, cross, scale)
