"""ctypes binding of libanpd_b200.so: argument marshalling only.

Every function here has the name of the C entry point it calls (include/anpd.h)
and does nothing but convert arguments and check the status.  There is no
Python or CPU implementation behind any call: if the shared library is missing
the import of `lib()` raises, and without a CUDA device the library itself
returns ANPD_ERR_CUDA.
"""
from __future__ import annotations

import ctypes as C
import os

import numpy as np

HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(HERE, "libanpd_b200.so")

K_MAX, N_MAX, ROWS = 7, 8, 8

OK, ERR_ARG, ERR_OOM, ERR_CAPACITY, ERR_RANGE, ERR_CUDA, ERR_STATE = 0, -1, -2, -3, -4, -5, -6


class AnpdError(RuntimeError):
    def __init__(self, status: int, what: str):
        super().__init__(f"{what}: status {status} ({status_string(status)})")
        self.status = status


class ModelConfig(C.Structure):
    _fields_ = [("n_layers", C.c_int), ("d_model", C.c_int), ("n_q_heads", C.c_int), ("n_kv_heads", C.c_int),
                ("head_dim", C.c_int), ("d_ffn", C.c_int), ("vocab", C.c_int),
                ("rope_theta", C.c_float), ("rms_eps", C.c_float)]


class NgramConfig(C.Structure):
    _fields_ = [("n_min", C.c_int), ("n_max", C.c_int), ("max_ctx", C.c_int), ("policy", C.c_int)]


class NgramEntry(C.Structure):
    _fields_ = [("key", C.c_int32 * (N_MAX - 1)), ("succ", C.c_int32), ("count", C.c_int32), ("last_pos", C.c_int32)]


class Stats(C.Structure):
    _fields_ = [("steps", C.c_int), ("drafted", C.c_int), ("accepted", C.c_int), ("generated", C.c_int),
                ("hist_accepted", C.c_int * 8), ("alt_wins", C.c_int), ("reserved", C.c_int), ("ms_prefill", C.c_double), ("ms_decode", C.c_double),
                ("bytes_per_step", C.c_double)]

    def as_dict(self) -> dict:
        return {"steps": self.steps, "drafted": self.drafted, "accepted": self.accepted, "generated": self.generated,
                "hist_accepted": list(self.hist_accepted), "alt_wins": self.alt_wins, "ms_prefill": self.ms_prefill, "ms_decode": self.ms_decode,
                "bytes_per_step": self.bytes_per_step}


class Profile(C.Structure):
    _fields_ = [("ms_gemm", C.c_double), ("n_gemm", C.c_int), ("ms_attn", C.c_double), ("n_attn", C.c_int),
                ("ms_other", C.c_double), ("n_other", C.c_int), ("ms_ngram", C.c_double), ("n_ngram", C.c_int),
                ("gemm_bytes", C.c_double)]


_P = C.c_void_p
_I32P = C.POINTER(C.c_int32)
_IP = C.POINTER(C.c_int)

# name -> (restype, argtypes); the list the ABI test checks against include/anpd.h
SIGNATURES = {
    "anpd_model_create": (C.c_int, [C.POINTER(ModelConfig), C.POINTER(_P), C.c_int, C.c_int, _P, C.POINTER(_P)]),
    "anpd_model_destroy": (C.c_int, [_P]),
    "anpd_kv_create": (C.c_int, [_P, C.c_int, C.c_int, C.c_int, C.POINTER(_P)]),
    "anpd_kv_destroy": (C.c_int, [_P]),
    "anpd_kv_len": (C.c_int, [_P, C.c_int, _IP]),
    "anpd_kv_truncate": (C.c_int, [_P, C.c_int, C.c_int]),
    "anpd_kv_set_candidates": (C.c_int, [_P, C.c_int]),
    "anpd_ngram_create": (C.c_int, [C.POINTER(NgramConfig), _P, C.POINTER(_P)]),
    "anpd_ngram_reset": (C.c_int, [_P]),
    "anpd_ngram_destroy": (C.c_int, [_P]),
    "anpd_ngram_len": (C.c_int, [_P, _IP]),
    "anpd_ngram_update": (C.c_int, [_P, _I32P, C.c_int]),
    "anpd_ngram_draft": (C.c_int, [_P, C.c_int, _I32P, _IP]),
    "anpd_ngram_dump": (C.c_int, [_P, C.c_int, C.POINTER(NgramEntry), C.c_int, _IP]),
    "anpd_ngram_dump_best": (C.c_int, [_P, C.c_int, C.POINTER(NgramEntry), C.c_int, _IP]),
    "anpd_prefill": (C.c_int, [_P, _P, C.c_int, _I32P, C.c_int, _I32P]),
    "anpd_verify": (C.c_int, [_P, _P, C.c_int32, _I32P, C.c_int, _IP, _I32P]),
    "anpd_verify_batch": (C.c_int, [_P, _P, _I32P, _I32P, _IP, _IP, _I32P]),
    "anpd_verify_logits": (C.c_int, [_P, _P, C.c_int32, _I32P, C.c_int, C.POINTER(C.c_float)]),
    "anpd_verify_two_candidates": (C.c_int, [_P, _P, C.c_int32, _I32P, C.c_int, _I32P, C.c_int, _IP, _I32P, _IP, C.POINTER(C.c_float)]),
    "anpd_verify_stage": (C.c_int, [_P, _P, _I32P, _I32P, _IP]),
    "anpd_verify_enqueue": (C.c_int, [_P, _P]),
    "anpd_verify_result": (C.c_int, [_P, _P, _IP, _I32P]),
    "anpd_generate": (C.c_int, [_P, _P, _P, _I32P, C.c_int, C.c_int, C.c_int, _I32P, _IP, C.POINTER(Stats)]),
    "anpd_generate_dev": (C.c_int, [_P, _P, _P, _P, C.c_int, C.c_int, C.c_int, _P, _IP, C.POINTER(Stats)]),
    "anpd_generate_batch": (C.c_int, [_P, _P, C.POINTER(_P), _I32P, C.c_int, C.c_int, C.c_int, _I32P, C.POINTER(Stats)]),
    "anpd_profile_enable": (C.c_int, [_P, C.c_int]),
    "anpd_profile_read": (C.c_int, [_P, C.POINTER(Profile), C.c_int]),
    "anpd_launch_count": (C.c_longlong, [C.c_int]),
    "anpd_debug_gemm": (C.c_int, [C.POINTER(C.c_uint16), C.c_int, C.c_int, C.POINTER(C.c_float), C.c_int,
                                  C.POINTER(C.c_float), C.c_int]),
    "anpd_gemm_static": (C.c_int, [_P, C.c_int, C.c_int, _P, C.c_int, _P, _P]),
    "anpd_status_string": (C.c_char_p, [C.c_int]),
}

_lib = None


def lib() -> C.CDLL:
    """The loaded shared library; raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(f"{LIB_PATH} is missing: build it with paper_2404_08698_b200.build.build() "
                              "(there is no fallback implementation)")
        handle = C.CDLL(LIB_PATH)
        for name, (res, args) in SIGNATURES.items():
            fn = getattr(handle, name)
            fn.restype, fn.argtypes = res, args
        _lib = handle
    return _lib


def status_string(status: int) -> str:
    return lib().anpd_status_string(status).decode()


def _check(status: int, what: str) -> None:
    if status != OK:
        raise AnpdError(status, what)


def _i32(a) -> np.ndarray:
    return np.ascontiguousarray(np.asarray(a, dtype=np.int32).reshape(-1))


def _ptr(a: np.ndarray, typ=_I32P):
    return a.ctypes.data_as(typ)


# ---- model ----------------------------------------------------------------------------------
def anpd_model_create(shape, tensors: list, stream: int = 0) -> int:
    """`shape`: object with the anpd_model_config fields.  `tensors`: torch tensors in the
    documented order, all on the host or all on one CUDA device, matrices all bf16 or all fp32
    (norm gains fp32).  Returns the handle."""
    cfg = ModelConfig(shape.n_layers, shape.d_model, shape.n_q_heads, shape.n_kv_heads, shape.head_dim,
                      shape.d_ffn, shape.vocab, shape.rope_theta, shape.rms_eps)
    import torch
    mats = [t for t in tensors if t.dim() == 2]
    bf16 = all(t.dtype == torch.bfloat16 for t in mats)
    assert bf16 or all(t.dtype == torch.float32 for t in mats)
    assert all(t.dtype == torch.float32 for t in tensors if t.dim() == 1)
    on_dev = all(t.is_cuda for t in tensors)
    assert on_dev or not any(t.is_cuda for t in tensors)
    keep = [t.contiguous() for t in tensors]
    arr = (_P * len(keep))(*[t.data_ptr() for t in keep])
    out = _P()
    _check(lib().anpd_model_create(C.byref(cfg), arr, int(bf16), int(on_dev), _P(stream), C.byref(out)), "anpd_model_create")
    return out.value


def anpd_model_destroy(m: int) -> None:
    _check(lib().anpd_model_destroy(_P(m)), "anpd_model_destroy")


# ---- KV -------------------------------------------------------------------------------------
def anpd_kv_create(m: int, max_len: int, batch: int = 1, shuffle_pages: bool = False) -> int:
    out = _P()
    _check(lib().anpd_kv_create(_P(m), max_len, batch, int(shuffle_pages), C.byref(out)), "anpd_kv_create")
    return out.value


def anpd_kv_destroy(kv: int) -> None:
    _check(lib().anpd_kv_destroy(_P(kv)), "anpd_kv_destroy")


def anpd_kv_len(kv: int, seq: int = 0) -> int:
    n = C.c_int()
    _check(lib().anpd_kv_len(_P(kv), seq, C.byref(n)), "anpd_kv_len")
    return n.value


def anpd_kv_truncate(kv: int, seq: int, length: int) -> None:
    _check(lib().anpd_kv_truncate(_P(kv), seq, length), "anpd_kv_truncate")


def anpd_kv_set_candidates(kv: int, candidates: int) -> None:
    _check(lib().anpd_kv_set_candidates(_P(kv), candidates), "anpd_kv_set_candidates")


# ---- n-gram ---------------------------------------------------------------------------------
def anpd_ngram_create(n_min: int, n_max: int, max_ctx: int, policy: int = 0, stream: int = 0) -> int:
    cfg = NgramConfig(n_min, n_max, max_ctx, policy)
    out = _P()
    _check(lib().anpd_ngram_create(C.byref(cfg), _P(stream), C.byref(out)), "anpd_ngram_create")
    return out.value


def anpd_ngram_reset(ctx: int) -> None:
    _check(lib().anpd_ngram_reset(_P(ctx)), "anpd_ngram_reset")


def anpd_ngram_destroy(ctx: int) -> None:
    _check(lib().anpd_ngram_destroy(_P(ctx)), "anpd_ngram_destroy")


def anpd_ngram_len(ctx: int) -> int:
    n = C.c_int()
    _check(lib().anpd_ngram_len(_P(ctx), C.byref(n)), "anpd_ngram_len")
    return n.value


def anpd_ngram_update(ctx: int, new_tokens) -> None:
    a = _i32(new_tokens)
    _check(lib().anpd_ngram_update(_P(ctx), _ptr(a), a.size), "anpd_ngram_update")


def anpd_ngram_draft(ctx: int, K: int) -> list[int]:
    buf = np.zeros(max(K, 1), dtype=np.int32)
    n = C.c_int()
    _check(lib().anpd_ngram_draft(_P(ctx), K, _ptr(buf), C.byref(n)), "anpd_ngram_draft")
    return buf[:n.value].tolist()


def _dump(fn, ctx: int, n: int, what: str):
    cnt = C.c_int()
    _check(fn(_P(ctx), n, None, 0, C.byref(cnt)), what)
    arr = (NgramEntry * max(cnt.value, 1))()
    _check(fn(_P(ctx), n, arr, cnt.value, C.byref(cnt)), what)
    return [(tuple(e.key[:n - 1]), e.succ, e.count, e.last_pos) for e in arr[:cnt.value]]


def anpd_ngram_dump(ctx: int, n: int):
    """[(context, successor, count, last_pos)] sorted."""
    return _dump(lib().anpd_ngram_dump, ctx, n, "anpd_ngram_dump")


def anpd_ngram_dump_best(ctx: int, n: int):
    return _dump(lib().anpd_ngram_dump_best, ctx, n, "anpd_ngram_dump_best")


# ---- verification ---------------------------------------------------------------------------
def anpd_prefill(m: int, kv: int, prompt, seq: int = 0) -> int:
    a = _i32(prompt)
    first = C.c_int32()
    _check(lib().anpd_prefill(_P(m), _P(kv), seq, _ptr(a), a.size, C.byref(first)), "anpd_prefill")
    return first.value


def anpd_verify(m: int, kv: int, last_tok: int, draft) -> tuple[int, int]:
    d = _i32(draft)
    acc, nxt = C.c_int(), C.c_int32()
    _check(lib().anpd_verify(_P(m), _P(kv), int(last_tok), _ptr(d) if d.size else None, d.size,
                             C.byref(acc), C.byref(nxt)), "anpd_verify")
    return acc.value, nxt.value


def _pack_batch(last_tok, drafts):
    lt = _i32(last_tok)
    B = lt.size
    dl = np.asarray([len(d) for d in drafts], dtype=np.int32)
    dr = np.zeros((B, K_MAX), dtype=np.int32)
    for b, d in enumerate(drafts):
        dr[b, :len(d)] = d
    return lt, dr, dl


def anpd_verify_batch(m: int, kv: int, last_tok, drafts) -> tuple[list[int], list[int]]:
    lt, dr, dl = _pack_batch(last_tok, drafts)
    acc = np.zeros(lt.size, dtype=np.int32)
    nxt = np.zeros(lt.size, dtype=np.int32)
    _check(lib().anpd_verify_batch(_P(m), _P(kv), _ptr(lt), _ptr(dr), _ptr(dl, _IP), _ptr(acc, _IP), _ptr(nxt)),
           "anpd_verify_batch")
    return acc.tolist(), nxt.tolist()


def anpd_verify_logits(m: int, kv: int, last_tok: int, draft, vocab: int) -> np.ndarray:
    d = _i32(draft)
    out = np.zeros((d.size + 1, vocab), dtype=np.float32)
    _check(lib().anpd_verify_logits(_P(m), _P(kv), int(last_tok), _ptr(d) if d.size else None, d.size,
                                    out.ctypes.data_as(C.POINTER(C.c_float))), "anpd_verify_logits")
    return out


def anpd_verify_two_candidates(m: int, kv: int, last_tok: int, draft_a, draft_b, vocab: int = 0):
    """(chosen, accepted_len, next_tok, logits or None); logits [(1 + len_a + len_b), vocab] when vocab > 0."""
    a, b = _i32(draft_a), _i32(draft_b)
    acc, nxt, chosen = C.c_int(), C.c_int32(), C.c_int()
    out = np.zeros((1 + a.size + b.size, vocab), dtype=np.float32) if vocab > 0 else None
    _check(lib().anpd_verify_two_candidates(_P(m), _P(kv), int(last_tok), _ptr(a) if a.size else None, a.size,
                                            _ptr(b) if b.size else None, b.size, C.byref(acc), C.byref(nxt), C.byref(chosen),
                                            out.ctypes.data_as(C.POINTER(C.c_float)) if out is not None else None),
           "anpd_verify_two_candidates")
    return chosen.value, acc.value, nxt.value, out


def anpd_verify_stage(m: int, kv: int, last_tok, drafts) -> None:
    lt, dr, dl = _pack_batch(last_tok, drafts)
    _check(lib().anpd_verify_stage(_P(m), _P(kv), _ptr(lt), _ptr(dr), _ptr(dl, _IP)), "anpd_verify_stage")


def anpd_verify_enqueue(m: int, kv: int) -> None:
    _check(lib().anpd_verify_enqueue(_P(m), _P(kv)), "anpd_verify_enqueue")


def anpd_verify_result(m: int, kv: int, batch: int = 1) -> tuple[list[int], list[int]]:
    acc = np.zeros(batch, dtype=np.int32)
    nxt = np.zeros(batch, dtype=np.int32)
    _check(lib().anpd_verify_result(_P(m), _P(kv), _ptr(acc, _IP), _ptr(nxt)), "anpd_verify_result")
    return acc.tolist(), nxt.tolist()


# ---- Algorithm 1 ----------------------------------------------------------------------------
def anpd_generate(m: int, kv: int, ctx: int, prompt, max_new: int, K: int) -> tuple[np.ndarray, dict]:
    p = _i32(prompt)
    out = np.zeros(max_new, dtype=np.int32)
    n_out = C.c_int()
    st = Stats()
    _check(lib().anpd_generate(_P(m), _P(kv), _P(ctx), _ptr(p), p.size, max_new, K, _ptr(out), C.byref(n_out),
                               C.byref(st)), "anpd_generate")
    return out[:n_out.value], st.as_dict()


def anpd_generate_dev(m: int, kv: int, ctx: int, prompt_dev, max_new: int, K: int, out_dev) -> dict:
    """prompt_dev / out_dev: int32 CUDA tensors (out_dev holds at least max_new elements)."""
    n_out = C.c_int()
    st = Stats()
    _check(lib().anpd_generate_dev(_P(m), _P(kv), _P(ctx), _P(prompt_dev.data_ptr()), prompt_dev.numel(), max_new, K,
                                   _P(out_dev.data_ptr()), C.byref(n_out), C.byref(st)), "anpd_generate_dev")
    return st.as_dict()


def anpd_generate_batch(m: int, kv: int, ctxs: list[int], prompts, max_new: int, K: int):
    p = np.ascontiguousarray(np.asarray(prompts, dtype=np.int32))
    B, plen = p.shape
    out = np.zeros((B, max_new), dtype=np.int32)
    st = (Stats * B)()
    arr = (_P * B)(*ctxs)
    _check(lib().anpd_generate_batch(_P(m), _P(kv), arr, _ptr(p), plen, max_new, K, _ptr(out), st), "anpd_generate_batch")
    return out, [s.as_dict() for s in st]


# ---- measurement ----------------------------------------------------------------------------
def anpd_profile_enable(m: int, on: bool) -> None:
    _check(lib().anpd_profile_enable(_P(m), int(on)), "anpd_profile_enable")


def anpd_profile_read(m: int, reset: bool = True) -> dict:
    pr = Profile()
    _check(lib().anpd_profile_read(_P(m), C.byref(pr), int(reset)), "anpd_profile_read")
    return {k: getattr(pr, k) for k, _ in Profile._fields_}


def anpd_launch_count(reset: bool = False) -> int:
    return int(lib().anpd_launch_count(int(reset)))


def anpd_debug_gemm(w_bf16, a, plain: int = 0) -> np.ndarray:
    """w_bf16: torch bf16 CPU tensor [N, K]; a: fp32 array [rows, K].  Returns out [rows, N] fp32.
    plain: 0 stream-K kernel, 1 plain cross-check kernel, 2 row-range kernel (8 rows)."""
    import torch
    N, K = w_bf16.shape
    wb = np.ascontiguousarray(w_bf16.contiguous().view(torch.int16).numpy().view(np.uint16))
    a = np.ascontiguousarray(np.asarray(a, dtype=np.float32))
    rows = a.shape[0]
    out = np.zeros((rows, N), dtype=np.float32)
    _check(lib().anpd_debug_gemm(wb.ctypes.data_as(C.POINTER(C.c_uint16)), N, K, a.ctypes.data_as(C.POINTER(C.c_float)), rows,
                                 out.ctypes.data_as(C.POINTER(C.c_float)), int(plain)), "anpd_debug_gemm")
    return out


def anpd_gemm_static(w_bf16_dev, a_dev, out_dev, stream: int = 0) -> None:
    """out_dev[rows, N] = a_dev[rows, K] @ w_bf16_dev[N, K]^T with no allocation inside the library.
    All three are CUDA tensors owned by the caller (bf16, fp32, fp32); out_dev is overwritten."""
    N, K = w_bf16_dev.shape
    rows = a_dev.shape[0]
    assert w_bf16_dev.is_cuda and a_dev.is_cuda and out_dev.is_cuda
    assert w_bf16_dev.is_contiguous() and a_dev.is_contiguous() and out_dev.is_contiguous()
    _check(lib().anpd_gemm_static(_P(w_bf16_dev.data_ptr()), N, K, _P(a_dev.data_ptr()), rows, _P(out_dev.data_ptr()),
                                  _P(stream)), "anpd_gemm_static")
