"""Thin ctypes binding of libsled.so: same names as include/sled.h, argument marshalling only.

Every step of the verification path runs inside the CUDA library; this module only turns
Python objects into the plain pointers and sizes the C boundary takes.  There is no CPU
fallback: loading fails loudly when the library has not been built.
"""
from __future__ import annotations

import ctypes as C
import os

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libsled.so")

SLED_OK = 0
SLED_ERR_ARG, SLED_ERR_UNKNOWN_CTX, SLED_ERR_DUP_CTX, SLED_ERR_K_RANGE, SLED_ERR_TOKEN_RANGE = -1, -2, -3, -4, -5
SLED_ERR_NO_PAGES, SLED_ERR_BATCH_TOO_LARGE, SLED_ERR_NONFINITE, SLED_ERR_DEVICE, SLED_ERR_NO_DEVICE = -6, -7, -8, -9, -10
SLED_ERR_BASE_LEN = -11
SLED_F32, SLED_BF16 = 0, 1
SLED_PENDING = 1
SLED_BATCH_STATIC, SLED_BATCH_CONTINUOUS = 0, 1

EXPORTS = (
    "sled_init", "sled_verify_batch", "sled_release", "sled_prefill", "sled_set_sampling", "sled_get_stats",
    "sled_get_stream", "sled_shutdown", "sled_strerror", "sled_accept_rows", "sled_accept_rows_static", "sled_attention_ragged",
    "sled_debug_load_kv", "sled_debug_read_kv", "sled_debug_copy_logits", "sled_debug_truncate", "sled_debug_truncate_batch", "sled_debug_arm_wait_timeout",
    "sled_debug_set_commit", "sled_debug_set_timing", "sled_debug_query_ctx", "sled_debug_shuffle_pages",
    "sled_kvm_create", "sled_kvm_destroy", "sled_kvm_open", "sled_kvm_reserve_batch", "sled_kvm_commit",
    "sled_kvm_release", "sled_kvm_query", "sled_kvm_free_pages", "sled_kvm_pack", "sled_kvm_reserve_batch_at",
    "sled_kvm_commit_tokens", "sled_kvm_history",
    "sled_server_config", "sled_submit", "sled_step", "sled_poll", "sled_queued",
    "sled_planner_create", "sled_planner_destroy", "sled_planner_push", "sled_planner_next_batch", "sled_planner_queued",
    "sled_debug_plan_attention",
)


class SledConfig(C.Structure):
    _fields_ = [(n, C.c_int32) for n in
                ("n_layers", "d_model", "n_q_heads", "n_kv_heads", "head_dim", "ffn_dim", "vocab")] + [
        ("rms_eps", C.c_float), ("rope_theta", C.c_float), ("weight_dtype", C.c_int32), ("kv_dtype", C.c_int32),
        ("page_size", C.c_int32), ("n_pages", C.c_int32), ("max_batch", C.c_int32), ("max_k", C.c_int32),
        ("max_step_tokens", C.c_int32), ("temperature", C.c_float), ("greedy", C.c_int32),
        ("probs_on_device", C.c_int32), ("device_index", C.c_int32), ("stream", C.c_void_p),
        ("draft_probs_dtype", C.c_int32), ("attention_impl", C.c_int32), ("linear_weight_bits", C.c_int32)]


class SledWeights(C.Structure):
    _fields_ = [("tok_emb", C.c_void_p), ("final_norm", C.c_void_p), ("lm_head", C.c_void_p)] + [
        (n, C.POINTER(C.c_void_p)) for n in
        ("attn_norm", "wq", "wk", "wv", "wo", "ffn_norm", "w_gate", "w_up", "w_down")] + [
        ("lm_head_scale", C.c_void_p)] + [
        (n + "_scale", C.POINTER(C.c_void_p)) for n in ("wq", "wk", "wv", "wo", "w_gate", "w_up", "w_down")]


class SledRequest(C.Structure):
    _fields_ = [("ctx_id", C.c_uint64), ("draft_tokens", C.c_void_p), ("draft_probs", C.c_void_p), ("k", C.c_int32),
                ("base_len", C.c_int64)]


class SledResult(C.Structure):
    _fields_ = [("n_accepted", C.c_int32), ("next_token", C.c_int32), ("status", C.c_int32)]


class SledStats(C.Structure):
    _fields_ = [(n, C.c_int64) for n in ("steps", "requests", "tokens_scored", "drafts_accepted", "tokens_committed")] + [
        (n, C.c_int32) for n in ("pages_total", "pages_free", "contexts_open")] + [
        ("kernels_launched", C.c_int64), ("kernels_last_step", C.c_int64)] + [
        (n, C.c_float) for n in ("ms_linear", "ms_attention", "ms_accept", "ms_other", "ms_step")] + [
        ("linear_launches_last_step", C.c_int32), ("attention_launches_last_step", C.c_int32), ("ms_idle", C.c_float)]


class SledError(RuntimeError):
    def __init__(self, code: int, what: str):
        super().__init__(f"{what}: {strerror(code)} ({code})")
        self.code = code


_lib = None


def lib():
    """Loads libsled.so (raises if it has not been built: nothing else can run the path)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: build it with paper_2506_09397_b200.build.build(); "
                               "there is no fallback implementation")
        L = C.CDLL(LIB_PATH)
        P, I32, I64, U64, F = C.c_void_p, C.c_int32, C.c_int64, C.c_uint64, C.c_float
        sig = {
            "sled_init": (C.c_int, [C.POINTER(SledWeights), C.POINTER(SledConfig), C.POINTER(P)]),
            "sled_verify_batch": (C.c_int, [P, C.POINTER(SledRequest), I32, U64, C.POINTER(SledResult)]),
            "sled_release": (C.c_int, [P, U64]),
            "sled_prefill": (C.c_int, [P, U64, P, I32]),
            "sled_set_sampling": (C.c_int, [P, F, I32]),
            "sled_get_stats": (C.c_int, [P, C.POINTER(SledStats)]),
            "sled_get_stream": (P, [P]),
            "sled_shutdown": (None, [P]),
            "sled_strerror": (C.c_char_p, [C.c_int]),
            "sled_accept_rows": (C.c_int, [P, P, P, P, P, P, I32, I32, F, I32, U64, C.POINTER(SledResult), P,
                                           C.POINTER(F)]),
            "sled_accept_rows_static": (C.c_int, [P, P, P, P, P, P, I32, I32, F, I32, U64, C.POINTER(SledResult), P]),
            "sled_attention_ragged": (C.c_int, [P, I32, P, P, I32, P, P, C.POINTER(F)]),
            "sled_debug_load_kv": (C.c_int, [P, U64, P, P, I32, I32]),
            "sled_debug_read_kv": (C.c_int, [P, U64, I32, P, P, I32]),
            "sled_debug_copy_logits": (C.c_int, [P, P, I32]),
            "sled_debug_truncate": (C.c_int, [P, U64, I64, I32]),
            "sled_debug_truncate_batch": (C.c_int, [P, P, P, P, I32]),
            "sled_debug_arm_wait_timeout": (C.c_int, [P, I32]),
            "sled_debug_set_commit": (C.c_int, [P, I32]),
            "sled_debug_set_timing": (C.c_int, [P, I32]),
            "sled_debug_query_ctx": (C.c_int, [P, U64, C.POINTER(I64), C.POINTER(I32), C.POINTER(I32), P, I32]),
            "sled_debug_shuffle_pages": (C.c_int, [P, U64]),
            "sled_kvm_create": (P, [I32, I32]),
            "sled_kvm_destroy": (None, [P]),
            "sled_kvm_open": (C.c_int, [P, U64, I64, I32]),
            "sled_kvm_reserve_batch": (C.c_int, [P, P, P, I32]),
            "sled_kvm_commit": (C.c_int, [P, U64, I32, I32]),
            "sled_kvm_release": (C.c_int, [P, U64]),
            "sled_kvm_query": (C.c_int, [P, U64, C.POINTER(I64), C.POINTER(I32), C.POINTER(I32), P, I32]),
            "sled_kvm_free_pages": (I32, [P]),
            "sled_kvm_pack": (C.c_int, [P, P, P, P, I32, P, P, P, P, P]),
            "sled_kvm_reserve_batch_at": (C.c_int, [P, P, P, P, I32]),
            "sled_kvm_commit_tokens": (C.c_int, [P, U64, I32, I32, P]),
            "sled_kvm_history": (C.c_int, [P, U64, C.POINTER(I64), C.POINTER(I32), P, I32]),
            "sled_server_config": (C.c_int, [P, I32, I32]),
            "sled_submit": (C.c_int, [P, C.POINTER(SledRequest), C.POINTER(U64)]),
            "sled_step": (C.c_int, [P, U64, I32, C.POINTER(I32)]),
            "sled_poll": (C.c_int, [P, U64, C.POINTER(SledResult)]),
            "sled_queued": (I32, [P]),
            "sled_planner_create": (P, [I32, I32, I32, I32]),
            "sled_planner_destroy": (None, [P]),
            "sled_planner_push": (C.c_int, [P, U64, U64, I32]),
            "sled_planner_next_batch": (I32, [P, I32, P, I32]),
            "sled_planner_queued": (I32, [P]),
            "sled_debug_plan_attention": (C.c_int, [P, P, I32, I32, I32, I32, C.c_int64, P]),
        }
        for name, (res, args) in sig.items():
            fn = getattr(L, name)
            fn.restype, fn.argtypes = res, args
        _lib = L
    return _lib


def strerror(code: int) -> str:
    return lib().sled_strerror(code).decode()


def _check(code: int, what: str) -> None:
    if code != SLED_OK:
        raise SledError(code, what)


def _settle(*tensors) -> None:
    """The library works on its own stream and does not wait for anybody else's: device tensors handed to
    it must be complete.  Torch fills them asynchronously on its current stream, so that stream is drained."""
    if any(isinstance(t, torch.Tensor) and t.is_cuda for t in tensors):
        torch.cuda.current_stream().synchronize()


def _addr(t) -> int:
    if t is None:
        return 0
    if isinstance(t, np.ndarray):
        assert t.flags["C_CONTIGUOUS"]
        return t.ctypes.data
    assert t.is_contiguous()
    return t.data_ptr()


_PER_LAYER = ("attn_norm", "wq", "wk", "wv", "wo", "ffn_norm", "w_gate", "w_up", "w_down")
_DT = {"fp32": SLED_F32, "bf16": SLED_BF16}


class Engine:
    """Owner of one sled_engine handle.  Methods mirror the C entry points one to one."""

    def __init__(self, shape, weights: dict, *, n_pages: int, max_batch: int, max_k: int, max_step_tokens: int,
                 temperature: float = 1.0, greedy: bool = False, probs_on_device: bool = False, device_index: int = 0,
                 page_size: int = 16, stream: int | None = None, draft_probs_dtype: str = "fp32",
                 attention_impl: int = 0, linear_weight_bits: int = 16):
        """linear_weight_bits = 8: weights["wq"] .. ["w_down"] and ["lm_head"] are uint8 tensors of e4m3 bytes and
        weights["wq_scale"] .. / ["lm_head_scale"] fp32 tensors with one scale per output row; 4: the same with two
        e2m1 codes per byte (uint8 tensors [N, K / 2])."""
        self.shape = shape
        cfg = SledConfig(shape.n_layers, shape.d_model, shape.n_q_heads, shape.n_kv_heads, shape.head_dim,
                         shape.ffn_dim, shape.vocab, shape.rms_eps, shape.rope_theta, _DT[shape.weight_dtype],
                         _DT[shape.kv_dtype], page_size, n_pages, max_batch, max_k, max_step_tokens, temperature,
                         int(greedy), int(probs_on_device), device_index, stream, _DT[draft_probs_dtype], attention_impl,
                         linear_weight_bits)
        w = SledWeights()
        w.tok_emb, w.final_norm, w.lm_head = _addr(weights["tok_emb"]), _addr(weights["final_norm"]), _addr(weights["lm_head"])
        keep = []
        for name in _PER_LAYER:
            arr = (C.c_void_p * shape.n_layers)(*[_addr(t) for t in weights[name]])
            keep.append(arr)
            setattr(w, name, C.cast(arr, C.POINTER(C.c_void_p)))
        if linear_weight_bits in (8, 4):
            w.lm_head_scale = _addr(weights["lm_head_scale"])
            for name in ("wq", "wk", "wv", "wo", "w_gate", "w_up", "w_down"):
                arr = (C.c_void_p * shape.n_layers)(*[_addr(t) for t in weights[name + "_scale"]])
                keep.append(arr)
                setattr(w, name + "_scale", C.cast(arr, C.POINTER(C.c_void_p)))
        h = C.c_void_p()
        _settle(weights["tok_emb"])
        _check(lib().sled_init(C.byref(w), C.byref(cfg), C.byref(h)), "sled_init")
        self.h = h
        self.cfg = cfg
        self.probs_on_device = probs_on_device

    # -- the three calls
    def verify_batch(self, requests, seed: int):
        """requests: list of (ctx_id, draft_tokens int32 host array [k], draft_probs [k, V] fp32 or None[, base_len]).
        Returns list of (n_accepted, next_token, status)."""
        n = len(requests)
        _settle(*[r[2] for r in requests])
        reqs = (SledRequest * max(n, 1))()
        keep = []
        for i, r in enumerate(requests):
            ctx, toks, probs = r[:3]
            reqs[i].base_len = r[3] if len(r) > 3 else 0
            toks = np.ascontiguousarray(np.asarray(toks, dtype=np.int32).reshape(-1))
            keep.append(toks)
            if probs is not None and not isinstance(probs, torch.Tensor):
                probs = np.ascontiguousarray(probs, dtype=np.float32)
                keep.append(probs)
            if isinstance(probs, torch.Tensor):
                assert probs.dtype == (torch.bfloat16 if self.cfg.draft_probs_dtype == SLED_BF16 else torch.float32)
            reqs[i].ctx_id = ctx
            reqs[i].draft_tokens = toks.ctypes.data if toks.size else None
            reqs[i].draft_probs = _addr(probs) if probs is not None and toks.size else None
            reqs[i].k = toks.size
        res = (SledResult * max(n, 1))()
        _check(lib().sled_verify_batch(self.h, reqs, n, seed, res), "sled_verify_batch")
        return [(res[i].n_accepted, res[i].next_token, res[i].status) for i in range(n)]

    def verify_batch_raw(self, reqs, n: int, seed: int, res) -> int:
        """Pre-marshalled arrays (SledRequest * n, SledResult * n): the bare call, for timing."""
        return lib().sled_verify_batch(self.h, reqs, n, seed, res)

    def release(self, ctx_id: int) -> None:
        _check(lib().sled_release(self.h, ctx_id), "sled_release")

    # -- the server loop
    def server_config(self, policy: int, batch_size: int = 0) -> None:
        _check(lib().sled_server_config(self.h, policy, batch_size), "sled_server_config")

    def submit(self, ctx_id: int, draft_tokens, draft_probs=None, base_len: int = 0) -> int:
        """Queues one request; returns its ticket.  draft_probs must stay alive until the ticket has been polled."""
        toks = np.ascontiguousarray(np.asarray(draft_tokens, dtype=np.int32).reshape(-1))
        _settle(draft_probs)
        r = SledRequest(ctx_id, toks.ctypes.data if toks.size else None,
                        _addr(draft_probs) if draft_probs is not None and toks.size else None, toks.size, base_len)
        t = C.c_uint64()
        _check(lib().sled_submit(self.h, C.byref(r), C.byref(t)), "sled_submit")
        return t.value

    def step(self, seed: int, flush: bool = False) -> int:
        n = C.c_int32()
        _check(lib().sled_step(self.h, seed, int(flush), C.byref(n)), "sled_step")
        return n.value

    def poll(self, ticket: int):
        """(n_accepted, next_token, status) once verified, None while queued."""
        r = SledResult()
        rc = lib().sled_poll(self.h, ticket, C.byref(r))
        if rc == SLED_PENDING:
            return None
        _check(rc, "sled_poll")
        return (r.n_accepted, r.next_token, r.status)

    def queued(self) -> int:
        return lib().sled_queued(self.h)

    def prefill(self, ctx_id: int, tokens) -> None:
        t = np.ascontiguousarray(np.asarray(tokens, dtype=np.int32))
        _check(lib().sled_prefill(self.h, ctx_id, t.ctypes.data, t.size), "sled_prefill")

    # -- the rest
    def set_sampling(self, temperature: float, greedy: bool) -> None:
        _check(lib().sled_set_sampling(self.h, temperature, int(greedy)), "sled_set_sampling")

    def stats(self) -> SledStats:
        s = SledStats()
        _check(lib().sled_get_stats(self.h, C.byref(s)), "sled_get_stats")
        return s

    def stream(self) -> int:
        return lib().sled_get_stream(self.h) or 0

    def load_kv(self, ctx_id: int, K, V, pending: int) -> None:
        n = K.shape[1]
        _settle(K, V)
        _check(lib().sled_debug_load_kv(self.h, ctx_id, _addr(K), _addr(V), n, pending), "sled_debug_load_kv")

    def read_kv(self, ctx_id: int, layer: int, n_tokens: int):
        s = self.shape
        dt = torch.bfloat16 if s.kv_dtype == "bf16" else torch.float32
        K = torch.empty(n_tokens, s.n_kv_heads, s.head_dim, dtype=dt)
        V = torch.empty_like(K)
        _check(lib().sled_debug_read_kv(self.h, ctx_id, layer, K.data_ptr(), V.data_ptr(), n_tokens), "sled_debug_read_kv")
        return K, V

    def logits(self, n_rows: int) -> np.ndarray:
        out = np.empty((n_rows, self.shape.vocab), dtype=np.float32)
        _check(lib().sled_debug_copy_logits(self.h, out.ctypes.data, n_rows), "sled_debug_copy_logits")
        return out

    def truncate(self, ctx_id: int, n_kv: int, pending: int) -> None:
        _check(lib().sled_debug_truncate(self.h, ctx_id, n_kv, pending), "sled_debug_truncate")

    def arm_wait_timeout(self, limit_us: int) -> None:
        _check(lib().sled_debug_arm_wait_timeout(self.h, limit_us), "sled_debug_arm_wait_timeout")

    def set_commit(self, on: bool) -> None:
        _check(lib().sled_debug_set_commit(self.h, int(on)), "sled_debug_set_commit")

    def set_timing(self, mode: int) -> None:
        """0 off, 1 device timestamps per launch (overlap untouched), 2 events between kernel groups (serialises)."""
        _check(lib().sled_debug_set_timing(self.h, int(mode)), "sled_debug_set_timing")

    def shuffle_pages(self, seed: int) -> None:
        _check(lib().sled_debug_shuffle_pages(self.h, seed), "sled_debug_shuffle_pages")

    def query_ctx(self, ctx_id: int):
        n_kv, pend, npg = C.c_int64(), C.c_int32(), C.c_int32()
        _check(lib().sled_debug_query_ctx(self.h, ctx_id, C.byref(n_kv), C.byref(pend), C.byref(npg), None, 0),
               "sled_debug_query_ctx")
        pages = np.zeros(max(npg.value, 1), dtype=np.int32)
        _check(lib().sled_debug_query_ctx(self.h, ctx_id, None, None, None, pages.ctypes.data, npg.value),
               "sled_debug_query_ctx")
        return n_kv.value, pend.value, pages[:npg.value].copy()

    def attention_ragged(self, layer: int, ctx_ids, q_len, q: torch.Tensor, out: torch.Tensor) -> float:
        ids = np.ascontiguousarray(np.asarray(ctx_ids, dtype=np.uint64))
        ql = np.ascontiguousarray(np.asarray(q_len, dtype=np.int32))
        ms = C.c_float()
        _settle(q, out)
        _check(lib().sled_attention_ragged(self.h, layer, ids.ctypes.data, ql.ctypes.data, ids.size, q.data_ptr(),
                                           out.data_ptr(), C.byref(ms)), "sled_attention_ragged")
        return ms.value

    def shutdown(self) -> None:
        if self.h:
            lib().sled_shutdown(self.h)
            self.h = None

    def __del__(self):
        try:
            self.shutdown()
        except Exception:
            pass


def accept_rows(logits: torch.Tensor, cu_rows, drafts, q_rows, ctx_ids, pos0, temperature: float, greedy: bool,
                seed: int, stream: int = 0):
    """sled_accept_rows: logits [rows, V] and q_rows [sum k, V] are CUDA tensors, the rest host arrays.
    Returns (list of (n_accepted, next_token, status), kernel milliseconds)."""
    cu = np.ascontiguousarray(np.asarray(cu_rows, dtype=np.int32))
    n = cu.size - 1
    d = np.ascontiguousarray(np.asarray(drafts, dtype=np.int32).reshape(-1))
    ids = np.ascontiguousarray(np.asarray(ctx_ids, dtype=np.uint64))
    p0 = np.ascontiguousarray(np.asarray(pos0, dtype=np.int64))
    res = (SledResult * n)()
    ms = C.c_float()
    _settle(logits, q_rows)
    _check(lib().sled_accept_rows(logits.data_ptr(), cu.ctypes.data, d.ctypes.data if d.size else None,
                                  _addr(q_rows) if q_rows is not None else None, ids.ctypes.data, p0.ctypes.data, n,
                                  logits.shape[1], temperature, int(greedy), seed, res, stream, C.byref(ms)),
           "sled_accept_rows")
    return [(res[i].n_accepted, res[i].next_token, res[i].status) for i in range(n)], ms.value


def accept_rows_static(logits: torch.Tensor, cu_rows, drafts, q_rows, ctx_ids, pos0, temperature: float,
                       greedy: bool, seed: int, stream: int = 0):
    """sled_accept_rows_static: same arguments and results as accept_rows, for callers that must not
    allocate device memory (the batch description goes into a fixed array inside the library, at most
    1024 requests / 8192 rows; calls on one device must not overlap).  Returns the result list."""
    cu = np.ascontiguousarray(np.asarray(cu_rows, dtype=np.int32))
    n = cu.size - 1
    d = np.ascontiguousarray(np.asarray(drafts, dtype=np.int32).reshape(-1))
    ids = np.ascontiguousarray(np.asarray(ctx_ids, dtype=np.uint64))
    p0 = np.ascontiguousarray(np.asarray(pos0, dtype=np.int64))
    res = (SledResult * max(n, 1))()
    _settle(logits, q_rows)
    _check(lib().sled_accept_rows_static(logits.data_ptr(), cu.ctypes.data, d.ctypes.data if d.size else None,
                                         _addr(q_rows) if q_rows is not None else None, ids.ctypes.data,
                                         p0.ctypes.data, n, logits.shape[1], temperature, int(greedy), seed, res,
                                         stream), "sled_accept_rows_static")
    return [(res[i].n_accepted, res[i].next_token, res[i].status) for i in range(n)]


class KvManager:
    """The host-side page manager alone (sled_kvm_*): needs no device."""

    def __init__(self, n_pages: int, page_size: int):
        self.h = lib().sled_kvm_create(n_pages, page_size)
        if not self.h:
            raise SledError(SLED_ERR_ARG, "sled_kvm_create")

    def open(self, ctx: int, n_kv: int, pending: int) -> int:
        return lib().sled_kvm_open(self.h, ctx, n_kv, pending)

    def reserve_batch(self, ctxs, extra, base_len=None) -> int:
        c = np.ascontiguousarray(np.asarray(ctxs, dtype=np.uint64))
        x = np.ascontiguousarray(np.asarray(extra, dtype=np.int32))
        if base_len is None:
            return lib().sled_kvm_reserve_batch(self.h, c.ctypes.data, x.ctypes.data, c.size)
        b = np.ascontiguousarray(np.asarray(base_len, dtype=np.int64))
        return lib().sled_kvm_reserve_batch_at(self.h, c.ctypes.data, x.ctypes.data, b.ctypes.data, c.size)

    def commit(self, ctx: int, n_keep: int, pending: int, kept=None) -> int:
        if kept is None:
            return lib().sled_kvm_commit(self.h, ctx, n_keep, pending)
        t = np.ascontiguousarray(np.asarray(kept, dtype=np.int32))
        return lib().sled_kvm_commit_tokens(self.h, ctx, n_keep, pending, t.ctypes.data if t.size else None)

    def history(self, ctx: int):
        start, n = C.c_int64(), C.c_int32()
        rc = lib().sled_kvm_history(self.h, ctx, C.byref(start), C.byref(n), None, 0)
        if rc:
            return rc, None
        toks = np.zeros(max(n.value, 1), dtype=np.int32)
        lib().sled_kvm_history(self.h, ctx, None, None, toks.ctypes.data, n.value)
        return 0, (start.value, [int(x) for x in toks[:n.value]])

    def release(self, ctx: int) -> int:
        return lib().sled_kvm_release(self.h, ctx)

    def query(self, ctx: int):
        n_kv, pend, npg = C.c_int64(), C.c_int32(), C.c_int32()
        rc = lib().sled_kvm_query(self.h, ctx, C.byref(n_kv), C.byref(pend), C.byref(npg), None, 0)
        if rc:
            return rc, None
        pages = np.zeros(max(npg.value, 1), dtype=np.int32)
        lib().sled_kvm_query(self.h, ctx, None, None, None, pages.ctypes.data, npg.value)
        return 0, (n_kv.value, pend.value, pages[:npg.value].copy())

    def free_pages(self) -> int:
        return lib().sled_kvm_free_pages(self.h)

    def pack(self, ctxs, ks, drafts):
        c = np.ascontiguousarray(np.asarray(ctxs, dtype=np.uint64))
        k = np.ascontiguousarray(np.asarray(ks, dtype=np.int32))
        n = c.size
        T = int(k.sum()) + n
        arrs = [np.ascontiguousarray(np.asarray(d, dtype=np.int32).reshape(-1)) for d in drafts]
        ptrs = (C.c_void_p * max(n, 1))(*[a.ctypes.data if a.size else None for a in arrs])
        cu = np.zeros(n + 1, np.int32)
        out = [np.zeros(max(T, 1), np.int32) for _ in range(4)]
        rc = lib().sled_kvm_pack(self.h, c.ctypes.data, k.ctypes.data, ptrs, n, cu.ctypes.data,
                                 *[o.ctypes.data for o in out])
        return rc, cu, [o[:T] for o in out]

    def __del__(self):
        try:
            if self.h:
                lib().sled_kvm_destroy(self.h)
                self.h = None
        except Exception:
            pass


class Planner:
    """The request queue and batch planner alone (sled_planner_*): needs no device."""

    def __init__(self, policy: int, batch_size: int, max_batch: int, max_step_tokens: int):
        self.h = lib().sled_planner_create(policy, batch_size, max_batch, max_step_tokens)
        if not self.h:
            raise SledError(SLED_ERR_ARG, "sled_planner_create")
        self.cap = max_batch

    def push(self, ticket: int, ctx: int, k: int) -> int:
        return lib().sled_planner_push(self.h, ticket, ctx, k)

    def next_batch(self, flush: bool = False, cap: int | None = None):
        cap = self.cap if cap is None else cap
        out = np.zeros(max(cap, 1), dtype=np.uint64)
        n = lib().sled_planner_next_batch(self.h, int(flush), out.ctypes.data, cap)
        return n if n < 0 else [int(x) for x in out[:n]]

    def queued(self) -> int:
        return lib().sled_planner_queued(self.h)

    def __del__(self):
        try:
            if self.h:
                lib().sled_planner_destroy(self.h)
                self.h = None
        except Exception:
            pass


def plan_attention(n_keys, q_tokens, n_kv_heads: int, group: int, resident_blocks: int, part_rows_cap: int):
    """Keys per attention work item of every request (sled_debug_plan_attention: host only, needs no device)."""
    nk = np.ascontiguousarray(n_keys, dtype=np.int64)
    qt = np.ascontiguousarray(q_tokens, dtype=np.int32)
    out = np.zeros(len(nk), dtype=np.int64)
    _check(lib().sled_debug_plan_attention(nk.ctypes.data, qt.ctypes.data, len(nk), n_kv_heads, group, resident_blocks,
                                           part_rows_cap, out.ctypes.data), "sled_debug_plan_attention")
    return [int(c) for c in out]
