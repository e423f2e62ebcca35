"""TEST INFRASTRUCTURE ONLY: Python face of the CPU oracle (oracle/sled_oracle.cpp).

Only tests, the smoke check and the benchmark's CPU-baseline leg may import this
module; the product path never does.  It compiles the C++ file with g++ on first
use and composes its functions into the server-side state machine of one
verification cycle (Section 3.2 of the paper: devices send draft tokens, the
server answers with the rejected position and the corrective token):

    prefill   -> KV of all prompt tokens but the last, which becomes *pending*
    verify    -> feed [pending, d_1..d_k], Eq. 1 acceptance, then commit the KV of
                 pending and of the accepted drafts, drop the rest, pending := next;
                 with base_len = m the context is first cut back to its first m tokens
                 (Section 3.3: a device whose timer ran out sends its drafts again,
                 extended, from the point it last heard about)
    release   -> forget the context

The arithmetic is all in the C++ file; this file only moves arrays.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from dataclasses import dataclass, field

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "sled_oracle.cpp")
_LIB = os.path.join(_HERE, "_build", "liboracle.so")


def build(force: bool = False) -> str:
    """Compile the oracle (g++, OpenMP, no contraction of a*b+c into fma)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        os.makedirs(os.path.dirname(_LIB), exist_ok=True)
        tmp = _LIB + f".{os.getpid()}.tmp"
        subprocess.check_call(
            ["g++", "-O2", "-std=c++17", "-fopenmp", "-ffp-contract=off", "-shared", "-fPIC", "-o", tmp, _SRC]
        )
        os.replace(tmp, _LIB)
    return _LIB


class _Cfg(C.Structure):
    _fields_ = [(n, C.c_int32) for n in
                ("n_layers", "d_model", "n_q_heads", "n_kv_heads", "head_dim", "ffn_dim", "vocab")] + [
        ("rms_eps", C.c_float), ("rope_theta", C.c_float), ("weight_dtype", C.c_int32), ("kv_dtype", C.c_int32)]


class _Weights(C.Structure):
    _fields_ = [("tok_emb", C.c_void_p), ("final_norm", C.c_void_p), ("lm_head", C.c_void_p)] + [
        (n, C.POINTER(C.c_void_p)) for n in
        ("attn_norm", "wq", "wk", "wv", "wo", "ffn_norm", "w_gate", "w_up", "w_down")]


class Margin(C.Structure):
    _fields_ = [("accept_rel", C.c_double), ("sample_rel", C.c_double), ("greedy_gap", C.c_double),
                ("draw_mass", C.c_double)]


_lib = None


def lib():
    global _lib
    if _lib is None:
        L = C.CDLL(build())
        L.orc_philox4x32_10.argtypes = [C.POINTER(C.c_uint32)] * 3
        L.orc_philox4x32_10.restype = None
        L.orc_uniforms.argtypes = [C.c_uint64, C.c_uint64, C.c_int64, C.POINTER(C.c_uint32), C.POINTER(C.c_uint32)]
        L.orc_uniforms.restype = None
        L.orc_fixed_exp.argtypes = [C.c_float]
        L.orc_fixed_exp.restype = C.c_uint64
        L.orc_fixed_softmax.argtypes = [C.c_void_p, C.c_int32, C.c_float, C.c_void_p, C.POINTER(C.c_uint64)]
        L.orc_fixed_softmax.restype = None
        L.orc_accept.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.c_int32, C.c_float, C.c_int32,
                                 C.c_uint64, C.c_uint64, C.c_int64, C.POINTER(C.c_int32), C.POINTER(C.c_int32),
                                 C.POINTER(Margin)]
        L.orc_accept.restype = C.c_int
        L.orc_forward_token.argtypes = [C.POINTER(_Cfg), C.POINTER(_Weights), C.c_int32, C.c_int64, C.c_void_p,
                                        C.c_void_p, C.c_int64, C.c_void_p, C.c_int32]
        L.orc_forward_token.restype = C.c_int
        L.orc_attend_one.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int64, C.c_int32, C.c_void_p]
        L.orc_attend_one.restype = None
        L.orc_round_bf16.argtypes = [C.c_double]
        L.orc_round_bf16.restype = C.c_float
        L.orc_num_threads.restype = C.c_int
        L.orc_set_threads.argtypes = [C.c_int]
        _lib = L
    return _lib


# ------------------------------------------------------------------ scalars --
def philox(key, ctr):
    k = (C.c_uint32 * 2)(*key)
    c = (C.c_uint32 * 4)(*ctr)
    o = (C.c_uint32 * 4)()
    lib().orc_philox4x32_10(k, c, o)
    return tuple(int(x) for x in o)


def uniforms(seed: int, ctx_id: int, abs_pos: int):
    a, s = C.c_uint32(), C.c_uint32()
    lib().orc_uniforms(seed, ctx_id, abs_pos, C.byref(a), C.byref(s))
    return a.value, s.value


def fixed_exp(x: float) -> int:
    return int(lib().orc_fixed_exp(float(np.float32(x))))


def fixed_softmax(z: np.ndarray, tau: float = 1.0):
    z = np.ascontiguousarray(z, dtype=np.float32)
    E = np.empty(z.shape[0], dtype=np.uint64)
    Z = C.c_uint64()
    lib().orc_fixed_softmax(z.ctypes.data, z.shape[0], tau, E.ctypes.data, C.byref(Z))
    return E, int(Z.value)


def accept(logits: np.ndarray, q, drafts, tau: float, greedy: bool, seed: int, ctx_id: int, pos0: int):
    """One request's decision.  logits [k+1, V] fp32; q [k, V] fp32 or None; drafts [k].
    Returns (status, n_accepted, next_token, Margin)."""
    logits = np.ascontiguousarray(logits, dtype=np.float32)
    k = logits.shape[0] - 1
    V = logits.shape[1]
    drafts = np.ascontiguousarray(drafts, dtype=np.int32).reshape(-1)
    assert drafts.shape[0] == k
    qp = None
    if q is not None and k > 0:
        q = np.ascontiguousarray(q, dtype=np.float32)
        assert q.shape == (k, V)
        qp = q.ctypes.data
    elif not greedy and k > 0:
        raise ValueError("sampling mode needs draft distributions")
    n_acc, nxt, mg = C.c_int32(), C.c_int32(), Margin()
    st = lib().orc_accept(logits.ctypes.data, qp, drafts.ctypes.data, k, V, tau, int(bool(greedy)), seed, ctx_id,
                          pos0, C.byref(n_acc), C.byref(nxt), C.byref(mg))
    return st, n_acc.value, nxt.value, mg


def attend_one(q: np.ndarray, keys: np.ndarray, values: np.ndarray) -> np.ndarray:
    q = np.ascontiguousarray(q, dtype=np.float32)
    keys = np.ascontiguousarray(keys, dtype=np.float32)
    values = np.ascontiguousarray(values, dtype=np.float32)
    out = np.empty(q.shape[0], dtype=np.float64)
    lib().orc_attend_one(q.ctypes.data, keys.ctypes.data, values.ctypes.data, keys.shape[0], q.shape[0],
                         out.ctypes.data)
    return out


def round_bf16(x: float) -> float:
    return float(lib().orc_round_bf16(float(x)))


def num_threads() -> int:
    return int(lib().orc_num_threads())


def set_threads(n: int) -> None:
    lib().orc_set_threads(int(n))


# -------------------------------------------------------------------- model --
_PER_LAYER = ("attn_norm", "wq", "wk", "wv", "wo", "ffn_norm", "w_gate", "w_up", "w_down")


def _ptr(a) -> int:
    """Address of a numpy array or of a CPU torch tensor (bf16 tensors have no numpy view)."""
    if isinstance(a, np.ndarray):
        assert a.flags["C_CONTIGUOUS"]
        return a.ctypes.data
    assert a.device.type == "cpu" and a.is_contiguous()
    return a.data_ptr()


@dataclass
class Context:
    n_kv: int                 # cached positions (= committed tokens - 1)
    pending: int              # last committed token, not yet in the cache
    K: np.ndarray             # [L, cap, Hkv, h] fp32 values on the cache format's grid
    V: np.ndarray
    tokens: list = field(default_factory=list)  # committed tokens from sequence index hist_start on; the last one is pending
    hist_start: int = 0       # 0 for prefilled contexts; the pending token's index when only the cache was given


class OracleModel:
    """Target model + per-context caches, driven one token at a time."""

    def __init__(self, shape, weights: dict, round_acts: bool = False):
        """shape: any object with the config attributes; weights: name -> array (per-layer names -> list).
        round_acts: the separately reported mode that rounds matrix-product inputs to bf16 (see the C++ file)."""
        self.shape = shape
        self.round_acts = int(bool(round_acts))
        wd = 1 if shape.weight_dtype == "bf16" else 0
        kd = 1 if shape.kv_dtype == "bf16" else 0
        self.cfg = _Cfg(shape.n_layers, shape.d_model, shape.n_q_heads, shape.n_kv_heads, shape.head_dim,
                        shape.ffn_dim, shape.vocab, shape.rms_eps, shape.rope_theta, wd, kd)
        self._keep = weights
        w = _Weights()
        w.tok_emb, w.final_norm, w.lm_head = _ptr(weights["tok_emb"]), _ptr(weights["final_norm"]), _ptr(weights["lm_head"])
        self._arrs = {}
        for name in _PER_LAYER:
            arr = (C.c_void_p * shape.n_layers)(*[_ptr(t) for t in weights[name]])
            self._arrs[name] = arr
            setattr(w, name, C.cast(arr, C.POINTER(C.c_void_p)))
        self.w = w
        self.ctx: dict[int, Context] = {}

    # -- cache plumbing
    def _new_cache(self, cap: int):
        s = self.shape
        shp = (s.n_layers, cap, s.n_kv_heads, s.head_dim)
        return np.zeros(shp, dtype=np.float32), np.zeros(shp, dtype=np.float32)

    def _grow(self, c: Context, need: int):
        cap = c.K.shape[1]
        if need <= cap:
            return
        K, V = self._new_cache(max(need, 2 * cap))
        K[:, :cap], V[:, :cap] = c.K, c.V
        c.K, c.V = K, V

    def forward_token(self, c: Context, token: int, pos: int) -> np.ndarray:
        self._grow(c, pos + 1)
        out = np.empty(self.shape.vocab, dtype=np.float32)
        rc = lib().orc_forward_token(C.byref(self.cfg), C.byref(self.w), int(token), int(pos), c.K.ctypes.data,
                                     c.V.ctypes.data, c.K.shape[1], out.ctypes.data, self.round_acts)
        assert rc == 0
        return out

    # -- the three calls
    def prefill(self, ctx_id: int, tokens) -> None:
        tokens = [int(t) for t in tokens]
        assert len(tokens) >= 1 and ctx_id not in self.ctx
        K, V = self._new_cache(max(16, len(tokens) + 16))
        c = Context(0, tokens[-1], K, V, list(tokens))
        for pos, t in enumerate(tokens[:-1]):
            self.forward_token(c, t, pos)
        c.n_kv = len(tokens) - 1
        self.ctx[ctx_id] = c

    def load_kv(self, ctx_id: int, K: np.ndarray, V: np.ndarray, pending: int) -> None:
        """Context whose cache content is given ([L, n, Hkv, h], values on the cache grid)."""
        assert ctx_id not in self.ctx
        n = K.shape[1]
        Kc, Vc = self._new_cache(n + 16)
        Kc[:, :n], Vc[:, :n] = K, V
        self.ctx[ctx_id] = Context(n, int(pending), Kc, Vc, [int(pending)], n)

    def release(self, ctx_id: int) -> None:
        del self.ctx[ctx_id]

    def score(self, ctx_id: int, drafts) -> np.ndarray:
        """Target logits at the k+1 positions [pending, d_1..d_k]; the cache rows written for
        them stay beyond n_kv until a commit keeps some."""
        c = self.ctx[ctx_id]
        feed = [c.pending] + [int(d) for d in drafts]
        return np.stack([self.forward_token(c, t, c.n_kv + j) for j, t in enumerate(feed)])

    def rebase(self, ctx_id: int, base_len: int) -> None:
        """Cuts the context back to its first base_len committed tokens: the last of them becomes pending again,
        the cache keeps the base_len - 1 entries before it.  Only as far back as the token history is known."""
        c = self.ctx[ctx_id]
        if not (c.hist_start + 1 <= base_len <= c.n_kv + 1):
            raise ValueError("base_len outside the known history")
        c.tokens = c.tokens[:base_len - c.hist_start]
        c.n_kv = base_len - 1
        c.pending = c.tokens[-1]

    def verify(self, ctx_id: int, drafts, q, seed: int, tau: float = 1.0, greedy: bool = False, commit: bool = True,
               base_len: int = 0):
        """Returns (status, n_accepted, next_token, logits [k+1, V], Margin).  base_len > 0: the drafts continue the
        first base_len tokens of the context (what the device had seen when it drafted), not its current end."""
        if base_len:
            self.rebase(ctx_id, base_len)
        c = self.ctx[ctx_id]
        logits = self.score(ctx_id, drafts)
        st, n_acc, nxt, mg = accept(logits, q, drafts, tau, greedy, seed, ctx_id, c.n_kv)
        if commit and st == 0:
            # KV of pending and of the accepted drafts is kept: truncating the length drops the rest
            c.n_kv += n_acc + 1
            c.tokens += [int(d) for d in drafts[:n_acc]] + [nxt]
            c.pending = nxt
        return st, n_acc, nxt, logits, mg
