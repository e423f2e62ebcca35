"""Seeded synthetic inputs shaped like the paper's workloads.

This module only draws random arrays (torch generators seeded per item); it holds
none of the verification arithmetic and imports neither the CUDA binding nor the
CPU oracle, so both can be fed from it.

What stands in for what (Section 4 of the paper evaluates with trained Llama
checkpoints, real edge devices and a public question set, none of which is used
here): random-initialised Llama-shaped weights, contexts whose cached keys and
values are either produced by a real prefill of random token ids (small shapes) or
drawn directly on the cache's number grid (large shapes), and per-device draft
lengths k_i that differ inside a batch, as dynamic drafting (Section 3.3) produces.
"""
from __future__ import annotations

from dataclasses import dataclass, replace

import numpy as np
import torch


@dataclass(frozen=True)
class ModelShape:
    name: str
    n_layers: int
    d_model: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    ffn_dim: int
    vocab: int
    rope_theta: float
    weight_dtype: str  # "fp32" | "bf16"
    kv_dtype: str      # "fp32" | "bf16"
    rms_eps: float = 1e-5

    @property
    def torch_wdtype(self):
        return torch.bfloat16 if self.weight_dtype == "bf16" else torch.float32

    @property
    def torch_kvdtype(self):
        return torch.bfloat16 if self.kv_dtype == "bf16" else torch.float32

    def streamed_params(self) -> int:
        """Weights every step reads once: all linear layers and the LM head."""
        s = self
        per_layer = s.d_model * s.n_q_heads * s.head_dim * 2 + 2 * s.d_model * s.n_kv_heads * s.head_dim \
            + 3 * s.d_model * s.ffn_dim
        return s.n_layers * per_layer + s.vocab * s.d_model

    def kv_bytes_per_token(self) -> int:
        el = 2 if self.kv_dtype == "bf16" else 4
        return 2 * self.n_layers * self.n_kv_heads * self.head_dim * el


TINY = ModelShape("tiny", 2, 256, 4, 4, 64, 688, 4096, 1e4, "fp32", "fp32")
# same shape with 16-bit storage: exercises the tensor-core path at a size the oracle can prefill
TINY_BF16 = replace(TINY, name="tiny_bf16", weight_dtype="bf16", kv_dtype="bf16")
# a small grouped-query shape with head_dim 128 (the 8B head geometry) the oracle can still prefill
SMALL_GQA = ModelShape("small_gqa", 2, 512, 8, 2, 128, 1408, 8192, 5e5, "bf16", "bf16")
LLAMA_1B = ModelShape("llama1b", 16, 2048, 32, 8, 64, 8192, 128256, 5e5, "bf16", "bf16")
LLAMA_8B = ModelShape("llama8b", 32, 4096, 32, 8, 128, 14336, 128256, 5e5, "bf16", "bf16")
SHAPES = {s.name: s for s in (TINY, TINY_BF16, SMALL_GQA, LLAMA_1B, LLAMA_8B)}

PER_LAYER = ("attn_norm", "wq", "wk", "wv", "wo", "ffn_norm", "w_gate", "w_up", "w_down")


def _gen(seed: int, *ids: int, device="cpu") -> torch.Generator:
    """One generator per (seed, item ids): items can be drawn in any order or skipped."""
    g = torch.Generator(device=device)
    key = seed & 0xFFFFFFFF
    for i in ids:
        key = (key * 1000003 + int(i) + 0x9E3779B9) & 0x7FFFFFFFFFFFFFFF
    g.manual_seed(key)
    return g


def make_weights(shape: ModelShape, seed: int = 0, device: str = "cpu") -> dict:
    """Linear weights ~ N(0, 0.02^2), row-major [out, in]; norm gains 1 + N(0, 0.1^2) so that a
    wrongly indexed gain shows.  Drawn in fp32 and rounded once to the storage type.  The stream
    of a torch generator depends on the device it lives on: arrays drawn on "cpu" and on "cuda"
    differ, each is reproducible."""
    s, dt = shape, shape.torch_wdtype

    def lin(n_out, n_in, *ids):
        return (torch.randn(n_out, n_in, generator=_gen(seed, *ids, device=device), device=device,
                            dtype=torch.float32) * 0.02).to(dt)

    def gain(*ids):
        return (1.0 + 0.1 * torch.randn(s.d_model, generator=_gen(seed, *ids, device=device), device=device,
                                        dtype=torch.float32)).to(dt)

    w = {"tok_emb": lin(s.vocab, s.d_model, 1), "final_norm": gain(2), "lm_head": lin(s.vocab, s.d_model, 3)}
    for name in PER_LAYER:
        w[name] = []
    for l in range(s.n_layers):
        w["attn_norm"].append(gain(10, l))
        w["wq"].append(lin(s.n_q_heads * s.head_dim, s.d_model, 11, l))
        w["wk"].append(lin(s.n_kv_heads * s.head_dim, s.d_model, 12, l))
        w["wv"].append(lin(s.n_kv_heads * s.head_dim, s.d_model, 13, l))
        w["wo"].append(lin(s.d_model, s.n_q_heads * s.head_dim, 14, l))
        w["ffn_norm"].append(gain(15, l))
        w["w_gate"].append(lin(s.ffn_dim, s.d_model, 16, l))
        w["w_up"].append(lin(s.ffn_dim, s.d_model, 17, l))
        w["w_down"].append(lin(s.d_model, s.ffn_dim, 18, l))
    return w


LINEAR_NAMES = ("wq", "wk", "wv", "wo", "w_gate", "w_up", "w_down")


def to_e4m3_rows(w: torch.Tensor):
    """Storage format of the 8-bit weight path: every row of a matrix divided by its scale = max|row| / 448 and
    rounded to the nearest e4m3 value.  Returns (bytes uint8 [N, K], scale fp32 [N])."""
    w32 = w.to(torch.float32)
    scale = w32.abs().amax(dim=1) / 448.0
    scale = torch.where(scale > 0, scale, torch.ones_like(scale))
    q = (w32 / scale[:, None]).to(torch.float8_e4m3fn)
    return q.view(torch.uint8).contiguous(), scale.contiguous()


def from_e4m3_rows(q: torch.Tensor, scale: torch.Tensor) -> torch.Tensor:
    """The matrix those bytes and scales stand for, in fp32 (scale * e4m3 value, one rounding)."""
    return q.view(torch.float8_e4m3fn).to(torch.float32) * scale[:, None]


E2M1_VALUES = (0.0, 0.5, 1.0, 1.5, 2.0, 3.0, 4.0, 6.0)   # magnitudes of the 4-bit float (1 sign, 2 exponent, 1 mantissa bit)


def to_e2m1_rows(w: torch.Tensor):
    """Storage format of the 4-bit weight path: every row divided by its scale = max|row| / 6 and rounded to the
    nearest e2m1 value (codes 0..7 = E2M1_VALUES, bit 3 = sign), two codes per byte, the even column in the low half.
    Returns (bytes uint8 [N, K / 2], scale fp32 [N]); K must be even."""
    w32 = w.to(torch.float32)
    assert w32.shape[1] % 2 == 0
    scale = w32.abs().amax(dim=1) / 6.0
    scale = torch.where(scale > 0, scale, torch.ones_like(scale))
    x = w32 / scale[:, None]
    grid = torch.tensor(E2M1_VALUES, device=w32.device)
    code = torch.bucketize(x.abs(), (grid[1:] + grid[:-1]) / 2).to(torch.uint8)      # nearest magnitude
    code = code | ((x < 0) & (code > 0)).to(torch.uint8) * 8
    return (code[:, 0::2] | (code[:, 1::2] << 4)).contiguous(), scale.contiguous()


def from_e2m1_rows(q: torch.Tensor, scale: torch.Tensor) -> torch.Tensor:
    """The matrix those nibbles and scales stand for, in fp32."""
    table = torch.tensor(E2M1_VALUES + tuple(-v for v in E2M1_VALUES), device=q.device)
    codes = torch.stack([q & 15, q >> 4], dim=2).reshape(q.shape[0], -1).long()
    return table[codes] * scale[:, None]


def quantize_linear_weights(w: dict, dequantised: bool = True, bits: int = 8):
    """(weights for the 8-bit - or, bits = 4, the 4-bit - path, the same model with its linear layers as fp32
    matrices - or None when `dequantised` is off).  The first holds e4m3 bytes (e2m1 nibbles) and `<name>_scale` for
    the linear layers and the LM head, everything else as in `w`; the second is what those bytes mean, for whoever
    wants to compute with them in another way."""
    to_rows, from_rows = (to_e4m3_rows, from_e4m3_rows) if bits == 8 else (to_e2m1_rows, from_e2m1_rows)
    q, deq = dict(w), (dict(w) if dequantised else None)
    b, sc = to_rows(w["lm_head"])
    q["lm_head"], q["lm_head_scale"] = b, sc
    if dequantised:
        deq["lm_head"] = from_rows(b, sc)
    for name in LINEAR_NAMES:
        pairs = [to_rows(t) for t in w[name]]
        q[name] = [p[0] for p in pairs]
        q[name + "_scale"] = [p[1] for p in pairs]
        if dequantised:
            deq[name] = [from_rows(*p) for p in pairs]
    return q, deq


def weights_to(w: dict, device: str) -> dict:
    return {k: ([t.to(device) for t in v] if isinstance(v, list) else v.to(device)) for k, v in w.items()}


def as_f32_numpy(t: torch.Tensor) -> np.ndarray:
    return t.detach().to("cpu", torch.float32).contiguous().numpy()


def make_prompt(vocab: int, n: int, seed: int, ctx_id: int) -> np.ndarray:
    """n uniform-random token ids."""
    return torch.randint(0, vocab, (n,), generator=_gen(seed, 100, ctx_id), dtype=torch.int64).to(torch.int32).numpy()


def make_kv(shape: ModelShape, n_tokens: int, seed: int, ctx_id: int, device: str = "cpu"):
    """Cache content drawn directly: K, V ~ N(0, 1) on the cache format's grid, [L, n, Hkv, h]."""
    shp = (shape.n_layers, n_tokens, shape.n_kv_heads, shape.head_dim)
    K = torch.randn(shp, generator=_gen(seed, 200, ctx_id, device=device), device=device, dtype=torch.float32)
    V = torch.randn(shp, generator=_gen(seed, 201, ctx_id, device=device), device=device, dtype=torch.float32)
    return K.to(shape.torch_kvdtype), V.to(shape.torch_kvdtype)


def make_drafts(vocab: int, k: int, seed: int, ctx_id: int, step: int = 0, sigma: float = 1.0, device: str = "cpu"):
    """A device's k draft tokens with their distributions: draft logits ~ N(0, sigma^2) iid,
    q = softmax(logits) (fp32 rows), d_j ~ q_j.  Returns (drafts int32 [k], q fp32 [k, V])."""
    if k == 0:
        return torch.zeros(0, dtype=torch.int32, device=device), torch.zeros(0, vocab, dtype=torch.float32, device=device)
    g = _gen(seed, 300, ctx_id, step, device=device)
    logits = torch.randn(k, vocab, generator=g, device=device, dtype=torch.float32) * sigma
    q = torch.softmax(logits, dim=-1)
    d = torch.multinomial(q, 1, generator=g).reshape(k).to(torch.int32)
    return d, q


def draw_k(batch: int, choices, seed: int) -> list:
    """Per-device draft length, iid uniform over `choices` (mixed lengths in one batch)."""
    idx = torch.randint(0, len(choices), (batch,), generator=_gen(seed, 400))
    return [int(choices[i]) for i in idx]


def draw_context_lengths(batch: int, lo: int, hi: int, seed: int) -> list:
    return [int(x) for x in torch.randint(lo, hi + 1, (batch,), generator=_gen(seed, 401))]


def draw_lognormal_kv_lengths(batch: int, median: int, sigma: float, lo: int, hi: int, seed: int) -> list:
    z = torch.randn(batch, generator=_gen(seed, 402), dtype=torch.float64)
    return [int(x) for x in torch.clamp((median * torch.exp(sigma * z)).round(), lo, hi)]


def make_accept_rows(n_requests: int, k: int, vocab: int, tau_draft: float, seed: int, device: str = "cpu",
                     rho: float = 0.8, sigma: float = 3.0):
    """Acceptance-only workload: per request k+1 rows of target logits z ~ N(0, sigma^2) and k rows of
    draft distributions q = softmax((rho z + sqrt(1-rho^2) z') / tau_draft), z' ~ N(0, sigma^2), d ~ q.
    Returns logits [n, k+1, V] fp32, q [n, k, V] fp32, drafts [n, k] int32."""
    g = _gen(seed, 500, device=device)
    z = torch.randn(n_requests, k + 1, vocab, generator=g, device=device, dtype=torch.float32) * sigma
    q = torch.empty(n_requests, k, vocab, device=device, dtype=torch.float32)
    d = torch.empty(n_requests, k, device=device, dtype=torch.int32)
    mix = (1.0 - rho * rho) ** 0.5
    for i in range(n_requests):  # per request to bound the temporary
        zp = torch.randn(k, vocab, generator=g, device=device, dtype=torch.float32) * sigma
        qi = torch.softmax((rho * z[i, :k] + mix * zp) / tau_draft, dim=-1)
        q[i] = qi
        d[i] = torch.multinomial(qi, 1, generator=g).reshape(k).to(torch.int32)
    return z, q, d


def correlated_draft(z_row: torch.Tensor, seed: int, ctx_id: int, j: int, rho: float = 0.8):
    """One draft position of a device whose draft model resembles the target: given the target's logits z at that
    position (from whichever implementation is being driven), draft logits = rho z + sqrt(1 - rho^2) std(z) noise,
    q = softmax(draft logits), d ~ q.  Returns (d int, q fp32 [V]) on z_row's device."""
    dev = z_row.device
    g = _gen(seed, 600, ctx_id, j, device=dev.type)
    z = z_row.to(torch.float32)
    noise = torch.randn(z.shape[0], generator=g, device=dev, dtype=torch.float32)
    q = torch.softmax(rho * z + (1.0 - rho * rho) ** 0.5 * z.std() * noise, dim=-1)
    d = int(torch.multinomial(q, 1, generator=g).item())
    return d, q
