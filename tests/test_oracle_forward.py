"""Pins of the oracle's target-model forward and of the verify / commit state machine."""
import math

import numpy as np
import pytest
import torch

from oracle import oracle as O
from paper_2506_09397_b200 import inputs as I


def _np_weights(w):
    """fp32 weights as numpy, bf16 weights stay torch CPU tensors (both give raw pointers)."""
    out = {}
    for k, v in w.items():
        conv = (lambda t: t.numpy() if t.dtype == torch.float32 else t)
        out[k] = [conv(t.contiguous()) for t in v] if isinstance(v, list) else conv(v.contiguous())
    return out


def _hf_model(shape, w):
    """The same network built from the transformers library's Llama, in fp64.  That code rotates
    the two halves of a head instead of adjacent pairs, so query/key rows are permuted per head
    (even rows first, then odd rows), which leaves every q.k product unchanged."""
    from transformers import LlamaConfig, LlamaForCausalLM

    cfg = LlamaConfig(hidden_size=shape.d_model, intermediate_size=shape.ffn_dim, num_hidden_layers=shape.n_layers,
                      num_attention_heads=shape.n_q_heads, num_key_value_heads=shape.n_kv_heads,
                      head_dim=shape.head_dim, vocab_size=shape.vocab, rms_norm_eps=shape.rms_eps,
                      rope_theta=shape.rope_theta, tie_word_embeddings=False, attention_bias=False, mlp_bias=False,
                      max_position_embeddings=4096, attn_implementation="eager")
    try:
        cfg.rope_parameters = {"rope_type": "default", "rope_theta": shape.rope_theta}
    except Exception:
        pass
    m = LlamaForCausalLM(cfg).to(torch.float64).eval()
    h = shape.head_dim
    perm = torch.cat([torch.arange(0, h, 2), torch.arange(1, h, 2)])

    def permute(wm, n_heads):
        return wm.double().reshape(n_heads, h, -1)[:, perm, :].reshape(n_heads * h, -1)

    sd = {"model.embed_tokens.weight": w["tok_emb"].double(), "model.norm.weight": w["final_norm"].double(),
          "lm_head.weight": w["lm_head"].double()}
    for l in range(shape.n_layers):
        p = f"model.layers.{l}."
        sd[p + "input_layernorm.weight"] = w["attn_norm"][l].double()
        sd[p + "self_attn.q_proj.weight"] = permute(w["wq"][l], shape.n_q_heads)
        sd[p + "self_attn.k_proj.weight"] = permute(w["wk"][l], shape.n_kv_heads)
        sd[p + "self_attn.v_proj.weight"] = w["wv"][l].double()
        sd[p + "self_attn.o_proj.weight"] = w["wo"][l].double()
        sd[p + "post_attention_layernorm.weight"] = w["ffn_norm"][l].double()
        sd[p + "mlp.gate_proj.weight"] = w["w_gate"][l].double()
        sd[p + "mlp.up_proj.weight"] = w["w_up"][l].double()
        sd[p + "mlp.down_proj.weight"] = w["w_down"][l].double()
    missing, unexpected = m.load_state_dict(sd, strict=False)
    assert not unexpected and all("rotary" in k or "inv_freq" in k for k in missing), (missing, unexpected)
    return m


@pytest.mark.parametrize("shape", [I.TINY, I.ModelShape("gqa_pin", 2, 128, 8, 2, 32, 320, 512, 5e5, "fp32", "fp32")])
def test_forward_matches_library_llama(shape):
    w = I.make_weights(shape, seed=3)
    toks = I.make_prompt(shape.vocab, 24, 3, 0)
    model = O.OracleModel(shape, _np_weights(w))
    model.prefill(0, list(toks) + [0])          # caches all 24, pending is a dummy
    c = model.ctx[0]
    mine = np.stack([model.forward_token(c, int(t), p) for p, t in enumerate(toks)])  # recompute: same logits per position
    hf = _hf_model(shape, w)
    with torch.no_grad():
        ref = hf(torch.tensor(toks, dtype=torch.long)[None]).logits[0].numpy()
    assert np.abs(ref).max() > 0.1
    assert np.max(np.abs(mine - ref)) < 5e-6     # fp32 rounding of the returned logits only


def _rne(t):
    """fp64 tensor -> nearest bf16 value (ties to even), kept in fp64: the library conversion."""
    return t.to(torch.float32).to(torch.bfloat16).to(torch.float64)


def _hf_logits_rounded(shape, w, toks, round_acts, skip=None):
    """Library Llama in fp64 with K and V rounded to the cache format and, if round_acts, the inputs of every
    matrix product rounded to bf16: the two normalised layer inputs, the rotated query, the attention
    output, the SwiGLU output and the final normalised vector."""
    from transformers.models.llama import modeling_llama as ML
    hf = _hf_model(shape, w)
    kv16 = shape.kv_dtype == "bf16"
    pre = lambda mod, args: (_rne(args[0]),) + tuple(args[1:])
    hooks = []
    # The library's RMSNorm and rotary table compute in fp32 whatever the model's type; their 1e-7 relative error
    # moves a few values across a bf16 rounding boundary and shows up as 1e-3 logit differences in single rows that
    # have nothing to do with the rounding points under test.  Both outputs are therefore recomputed in fp64 (the
    # library's own versions are already compared with the oracle's, to fp32 accuracy, by
    # test_forward_matches_library_llama); attention, masking, head grouping, the rotation itself, the MLP and the
    # residual structure remain the library's.
    def norm64(mod, args, out):
        x = args[0]
        return mod.weight * (x * torch.rsqrt(x.pow(2).mean(-1, keepdim=True) + mod.variance_epsilon))

    def rotary64(mod, args, out):
        pos = torch.arange(out[0].shape[1], dtype=torch.float64)[None]      # the whole prompt is fed at positions 0..n-1
        inv = shape.rope_theta ** (-torch.arange(0, shape.head_dim, 2, dtype=torch.float64) / shape.head_dim)
        ang = pos[:, :, None] * inv[None, None, :]
        ang = torch.cat([ang, ang], dim=-1)                                 # the library's two-halves layout
        assert out[0].shape == ang.shape
        return ang.cos(), ang.sin()
    hooks.append(hf.model.rotary_emb.register_forward_hook(rotary64))
    for layer in hf.model.layers:
        hooks.append(layer.input_layernorm.register_forward_hook(norm64))
        hooks.append(layer.post_attention_layernorm.register_forward_hook(norm64))
    hooks.append(hf.model.norm.register_forward_hook(norm64))
    if round_acts:
        for layer in hf.model.layers:
            points = {"attn_in": (layer.self_attn.q_proj, layer.self_attn.k_proj, layer.self_attn.v_proj),
                      "attn_out": (layer.self_attn.o_proj,), "ffn_in": (layer.mlp.gate_proj, layer.mlp.up_proj),
                      "swiglu": (layer.mlp.down_proj,)}
            for name, lins in points.items():
                if name != skip:
                    for lin in lins:
                        hooks.append(lin.register_forward_pre_hook(pre))
        if skip != "final":
            hooks.append(hf.lm_head.register_forward_pre_hook(pre))
    inner = ML.eager_attention_forward
    seen = []

    def attention(module, query, key, value, *a, **kw):
        seen.append(1)
        if round_acts and skip != "query":
            query = _rne(query)
        if kv16:
            key, value = _rne(key), _rne(value)
        return inner(module, query, key, value, *a, **kw)

    ML.eager_attention_forward = attention
    try:
        with torch.no_grad():
            ref = hf(torch.tensor(toks, dtype=torch.long)[None]).logits[0].numpy()
    finally:
        ML.eager_attention_forward = inner
        for h in hooks:
            h.remove()
    assert len(seen) == shape.n_layers          # the wrapped attention was the one that ran
    return ref


@pytest.mark.parametrize("round_acts", [False, True])
@pytest.mark.parametrize("shape", [I.TINY_BF16, I.ModelShape("gqa_pin16", 3, 128, 8, 2, 32, 320, 512, 5e5, "bf16", "bf16")])
def test_16bit_modes_match_library_llama_with_the_same_rounding_points(shape, round_acts):
    w = I.make_weights(shape, seed=4)
    toks = I.make_prompt(shape.vocab, 20, 4, 0)
    model = O.OracleModel(shape, _np_weights(w), round_acts=round_acts)
    model.prefill(0, list(toks) + [0])
    c = model.ctx[0]
    mine = np.stack([model.forward_token(c, int(t), p) for p, t in enumerate(toks)])
    ref = _hf_logits_rounded(shape, w, toks, round_acts)
    assert np.abs(ref).max() > 0.1
    row_err = np.max(np.abs(mine - ref), axis=1)
    if not round_acts:
        assert row_err.max() < 5e-6
    else:
        # The library's attention takes its softmax in fp32: a 1e-7 error in an attention output now and then crosses
        # a bf16 rounding boundary (about 3e-5 of the rounded values), which moves that token's logits by 1e-3.
        # A rounding point that is missing, misplaced or of the wrong kind moves EVERY row by that much; so: nearly
        # all rows agree to fp32 accuracy, and no row is off by more than single flips explain.
        assert np.mean(row_err < 5e-6) >= 0.8, row_err
        assert row_err.max() < 1e-2, row_err
    # the two modes are different functions (so the comparison above can tell them apart) ...
    other = _hf_logits_rounded(shape, w, toks, not round_acts)
    assert np.mean(np.max(np.abs(mine - other), axis=1) < 5e-6) <= 0.1
    # ... as is the rounded mode with any one of its six rounding points left out
    if round_acts and shape.n_layers == 2:
        for point in ("attn_in", "query", "attn_out", "ffn_in", "swiglu", "final"):
            less = _hf_logits_rounded(shape, w, toks, True, skip=point)
            assert np.mean(np.max(np.abs(mine - less), axis=1) < 5e-6) <= 0.2, point
    # ... and so is a forward that keeps K and V unrounded
    if not round_acts:
        exact = _hf_logits_rounded(I.ModelShape(shape.name, shape.n_layers, shape.d_model, shape.n_q_heads,
                                                shape.n_kv_heads, shape.head_dim, shape.ffn_dim, shape.vocab,
                                                shape.rope_theta, "bf16", "fp32"), w, toks, False)
        assert np.max(np.abs(mine - exact)) > 1e-5


def test_bf16_rounding_is_round_to_nearest_even():
    rng = np.random.default_rng(5)
    xs = np.concatenate([rng.standard_normal(20000) * np.exp(rng.uniform(-20, 20, 20000)),
                         [0.0, -0.0, 1.0, -1.0, 3.0e38, -3.0e38, 1e-40, float("inf"), float("-inf")]]).astype(np.float32)
    want = torch.from_numpy(xs).to(torch.bfloat16).to(torch.float32).numpy()
    got = np.array([O.round_bf16(float(x)) for x in xs], dtype=np.float32)
    assert np.array_equal(got.view(np.uint32), want.view(np.uint32))
    assert math.isnan(O.round_bf16(float("nan")))
    # exact ties (the 8th fraction bit set, nothing below it): the neighbour with an even last kept bit wins
    for base, tie, even in ((1.0, 1.0 + 2**-8, 1.0), (1.0, 1.0 + 3 * 2**-8, 1.0 + 2**-6), (-2.0, -2.0 - 2**-7, -2.0),
                            (0.5, 0.5 + 3 * 2**-9, 0.5 + 2**-7)):
        assert O.round_bf16(tie) == even, (tie, O.round_bf16(tie), even)
        assert O.round_bf16(tie) == float(torch.tensor(tie, dtype=torch.float32).to(torch.bfloat16))
    # truncation, or rounding half away from zero, would each fail one of the ties above
    trunc = lambda x: float(np.array([x], np.float32).view(np.uint32)[0] & 0xFFFF0000 and
                            np.array([np.array([x], np.float32).view(np.uint32)[0] & 0xFFFF0000], np.uint32).view(np.float32)[0])
    assert trunc(1.0 + 3 * 2**-8) != O.round_bf16(1.0 + 3 * 2**-8)
    # just above / below a tie goes to the nearer neighbour
    assert O.round_bf16(1.0 + 2**-8 + 2**-20) == 1.0 + 2**-7
    assert O.round_bf16(1.0 + 3 * 2**-8 - 2**-20) == 1.0 + 2**-7


def test_cached_values_are_on_the_bf16_grid():
    shape = I.TINY_BF16
    w = I.make_weights(shape, seed=1)
    model = O.OracleModel(shape, _np_weights(w))
    model.prefill(0, [5, 9, 11, 2])
    c = model.ctx[0]
    K = torch.from_numpy(c.K[:, :3])
    # stored values are already on the bf16 grid
    assert torch.equal(K.to(torch.bfloat16).float(), K)
    assert float(K.abs().max()) > 0


def test_attend_one_against_torch():
    rng = np.random.default_rng(0)
    h, n = 64, 37
    q = rng.standard_normal(h).astype(np.float32)
    K = rng.standard_normal((n, h)).astype(np.float32)
    V = rng.standard_normal((n, h)).astype(np.float32)
    ref = torch.nn.functional.scaled_dot_product_attention(
        torch.tensor(q, dtype=torch.float64)[None, None], torch.tensor(K, dtype=torch.float64)[None],
        torch.tensor(V, dtype=torch.float64)[None])[0, 0].numpy()
    assert np.max(np.abs(O.attend_one(q, K, V) - ref)) < 1e-12
    # one key: the output is its value; equal keys: the mean of the values
    assert np.allclose(O.attend_one(q, K[:1], V[:1]), V[0])
    assert np.allclose(O.attend_one(q, np.repeat(K[:1], 5, 0), V[:5]), V[:5].mean(0))


@pytest.fixture(scope="module")
def tiny():
    w = I.make_weights(I.TINY, seed=0)
    return _np_weights(w)


def test_greedy_verification_reproduces_autoregressive_argmax(tiny):
    shape = I.TINY
    prompt = list(I.make_prompt(shape.vocab, 12, 0, 1))
    a = O.OracleModel(shape, tiny)
    a.prefill(1, prompt)
    gen = []
    for _ in range(6):                           # plain decoding: k = 0 greedy steps
        st, n_acc, nxt, _, _ = a.verify(1, [], None, seed=0, greedy=True)
        assert (st, n_acc) == (0, 0)
        gen.append(nxt)
    b = O.OracleModel(shape, tiny)
    b.prefill(1, prompt)
    st, n_acc, nxt, _, _ = b.verify(1, gen[:5], None, seed=0, greedy=True)
    assert (n_acc, nxt) == (5, gen[5])           # all accepted, bonus token = the next argmax
    for r in range(5):                           # corrupt draft r+1: rejected there, corrected to the argmax
        c = O.OracleModel(shape, tiny)
        c.prefill(1, prompt)
        bad = list(gen[:5])
        bad[r] = (bad[r] + 1) % shape.vocab
        st, n_acc, nxt, _, _ = c.verify(1, bad, None, seed=0, greedy=True)
        assert (n_acc, nxt) == (r, gen[r])
        assert c.ctx[1].tokens == prompt + gen[:r + 1]
        assert c.ctx[1].n_kv == len(prompt) - 1 + r + 1


def test_rollback_is_transparent(tiny):
    shape = I.TINY
    prompt = list(I.make_prompt(shape.vocab, 10, 0, 2))
    a = O.OracleModel(shape, tiny)
    a.prefill(2, prompt)
    d, q = I.make_drafts(shape.vocab, 4, 0, 2)
    st, n_acc, nxt, _, _ = a.verify(2, d.numpy(), q.numpy(), seed=5)
    assert st == 0 and n_acc < 4                 # some drafts rolled back (independent q: nearly always)
    history = a.ctx[2].tokens
    assert history == prompt + [int(x) for x in d[:n_acc]] + [nxt]
    b = O.OracleModel(shape, tiny)               # fresh context with the committed history
    b.prefill(2, history)
    d2, q2 = I.make_drafts(shape.vocab, 3, 0, 2, step=1)
    ra = a.verify(2, d2.numpy(), q2.numpy(), seed=6)
    rb = b.verify(2, d2.numpy(), q2.numpy(), seed=6)
    assert ra[:3] == rb[:3]
    assert np.array_equal(ra[3], rb[3])          # bit-identical logits: stale cache rows were never read


def test_sampling_positions_do_not_collide_across_steps(tiny):
    # the uniforms of consecutive steps of one context use distinct counters
    shape = I.TINY
    a = O.OracleModel(shape, tiny)
    a.prefill(3, [1, 2, 3])
    seen = set()
    for step in range(4):
        c = a.ctx[3]
        d, q = I.make_drafts(shape.vocab, 2, 0, 3, step=step)
        pos0 = c.n_kv
        st, n_acc, nxt, _, _ = a.verify(3, d.numpy(), q.numpy(), seed=1)
        for j in range(n_acc + 1):
            assert pos0 + j + 1 not in seen
            seen.add(pos0 + j + 1)


def test_resent_drafts_continue_the_devices_view(tiny):
    # Section 3.3: after a timeout the device sends its drafts again, extended.  If the server had in fact
    # processed the first request, it must go back to the length the device still believes in (base_len);
    # the outcome must be that of a context that never saw the first request.
    shape = I.TINY
    prompt = list(I.make_prompt(shape.vocab, 9, 0, 4))
    a = O.OracleModel(shape, tiny)
    a.prefill(4, prompt)
    d1, q1 = I.make_drafts(shape.vocab, 3, 0, 4)
    a.verify(4, d1.numpy(), q1.numpy(), seed=1)                   # processed; its answer is lost on the way back
    assert a.ctx[4].n_kv + 1 > len(prompt)
    d2, q2 = I.make_drafts(shape.vocab, 5, 0, 4, step=1)          # the resent, longer draft from the old position
    ra = a.verify(4, d2.numpy(), q2.numpy(), seed=2, base_len=len(prompt))
    b = O.OracleModel(shape, tiny)
    b.prefill(4, prompt)
    rb = b.verify(4, d2.numpy(), q2.numpy(), seed=2)
    assert ra[:3] == rb[:3] and np.array_equal(ra[3], rb[3])
    assert a.ctx[4].tokens == b.ctx[4].tokens and a.ctx[4].n_kv == b.ctx[4].n_kv and a.ctx[4].pending == b.ctx[4].pending
    # every admissible base_len gives the state of a fresh context with that history; base_len = current length is a no-op
    full = list(a.ctx[4].tokens)
    for m in range(1, len(full) + 1):
        c = O.OracleModel(shape, tiny)
        c.prefill(4, full)
        c.rebase(4, m)
        assert (c.ctx[4].tokens, c.ctx[4].n_kv, c.ctx[4].pending) == (full[:m], m - 1, full[m - 1])
    for bad in (0, len(full) + 1):
        c = O.OracleModel(shape, tiny)
        c.prefill(4, full)
        with pytest.raises(ValueError):
            c.rebase(4, bad)
    # a context whose cache was given without its tokens can only go back to where its known history starts
    K, V = I.make_kv(shape, 6, 0, 1)
    c = O.OracleModel(shape, tiny)
    c.load_kv(5, K.numpy(), V.numpy(), pending=3)
    c.verify(5, d1.numpy(), q1.numpy(), seed=1)
    c.rebase(5, 7)
    assert (c.ctx[5].n_kv, c.ctx[5].pending) == (6, 3)
    with pytest.raises(ValueError):
        c.rebase(5, 6)
