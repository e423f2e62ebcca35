"""Pins of the oracle's target-model forward and of the verify / commit state machine."""
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


def test_bf16_rounding_matches_torch():
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
