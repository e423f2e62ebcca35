"""End-to-end agreement of the GPU path with the oracle on a thousand requests per case: how often the two return
the same (n_accepted, next_token), and that every difference sits where the measured logit deviation of that very
request can move the deciding comparison.

The target distributions are made peaked (the LM head of the random-init model is scaled up so that the most likely
token carries a few tenths of the mass, as a trained model's does); the drafts come from distributions correlated
with the oracle's own logits, so that drafts are accepted and rejected at realistic rates.  What to expect:
  * fp32 weights: logits agree to ~1e-5, decisions practically always (>= 99.9 % asserted);
  * bf16 weights: every matrix product sees its input rounded to 16 bits, which moves a logit by about half a percent
    of the logits' spread (no less in the oracle's own 16-bit mode).  Greedy: the decision differs where the top two
    logits are closer than that, about one request in seventy for logits that are spread like these.  Sampling: the
    token is picked by where a uniform number falls in the cumulative distribution, every boundary of which moves
    by up to e^(2 eps) - 1 of the mass, so a good tenth of the draws land on the other side of a boundary.
    The rates are reported; asserted are lower bounds a little under what was measured, and - the point - that each
    single difference is one the logit deviation measured on that very request can cause.
"""
import numpy as np
import pytest
import torch

from oracle import oracle as O
from paper_2506_09397_b200 import binding as B
from paper_2506_09397_b200 import inputs as I
from util import oracle_weights, rel_margin_ok

pytestmark = pytest.mark.gpu

N_CTX, ROUNDS, K = 100, 10, 4          # 1000 requests per case


def _run_case(shape, greedy, tau, head_scale, seed, weight_bits=16):
    w = I.make_weights(shape, seed=seed)
    w["lm_head"] = (w["lm_head"].float() * head_scale).to(w["lm_head"].dtype)
    w_eng, w_orc, shape_orc = w, w, shape
    if weight_bits == 8:   # the engine on e4m3 bytes + row scales, the oracle on the fp32 matrices they stand for
        import dataclasses
        w_eng, deq = I.quantize_linear_weights(w)
        w_orc = {k: ([t.float() for t in v] if isinstance(v, list) else v.float()) for k, v in deq.items()}
        shape_orc = dataclasses.replace(shape, weight_dtype="fp32")
    eng = B.Engine(shape, w_eng, n_pages=N_CTX * 6 + 8, max_batch=N_CTX, max_k=K, max_step_tokens=N_CTX * (K + 1),
                   temperature=tau, greedy=greedy, linear_weight_bits=weight_bits)
    orc = O.OracleModel(shape_orc, oracle_weights(w_orc))
    for c in range(N_CTX):
        p = I.make_prompt(shape.vocab, 6 + c % 11, seed, c)
        eng.prefill(c, p)
        orc.prefill(c, p)
    n_req = n_same = 0
    misses, top1, acc = [], [], 0
    for r in range(ROUNDS):
        reqs = []
        for c in range(N_CTX):
            ctx = orc.ctx[c]
            d, q, tok = np.zeros(K, np.int32), np.zeros((K, shape.vocab), np.float32), ctx.pending
            for j in range(K):                    # drafts from distributions built on the oracle's own logits
                z = orc.forward_token(ctx, int(tok), ctx.n_kv + j)
                tok, qj = I.correlated_draft(torch.from_numpy(z / np.float32(tau)), seed, c, r * K + j, rho=0.97)
                d[j], q[j] = tok, qj.numpy()
            reqs.append((c, d, q))
        got = eng.verify_batch([(c, d, None if greedy else q) for c, d, q in reqs], seed=r)
        glog = eng.logits(N_CTX * (K + 1))
        for i, (c, d, q) in enumerate(reqs):
            pos0 = orc.ctx[c].n_kv
            st, n_acc, nxt, ol, mg = orc.verify(c, d, None if greedy else q, r, tau, greedy, commit=False)
            mine = glog[i * (K + 1):(i + 1) * (K + 1)]
            g = got[i]
            st2, n2, x2, _ = O.accept(mine, None if greedy else q, d, tau, greedy, r, c, pos0)
            assert (n2, x2, 0) == g                                   # always: the oracle's rule on the GPU's logits
            n_req += 1
            acc += g[0]
            e = np.exp((ol[0] - ol[0].max()).astype(np.float64) / tau)
            top1.append(float(e.max() / e.sum()))
            if (n_acc, nxt) == g[:2]:
                n_same += 1
            else:
                upto = max(n_acc, g[0]) + 1
                eps = float(np.max(np.abs(mine[:upto] - ol[:upto])))
                misses.append((c, r, (n_acc, nxt), g[:2], eps, mg.accept_rel, mg.sample_rel, mg.draw_mass, mg.greedy_gap))
                assert rel_margin_ok(mg, eps), misses[-1]
            oc = orc.ctx[c]                                           # both sides continue from the GPU's decision
            oc.n_kv += g[0] + 1
            oc.tokens += [int(x) for x in d[:g[0]]] + [g[1]]
            oc.pending = g[1]
    eng.shutdown()
    rate = n_same / n_req
    print(f"{shape.name} {'greedy' if greedy else f'sampling tau={tau}'}: {n_same}/{n_req} requests agree ({100 * rate:.2f} %), "
          f"acceptance {acc / (n_req * K):.2f}, mean top-1 mass {np.mean(top1):.2f}")
    for m in misses:
        print("   differs:", m)
    assert 0.1 < np.mean(top1) < 0.95 and 0.05 < acc / (n_req * K) < 0.98     # peaked, and both outcomes occur
    return rate


def test_fp32_sampling_agrees():
    assert _run_case(I.TINY, False, 0.7, 14.0, 21) >= 0.999


def test_bf16_greedy_every_difference_is_explained():
    assert _run_case(I.SMALL_GQA, True, 1.0, 9.0, 22) >= 0.97       # measured 98.5 %


def test_bf16_sampling_every_difference_is_explained():
    assert _run_case(I.SMALL_GQA, False, 1.0, 9.0, 23) >= 0.8       # measured 86.6 %


def test_8bit_weights_greedy_every_difference_is_explained():
    # the 8-bit weight path (activations as two e4m3 parts on fp8 MMAs) against the oracle on the same bytes: as with
    # bf16 weights, decisions differ only where the top two logits are closer than the measured deviation
    assert _run_case(I.SMALL_GQA, True, 1.0, 9.0, 24, weight_bits=8) >= 0.97
