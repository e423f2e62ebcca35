"""The 8-bit and 4-bit weight paths (linear_weight_bits = 8: e4m3 bytes, 4: e2m1 nibbles two to a byte, each with one
fp32 scale per output row) against the oracle
run on the matrices those bytes stand for.  No weight is quantised on the device: both sides are given the same bytes
and scales.  The device feeds its bf16 activations to fp8 MMAs as two e4m3 parts per element (eight significant
bits, like bf16) and sums in fp32, so the comparison is the bf16 path's, with the same tolerance."""
import dataclasses

import numpy as np
import pytest
import torch

from oracle import oracle as O
from paper_2506_09397_b200 import binding as B
from paper_2506_09397_b200 import inputs as I
from test_gpu_forward import TOL, _verify_both

pytestmark = pytest.mark.gpu


def _both_sides(shape, w_bf16, bits=8, **eng_args):
    """Engine on the bytes, oracle on the fp32 matrices they mean (embedding and gains widened exactly)."""
    q, deq = I.quantize_linear_weights(w_bf16, bits=bits)
    eng = B.Engine(shape, q, linear_weight_bits=bits, **eng_args)
    f32 = {k: ([t.float().numpy() for t in v] if isinstance(v, list) else v.float().numpy())
           for k, v in deq.items() if not k.endswith("_scale")}
    orc = O.OracleModel(dataclasses.replace(shape, weight_dtype="fp32"), f32)
    return eng, orc


def test_every_byte_pattern_is_decoded():
    # LM-head row n holds byte n in every column (scale 1): its logit is e4m3(n) x (sum of the normalised hidden
    # state).  All 254 patterns - subnormals and both zeros among them - against the oracle's fp32 matrix.
    shape = I.ModelShape("w8_bytes", 1, 256, 4, 2, 64, 512, 256, 5e5, "bf16", "bf16")
    w = I.make_weights(shape, seed=3)
    q, deq = I.quantize_linear_weights(w)
    pattern = torch.arange(256, dtype=torch.uint8)
    pattern[0x7f] = 0
    pattern[0xff] = 0
    q["lm_head"] = pattern[:, None].repeat(1, shape.d_model).contiguous()
    q["lm_head_scale"] = torch.ones(256)
    deq["lm_head"] = I.from_e4m3_rows(q["lm_head"], q["lm_head_scale"])
    values = deq["lm_head"][:, 0]
    assert float(values[0x01]) == 2.0 ** -9 and float(values[0x7e]) == 448.0 and float(values[0x88]) == -(2.0 ** -6)
    eng = B.Engine(shape, q, linear_weight_bits=8, n_pages=8, max_batch=2, max_k=2, max_step_tokens=8)
    f32 = {k: ([t.float().numpy() for t in v] if isinstance(v, list) else v.float().numpy())
           for k, v in deq.items() if not k.endswith("_scale")}
    orc = O.OracleModel(dataclasses.replace(shape, weight_dtype="fp32"), f32)
    p = I.make_prompt(shape.vocab, 5, 3, 1)
    eng.prefill(1, p)
    orc.prefill(1, p)
    d, qq = I.make_drafts(shape.vocab, 2, 3, 1)
    eng.set_commit(False)
    eng.verify_batch([(1, d.numpy(), qq.numpy())], 0)
    glog = eng.logits(3)
    st, n_acc, nxt, ol, mg = orc.verify(1, d.numpy(), qq.numpy(), 0, commit=False)
    hidden_sum = ol[:, 0x38] / float(values[0x38])                     # byte 0x38 is 1.0
    assert np.all(np.abs(hidden_sum) > 1.0), hidden_sum
    mag = np.maximum(np.abs(values.numpy()), 2.0 ** -9)
    for row in range(3):
        want = values.numpy() * hidden_sum[row]
        assert np.max(np.abs(ol[row] - want)) <= 1e-3 * np.max(np.abs(want))          # the oracle itself
        # a wrongly decoded byte is off by an eighth of its value at least; bf16 inputs cost far less
        assert np.all(np.abs(glog[row] - want) <= mag * (2e-2 * np.abs(hidden_sum[row]) + 0.05)), row
    eng.shutdown()


def test_every_nibble_pattern_is_decoded():
    # LM-head row n holds code n % 16 in every column (scale 1): its logit is e2m1(n % 16) x (sum of the normalised
    # hidden state); rows 16.. put the code in the even or the odd columns only (low / high half of a byte)
    shape = I.ModelShape("w4_nibbles", 1, 256, 4, 2, 64, 512, 256, 5e5, "bf16", "bf16")
    w = I.make_weights(shape, seed=3)
    q, deq = I.quantize_linear_weights(w, bits=4)
    rows = torch.arange(256, dtype=torch.uint8)
    code = rows % 16
    low = torch.where((rows < 16) | (rows % 2 == 0), code, torch.zeros_like(code))
    high = torch.where((rows < 16) | (rows % 2 == 1), code, torch.zeros_like(code))
    q["lm_head"] = (low | (high << 4))[:, None].repeat(1, shape.d_model // 2).contiguous()
    q["lm_head_scale"] = torch.ones(256)
    deq["lm_head"] = I.from_e2m1_rows(q["lm_head"], q["lm_head_scale"])
    assert [float(v) for v in deq["lm_head"][:16, 0]] == [0, .5, 1, 1.5, 2, 3, 4, 6, 0, -.5, -1, -1.5, -2, -3, -4, -6]
    assert float(deq["lm_head"][19, 0]) == 0.0 and float(deq["lm_head"][19, 1]) == 1.5      # odd row: high half only
    eng = B.Engine(shape, q, linear_weight_bits=4, n_pages=8, max_batch=2, max_k=2, max_step_tokens=8)
    f32 = {k: ([t.float().numpy() for t in v] if isinstance(v, list) else v.float().numpy())
           for k, v in deq.items() if not k.endswith("_scale")}
    orc = O.OracleModel(dataclasses.replace(shape, weight_dtype="fp32"), f32)
    p = I.make_prompt(shape.vocab, 5, 3, 1)
    eng.prefill(1, p)
    orc.prefill(1, p)
    d, qq = I.make_drafts(shape.vocab, 2, 3, 1)
    eng.set_commit(False)
    eng.verify_batch([(1, d.numpy(), qq.numpy())], 0)
    glog = eng.logits(3)
    st, n_acc, nxt, ol, mg = orc.verify(1, d.numpy(), qq.numpy(), 0, commit=False)
    values = deq["lm_head"].numpy()
    mag = np.abs(values).max(axis=1)                                    # |e2m1(code)| of each row
    checked = 0
    for row in range(3):
        # the three sums a logit can be a multiple of: all columns, the even ones, the odd ones (rows 2, 18, 19)
        sums = np.array([ol[row, 2] / 1.0, ol[row, 18] / 1.0, ol[row, 19] / 1.5])
        if not np.all(np.abs(sums) > 1.5):       # a sum near zero tells a wrong code from rounding noise badly
            continue
        checked += 1
        which = np.where(np.arange(256) < 16, 0, 1 + np.arange(256) % 2)
        want = np.where(np.arange(256) % 2 == 1, values[:, 1], values[:, 0]) * sums[which]
        assert np.max(np.abs(ol[row] - want)) <= 1e-3 * np.max(np.abs(want))          # the oracle itself
        # a wrongly decoded code is off by a quarter of its value at least, a swapped half by all of it; the
        # bf16 inputs cost far less
        assert np.all(np.abs(glog[row] - want) <= mag * (2e-2 * np.abs(sums[which]) + 0.15)), row
    assert checked >= 1
    eng.shutdown()


@pytest.mark.parametrize("n_req,k,attention_impl,bits", [(4, 4, 0, 8), (16, 8, 0, 8), (40, 8, 0, 8), (5, 8, 1, 8),
                                                         (4, 4, 0, 4), (16, 8, 0, 4), (40, 8, 0, 4)])
def test_steps_with_8bit_weights_match_the_oracle(n_req, k, attention_impl, bits):
    # narrow and wide steps (20, 144 and 360 tokens: token tiles of 32, 160 and 3 x 128), prefill in chunks, commit
    shape = I.SMALL_GQA
    w = I.make_weights(shape, seed=5)
    eng, orc = _both_sides(shape, w, bits=bits, n_pages=4 * n_req + 32, max_batch=n_req, max_k=8, max_step_tokens=max(n_req * (k + 1), 64),
                           attention_impl=attention_impl)   # 1: the tcgen05 attention kernel in front of the merge + split
    checked = sorted({0, n_req // 2, n_req - 1})
    for c in range(n_req):
        p = I.make_prompt(shape.vocab, 3 + (5 * c) % 31, 5, c)
        eng.prefill(c, p)
        if c in checked:
            orc.prefill(c, p)
    explain = []
    for step in range(2):
        reqs = [(c,) + tuple(I.make_drafts(shape.vocab, k, 5, c, step)) for c in range(n_req)]
        if step == 0:
            # every request on the device, the checked ones on both sides
            eng.set_commit(False)
            eng.verify_batch([(c, d.numpy(), q.numpy()) for c, d, q in reqs], step)
            eng.set_commit(True)
        _verify_both(eng, orc, [r for r in reqs if r[0] in checked], seed=step, tau=1.0, greedy=False, tol=TOL["bf16"],
                     explain=explain)
    eng.shutdown()


@pytest.mark.parametrize("bits", [8, 4])
def test_8bit_weights_with_ragged_matrix_shapes(bits):
    # inner sizes that are not multiples of the 128-wide k-slab (320 = 2.5 slabs, 784 = 6.125) and row counts that are
    # not multiples of the 128-row weight tile (960, 320, 1568, 4200): the last slab and the last tile are partly empty
    shape = I.ModelShape("odd_w8", 2, 320, 5, 5, 64, 784, 4200, 5e5, "bf16", "bf16")
    w = I.make_weights(shape, seed=7)
    eng, orc = _both_sides(shape, w, bits=bits, n_pages=200, max_batch=12, max_k=8, max_step_tokens=108)
    for c in range(12):
        p = I.make_prompt(shape.vocab, 2 + (5 * c) % 23, 7, c)
        eng.prefill(c, p)
        if c % 4 == 0:
            orc.prefill(c, p)
    explain = []
    reqs = [(c,) + tuple(I.make_drafts(shape.vocab, 5 + c % 4, 7, c)) for c in range(12)]
    eng.set_commit(False)
    eng.verify_batch([(c, d.numpy(), q.numpy()) for c, d, q in reqs], 1)
    eng.set_commit(True)
    _verify_both(eng, orc, [r for r in reqs if r[0] % 4 == 0], seed=1, tau=1.0, greedy=False, tol=TOL["bf16"], explain=explain)
    eng.shutdown()


def test_8bit_weights_need_scales_and_bf16():
    shape = I.SMALL_GQA
    w = I.make_weights(shape, seed=5)
    with pytest.raises(B.SledError):
        B.Engine(I.TINY, I.quantize_linear_weights(I.make_weights(I.TINY, 0))[0], linear_weight_bits=8, n_pages=8,
                 max_batch=1, max_k=1, max_step_tokens=8)      # fp32 model
    with pytest.raises(B.SledError):
        B.Engine(shape, w, linear_weight_bits=2, n_pages=8, max_batch=1, max_k=1, max_step_tokens=8)   # no such width
    with pytest.raises(B.SledError):
        B.Engine(I.TINY, I.quantize_linear_weights(I.make_weights(I.TINY, 0), bits=4)[0], linear_weight_bits=4, n_pages=8,
                 max_batch=1, max_k=1, max_step_tokens=8)      # fp32 model
