"""Ragged verification attention over the paged cache vs the oracle's one-query attention."""
import numpy as np
import pytest
import torch

from oracle import oracle as O
from paper_2506_09397_b200 import binding as B
from paper_2506_09397_b200 import inputs as I

pytestmark = pytest.mark.gpu


def _attn_shape(h, hq, hkv, kv="bf16"):
    # a one-layer model: only the cache geometry matters for the attention-only entry
    return I.ModelShape("attn_only", 1, 64, hq, hkv, h, 64, 64, 5e5, "bf16" if kv == "bf16" else "fp32", kv)


@pytest.mark.parametrize("h,hq,hkv,kv,impl", [(128, 32, 8, "bf16", 0), (128, 32, 8, "bf16", 1), (64, 32, 8, "bf16", 0),
                                              (64, 4, 4, "fp32", 0)])
def test_ragged_attention_matches_oracle(h, hq, hkv, kv, impl):
    # impl 1: the tcgen05 kernel (head_dim 128, at most 48 query rows per request); 0: the warp-level kernels
    shape = _attn_shape(h, hq, hkv, kv)
    w = I.make_weights(shape, 0)
    lens = [128, 131, 700, 2048, 5000, 9, 16, 17, 1023, 3000]     # total cached tokens incl. the new ones
    qlens = [2, 9, 5, 3, 8, 9, 4, 1, 7, 6]
    n_pages = sum((n + 15) // 16 for n in lens) + 4
    eng = B.Engine(shape, w, n_pages=n_pages, max_batch=16, max_k=8, max_step_tokens=128, attention_impl=impl)
    eng.shuffle_pages(1)
    Ks, Vs = {}, {}
    for i, n in enumerate(lens):
        K, V = I.make_kv(shape, n, 4, i)
        eng.load_kv(100 + i, K, V, pending=0)
        Ks[i], Vs[i] = K[0].float().numpy(), V[0].float().numpy()
    T = sum(qlens)
    adt = torch.bfloat16 if kv == "bf16" else torch.float32
    g = torch.Generator().manual_seed(3)
    q = torch.randn(T, hq, h, generator=g).to(adt)
    out = torch.zeros(T, hq, h, dtype=adt, device="cuda")
    eng.attention_ragged(0, [100 + i for i in range(len(lens))], qlens, q.cuda(), out)
    out = out.float().cpu().numpy()
    rng = np.random.default_rng(0)
    t = 0
    worst = 0.0
    for i, (n, ql) in enumerate(zip(lens, qlens)):
        for j in range(ql):
            n_vis = n - ql + j + 1
            for head in rng.choice(hq, size=3, replace=False):
                kvh = head // (hq // hkv)
                ref = O.attend_one(q[t + j, head].float().numpy(), Ks[i][:n_vis, kvh], Vs[i][:n_vis, kvh])
                worst = max(worst, float(np.max(np.abs(out[t + j, head] - ref)) / max(1e-2, float(np.abs(ref).max()))))
        t += ql
    # error relative to the size of the output row: bf16 output and probability rounding is 2^-9 relative
    assert worst <= (1e-2 if kv == "bf16" else 2e-5), worst
    eng.shutdown()
