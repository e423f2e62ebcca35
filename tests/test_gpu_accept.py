"""Acceptance kernel vs the oracle: bit-exact n_accepted / next_token on identical logits."""
import numpy as np
import pytest
import torch

from oracle import oracle as O
from paper_2506_09397_b200 import binding as B
from paper_2506_09397_b200 import inputs as I

pytestmark = pytest.mark.gpu


def _run_both(z, q, d, ks, tau, greedy, seed, ctx0=1000, pos0_base=17):
    """z [n, kmax+1, V], q [n, kmax, V], d [n, kmax] CPU tensors; request i uses its first ks[i] drafts."""
    n, V = z.shape[0], z.shape[2]
    rows, qrows, drafts, cu = [], [], [], [0]
    for i in range(n):
        k = ks[i]
        rows.append(z[i, :k + 1])
        qrows.append(q[i, :k])
        drafts += [int(x) for x in d[i, :k]]
        cu.append(cu[-1] + k + 1)
    logits = torch.cat(rows).contiguous()
    qcat = torch.cat(qrows).contiguous() if sum(ks) else torch.zeros(0, V)
    ctx = [ctx0 + 7 * i for i in range(n)]
    pos0 = [pos0_base + 3 * i for i in range(n)]
    got, ms = B.accept_rows(logits.cuda(), cu, drafts, None if greedy else qcat.cuda(), ctx, pos0, tau, greedy, seed)
    want = []
    for i in range(n):
        k = ks[i]
        st, n_acc, nxt, _ = O.accept(rows[i].numpy(), None if greedy or k == 0 else qrows[i].numpy(),
                                     np.array(drafts[cu[i] - i:cu[i] - i + k], np.int32), tau, greedy, seed, ctx[i], pos0[i])
        want.append((n_acc, nxt, 0 if st == 0 else B.SLED_ERR_NONFINITE))
    return got, want


@pytest.mark.parametrize("tau,greedy", [(1.0, False), (0.7, False), (1.0, True)])
def test_full_vocab_rows(tau, greedy):
    n, k, V = 24, 7, 128256
    z, q, d = I.make_accept_rows(n, k, V, tau_draft=1.0, seed=3)
    ks = [int(x) for x in np.random.default_rng(1).integers(0, k + 1, n)]
    ks[0], ks[1] = k, 0
    got, want = _run_both(z, q, d, ks, tau, greedy, seed=11)
    assert got == want
    if not greedy:
        assert len({g[0] for g in got}) > 1        # both acceptances and rejections occurred


@pytest.mark.parametrize("V", [1, 5, 1000, 4096, 4097, 33000])
def test_ragged_vocab_sizes(V):
    n, k = 16, 4
    z, q, d = I.make_accept_rows(n, k, V, tau_draft=1.0, seed=V, sigma=1.5)
    got, want = _run_both(z, q, d, [k] * n, 1.3, False, seed=5)
    assert got == want
    got, want = _run_both(z, q, d, [k] * n, 1.0, True, seed=5)
    assert got == want


def test_many_seeds_small_vocab():
    # many decisions on a small vocabulary: exercises accept/reject boundaries and the CDF search
    n, k, V = 512, 3, 64
    z, q, d = I.make_accept_rows(n, k, V, tau_draft=1.0, seed=9, sigma=1.0)
    for seed in range(4):
        got, want = _run_both(z, q, d, [k] * n, 1.0, False, seed=seed)
        assert got == want
    accepted = sum(g[0] for g in got)
    assert 0 < accepted < n * k


def test_degenerate_rows():
    V = 5000
    z = torch.zeros(4, 3, V)
    q = torch.full((4, 2, V), 1.0 / V)
    d = torch.zeros(4, 2, dtype=torch.int32)
    # request 0: q(d) = 0 -> always accepted; request 1: p == q everywhere except rounding -> residual may vanish
    q[0, :, 0] = 0.0
    # request 2: a +inf logit in the first row; request 3: NaN only in a row behind a certain rejection
    z[2, 0, 17] = float("inf")
    z[3, 0, 1] = 60.0              # p concentrated on token 1, draft is token 0 with q = 1
    q[3, 0] = 0.0
    q[3, 0, 0] = 1.0
    z[3, 1:, :] = float("nan")
    got, want = _run_both(z, q, d, [2, 2, 2, 2], 1.0, False, seed=1)
    assert got == want
    assert got[2] == (0, -1, B.SLED_ERR_NONFINITE)
    assert got[3][:2] == (0, 1) and got[3][2] == 0
    z[:, :, 7] = 3.0
    z[:, :, 3] = 3.0               # tie: lowest index wins
    z[2, 0, 17] = 0.0
    z[3] = 0.0
    got, want = _run_both(z, q, d, [2, 2, 2, 2], 1.0, True, seed=1)
    assert got == want and all(g[1] == 3 for g in got[:3]) and got[3] == (2, 0, 0)   # all-equal row: index 0


def test_draft_rows_at_an_odd_address():
    # draft rows are the caller's memory: a 4-byte aligned address that is not 16-byte aligned must work
    n, k, V = 8, 3, 4096
    z, q, d = I.make_accept_rows(n, k, V, tau_draft=1.0, seed=12, sigma=1.5)
    logits = z.reshape(n * (k + 1), V).contiguous().cuda()
    cu = [(k + 1) * i for i in range(n + 1)]
    ctx, pos0 = list(range(50, 50 + n)), [9] * n
    drafts = d.reshape(-1).numpy()
    qa = q.reshape(n * k, V).contiguous().cuda()
    buf = torch.zeros(n * k * V + 1, device="cuda")
    buf[1:] = qa.reshape(-1)
    qb = buf[1:].view(n * k, V)
    assert qb.data_ptr() % 16 == 4
    want, _ = B.accept_rows(logits, cu, drafts, qa, ctx, pos0, 1.0, False, seed=2)
    got, _ = B.accept_rows(logits, cu, drafts, qb, ctx, pos0, 1.0, False, seed=2)
    assert got == want
    assert any(g[0] < k for g in got)            # some request reached the residual pass that reads the row
