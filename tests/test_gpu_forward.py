"""Whole verification step on the GPU vs the oracle: logits within tolerance, decisions equal
(or explained by a deciding margin below the tolerance), cache commit / rollback."""
import numpy as np
import pytest
import torch

from oracle import oracle as O
from paper_2506_09397_b200 import binding as B
from paper_2506_09397_b200 import inputs as I
from util import oracle_weights, rel_margin_ok

pytestmark = pytest.mark.gpu

TOL = {"fp32": 1e-4, "bf16": 2e-2}   # max |logit difference| allowed per weight type


def _engine(shape, w, **kw):
    args = dict(n_pages=256, max_batch=16, max_k=8, max_step_tokens=160)
    args.update(kw)
    return B.Engine(shape, w, **args)


def _verify_both(eng, orc, reqs, seed, tau, greedy, tol, explain):
    """reqs: list of (ctx, drafts tensor, q tensor).  Runs one step on both sides and compares."""
    got = eng.verify_batch([(c, d.numpy(), None if greedy else q.numpy()) for c, d, q in reqs], seed)
    T = sum(len(d) + 1 for _, d, _ in reqs)
    glog = eng.logits(T)
    row = 0
    for (c, d, q), g in zip(reqs, got):
        k = len(d)
        pos0 = orc.ctx[c].n_kv
        st, n_acc, nxt, ologits, mg = orc.verify(c, d.numpy(), None if greedy else q.numpy(), seed, tau, greedy, commit=False)
        mine = glog[row:row + k + 1]
        row += k + 1
        assert np.max(np.abs(mine - ologits)) <= tol, (c, float(np.max(np.abs(mine - ologits))))
        # bit-exact given identical logits: the oracle's rule on the GPU's logits
        st2, n2, x2, _ = O.accept(mine, None if greedy or k == 0 else q.numpy(), d.numpy(), tau, greedy, seed, c, pos0)
        assert (n2, x2) == g[:2] and g[2] == 0
        if (n_acc, nxt) != g[:2]:
            # the two sides may differ only where the logit deviation measured on the rows either side looked at can
            # move the deciding comparison
            upto = max(n_acc, g[0]) + 1
            eps = float(np.max(np.abs(mine[:upto] - ologits[:upto])))
            assert rel_margin_ok(mg, eps), (c, (n_acc, nxt), g, eps, mg.accept_rel, mg.sample_rel, mg.greedy_gap, mg.draw_mass)
            explain.append(c)
        # the oracle follows the GPU's decision so that both sides keep the same history
        oc = orc.ctx[c]
        oc.n_kv += g[0] + 1
        oc.tokens += [int(x) for x in d[:g[0]]] + [g[1]]
        oc.pending = g[1]
    return got


@pytest.mark.parametrize("shape_name", ["tiny", "tiny_bf16", "small_gqa"])
def test_prefilled_contexts_multi_step(shape_name):
    shape = I.SHAPES[shape_name]
    tol = TOL[shape.weight_dtype]
    w = I.make_weights(shape, seed=0)
    eng = _engine(shape, w)
    orc = O.OracleModel(shape, oracle_weights(w))
    ctxs = [11, 12, 13, 14]
    lens = [64, 64, 64, 64] if shape_name == "tiny" else [33, 5, 64, 18]
    for c, n in zip(ctxs, lens):
        p = I.make_prompt(shape.vocab, n, 0, c)
        eng.prefill(c, p)
        orc.prefill(c, p)
    # cache written by the prefill: on the format's grid and close to the oracle's
    K, V = eng.read_kv(ctxs[0], shape.n_layers - 1, lens[0] - 1)
    ok = orc.ctx[ctxs[0]].K[shape.n_layers - 1, :lens[0] - 1]
    assert np.max(np.abs(K.float().numpy() - ok)) <= (2e-2 if shape.kv_dtype == "bf16" else 1e-5)
    explain = []
    for step in range(4):
        ks = [4, 4, 4, 4] if (shape_name == "tiny" and step == 0) else I.draw_k(4, [0, 1, 3, 5, 8], seed=step)
        reqs = []
        for c, k in zip(ctxs, ks):
            d, q = I.make_drafts(shape.vocab, k, 0, c, step)
            reqs.append((c, d, q))
        greedy = step == 3
        eng.set_sampling(1.0 if step < 2 else 0.8, greedy)
        _verify_both(eng, orc, reqs, seed=step, tau=1.0 if step < 2 else 0.8, greedy=greedy, tol=tol, explain=explain)
        for c in ctxs:   # commit / rollback bookkeeping agrees
            n_kv, pending, pages = eng.query_ctx(c)
            assert (n_kv, pending) == (orc.ctx[c].n_kv, orc.ctx[c].pending)
            assert len(pages) == (n_kv + 15) // 16
    assert len(explain) <= 8          # each one was checked to sit within the deciding margin
    st = eng.stats()
    assert st.steps == 4 and st.kernels_last_step > 0 and st.tokens_committed > 0
    for c in ctxs:
        eng.release(c)
    assert eng.stats().pages_free == 256
    eng.shutdown()


def test_greedy_accepts_its_own_continuation():
    # generate with k = 0 steps, then verify that continuation as drafts: all accepted + bonus
    shape = I.TINY
    w = I.make_weights(shape, seed=0)
    eng = _engine(shape, w, greedy=True)
    p = I.make_prompt(shape.vocab, 20, 0, 1)
    eng.prefill(1, p)
    gen = []
    for _ in range(7):
        (n_acc, nxt, st), = eng.verify_batch([(1, [], None)], 0)
        assert (n_acc, st) == (0, 0)
        gen.append(nxt)
    eng.prefill(2, p)
    (n_acc, nxt, st), = eng.verify_batch([(2, gen[:6], None)], 0)
    assert (n_acc, nxt) == (6, gen[6])
    eng.prefill(3, p)
    bad = list(gen[:6])
    bad[2] = (bad[2] + 1) % shape.vocab
    (n_acc, nxt, st), = eng.verify_batch([(3, bad, None)], 0)
    assert (n_acc, nxt) == (2, gen[2])
    assert eng.query_ctx(3)[0] == 19 + 3
    eng.shutdown()


def test_batch_composition_does_not_change_a_request():
    shape = I.SMALL_GQA
    w = I.make_weights(shape, seed=1)
    eng = _engine(shape, w)
    eng.set_commit(False)
    for c, n in [(1, 40), (2, 9), (3, 70)]:
        eng.prefill(c, I.make_prompt(shape.vocab, n, 1, c))
    reqs = {c: I.make_drafts(shape.vocab, k, 1, c) for c, k in [(1, 5), (2, 8), (3, 2)]}
    alone = {}
    for c, (d, q) in reqs.items():
        alone[c] = (eng.verify_batch([(c, d.numpy(), q.numpy())], 7)[0], eng.logits(len(d) + 1))
    order = [3, 1, 2]
    got = eng.verify_batch([(c, reqs[c][0].numpy(), reqs[c][1].numpy()) for c in order], 7)
    lg = eng.logits(sum(len(reqs[c][0]) + 1 for c in order))
    row = 0
    for c, g in zip(order, got):
        k = len(reqs[c][0])
        assert np.max(np.abs(lg[row:row + k + 1] - alone[c][1])) <= 2e-3   # same math, different tile shapes
        row += k + 1
        assert g == alone[c][0]
    eng.shutdown()


@pytest.mark.parametrize("attention_impl", [0, 1])
def test_synthetic_cache_and_long_context_split(attention_impl):
    # cache content loaded directly; one context long enough that its keys are split over several blocks
    # (attention_impl 1: the same step with the tcgen05 attention kernel)
    shape = I.SMALL_GQA
    w = I.make_weights(shape, seed=2)
    eng = _engine(shape, w, n_pages=400, attention_impl=attention_impl)
    eng.shuffle_pages(5)
    orc = O.OracleModel(shape, oracle_weights(w))
    lens = {21: 1500, 22: 300, 23: 17}
    for c, n in lens.items():
        K, V = I.make_kv(shape, n, 2, c)
        K, V = K * 0.3, V * 0.3
        eng.load_kv(c, K.contiguous(), V.contiguous(), pending=5)
        orc.load_kv(c, K.float().numpy(), V.float().numpy(), pending=5)
        Kb, Vb = eng.read_kv(c, 1, n)
        assert torch.equal(Kb, K[1]) and torch.equal(Vb, V[1])   # paged gather == the contiguous cache
    reqs = []
    for c, k in zip(lens, [8, 3, 6]):
        d, q = I.make_drafts(shape.vocab, k, 2, c)
        reqs.append((c, d, q))
    explain = []
    _verify_both(eng, orc, reqs, seed=3, tau=1.0, greedy=False, tol=2e-2, explain=explain)
    eng.shutdown()


def test_large_step_uses_several_token_tiles():
    # more than 256 tokens in one step: the linear layers run as several token tiles per weight tile
    # (and tiles shared between blocks); a long prefill chunk goes the same way
    shape = I.SMALL_GQA
    w = I.make_weights(shape, seed=4)
    eng = _engine(shape, w, n_pages=600, max_batch=40, max_k=8, max_step_tokens=400)
    orc = O.OracleModel(shape, oracle_weights(w))
    ctxs = list(range(40))
    for c in ctxs:
        n = 3 + (7 * c) % 29
        p = I.make_prompt(shape.vocab, n, 4, c)
        eng.prefill(c, p)
        if c % 9 == 0:
            orc.prefill(c, p)
    reqs = []
    for c in ctxs:
        d, q = I.make_drafts(shape.vocab, 8 if c % 3 else 5, 4, c)
        reqs.append((c, d, q))
    T = sum(len(d) + 1 for _, d, _ in reqs)
    assert T > 256
    eng.set_commit(False)
    got = eng.verify_batch([(c, d.numpy(), q.numpy()) for c, d, q in reqs], 9)
    glog = eng.logits(T)
    row = 0
    for (c, d, q), g in zip(reqs, got):
        k = len(d)
        if c in orc.ctx:
            st, n_acc, nxt, ol, mg = orc.verify(c, d.numpy(), q.numpy(), 9, commit=False)
            assert np.max(np.abs(glog[row:row + k + 1] - ol)) <= 2e-2
            st2, n2, x2, _ = O.accept(glog[row:row + k + 1], q.numpy(), d.numpy(), 1.0, False, 9, c, orc.ctx[c].n_kv)
            assert (n2, x2, 0) == g
        row += k + 1
    # a prompt longer than one step: prefilled in chunks of max_step_tokens (> 256 tokens per chunk)
    long_prompt = I.make_prompt(shape.vocab, 700, 4, 99)
    eng.prefill(99, long_prompt)
    orc.prefill(99, long_prompt)
    K, V = eng.read_kv(99, shape.n_layers - 1, 699)
    assert np.max(np.abs(K.float().numpy() - orc.ctx[99].K[shape.n_layers - 1, :699])) <= 2e-2
    d, q = I.make_drafts(shape.vocab, 4, 4, 99)
    eng.set_commit(True)
    _verify_both(eng, orc, [(99, d, q)], seed=2, tau=1.0, greedy=False, tol=2e-2, explain=[])
    eng.shutdown()


def test_large_step_ragged_matrix_shapes():
    # more than 128 tokens with matrices whose row counts are not multiples of the 128-row weight tile and whose
    # inner sizes are not multiples of the 64-wide k-slab: an even number of weight tiles runs as CTA pairs (QKV: 960
    # rows -> 8 tiles, the last one half empty), an odd number as single CTAs (O and down: 3 tiles, gate/up: 13,
    # LM head: 33); the down projection has a k tail (776 = 12 slabs + 8)
    shape = I.ModelShape("odd_bf16", 2, 320, 5, 5, 64, 776, 4200, 5e5, "bf16", "bf16")
    w = I.make_weights(shape, seed=6)
    eng = _engine(shape, w, n_pages=400, max_batch=30, max_k=8, max_step_tokens=300)
    orc = O.OracleModel(shape, oracle_weights(w))
    ctxs = list(range(30))
    for c in ctxs:
        p = I.make_prompt(shape.vocab, 2 + (5 * c) % 23, 6, c)
        eng.prefill(c, p)
        if c % 7 == 0:
            orc.prefill(c, p)
    reqs = [(c,) + tuple(I.make_drafts(shape.vocab, 5 + c % 4, 6, c)) for c in ctxs]
    T = sum(len(d) + 1 for _, d, _ in reqs)
    assert T > 128
    eng.set_commit(False)
    got = eng.verify_batch([(c, d.numpy(), q.numpy()) for c, d, q in reqs], 5)
    glog = eng.logits(T)
    row = 0
    for (c, d, q), g in zip(reqs, got):
        k = len(d)
        if c in orc.ctx:
            st, n_acc, nxt, ol, mg = orc.verify(c, d.numpy(), q.numpy(), 5, commit=False)
            assert np.max(np.abs(glog[row:row + k + 1] - ol)) <= 2e-2
            st2, n2, x2, _ = O.accept(glog[row:row + k + 1], q.numpy(), d.numpy(), 1.0, False, 5, c, orc.ctx[c].n_kv)
            assert (n2, x2, 0) == g
        row += k + 1
    eng.shutdown()


def test_edge_batches():
    # empty batch, a batch of plain decoding steps (k = 0 everywhere), the largest allowed batch, page reuse
    shape = I.TINY
    w = I.make_weights(shape, seed=0)
    eng = _engine(shape, w, n_pages=16, max_batch=3, max_k=4, max_step_tokens=15)
    orc = O.OracleModel(shape, oracle_weights(w))
    assert eng.verify_batch([], 0) == []
    for c in (1, 2, 3):
        p = I.make_prompt(shape.vocab, 1 if c == 1 else 17 + c, 0, c)     # context 1: only a pending token, empty cache
        eng.prefill(c, p)
        orc.prefill(c, p)
    explain = []
    got = _verify_both(eng, orc, [(c, torch.zeros(0, dtype=torch.int32), torch.zeros(0, shape.vocab)) for c in (1, 2, 3)],
                       seed=1, tau=1.0, greedy=False, tol=1e-4, explain=explain)
    assert all(g[0] == 0 for g in got)
    reqs = []
    for c in (1, 2, 3):                                                   # max_batch requests of max_k drafts = max_step_tokens
        d, q = I.make_drafts(shape.vocab, 4, 0, c, step=1)
        reqs.append((c, d, q))
    eng.set_sampling(0.9, False)
    _verify_both(eng, orc, reqs, seed=2, tau=0.9, greedy=False, tol=1e-4, explain=explain)
    for c in (1, 2, 3):
        assert eng.query_ctx(c)[0] == orc.ctx[c].n_kv
    used = 16 - eng.stats().pages_free
    assert used == sum((orc.ctx[c].n_kv + 15) // 16 for c in (1, 2, 3))
    eng.release(2)
    p = I.make_prompt(shape.vocab, 40, 0, 4)                               # takes over the pages just returned
    eng.prefill(4, p)
    orc.release(2)
    orc.prefill(4, p)
    d, q = I.make_drafts(shape.vocab, 3, 0, 4)
    eng.set_sampling(1.0, True)
    _verify_both(eng, orc, [(4, d, q), (1,) + tuple(I.make_drafts(shape.vocab, 2, 0, 1, step=2))], seed=3, tau=1.0,
                 greedy=True, tol=1e-4, explain=explain)
    st = eng.stats()
    assert st.steps == 3 and st.requests == 8 and st.contexts_open == 3
    eng.shutdown()


def test_errors_leave_everything_unchanged():
    shape = I.TINY
    w = I.make_weights(shape, seed=0)
    eng = _engine(shape, w, n_pages=8, max_batch=2, max_k=4, max_step_tokens=10)
    eng.prefill(1, I.make_prompt(shape.vocab, 30, 0, 1))
    eng.prefill(2, I.make_prompt(shape.vocab, 30, 0, 2))
    before = (eng.query_ctx(1), eng.query_ctx(2), eng.stats().pages_free)
    d, q = I.make_drafts(shape.vocab, 4, 0, 1)

    def code(reqs):
        with pytest.raises(B.SledError) as ei:
            eng.verify_batch(reqs, 0)
        return ei.value.code

    assert code([(9, d.numpy(), q.numpy())]) == B.SLED_ERR_UNKNOWN_CTX
    assert code([(1, d.numpy(), q.numpy()), (1, d.numpy(), q.numpy())]) == B.SLED_ERR_DUP_CTX
    assert code([(1, np.arange(5), np.zeros((5, shape.vocab), np.float32))]) == B.SLED_ERR_K_RANGE
    assert code([(1, np.array([shape.vocab]), q.numpy()[:1])]) == B.SLED_ERR_TOKEN_RANGE
    assert code([(1, d.numpy(), None)]) == B.SLED_ERR_ARG
    assert code([(1, d.numpy(), q.numpy())] * 3) == B.SLED_ERR_BATCH_TOO_LARGE
    with pytest.raises(B.SledError) as ei:
        eng.prefill(3, I.make_prompt(shape.vocab, 16 * 8, 0, 3))
    assert ei.value.code == B.SLED_ERR_NO_PAGES
    with pytest.raises(B.SledError) as ei:
        eng.prefill(1, [1, 2])
    assert ei.value.code == B.SLED_ERR_DUP_CTX
    after = (eng.query_ctx(1), eng.query_ctx(2), eng.stats().pages_free)
    assert str(before) == str(after)
    eng.release(1)
    with pytest.raises(B.SledError):
        eng.verify_batch([(1, d.numpy(), q.numpy())], 0)
    eng.shutdown()


@pytest.mark.parametrize("T_want", [163, 190, 225, 262, 300, 389, 520, 1030])
def test_wide_steps_on_cta_pairs(T_want):
    # more than 160 tokens: every linear layer of this shape (even numbers of weight tiles) runs on the persistent
    # CTA pairs; the step sizes give one to five token tiles with ragged last tiles of different widths, K-slice
    # counts that change with the step size, and fewer units than pairs (most pairs leave without work)
    shape = I.SMALL_GQA
    w = I.make_weights(shape, seed=12)
    n_req = (T_want + 8) // 9
    eng = _engine(shape, w, n_pages=4 * n_req + 8, max_batch=n_req, max_k=8, max_step_tokens=T_want + 8)
    orc = O.OracleModel(shape, oracle_weights(w))
    checked = {0, n_req // 2, n_req - 1}
    n_kv = {}
    for c in range(n_req):
        p = I.make_prompt(shape.vocab, 3 + (7 * c) % 29, 12, c)
        eng.prefill(c, p)
        n_kv[c] = len(p) - 1                                               # the prompt's last token waits as "pending"
        if c in checked:
            orc.prefill(c, p)
    ks = [8] * n_req
    ks[-1] = T_want - 9 * (n_req - 1) - 1                                  # the last request fills the step to T_want exactly
    assert 0 <= ks[-1] <= 8
    reqs = [(c,) + tuple(I.make_drafts(shape.vocab, ks[c], 12, c)) for c in range(n_req)]
    T = sum(len(d) + 1 for _, d, _ in reqs)
    assert T == T_want
    eng.set_commit(False)
    got = eng.verify_batch([(c, d.numpy(), q.numpy()) for c, d, q in reqs], 4)
    glog = eng.logits(T)
    row = 0
    for (c, d, q), g in zip(reqs, got):
        k = len(d)
        if c in checked:
            st, n_acc, nxt, ol, mg = orc.verify(c, d.numpy(), q.numpy(), 4, commit=False)
            assert np.max(np.abs(glog[row:row + k + 1] - ol)) <= 2e-2
        st2, n2, x2, _ = O.accept(glog[row:row + k + 1], q.numpy(), d.numpy(), 1.0, False, 4, c, n_kv[c])
        assert (n2, x2, 0) == g
        row += k + 1
    eng.shutdown()


def test_step_between_128_and_160_tokens():
    # 129..160 tokens: the widest single token tile of the linear layers (160 columns, partly filled)
    shape = I.SMALL_GQA
    w = I.make_weights(shape, seed=8)
    eng = _engine(shape, w, n_pages=300, max_batch=20, max_k=8, max_step_tokens=160)
    orc = O.OracleModel(shape, oracle_weights(w))
    ctxs = list(range(20))
    for c in ctxs:
        p = I.make_prompt(shape.vocab, 4 + (11 * c) % 37, 8, c)
        eng.prefill(c, p)
        if c % 6 == 0:
            orc.prefill(c, p)
    reqs = [(c,) + tuple(I.make_drafts(shape.vocab, 6 if c % 2 else 7, 8, c)) for c in ctxs]
    T = sum(len(d) + 1 for _, d, _ in reqs)
    assert 128 < T <= 160
    eng.set_commit(False)
    got = eng.verify_batch([(c, d.numpy(), q.numpy()) for c, d, q in reqs], 3)
    glog = eng.logits(T)
    row = 0
    for (c, d, q), g in zip(reqs, got):
        k = len(d)
        if c in orc.ctx:
            st, n_acc, nxt, ol, mg = orc.verify(c, d.numpy(), q.numpy(), 3, commit=False)
            assert np.max(np.abs(glog[row:row + k + 1] - ol)) <= 2e-2
            st2, n2, x2, _ = O.accept(glog[row:row + k + 1], q.numpy(), d.numpy(), 1.0, False, 3, c, orc.ctx[c].n_kv)
            assert (n2, x2, 0) == g
        row += k + 1
    eng.shutdown()


def test_resent_request_goes_back_to_base_len():
    # a device's answer is lost; it sends its drafts again, extended, naming the length it still believes in
    shape = I.SMALL_GQA
    w = I.make_weights(shape, seed=9)
    eng = _engine(shape, w)
    orc = O.OracleModel(shape, oracle_weights(w))
    lens = {31: 23, 32: 40, 33: 17}
    for c, n in lens.items():
        p = I.make_prompt(shape.vocab, n, 9, c)
        eng.prefill(c, p)
        orc.prefill(c, p)
    reqs = [(c,) + tuple(I.make_drafts(shape.vocab, 4, 9, c)) for c in lens]
    explain = []
    _verify_both(eng, orc, reqs, seed=1, tau=1.0, greedy=False, tol=2e-2, explain=explain)
    grown = {c: eng.query_ctx(c)[0] for c in lens}
    assert all(grown[c] >= lens[c] for c in lens)
    # context 31 resends from its old length with more drafts, 32 continues normally, 33 names its current length (no-op)
    d31, q31 = I.make_drafts(shape.vocab, 7, 9, 31, step=1)
    d32, q32 = I.make_drafts(shape.vocab, 3, 9, 32, step=1)
    d33, q33 = I.make_drafts(shape.vocab, 2, 9, 33, step=1)
    base = {31: lens[31], 32: 0, 33: grown[33] + 1}
    batch = [(31, d31, q31), (32, d32, q32), (33, d33, q33)]
    got = eng.verify_batch([(c, d.numpy(), q.numpy(), base[c]) for c, d, q in batch], 2)
    glog = eng.logits(sum(len(d) + 1 for _, d, _ in batch))
    row = 0
    for (c, d, q), g in zip(batch, got):
        k = len(d)
        if base[c]:
            orc.rebase(c, base[c])
        pos0 = orc.ctx[c].n_kv
        if c == 31:
            assert pos0 == lens[31] - 1
        st, n_acc, nxt, ol, mg = orc.verify(c, d.numpy(), q.numpy(), 2, commit=False)
        mine = glog[row:row + k + 1]
        row += k + 1
        assert np.max(np.abs(mine - ol)) <= 2e-2
        st2, n2, x2, _ = O.accept(mine, q.numpy(), d.numpy(), 1.0, False, 2, c, pos0)
        assert (n2, x2, 0) == g
        assert eng.query_ctx(c)[:2] == (pos0 + g[0] + 1, g[1])
    # out-of-range base_len: refused, nothing changes (context 32 in the same batch included)
    before = [str(eng.query_ctx(c)) for c in lens]
    for bad in (eng.query_ctx(31)[0] + 2, 10**6):
        with pytest.raises(B.SledError) as ei:
            eng.verify_batch([(32, d32.numpy(), q32.numpy(), 0), (31, d31.numpy(), q31.numpy(), bad)], 3)
        assert ei.value.code == B.SLED_ERR_BASE_LEN
    assert before == [str(eng.query_ctx(c)) for c in lens]
    # a context opened from cache content alone cannot go back before the point where its tokens are known
    K, V = I.make_kv(shape, 20, 9, 40)
    eng.load_kv(40, (K * 0.3).contiguous(), (V * 0.3).contiguous(), pending=5)
    with pytest.raises(B.SledError) as ei:
        eng.verify_batch([(40, d33.numpy(), q33.numpy(), 20)], 3)
    assert ei.value.code == B.SLED_ERR_BASE_LEN
    assert eng.verify_batch([(40, d33.numpy(), q33.numpy(), 21)], 3)[0][2] == 0
    eng.shutdown()


@pytest.mark.parametrize("where", ["host", "device"])
def test_draft_rows_in_bf16(where):
    # rows sent in 16 bits (half the request bytes): the decision must be the oracle's rule applied to the GPU's
    # logits and to the rows as sent (a bf16 value widens to fp32 exactly)
    shape = I.SMALL_GQA
    w = I.make_weights(shape, seed=10)
    eng = _engine(shape, w, draft_probs_dtype="bf16")
    ctxs = [51, 52, 53, 54]
    for c in ctxs:
        eng.prefill(c, I.make_prompt(shape.vocab, 12 + c % 7, 10, c))
    eng.set_commit(False)
    reqs, rows = [], []
    for c, k in zip(ctxs, [5, 0, 8, 3]):
        d, q = I.make_drafts(shape.vocab, k, 10, c)
        q16 = q.to(torch.bfloat16).contiguous()
        rows.append(q16.float().numpy())
        reqs.append((c, d.numpy(), q16.cuda() if where == "device" else q16))
    got = eng.verify_batch(reqs, 4)
    glog = eng.logits(sum(len(r[1]) + 1 for r in reqs))
    row = 0
    for (c, d, _), qf, g in zip(reqs, rows, got):
        k = len(d)
        st2, n2, x2, _ = O.accept(glog[row:row + k + 1], qf if k else None, d, 1.0, False, 4, c, eng.query_ctx(c)[0])
        assert (n2, x2, 0) == g
        row += k + 1
    assert any(g[0] < len(r[1]) for r, g in zip(reqs, got))      # a rejection happened: the residual read a 16-bit row
    eng.shutdown()


def test_a_wait_that_runs_out_fails_the_step_and_nothing_else():
    # every device-side wait is bounded; this arms the give-up path on purpose (a kernel waits 2 ms on a barrier
    # nobody signals and returns with its error code): the step must come back as a device error with every
    # context untouched, and the next step on the same engine must be an ordinary, correct one
    shape = I.SMALL_GQA
    w = I.make_weights(shape, seed=12)
    eng = _engine(shape, w)
    orc = O.OracleModel(shape, oracle_weights(w))
    ctxs = [71, 72, 73]
    for c in ctxs:
        p = I.make_prompt(shape.vocab, 15 + c % 5, 12, c)
        eng.prefill(c, p)
        orc.prefill(c, p)
    reqs = [(c,) + tuple(I.make_drafts(shape.vocab, 5, 12, c)) for c in ctxs]
    explain = []
    _verify_both(eng, orc, reqs, seed=1, tau=1.0, greedy=False, tol=2e-2, explain=explain)
    before = [str(eng.query_ctx(c)) for c in ctxs] + [eng.stats().pages_free, eng.stats().steps]
    reqs = [(c,) + tuple(I.make_drafts(shape.vocab, 4, 12, c, step=1)) for c in ctxs]
    eng.arm_wait_timeout(2000)
    with pytest.raises(B.SledError) as ei:
        eng.verify_batch([(c, d.numpy(), q.numpy()) for c, d, q in reqs], 2)
    assert ei.value.code == B.SLED_ERR_DEVICE
    assert before == [str(eng.query_ctx(c)) for c in ctxs] + [eng.stats().pages_free, eng.stats().steps]
    _verify_both(eng, orc, reqs, seed=2, tau=1.0, greedy=False, tol=2e-2, explain=explain)   # the same requests, now served
    eng.shutdown()
    # the fp32 configuration has no such waits: arming is refused
    eng32 = _engine(I.TINY, I.make_weights(I.TINY, seed=0))
    with pytest.raises(B.SledError):
        eng32.arm_wait_timeout(1000)
    eng32.shutdown()
