"""The server loop (queue -> batch planner -> verification step, Section 3.4) against direct calls of the step:
the same batches, formed by the plain-list restatement of the planner's rules, must give the same results."""
import numpy as np
import pytest

from oracle import planner as PM
from paper_2506_09397_b200 import binding as B
from paper_2506_09397_b200 import inputs as I

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("policy,batch_size", [(B.SLED_BATCH_CONTINUOUS, 0), (B.SLED_BATCH_STATIC, 3)])
def test_queue_step_poll_equals_direct_verification(policy, batch_size):
    shape = I.SMALL_GQA
    w = I.make_weights(shape, seed=11)
    kw = dict(n_pages=256, max_batch=4, max_k=8, max_step_tokens=24)
    served, direct = B.Engine(shape, w, **kw), B.Engine(shape, w, **kw)
    served.server_config(policy, batch_size)
    model = PM.PlannerModel(policy, batch_size, kw["max_batch"], kw["max_step_tokens"])
    ctxs = list(range(60, 67))
    for c in ctxs:
        p = I.make_prompt(shape.vocab, 10 + c % 9, 11, c)
        served.prefill(c, p)
        direct.prefill(c, p)
    rng = np.random.default_rng(3)
    payload, results, expected = {}, {}, {}
    round_of = {c: 0 for c in ctxs}

    def step(flush):
        seed = 100 + len(expected)
        want_batch = model.next_batch(flush)
        n = served.step(seed, flush)
        assert n == len(want_batch)
        if want_batch:
            got = direct.verify_batch([payload[t] for t in want_batch], seed)
            for t, g in zip(want_batch, got):
                expected[t] = g

    for it in range(40):
        for _ in range(int(rng.integers(0, 4))):
            c = int(rng.choice(ctxs))
            d, q = I.make_drafts(shape.vocab, int(rng.integers(0, 9)), 11, c, step=round_of[c])
            round_of[c] += 1
            q = q.numpy()
            t = served.submit(c, d.numpy(), q)
            payload[t] = (c, d.numpy(), q)
            assert model.push(t, c, len(d))
            assert served.poll(t) is None                       # queued, not verified yet
        step(flush=False)
    while served.queued():
        step(flush=True)
    assert len(expected) == len(payload) > 20
    for t in payload:
        results[t] = served.poll(t)
    assert results == expected
    for c in ctxs:                                              # both engines went through the same history
        assert str(served.query_ctx(c)) == str(direct.query_ctx(c))
    with pytest.raises(B.SledError):
        served.poll(next(iter(payload)))                        # a polled ticket is forgotten
    served.shutdown()
    direct.shutdown()


def test_requests_of_a_released_context_get_their_own_error():
    shape = I.TINY
    w = I.make_weights(shape, seed=0)
    eng = B.Engine(shape, w, n_pages=64, max_batch=4, max_k=4, max_step_tokens=20)
    for c in (1, 2):
        eng.prefill(c, I.make_prompt(shape.vocab, 12, 0, c))
    d, q = I.make_drafts(shape.vocab, 3, 0, 1)
    t1 = eng.submit(1, d.numpy(), q.numpy())
    t2 = eng.submit(2, d.numpy(), q.numpy())
    t3 = eng.submit(2, d.numpy(), q.numpy(), base_len=40)        # beyond the context's end
    eng.release(1)
    assert eng.step(0) == 1                                      # context 2's first request runs
    assert eng.poll(t1) == (0, -1, B.SLED_ERR_UNKNOWN_CTX)
    assert eng.poll(t2)[2] == 0
    assert eng.poll(t3) is None and eng.step(1) == 0
    assert eng.poll(t3) == (0, -1, B.SLED_ERR_BASE_LEN)
    with pytest.raises(B.SledError) as ei:
        eng.submit(9, d.numpy(), q.numpy())
    assert ei.value.code == B.SLED_ERR_UNKNOWN_CTX
    eng.shutdown()
