"""The server's request queue and batch planner (Section 3.4): the library's planner against the plain-list
restatement of its rules, and both against the properties the rules imply."""
import numpy as np
import pytest

from oracle import planner as PM
from paper_2506_09397_b200 import binding as B


def _trace(rng, n_events, n_ctx, max_k):
    """Random interleaving of arrivals and planner calls: ('push', ticket, ctx, k) / ('batch', flush)."""
    ticket = 0
    for _ in range(n_events):
        if rng.random() < 0.7:
            ticket += 1
            yield ("push", ticket, int(rng.integers(0, n_ctx)), int(rng.integers(0, max_k + 1)))
        else:
            yield ("batch", bool(rng.random() < 0.15))


@pytest.mark.parametrize("policy,batch_size,max_batch,max_tokens,n_ctx", [
    (PM.STATIC, 4, 8, 72, 30), (PM.STATIC, 8, 8, 40, 50), (PM.STATIC, 1, 4, 9, 3),
    (PM.CONTINUOUS, 0, 6, 30, 12), (PM.CONTINUOUS, 0, 16, 1000, 5), (PM.CONTINUOUS, 0, 3, 9, 40)])
def test_library_planner_equals_the_restated_rules(policy, batch_size, max_batch, max_tokens, n_ctx):
    rng = np.random.default_rng(policy * 100 + max_batch)
    lib, ref = B.Planner(policy, batch_size, max_batch, max_tokens), PM.PlannerModel(policy, batch_size, max_batch, max_tokens)
    info, order, emitted = {}, [], []
    events = list(_trace(rng, 4000, n_ctx, 8))
    i = 0
    while i < len(events) or lib.queued():
        ev = events[i] if i < len(events) else ("batch", True)          # after the trace: flush until the queue is empty
        i += 1
        if ev[0] == "push":
            _, t, ctx, k = ev
            assert (lib.push(t, ctx, k) == 0) == ref.push(t, ctx, k)
            info[t] = (ctx, k)
            order.append(t)
            continue
        got, want = lib.next_batch(ev[1]), ref.next_batch(ev[1])
        assert got == want
        assert lib.queued() == len(ref.queue)
        if not got:
            continue
        emitted += got
        # what the rules imply, checked on the outcome itself
        ctxs = [info[t][0] for t in got]
        assert len(set(ctxs)) == len(ctxs)                                   # one request per context and step
        assert sum(info[t][1] + 1 for t in got) <= max_tokens                # the step's token capacity
        assert len(got) <= (batch_size if policy == PM.STATIC else max_batch)
        assert got == sorted(got)                                            # arrival order inside a batch
        if policy == PM.STATIC and not ev[1] and len(got) < batch_size:      # a short static batch: only when the step is full
            left = [t for t in order if t not in set(emitted)]
            nxt = next((t for t in left if info[t][0] not in set(ctxs)), None)
            assert nxt is not None and sum(info[t][1] + 1 for t in got) + info[nxt][1] + 1 > max_tokens
    assert sorted(emitted) == order and lib.queued() == 0                    # every request exactly once
    # requests of one context leave in the order they came
    last = {}
    for t in emitted:
        ctx = info[t][0]
        assert last.get(ctx, 0) < t
        last[ctx] = t


def test_static_batching_waits_for_its_batch():
    p = B.Planner(B.SLED_BATCH_STATIC, 3, 8, 100)
    assert p.push(1, 10, 2) == 0 and p.push(2, 11, 2) == 0
    assert p.next_batch() == []                      # two of three: wait (the paper's fixed batch size)
    assert p.push(3, 10, 4) == 0                     # same device again: does not count towards the three
    assert p.next_batch() == []
    assert p.push(4, 12, 0) == 0
    assert p.next_batch() == [1, 2, 4]
    assert p.next_batch() == [] and p.next_batch(flush=True) == [3]
    assert p.queued() == 0


def test_continuous_batching_takes_what_is_there():
    p = B.Planner(B.SLED_BATCH_CONTINUOUS, 0, 4, 20)
    assert p.next_batch() == []
    for t, (ctx, k) in enumerate([(1, 8), (2, 8), (3, 8), (4, 0)], start=1):
        assert p.push(t, ctx, k) == 0
    assert p.next_batch() == [1, 2]                  # the third would not fit 20 tokens, and nothing overtakes it
    assert p.next_batch() == [3, 4]
    assert p.push(9, 1, 30) == B.SLED_ERR_K_RANGE    # could never be scheduled
    assert p.push(10, 1, 3) == 0
    assert p.next_batch(cap=0) == B.SLED_ERR_ARG and p.queued() == 1


def test_planner_refuses_bad_configurations():
    for args in ((7, 1, 4, 10), (B.SLED_BATCH_STATIC, 0, 4, 10), (B.SLED_BATCH_STATIC, 5, 4, 10),
                 (B.SLED_BATCH_CONTINUOUS, 0, 0, 10), (B.SLED_BATCH_CONTINUOUS, 0, 4, 0)):
        with pytest.raises(B.SledError):
            B.Planner(*args)


# ---- the cut of a step's requests into attention work items (host only) ----------------------------------------
def _bench_like(b, seed=0):
    from paper_2506_09397_b200 import inputs as I
    ks = I.draw_k(b, [3, 5, 8], seed)
    ctx = I.draw_context_lengths(b, 512, 4096, seed)
    return [c + k + 1 for c, k in zip(ctx, ks)], [k + 1 for k in ks]


@pytest.mark.parametrize("b", [1, 3, 16, 36, 64, 128])
def test_attention_plan_is_a_valid_cut(b):
    # every request in equal parts of whole 64-key tiles, at least two tiles a part when it is cut, the partial
    # results within the room that there is
    n_keys, q_tok = _bench_like(b, seed=b)
    for cap in (1 << 20, 400, 0):
        chunks = B.plan_attention(n_keys, q_tok, 8, 4, 296, cap)
        part_rows = 0
        for n, q, c in zip(n_keys, q_tok, chunks):
            parts = -(-n // c)
            assert c % 64 == 0 and c > 0
            assert (parts - 1) * c < n <= parts * c
            if parts > 1:
                assert c >= 128
                assert c - 64 < -(-n // parts) + 63           # equal parts: no part a whole tile longer than need be
                part_rows += parts * q
        assert part_rows <= cap
        if cap == 0:
            assert all(c >= n for n, c in zip(n_keys, chunks))


def test_attention_plan_follows_what_was_measured():
    # the configurations that were timed with forced chunk lengths (8B shape, contexts 512..4096, 296 resident blocks):
    # one wave of items for 16 requests; at 36 and 64 requests the long contexts are cut and the short ones are not;
    # at 128 requests nothing is cut
    n_keys, q_tok = _bench_like(16)
    chunks = B.plan_attention(n_keys, q_tok, 8, 4, 296, 1 << 20)
    assert sum(-(-n // c) for n, c in zip(n_keys, chunks)) * 8 <= 296
    for b in (36, 64):
        n_keys, q_tok = _bench_like(b)
        chunks = B.plan_attention(n_keys, q_tok, 8, 4, 296, 1 << 20)
        cut = [n for n, c in zip(n_keys, chunks) if c < n]
        whole = [n for n, c in zip(n_keys, chunks) if c >= n]
        assert cut and whole and sum(cut) / len(cut) > 1.3 * sum(whole) / len(whole)
        assert 296 < sum(-(-n // c) for n, c in zip(n_keys, chunks)) * 8 <= 4 * 296
    n_keys, q_tok = _bench_like(128)
    chunks = B.plan_attention(n_keys, q_tok, 8, 4, 296, 1 << 20)
    assert all(c >= n for n, c in zip(n_keys, chunks))


@pytest.mark.parametrize("b,seed", [(8, 1), (24, 2), (40, 3), (64, 4), (100, 5)])
def test_attention_plan_ends_no_later_than_its_candidates(b, seed):
    # by the planner's own model (restated with plain lists), the chosen cut ends no later than any cut of its
    # candidate family: every request in equal parts of about one cost, that cost doubling from 4 key tiles up to
    # "nobody is cut" (candidates of more than four items per resident block are not considered)
    n_keys, q_tok = _bench_like(b, seed)
    chosen = B.plan_attention(n_keys, q_tok, 8, 4, 296, 1 << 20)
    t_chosen = PM.attention_plan_end_time(n_keys, q_tok, chosen, 8, 4, 296)
    costs = []
    for n, q in zip(n_keys, q_tok):
        rows = q * 4
        costs.append(-(-n // 64) * ((rows + 63) // 64) * (1.93 if rows > 32 else 1.15 if rows > 16 else 1.0))
    per_item, seen = 4.0, 0
    while True:
        whole = per_item >= max(costs)
        alt = []
        for n, c in zip(n_keys, costs):
            tiles = -(-n // 64)
            parts = 1 if whole else max(1, min(int(np.ceil(c / per_item)), max(1, tiles // 2)))
            alt.append(-(-tiles // parts) * 64)
        n_items = sum(-(-n // c) for n, c in zip(n_keys, alt)) * 8
        if whole or n_items <= 4 * 296:
            seen += 1
            assert t_chosen <= PM.attention_plan_end_time(n_keys, q_tok, alt, 8, 4, 296) * (1 + 1e-9), per_item
        if whole:
            break
        per_item *= 2.0
    assert seen >= 2


def test_attention_plan_refuses_bad_arguments():
    with pytest.raises(B.SledError):
        B.plan_attention([100, 0], [2, 2], 8, 4, 296, 100)
    with pytest.raises(B.SledError):
        B.plan_attention([100], [2], 0, 4, 296, 100)
