"""Pins of the oracle's acceptance rule (Eq. 1 and the residual resampling of Section 3.1)
against closed forms, brute force and the losslessness invariant."""
import math

import numpy as np
import pytest
from scipy import stats

from oracle import oracle as O


# ------------------------------------------------------------ fixed-point exp --
def test_fixed_exp_special_values():
    assert O.fixed_exp(0.0) == 2**40
    assert O.fixed_exp(-30.5) == 0
    assert O.fixed_exp(float("nan")) == 0
    assert O.fixed_exp(-1e30) == 0
    assert O.fixed_exp(float("-inf")) == 0


def test_fixed_exp_accuracy_and_monotone():
    xs = np.linspace(-29.9, 0.0, 20001).astype(np.float32)
    prev = -1
    for x in xs:
        e = O.fixed_exp(float(x))
        exact = math.exp(float(x)) * 2**40
        # within 2 ulp of fp32 relative accuracy plus the truncation to an integer
        assert abs(e - exact) <= exact * 2.5e-7 + 1.0, (x, e, exact)
        assert e >= prev - max(1, int(prev * 2.5e-7))  # monotone up to the rounding noise
        prev = e


def test_fixed_softmax_sum_is_exact():
    rng = np.random.default_rng(0)
    z = (rng.standard_normal(5000) * 3).astype(np.float32)
    E, Z = O.fixed_softmax(z, 0.7)
    assert Z == sum(int(e) for e in E)
    inv_tau = np.float32(1.0) / np.float32(0.7)
    s = z * inv_tau
    p = np.exp((s - s.max()).astype(np.float64))
    p /= p.sum()
    assert np.max(np.abs(E.astype(np.float64) / Z - p)) < 1e-7
    assert int(E[np.argmax(s)]) == 2**40


# --------------------------------------------- brute-force restatement in exact integers --
def brute_decision(logits, q, drafts, tau, seed, ctx, pos0):
    """Eq. 1 + residual with Python integers / Fractions, using only the published pieces
    (the uniforms and the integer numerators E) as inputs."""
    k = len(drafts)
    for j in range(k + 1):
        E, Z = O.fixed_softmax(logits[j], tau)
        E = [int(e) for e in E]
        ua, us = O.uniforms(seed, ctx, pos0 + j + 1)
        qrow = None
        if j < k:
            qrow = q[j]
            d = int(drafts[j])
            # u < p/q  <=>  U * q_d * Z < E_d * 2^24 ; evaluated as the spec says, in doubles
            lhs = (float(ua) * float(qrow[d])) * float(Z)
            rhs = float(E[d]) * 16777216.0
            if lhs < rhs:
                continue
        R = E
        if qrow is not None:
            R = [max(E[v] - int(float(qrow[v]) * float(Z)), 0) for v in range(len(E))]
            if sum(R) == 0:
                R = E
        W = sum(R)
        tgt = (us * W) >> 32
        run = 0
        for v, r in enumerate(R):
            run += r
            if run > tgt:
                return j, v
    raise AssertionError


def test_against_integer_restatement():
    rng = np.random.default_rng(1)
    V = 97
    for trial in range(300):
        k = int(rng.integers(0, 5))
        logits = (rng.standard_normal((k + 1, V)) * 2).astype(np.float32)
        ql = rng.standard_normal((k, V)) + 0.7 * logits[:k]
        q = np.exp(ql - ql.max(axis=1, keepdims=True)) if k else np.zeros((0, V))
        q = (q / q.sum(axis=1, keepdims=True)).astype(np.float32) if k else q.astype(np.float32)
        drafts = np.array([rng.choice(V, p=q[j].astype(np.float64) / q[j].astype(np.float64).sum()) for j in range(k)],
                          dtype=np.int32)
        tau = float(rng.choice([0.7, 1.0, 1.3]))
        st, n_acc, nxt, _ = O.accept(logits, q if k else None, drafts, tau, False, trial, 1000 + trial, 5 * trial)
        assert st == 0
        assert (n_acc, nxt) == brute_decision(logits, q, drafts, tau, trial, 1000 + trial, 5 * trial)


def test_k0_is_ordinary_sampling():
    # with no drafts the step is inverse-CDF sampling of softmax(z / tau) with the sampling uniform
    rng = np.random.default_rng(2)
    V = 50
    for trial in range(200):
        z = (rng.standard_normal((1, V)) * 3).astype(np.float32)
        st, n_acc, nxt, _ = O.accept(z, None, np.zeros(0, np.int32), 0.9, False, 11, trial, 40)
        _, us = O.uniforms(11, trial, 41)
        s = (z[0] * (np.float32(1.0) / np.float32(0.9))).astype(np.float64)
        p = np.exp(s - s.max())
        cdf = np.cumsum(p / p.sum())
        direct = int(np.searchsorted(cdf, us / 2**32, side="right"))
        assert st == 0 and n_acc == 0
        # the fixed-point CDF differs from the float one by < 1e-7: allow a neighbour only when that close
        if nxt != direct:
            u = us / 2**32
            assert min(abs(u - cdf[min(nxt, direct)]), abs(u - cdf[max(nxt, direct) - 1])) < 1e-6


# ----------------------------------------------------------------- closed forms --
def test_q_equals_p_always_accepts():
    rng = np.random.default_rng(3)
    V, k = 64, 4
    z = (rng.standard_normal((k + 1, V)) * 2).astype(np.float32)
    q = np.stack([(lambda E, Z: (E.astype(np.float64) / Z))(*O.fixed_softmax(z[j], 1.0)) for j in range(k)]).astype(np.float32)
    for seed in range(300):
        drafts = rng.integers(0, V, k).astype(np.int32)
        st, n_acc, nxt, _ = O.accept(z, q, drafts, 1.0, False, seed, 9, 100)
        assert (st, n_acc) == (0, k)


def test_disjoint_support_always_rejects_and_samples_p():
    V = 16
    z = np.full((2, V), -200.0, np.float32)
    z[:, :8] = np.linspace(-1, 1, 8)          # p lives on tokens 0..7
    q = np.zeros((1, V), np.float32)
    q[0, 8:] = 1 / 8                            # q lives on tokens 8..15
    p = np.exp(z[0, :8].astype(np.float64)); p /= p.sum()
    counts = np.zeros(8)
    n = 40000
    for i in range(n):
        st, n_acc, nxt, _ = O.accept(z, q, np.array([8 + i % 8], np.int32), 1.0, False, 3, i, 0)
        assert st == 0 and n_acc == 0 and nxt < 8
        counts[nxt] += 1
    chi2 = ((counts - n * p) ** 2 / (n * p)).sum()
    assert chi2 < stats.chi2.ppf(1 - 1e-3, 7)


def test_zero_draft_probability_of_the_draft_token():
    # q(d) = 0 with p(d) > 0: ratio is infinite, accept
    V = 8
    z = np.zeros((2, V), np.float32)
    q = np.zeros((1, V), np.float32); q[0, 1] = 1.0
    st, n_acc, _, _ = O.accept(z, q, np.array([0], np.int32), 1.0, False, 0, 0, 0)
    assert (st, n_acc) == (0, 1)


def test_greedy_rule_and_ties():
    V = 10
    z = np.zeros((3, V), np.float32)
    z[0, [4, 7]] = 5.0   # tie: lowest index wins
    z[1, 2] = 1.0
    z[2, 9] = 1.0
    assert O.accept(z, None, np.array([4, 2], np.int32), 1.0, True, 0, 0, 0)[1:3] == (2, 9)
    assert O.accept(z, None, np.array([7, 2], np.int32), 1.0, True, 0, 0, 0)[1:3] == (0, 4)
    assert O.accept(z, None, np.array([4, 3], np.int32), 1.0, True, 0, 0, 0)[1:3] == (1, 2)


def test_nonfinite_logit_is_reported():
    z = np.zeros((2, 8), np.float32)
    z[0, 3] = np.inf
    st, n_acc, nxt, _ = O.accept(z, np.full((1, 8), 0.125, np.float32), np.array([1], np.int32), 1.0, False, 0, 0, 0)
    assert (st, n_acc, nxt) == (1, 0, -1)
    z[0, 3] = np.nan
    assert O.accept(z, None, np.array([1], np.int32), 1.0, True, 0, 0, 0)[0] == 1


def test_rows_after_the_decision_are_not_looked_at():
    V = 8
    z = np.zeros((3, V), np.float32)
    z[0, 0] = 50.0               # p concentrated on token 0
    z[2, :] = np.nan             # never reached if draft 1 is rejected
    q = np.zeros((2, V), np.float32); q[:, 5] = 1.0
    st, n_acc, nxt, _ = O.accept(z, q, np.array([5, 5], np.int32), 1.0, False, 0, 0, 0)
    assert (st, n_acc, nxt) == (0, 0, 0)


# ------------------------------------------------ losslessness (Section 3.1's claim) --
def _softmax64(z):
    p = np.exp(z.astype(np.float64) - z.max())
    return p / p.sum()


@pytest.mark.parametrize("tau", [1.0, 0.7])
def test_first_committed_token_follows_target(tau):
    rng = np.random.default_rng(4)
    V, n = 32, 150000
    z = (rng.standard_normal((2, V)) * 1.5).astype(np.float32)
    p = _softmax64(z[0] * (np.float32(1) / np.float32(tau)))
    q64 = _softmax64((rng.standard_normal(V) * 1.5).astype(np.float32))
    q = q64.astype(np.float32)[None, :]
    draws = rng.choice(V, size=n, p=q64)        # the device's draft, from an independent generator
    counts = np.zeros(V)
    acc = 0
    for i in range(n):
        st, n_acc, nxt, _ = O.accept(z, q, np.array([draws[i]], np.int32), tau, False, 17, i, 3)
        counts[draws[i] if n_acc >= 1 else nxt] += 1
        acc += n_acc >= 1
    chi2 = ((counts - n * p) ** 2 / (n * p)).sum()
    assert chi2 < stats.chi2.ppf(1 - 1e-3, V - 1), chi2
    # acceptance probability has the closed form sum_v min(p_v, q_v)
    a = np.minimum(p, q64).sum()
    assert abs(acc / n - a) < 4.5 * math.sqrt(a * (1 - a) / n)


def test_second_committed_token_follows_target_given_first_accepted():
    rng = np.random.default_rng(5)
    V, n = 24, 150000
    z = (rng.standard_normal((3, V)) * 1.2).astype(np.float32)
    p2 = _softmax64(z[1])
    q64 = np.stack([_softmax64((rng.standard_normal(V) * 1.2).astype(np.float32)) for _ in range(2)])
    q = q64.astype(np.float32)
    d1 = rng.choice(V, size=n, p=q64[0])
    d2 = rng.choice(V, size=n, p=q64[1])
    counts = np.zeros(V)
    joint = np.zeros((2, V))   # second token split by parity of the first: independence check
    m = 0
    for i in range(n):
        st, n_acc, nxt, _ = O.accept(z, q, np.array([d1[i], d2[i]], np.int32), 1.0, False, 23, i, 9)
        if n_acc >= 1:
            tok = d2[i] if n_acc == 2 else nxt
            counts[tok] += 1
            joint[d1[i] % 2, tok] += 1
            m += 1
    assert m > n // 4
    chi2 = ((counts - m * p2) ** 2 / (m * p2)).sum()
    assert chi2 < stats.chi2.ppf(1 - 1e-3, V - 1), chi2
    for half in range(2):
        mh = joint[half].sum()
        c2 = ((joint[half] - mh * p2) ** 2 / (mh * p2)).sum()
        assert c2 < stats.chi2.ppf(1 - 1e-3, V - 1)


def test_chi_square_detects_a_planted_mistake():
    # the same test must FAIL for a wrong residual (resampling from p instead of norm(max(p-q,0))):
    # emulate that mistake on the CPU by handing the oracle q = 0 at the rejection only
    rng = np.random.default_rng(6)
    V, n = 32, 60000
    z = (rng.standard_normal((2, V)) * 1.5).astype(np.float32)
    p = _softmax64(z[0])
    q64 = _softmax64((rng.standard_normal(V) * 1.5).astype(np.float32))
    q = q64.astype(np.float32)[None, :]
    draws = rng.choice(V, size=n, p=q64)
    counts = np.zeros(V)
    for i in range(n):
        st, n_acc, nxt, _ = O.accept(z, q, np.array([draws[i]], np.int32), 1.0, False, 17, i, 3)
        if n_acc == 0:   # wrong rule: draw the corrective token from p itself
            nxt = O.accept(z[:1], None, np.zeros(0, np.int32), 1.0, False, 99, i, 3)[2]
        counts[draws[i] if n_acc >= 1 else nxt] += 1
    chi2 = ((counts - n * p) ** 2 / (n * p)).sum()
    assert chi2 > stats.chi2.ppf(1 - 1e-3, V - 1)


# ------------------------------------------------ draft rows sent in 16 bits: how far from lossless --
def _law_with_reported_q(p, q_true, q_sent):
    """Distribution of the first committed token when the device draws d ~ q_true but the server applies Eq. 1 and
    the residual with q_sent (all exact fp64): sum_d q_true(d) [a_d 1{x=d} + (1 - a_d) res(x)], a_d = min(1, p_d /
    q_sent_d), res = norm(max(p - q_sent, 0))."""
    a = np.minimum(1.0, p / q_sent)
    res = np.maximum(p - q_sent, 0.0)
    res = res / res.sum()
    return q_true * a + (q_true * (1.0 - a)).sum() * res


def test_bf16_draft_rows_deviate_by_their_rounding_and_no_more():
    import torch
    rng = np.random.default_rng(8)
    worst = 0.0
    for trial in range(200):
        V = int(rng.integers(8, 400))
        p = _softmax64((rng.standard_normal(V) * 2).astype(np.float32))
        q = _softmax64((0.8 * np.log(p) + 0.6 * rng.standard_normal(V) * 2).astype(np.float32))
        q16 = torch.from_numpy(q.astype(np.float32)).to(torch.bfloat16).to(torch.float64).numpy()
        exact = _law_with_reported_q(p, q, q)
        assert np.abs(exact - p).sum() < 1e-12                # with the true q the rule is lossless (Section 3.1)
        tv = 0.5 * np.abs(_law_with_reported_q(p, q, q16) - p).sum()
        assert 0.0 < tv <= 2.0 ** -8                          # rounded q: off by at most the relative rounding step
        worst = max(worst, tv)
    assert worst > 2.0 ** -14                                  # the bound is not vacuous: the deviation is real
    # the oracle applied to 16-bit rows follows that law, not p: the chi-square test against the predicted law passes
    V, n = 24, 120000
    z = (rng.standard_normal((2, V)) * 1.5).astype(np.float32)
    p = _softmax64(z[0])
    q64 = _softmax64((rng.standard_normal(V) * 1.5).astype(np.float32))
    q16 = torch.from_numpy(q64.astype(np.float32)).to(torch.bfloat16).to(torch.float32).numpy()
    law = _law_with_reported_q(p, q64, q16.astype(np.float64))
    draws = rng.choice(V, size=n, p=q64)
    counts = np.zeros(V)
    for i in range(n):
        st, n_acc, nxt, _ = O.accept(z, q16[None, :], np.array([draws[i]], np.int32), 1.0, False, 31, i, 3)
        counts[draws[i] if n_acc >= 1 else nxt] += 1
    chi2 = ((counts - n * law) ** 2 / (n * law)).sum()
    assert chi2 < stats.chi2.ppf(1 - 1e-3, V - 1), chi2
