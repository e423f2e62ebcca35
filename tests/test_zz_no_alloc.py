"""The allocation-free acceptance entry point against the ordinary one.

sled_accept_rows_static exists for callers that cannot call cudaMalloc (their GPU memory belongs to
another allocator, or an allocation would stall their latency path).  It keeps its device-side batch
description in a fixed array of the library, which every call reuses: so the check runs two calls in a
row, the second smaller than the first, and each must equal what sled_accept_rows returns (the
decisions are integers: equality is exact)."""
import numpy as np
import pytest
import torch

from paper_2506_09397_b200 import binding as B
from paper_2506_09397_b200 import inputs as I

pytestmark = pytest.mark.gpu


def _pack(z, q, d, ks):
    rows, qrows, drafts, cu = [], [], [], [0]
    for i, k in enumerate(ks):
        rows.append(z[i, :k + 1])
        qrows.append(q[i, :k])
        drafts += [int(x) for x in d[i, :k]]
        cu.append(cu[-1] + k + 1)
    return torch.cat(rows).contiguous().cuda(), torch.cat(qrows).contiguous().cuda(), drafts, cu


def test_two_calls_in_a_row_match_the_allocating_entry_point():
    n, k, V = 40, 6, 33000
    z, q, d = I.make_accept_rows(n, k, V, tau_draft=1.0, seed=21, sigma=2.0)
    rng = np.random.default_rng(4)
    first = [int(x) for x in rng.integers(0, k + 1, n)]
    second = [int(x) for x in rng.integers(0, k + 1, 9)]          # fewer requests: stale entries must not matter
    for call, ks in enumerate((first, second)):
        logits, qcat, drafts, cu = _pack(z[:len(ks)], q[:len(ks)], d[:len(ks)], ks)
        ctx = [500 + 3 * i for i in range(len(ks))]
        pos0 = [40 + i for i in range(len(ks))]
        for greedy, tau in ((False, 0.9), (True, 1.0)):
            want, _ = B.accept_rows(logits, cu, drafts, None if greedy else qcat, ctx, pos0, tau, greedy, seed=call + 1)
            got = B.accept_rows_static(logits, cu, drafts, None if greedy else qcat, ctx, pos0, tau, greedy, seed=call + 1)
            assert got == want
            assert all(s == 0 for _, _, s in got)
    assert len({g[0] for g in got}) >= 1


def test_sizes_beyond_the_fixed_maximum_are_refused():
    V = 8
    logits = torch.zeros(4, V, device="cuda")
    n = 1025                                                      # one more request than the array holds
    cu = np.arange(n + 1, dtype=np.int32)
    with pytest.raises(B.SledError) as ei:
        B.accept_rows_static(logits, cu, [], None, np.zeros(n, np.uint64), np.zeros(n, np.int64), 1.0, True, 0)
    assert ei.value.code == B.SLED_ERR_BATCH_TOO_LARGE
    cu = np.array([0, 8193], dtype=np.int32)                      # one request with too many rows
    with pytest.raises(B.SledError) as ei:
        B.accept_rows_static(logits, cu, np.zeros(8192, np.int32), None, np.zeros(1, np.uint64), np.zeros(1, np.int64),
                             1.0, True, 0)
    assert ei.value.code == B.SLED_ERR_BATCH_TOO_LARGE


def test_bad_descriptions_are_refused_before_anything_is_read():
    V = 8
    logits = torch.zeros(4, V, device="cuda")
    ids, p0 = np.zeros(1, np.uint64), np.zeros(1, np.int64)
    for fn in (lambda *a: B.accept_rows_static(*a), lambda *a: B.accept_rows(*a)[0]):
        with pytest.raises(B.SledError) as ei:       # drafts are read in greedy mode too: a missing array is an error
            fn(logits, np.array([0, 3], np.int32), [], None, ids, p0, 1.0, True, 0)
        assert ei.value.code == B.SLED_ERR_ARG
        with pytest.raises(B.SledError) as ei:       # the first row offset must be 0
            fn(logits, np.array([1, 3], np.int32), [0], None, ids, p0, 1.0, True, 0)
        assert ei.value.code == B.SLED_ERR_ARG
        with pytest.raises(B.SledError) as ei:       # a request without rows
            fn(logits, np.array([0, 0], np.int32), [], None, ids, p0, 1.0, True, 0)
        assert ei.value.code == B.SLED_ERR_ARG
