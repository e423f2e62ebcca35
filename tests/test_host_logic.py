"""Host-side logic of the CUDA library that needs no device: exported symbols, the page manager's
invariants under random verify / release sequences, ragged packing, and error returns."""
import ctypes as C
import os
import re

import numpy as np
import pytest

from paper_2506_09397_b200 import binding as B
from paper_2506_09397_b200 import build as builder

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def built():
    builder.build()


def test_library_exports_every_declared_symbol():
    header = open(os.path.join(ROOT, "include", "sled.h")).read()
    declared = set(re.findall(r"^(?:int|void|void\*|const char\*|int32_t|sled_kvm\*|sled_planner\*)\s+(sled_[a-z_0-9]+)\(", header, re.M))
    assert len(declared) > 20
    assert declared == set(B.EXPORTS)
    raw = C.CDLL(B.LIB_PATH)
    for name in declared:
        assert hasattr(raw, name), name


def test_strerror_and_null_arguments():
    L = B.lib()
    assert B.strerror(0) == "ok"
    assert "fallback" in B.strerror(B.SLED_ERR_NO_DEVICE)
    assert L.sled_init(None, None, None) == B.SLED_ERR_ARG
    assert L.sled_verify_batch(None, None, 0, 0, None) == B.SLED_ERR_ARG
    assert L.sled_release(None, 0) == B.SLED_ERR_ARG


def test_init_without_a_device_fails_loudly():
    import torch
    if torch.cuda.is_available():
        pytest.skip("a device is present")
    from paper_2506_09397_b200 import inputs as I
    w = I.make_weights(I.TINY, 0)
    with pytest.raises(B.SledError) as ei:
        B.Engine(I.TINY, w, n_pages=64, max_batch=4, max_k=4, max_step_tokens=32)
    assert ei.value.code == B.SLED_ERR_NO_DEVICE


def _check_invariants(m, live, n_pages, ps):
    owned = []
    for ctx, (n_kv, pending) in live.items():
        rc, q = m.query(ctx)
        assert rc == 0
        assert q[0] == n_kv and q[1] == pending
        assert len(q[2]) == (n_kv + ps - 1) // ps          # exactly the pages its tokens need
        owned += list(q[2])
    assert len(owned) == len(set(owned))                     # no page owned twice
    assert all(0 <= p < n_pages for p in owned)
    assert len(owned) + m.free_pages() == n_pages            # free + owned = pool


def test_page_manager_random_walk():
    rng = np.random.default_rng(0)
    n_pages, ps = 40, 16
    m = B.KvManager(n_pages, ps)
    live = {}
    nxt = 1
    for step in range(3000):
        op = rng.integers(0, 10)
        if op < 2 and len(live) < 8:
            n_kv = int(rng.integers(0, 70))
            rc = m.open(nxt, n_kv, 7)
            need = (n_kv + ps - 1) // ps
            if rc == 0:
                live[nxt] = (n_kv, 7)
            else:
                assert rc == B.SLED_ERR_NO_PAGES and need > m.free_pages()
            nxt += 1
        elif op < 8 and live:
            ids = list(rng.choice(list(live), size=min(len(live), int(rng.integers(1, 5))), replace=False))
            ks = [int(rng.integers(0, 9)) for _ in ids]
            free_before = m.free_pages()
            rc = m.reserve_batch(ids, [k + 1 for k in ks])
            if rc != 0:
                assert rc == B.SLED_ERR_NO_PAGES and m.free_pages() == free_before
                _check_invariants(m, live, n_pages, ps)       # a failed reservation changed nothing
                continue
            rc, cu, (tok, req, pos, slot) = m.pack(ids, ks, [np.arange(k) + 100 for k in ks])
            assert rc == 0 and cu[-1] == sum(k + 1 for k in ks)
            for i, ctx in enumerate(ids):
                n_kv, pending = live[ctx]
                rows = slice(cu[i], cu[i + 1])
                assert tok[rows][0] == pending and list(tok[rows][1:]) == list(np.arange(ks[i]) + 100)
                assert list(pos[rows]) == list(range(n_kv, n_kv + ks[i] + 1))
                assert all(req[rows] == i)
                pages = m.query(ctx)[1][2]
                assert list(slot[rows]) == [pages[p // ps] * ps + p % ps for p in range(n_kv, n_kv + ks[i] + 1)]
            for ctx, k in zip(ids, ks):
                n_acc = int(rng.integers(0, k + 1))
                assert m.commit(ctx, n_acc + 1, 50 + n_acc) == 0
                live[ctx] = (live[ctx][0] + n_acc + 1, 50 + n_acc)
        elif live:
            ctx = int(rng.choice(list(live)))
            assert m.release(ctx) == 0
            del live[ctx]
        _check_invariants(m, live, n_pages, ps)
    for ctx in list(live):
        m.release(ctx)
    assert m.free_pages() == n_pages


def test_page_manager_errors():
    m = B.KvManager(4, 16)
    assert m.open(1, 10, 0) == 0
    assert m.open(1, 10, 0) == B.SLED_ERR_DUP_CTX
    assert m.reserve_batch([1, 1], [1, 1]) == B.SLED_ERR_DUP_CTX
    assert m.reserve_batch([2], [1]) == B.SLED_ERR_UNKNOWN_CTX
    assert m.reserve_batch([1], [16 * 4]) == B.SLED_ERR_NO_PAGES
    assert m.commit(1, 1, 0) == B.SLED_ERR_ARG            # nothing reserved
    assert m.release(9) == B.SLED_ERR_UNKNOWN_CTX
    assert m.reserve_batch([1], [7]) == 0
    assert m.commit(1, 8, 0) == B.SLED_ERR_ARG            # more than reserved
    assert m.commit(1, 6, 3) == 0
    assert m.query(1)[1][:2] == (16, 3)
    assert m.free_pages() == 3                              # 16 tokens fit one page: the second went back


def test_page_manager_goes_back_to_a_base_length():
    # Random walk with requests that continue an earlier length of their context (a resent draft): the manager is
    # compared, after every operation, with plain Python lists holding each context's token history.
    rng = np.random.default_rng(7)
    n_pages, ps = 48, 16
    m = B.KvManager(n_pages, ps)
    hist = {}                                               # ctx -> (hist_start, [tokens from there on]); last = pending
    nxt = 1
    n_back = 0
    for step in range(3000):
        op = rng.integers(0, 10)
        if op < 2 and len(hist) < 6:
            n_kv = int(rng.integers(0, 60))
            if m.open(nxt, n_kv, 7) == 0:
                hist[nxt] = (n_kv, [7])
            nxt += 1
        elif op < 9 and hist:
            ids = [int(x) for x in rng.choice(list(hist), size=min(len(hist), int(rng.integers(1, 4))), replace=False)]
            ks = [int(rng.integers(0, 9)) for _ in ids]
            base = []
            for ctx in ids:
                start, toks = hist[ctx]
                n = start + len(toks)                       # committed tokens
                r = rng.integers(0, 4)
                base.append(0 if r == 0 else int(rng.integers(start + 1, n + 1)) if r < 3 else
                            int(rng.choice([start, n + 1])))   # the last two are out of range
            free_before = m.free_pages()
            before = {ctx: m.query(ctx)[1] for ctx in ids}
            rc = m.reserve_batch(ids, [k + 1 for k in ks], base)
            bad = any(b != 0 and not (hist[c][0] + 1 <= b <= hist[c][0] + len(hist[c][1])) for c, b in zip(ids, base))
            if bad:
                assert rc == B.SLED_ERR_BASE_LEN
            if rc != 0:
                assert rc in (B.SLED_ERR_BASE_LEN, B.SLED_ERR_NO_PAGES) and m.free_pages() == free_before
                for ctx in ids:                             # a refused batch changed nothing
                    q = m.query(ctx)[1]
                    assert q[:2] == before[ctx][:2] and list(q[2]) == list(before[ctx][2])
                    assert m.history(ctx)[1] == (hist[ctx][0], hist[ctx][1])
                continue
            for ctx, b in zip(ids, base):
                if b:
                    start, toks = hist[ctx]
                    n_back += b < start + len(toks)
                    hist[ctx] = (start, toks[:b - start])
            for ctx, k in zip(ids, ks):
                start, toks = hist[ctx]
                n_kv, pending = start + len(toks) - 1, toks[-1]
                q = m.query(ctx)[1]
                assert q[:2] == (n_kv, pending) and len(q[2]) == (n_kv + k + 1 + ps - 1) // ps
                drafts = [int(x) for x in rng.integers(100, 200, k)]
                n_acc = int(rng.integers(0, k + 1))
                new = int(rng.integers(200, 300))
                assert m.commit(ctx, n_acc + 1, new, drafts) == 0
                hist[ctx] = (start, toks + drafts[:n_acc] + [new])
        elif hist:
            ctx = int(rng.choice(list(hist)))
            assert m.release(ctx) == 0
            del hist[ctx]
        live = {c: (s + len(t) - 1, t[-1]) for c, (s, t) in hist.items()}
        _check_invariants(m, live, n_pages, ps)
        for c, (s, t) in hist.items():
            assert m.history(c)[1] == (s, t)
    assert n_back > 100                                      # the walk did go back many times
    # a commit that does not say which tokens were kept restarts the known history at the new pending token
    m2 = B.KvManager(8, 16)
    assert m2.open(1, 3, 9) == 0 and m2.reserve_batch([1], [4]) == 0
    assert m2.commit(1, 3, 5) == 0
    assert m2.history(1)[1] == (6, [5])
    assert m2.reserve_batch([1], [1], [6]) == B.SLED_ERR_BASE_LEN and m2.reserve_batch([1], [1], [7]) == 0


def test_e4m3_storage_format_round_trip():
    # what inputs.to_e4m3_rows stores is within half a step of the row-scaled value, the largest entry of a row lands
    # on the largest e4m3 number, and the NaN patterns never occur
    import torch
    from paper_2506_09397_b200 import inputs as I
    w = torch.randn(64, 256, generator=torch.Generator().manual_seed(1)) * 0.02
    b, sc = I.to_e4m3_rows(w)
    back = I.from_e4m3_rows(b, sc)
    assert b.dtype == torch.uint8 and not bool(((b & 0x7f) == 0x7f).any())
    assert torch.all((back - w).abs() <= w.abs() * 2.0 ** -4 + sc[:, None] * 2.0 ** -10)
    assert torch.allclose(back.abs().amax(dim=1), w.abs().amax(dim=1))
    table = I.from_e4m3_rows(torch.arange(256, dtype=torch.uint8)[:, None], torch.ones(256))[:, 0]
    assert float(table[0x01]) == 2.0 ** -9 and float(table[0x08]) == 2.0 ** -6 and float(table[0x38]) == 1.0
    assert float(table[0x7e]) == 448.0 and float(table[0xb8]) == -1.0


def test_e2m1_storage_format_round_trip():
    # what inputs.to_e2m1_rows stores: the nearest of the sixteen e2m1 values to the row-scaled entry (neighbouring
    # values are at most 2 apart, so within 1 of it), the row's largest entry on +-6, the even column in the low half
    # of a byte; the code table is the 4-bit float's definition (exponent bias 1, one mantissa bit, subnormal 0.5)
    import torch
    from paper_2506_09397_b200 import inputs as I
    w = torch.randn(64, 256, generator=torch.Generator().manual_seed(2)) * 0.02
    b, sc = I.to_e2m1_rows(w)
    back = I.from_e2m1_rows(b, sc)
    assert b.dtype == torch.uint8 and tuple(b.shape) == (64, 128)
    assert torch.all((back - w).abs() <= sc[:, None] * 1.0 + 1e-9)
    assert torch.allclose(back.abs().amax(dim=1), w.abs().amax(dim=1))
    small = (w.abs() <= sc[:, None] * 2.0)                      # up to 2 the values are half a unit apart
    assert torch.all((back - w).abs()[small] <= (sc[:, None] * 0.25 + 1e-9).expand_as(w)[small])
    table = I.from_e2m1_rows(torch.arange(16, dtype=torch.uint8)[:, None], torch.ones(16))
    for code in range(16):
        e, m, sign = (code >> 1) & 3, code & 1, -1.0 if code & 8 else 1.0
        want = sign * (0.5 * m if e == 0 else (1 + 0.5 * m) * 2.0 ** (e - 1))
        assert float(table[code, 0]) == want and float(table[code, 1]) == 0.0     # high half empty
    one = I.from_e2m1_rows(torch.tensor([[0x2f]], dtype=torch.uint8), torch.ones(1))
    assert one.tolist() == [[-6.0, 1.0]]                       # low half first
