"""Pins for block-query attention over the target's paged KV plus the block (Sec. 3.3.2)."""
import itertools
import math

import numpy as np
import pytest

from oracle import hspec_oracle as O


def _case(rng, k, Hq, Hkv, dh, ctx, page=16, extra_pages=2):
    n_pages = (ctx + page - 1) // page
    pool_pages = n_pages + extra_pages
    perm = rng.permutation(pool_pages)
    page_row = perm[:max(n_pages, 1)].astype(np.int32)
    k_pool = rng.standard_normal((pool_pages, page, Hkv, dh))
    v_pool = rng.standard_normal((pool_pages, page, Hkv, dh))
    q = rng.standard_normal((k, Hq, dh))
    kb, vb = rng.standard_normal((k, Hkv, dh)), rng.standard_normal((k, Hkv, dh))
    return q, k_pool, v_pool, page_row, kb, vb


def _enumerate(q, k_pool, v_pool, page_row, ctx, kb, vb, window):
    """Scalar-loop enumeration of the definition: no slicing, no shared helper."""
    k, Hq, dh = q.shape
    Hkv = kb.shape[1]
    page = k_pool.shape[1]
    out = np.zeros((k, Hq, dh))
    for i in range(k):
        for hq in range(Hq):
            h = hq // (Hq // Hkv)
            entries = []                                 # (score, value vector)
            for p in range(ctx):
                if window > 0 and not (0 <= (ctx + i) - p < window):
                    continue
                kk = k_pool[page_row[p // page], p % page, h]
                vv = v_pool[page_row[p // page], p % page, h]
                entries.append((sum(q[i, hq, d] * kk[d] for d in range(dh)) / math.sqrt(dh), vv))
            for j in range(i + 1):
                if window > 0 and not (0 <= i - j < window):
                    continue
                entries.append((sum(q[i, hq, d] * kb[j, h, d] for d in range(dh)) / math.sqrt(dh), vb[j, h]))
            z = sum(math.exp(s) for s, _ in entries)
            for s, vv in entries:
                out[i, hq] += math.exp(s) / z * vv
    return out


@pytest.mark.parametrize("ctx,window,Hkv", list(itertools.product([0, 1, 15, 16, 17, 40], [0, 1, 7, 64], [1, 2, 4])))
def test_matches_enumeration(rng, ctx, window, Hkv):
    q, k_pool, v_pool, page_row, kb, vb = _case(rng, 5, 4, Hkv, 8, ctx)
    got = O.attention_paged(q, k_pool, v_pool, page_row, ctx, kb, vb, window=window)
    np.testing.assert_allclose(got, _enumerate(q, k_pool, v_pool, page_row, ctx, kb, vb, window), rtol=1e-10, atol=1e-12)


def test_paged_equals_contiguous_bitwise(rng):
    q, k_pool, v_pool, page_row, kb, vb = _case(rng, 3, 4, 2, 8, 37)
    Kc, Vc = O.gather_kv(k_pool, page_row, 37), O.gather_kv(v_pool, page_row, 37)
    for p in (0, 15, 16, 36):
        np.testing.assert_array_equal(Kc[p], k_pool[page_row[p // 16], p % 16])
    a = O.attention_paged(q, k_pool, v_pool, page_row, 37, kb, vb)
    b = O.attention_contiguous(q, Kc, Vc, kb, vb)
    np.testing.assert_array_equal(a, b)


def test_gather_preserves_bf16_bits(rng):
    pool = rng.integers(0, 65536, (5, 16, 2, 4), dtype=np.uint16)
    row = np.array([3, 0, 4], dtype=np.int32)
    got = O.gather_kv(pool, row, 40)
    assert got.dtype == np.uint16
    np.testing.assert_array_equal(got[:16], pool[3])
    np.testing.assert_array_equal(got[16:32], pool[0])
    np.testing.assert_array_equal(got[32:40], pool[4, :8])


def test_two_part_online_softmax_merge(rng):
    # softmax over the union == merging (max, sum, weighted V) of the prefix part and the block part
    q, k_pool, v_pool, page_row, kb, vb = _case(rng, 4, 2, 1, 8, 23)
    full = O.attention_paged(q, k_pool, v_pool, page_row, 23, kb, vb)
    Kc, Vc = O.gather_kv(k_pool, page_row, 23), O.gather_kv(v_pool, page_row, 23)
    for i in range(4):
        for hq in range(2):
            s1 = Kc[:, 0] @ q[i, hq] / math.sqrt(8)
            s2 = kb[:i + 1, 0] @ q[i, hq] / math.sqrt(8)
            m1, m2 = s1.max(), s2.max()
            l1, l2 = np.exp(s1 - m1).sum(), np.exp(s2 - m2).sum()
            o1, o2 = np.exp(s1 - m1) @ Vc[:, 0] / l1, np.exp(s2 - m2) @ vb[:i + 1, 0] / l2
            m = max(m1, m2)
            w1, w2 = l1 * math.exp(m1 - m), l2 * math.exp(m2 - m)
            np.testing.assert_allclose(full[i, hq], (w1 * o1 + w2 * o2) / (w1 + w2), rtol=1e-10)


def test_equal_keys_give_mean_of_visible_values(rng):
    q, k_pool, v_pool, page_row, kb, vb = _case(rng, 3, 2, 1, 8, 20)
    k_pool[:] = 0.25
    kb[:] = 0.25
    got = O.attention_paged(q, k_pool, v_pool, page_row, 20, kb, vb)
    Vc = O.gather_kv(v_pool, page_row, 20)
    for i in range(3):
        ref = (Vc[:, 0].sum(0) + vb[:i + 1, 0].sum(0)) / (20 + i + 1)
        np.testing.assert_allclose(got[i, 0], ref, rtol=1e-10)


def test_empty_context_first_row_returns_its_own_value(rng):
    q, k_pool, v_pool, page_row, kb, vb = _case(rng, 3, 4, 2, 8, 0)
    got = O.attention_paged(q, k_pool, v_pool, page_row, 0, kb, vb)
    for hq in range(4):
        np.testing.assert_array_equal(got[0, hq], vb[0, hq // 2])


def test_scale_is_inverse_sqrt_head_dim(rng):
    # one prefix key + the row's own key: weights are a logistic of the score gap / sqrt(dh)
    dh = 16
    q = rng.standard_normal((1, 1, dh))
    k_pool, v_pool = rng.standard_normal((1, 16, 1, dh)), rng.standard_normal((1, 16, 1, dh))
    kb, vb = rng.standard_normal((1, 1, dh)), rng.standard_normal((1, 1, dh))
    got = O.attention_paged(q, k_pool, v_pool, np.array([0]), 1, kb, vb)
    gap = (q[0, 0] @ k_pool[0, 0, 0] - q[0, 0] @ kb[0, 0]) / math.sqrt(dh)
    w = 1 / (1 + math.exp(-gap))
    np.testing.assert_allclose(got[0, 0], w * v_pool[0, 0, 0] + (1 - w) * vb[0, 0], rtol=1e-10)


def test_prefix_permutation_invariance_and_window_limits(rng):
    q, k_pool, v_pool, page_row, kb, vb = _case(rng, 4, 4, 2, 8, 33)
    Kc, Vc = O.gather_kv(k_pool, page_row, 33), O.gather_kv(v_pool, page_row, 33)
    base = O.attention_contiguous(q, Kc, Vc, kb, vb)
    perm = rng.permutation(33)
    np.testing.assert_allclose(O.attention_contiguous(q, Kc[perm], Vc[perm], kb, vb), base, rtol=1e-10)
    # a window that covers everything is the full attention
    np.testing.assert_array_equal(O.attention_contiguous(q, Kc, Vc, kb, vb, window=33 + 4), base)
    # window 1: each row sees only itself
    w1 = O.attention_contiguous(q, Kc, Vc, kb, vb, window=1)
    for i in range(4):
        np.testing.assert_allclose(w1[i, 3], vb[i, 1], rtol=1e-12)


def test_gqa_equals_replicated_mha(rng):
    q, k_pool, v_pool, page_row, kb, vb = _case(rng, 3, 4, 2, 8, 19)
    got = O.attention_paged(q, k_pool, v_pool, page_row, 19, kb, vb)
    rep = lambda t: np.repeat(t, 2, axis=-2)
    mha = O.attention_paged(q, rep(k_pool), rep(v_pool), page_row, 19, rep(kb), rep(vb))
    np.testing.assert_allclose(got, mha, rtol=1e-12)


def test_nan_in_unmapped_slots_does_not_leak(rng):
    q, k_pool, v_pool, page_row, kb, vb = _case(rng, 3, 2, 1, 8, 21)
    clean = O.attention_paged(q, k_pool, v_pool, page_row, 21, kb, vb)
    k2, v2 = k_pool.copy(), v_pool.copy()
    k2[page_row[1], 5:] = np.nan      # tail of the last (partly filled) page
    v2[page_row[1], 5:] = np.nan
    unmapped = [p for p in range(k_pool.shape[0]) if p not in page_row[:2]]
    k2[unmapped] = np.nan
    v2[unmapped] = np.nan
    got = O.attention_paged(q, k2, v2, page_row, 21, kb, vb)
    assert np.isfinite(got).all()
    np.testing.assert_array_equal(got, clean)
