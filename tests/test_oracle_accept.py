"""Pins for oracle/accept_oracle.py: closed forms, brute force on tiny inputs, invariants (no GPU)."""
import math

import numpy as np
import pytest

from oracle import accept_oracle as ao


# --------------------------------------------------------------------------- token_probs

def test_token_probs_rows_sum_to_one_and_uniform():
    rng = np.random.default_rng(1)
    z = rng.normal(size=(5, 37)) * 3
    total = sum(ao.token_probs(z, np.full(5, v)) for v in range(37))
    np.testing.assert_allclose(total, 1.0, rtol=0, atol=1e-12)
    np.testing.assert_allclose(ao.token_probs(np.zeros((3, 8)), [0, 3, 7]), 1 / 8, rtol=0, atol=1e-15)


def test_token_probs_shift_invariance_and_logistic():
    rng = np.random.default_rng(2)
    z = rng.normal(size=(4, 11))
    ids = rng.integers(0, 11, size=4)
    np.testing.assert_allclose(ao.token_probs(z + 123.0, ids), ao.token_probs(z, ids), rtol=1e-12)
    # two tokens: softmax is the logistic function of the difference
    d = np.array([-3.0, 0.0, 0.5, 40.0])
    z2 = np.stack([d, np.zeros_like(d)], axis=1)
    np.testing.assert_allclose(ao.token_probs(z2, np.zeros(4, dtype=int)), 1 / (1 + np.exp(-d)), rtol=1e-12)


# --------------------------------------------------------------------------- accept_lengths

def _accept_loop(pt, pd, al):
    out = []
    for b in range(len(pt)):
        n = 0
        for i in range(len(pt[b])):
            r = np.float32(pt[b][i]) / np.float32(pd[b][i])
            if not (min(np.float32(1.0), r) >= np.float32(al[b][i])):
                break
            n += 1
        out.append(n)
    return out


def test_accept_matches_python_loop():
    rng = np.random.default_rng(3)
    for k in (1, 5, 16):
        pt = rng.uniform(0.0, 1.0, size=(64, k)).astype(np.float32)
        pd = rng.uniform(0.05, 1.0, size=(64, k)).astype(np.float32)
        al = rng.uniform(0.0, 1.0, size=(64, k)).astype(np.float32)
        assert ao.accept_lengths(pt, pd, al).tolist() == _accept_loop(pt, pd, al)


def test_accept_special_cases():
    rng = np.random.default_rng(4)
    k = 7
    pt = rng.uniform(0.1, 1.0, size=(9, k)).astype(np.float32)
    pd = rng.uniform(0.1, 1.0, size=(9, k)).astype(np.float32)
    assert ao.accept_lengths(pt, pd, np.zeros((9, k))).tolist() == [k] * 9                     # alpha = 0
    al = rng.uniform(0.0, 0.999, size=(9, k)).astype(np.float32)
    assert ao.accept_lengths(np.maximum(pt, pd), pd, al).tolist() == [k] * 9                   # P_T >= P_D
    first = (pt[:, 0] / pd[:, 0]).clip(max=1.0)
    al2 = al.copy()
    al2[:, 0] = np.nextafter(first, np.float32(2.0))                                          # just above the first ratio
    ok = first < 1.0
    assert (ao.accept_lengths(pt, pd, al2)[ok] == 0).all()
    # P_D = 0: +inf ratio is accepted, 0 / 0 is rejected
    assert ao.accept_lengths([[0.5, 0.5]], [[0.0, 0.5]], [[0.9, 0.0]]).tolist() == [2]
    assert ao.accept_lengths([[0.0, 0.5]], [[0.0, 0.5]], [[0.0, 0.0]]).tolist() == [0]


def test_accept_prefix_property():
    """The count for the first j positions is min(count for all k, j)."""
    rng = np.random.default_rng(5)
    pt = rng.uniform(0.0, 1.0, size=(40, 12)).astype(np.float32)
    pd = rng.uniform(0.05, 1.0, size=(40, 12)).astype(np.float32)
    al = rng.uniform(0.0, 1.0, size=(40, 12)).astype(np.float32)
    full = ao.accept_lengths(pt, pd, al)
    for j in (1, 4, 9):
        np.testing.assert_array_equal(ao.accept_lengths(pt[:, :j], pd[:, :j], al[:, :j]), np.minimum(full, j))


def test_accept_expected_length_closed_form():
    """With alpha ~ U(0,1) position i is accepted with probability r_i = min(1, P_T/P_D), so
    E[n] = sum_j prod_{i<=j} r_i (the geometric-like sum behind the acceptance-length figures)."""
    rng = np.random.default_rng(6)
    k, trials = 6, 200000
    r = np.array([0.9, 0.8, 1.0, 0.5, 0.7, 0.6], dtype=np.float32)
    pd = np.full((trials, k), 0.5, dtype=np.float32)
    pt = np.broadcast_to(r * np.float32(0.5), (trials, k))
    al = rng.uniform(0.0, 1.0, size=(trials, k)).astype(np.float32)
    expect = float(np.cumprod(r.astype(np.float64)).sum())
    got = ao.accept_lengths(pt, pd, al).mean()
    assert abs(got - expect) < 4 * math.sqrt(k * k / trials)


# --------------------------------------------------------------------------- markov_head

def _markov_brute(z, W_in, W_out, last, id_map=None):
    B, k, Vd = z.shape
    table = [[sum(float(W_out[v][j]) * float(W_in[u][j]) for j in range(W_in.shape[1])) for u in range(W_in.shape[0])]
             for v in range(Vd)]                      # table[v][u]: boost of token v after token u
    ids = []
    for b in range(B):
        prev, row_ids = int(last[b]), []
        for i in range(k):
            best, best_v = None, -1
            for v in range(Vd):
                val = float(z[b, i, v]) + table[v][prev]
                if best is None or val > best:
                    best, best_v = val, v
            row_ids.append(best_v)
            prev = best_v if id_map is None else int(id_map[best_v])
        ids.append(row_ids)
    return ids


def test_markov_matches_dense_table_brute_force():
    rng = np.random.default_rng(7)
    B, k, V, r = 3, 5, 13, 4
    z = rng.normal(size=(B, k, V))
    W_in, W_out = rng.normal(size=(V, r)), rng.normal(size=(V, r))
    last = rng.integers(0, V, size=B)
    ids, adj, margin = ao.markov_head(z, W_in, W_out, last)
    assert ids.tolist() == _markov_brute(z, W_in, W_out, last)
    assert (margin >= 0).all()
    # the adjusted logits are the plain ones plus the table column of the predecessor
    prev = np.concatenate([last[:, None], ids[:, :-1]], axis=1)
    np.testing.assert_allclose(adj, z + np.einsum("vr,bkr->bkv", W_out, W_in[prev]), rtol=1e-12, atol=1e-12)


def test_markov_pruned_vocabulary_brute_force():
    rng = np.random.default_rng(8)
    B, k, V, Vd, r = 2, 4, 17, 6, 3
    id_map = np.sort(rng.choice(V, size=Vd, replace=False))
    z = rng.normal(size=(B, k, Vd))
    W_in, W_out = rng.normal(size=(V, r)), rng.normal(size=(Vd, r))
    last = rng.integers(0, V, size=B)
    ids, _, _ = ao.markov_head(z, W_in, W_out, last, id_map=id_map)
    assert ids.tolist() == _markov_brute(z, W_in, W_out, last, id_map=id_map)


def test_markov_zero_table_is_plain_argmax_and_ties_go_low():
    rng = np.random.default_rng(9)
    z = rng.normal(size=(4, 6, 9))
    ids, adj, _ = ao.markov_head(z, rng.normal(size=(9, 5)), np.zeros((9, 5)), np.zeros(4, dtype=int))
    np.testing.assert_array_equal(ids, z.argmax(-1))
    np.testing.assert_array_equal(adj, z)
    ids, _, margin = ao.markov_head(np.zeros((1, 2, 5)), np.zeros((5, 2)), np.zeros((5, 2)), [0])
    assert ids.tolist() == [[0, 0]] and (margin == 0).all()


def test_markov_constructed_chain():
    """One-hot factors of rank V make the table a shifted identity: after token u the boost goes to u + 1.
    With flat logits the drafted block is last+1, last+2, ... (mod V)."""
    V, k = 7, 10
    W_in = np.eye(V)
    W_out = 5.0 * np.roll(np.eye(V), 1, axis=0)        # row v has its one at column v - 1
    ids, _, margin = ao.markov_head(np.zeros((2, k, V)), W_in, W_out, [2, 6])
    assert ids[0].tolist() == [(3 + i) % V for i in range(k)]
    assert ids[1].tolist() == [(0 + i) % V for i in range(k)]
    np.testing.assert_allclose(margin, 5.0)


def test_markov_locality():
    rng = np.random.default_rng(10)
    B, k, V, r = 2, 8, 11, 3
    z = rng.normal(size=(B, k, V))
    W_in, W_out = rng.normal(size=(V, r)), rng.normal(size=(V, r))
    last = rng.integers(0, V, size=B)
    ids0, _, _ = ao.markov_head(z, W_in, W_out, last)
    z2 = z.copy()
    z2[:, 5] += rng.normal(size=(B, V)) * 10
    ids1, _, _ = ao.markov_head(z2, W_in, W_out, last)
    np.testing.assert_array_equal(ids0[:, :5], ids1[:, :5])


# --------------------------------------------------------------------------- kv_inject_rows / scatter_kv

def test_scatter_then_gather_round_trip_and_untouched_rows():
    from oracle import hspec_oracle as O
    rng = np.random.default_rng(11)
    pool = rng.normal(size=(9, 16, 2, 8)).astype(np.float32)
    before = pool.copy()
    page_row = np.array([5, 2, 7, 0])
    pos = np.array([3, 17, 18, 40])
    rows = rng.normal(size=(4, 2, 8)).astype(np.float32)
    ao.scatter_kv(pool, page_row, pos, rows)
    got = O.gather_kv(pool, page_row, 41)
    np.testing.assert_array_equal(got[pos], rows)
    mask = np.ones(41, dtype=bool); mask[pos] = False
    np.testing.assert_array_equal(got[mask], O.gather_kv(before, page_row, 41)[mask])
    untouched = [p for p in range(9) if p not in page_row]
    np.testing.assert_array_equal(pool[untouched], before[untouched])


def test_kv_inject_rows_rotation_properties():
    rng = np.random.default_rng(12)
    T, Hkv, dh = 5, 2, 16
    kv = rng.normal(size=(T, 2, Hkv, dh))
    ones = np.ones(dh)
    K0, V0 = ao.kv_inject_rows(kv, ones, np.zeros(T, dtype=int), 1.0e4, k_norm=False)
    np.testing.assert_array_equal(K0, kv[:, 0])                      # position 0: no rotation
    np.testing.assert_array_equal(V0, kv[:, 1])                      # values are never touched
    pos = np.array([1, 7, 100, 4095, 31999])
    K, _ = ao.kv_inject_rows(kv, ones, pos, 1.0e4, k_norm=False)
    np.testing.assert_allclose(np.linalg.norm(K, axis=-1), np.linalg.norm(kv[:, 0], axis=-1), rtol=1e-12)
    # with the norm on, every key head has unit RMS times the gain
    Kn, _ = ao.kv_inject_rows(kv, 2.0 * ones, pos, 1.0e4, eps=0.0, k_norm=True)
    np.testing.assert_allclose(np.sqrt(np.mean(Kn * Kn, axis=-1)), 2.0, rtol=1e-12)


def test_kv_inject_rows_relative_position_law():
    """<RoPE(a, p), RoPE(b, p + d)> depends on d only (up to the float32 rounding of the angles)."""
    rng = np.random.default_rng(13)
    a = rng.normal(size=(1, 2, 1, 32)); b = rng.normal(size=(1, 2, 1, 32))
    ones = np.ones(32)
    dots = []
    for p in (0, 5, 64, 1000):
        Ka, _ = ao.kv_inject_rows(a, ones, [p], 1.0e6, k_norm=False)
        Kb, _ = ao.kv_inject_rows(b, ones, [p + 9], 1.0e6, k_norm=False)
        dots.append(float(np.sum(Ka * Kb)))
    np.testing.assert_allclose(dots, dots[0], rtol=0, atol=2e-3)


def test_kv_inject_keys_match_the_step_oracles_rope():
    """The injected key of position p equals what the draft step's own RoPE gives a block key at that position."""
    from oracle import hspec_oracle as O
    rng = np.random.default_rng(14)
    kv = rng.normal(size=(3, 2, 2, 16))
    pos = np.array([2, 50, 777])
    K, _ = ao.kv_inject_rows(kv, np.ones(16), pos, 1.0e6, k_norm=False)
    for t in range(3):
        np.testing.assert_allclose(K[t], O.rope(kv[t, 0], int(pos[t]), 1.0e6), rtol=1e-12, atol=1e-12)
