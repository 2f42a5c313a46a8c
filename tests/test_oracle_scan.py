"""Pins for the selective scan with injected initial state (Sec. 3.3.1)."""
import itertools

import numpy as np
import pytest

from oracle import hspec_oracle as O


def _case(rng, k, H, P, N, G, zero_init=False):
    S0 = np.zeros((H, P, N)) if zero_init else rng.standard_normal((H, P, N))
    x = rng.standard_normal((k, H, P))
    Bm, Cm = rng.standard_normal((k, G, N)), rng.standard_normal((k, G, N))
    dt = rng.uniform(1e-3, 1e-1, (k, H))
    a = np.exp(-dt * rng.uniform(1.0, 7.4, H))
    Dskip = rng.standard_normal(H)
    return S0, x, Bm, Cm, dt, a, Dskip


@pytest.mark.parametrize("k,N,G", list(itertools.product([1, 3, 5, 8], [1, 4], [1, 2])))
def test_sequential_equals_quadratic(rng, k, N, G):
    args = _case(rng, k, 4, 4, N, G)
    y_seq, _ = O.scan_sequential(*args)
    np.testing.assert_allclose(y_seq, O.scan_quadratic(*args), rtol=1e-11, atol=1e-12)


def test_brute_force_scalar_loops(rng):
    # every index written out, no numpy broadcasting: catches a swapped P/N or group index
    k, H, P, N, G = 3, 4, 2, 3, 2
    S0, x, Bm, Cm, dt, a, Dskip = _case(rng, k, H, P, N, G)
    y, S_fin = O.scan_sequential(S0, x, Bm, Cm, dt, a, Dskip)
    S = S0.copy()
    for i in range(k):
        for h in range(H):
            g = h // (H // G)
            for p in range(P):
                acc = 0.0
                for n in range(N):
                    S[h, p, n] = a[i, h] * S[h, p, n] + dt[i, h] * x[i, h, p] * Bm[i, g, n]
                    acc += Cm[i, g, n] * S[h, p, n]
                assert y[i, h, p] == pytest.approx(acc + Dskip[h] * x[i, h, p], rel=1e-12)
    np.testing.assert_allclose(S_fin, S, rtol=1e-12)


def test_zero_initial_state_is_plain_recurrence(rng):
    S0, x, Bm, Cm, dt, a, Dskip = _case(rng, 6, 4, 4, 4, 2, zero_init=True)
    y, _ = O.scan_sequential(S0, x, Bm, Cm, dt, a, Dskip)
    # plain Mamba-2 forward (no injected state), head by head, as a running sum
    for h in range(4):
        g = h // 2
        S = np.zeros((4, 4))
        for i in range(6):
            S = a[i, h] * S + np.outer(dt[i, h] * x[i, h], Bm[i, g])
            np.testing.assert_allclose(y[i, h], S @ Cm[i, g] + Dskip[h] * x[i, h], rtol=1e-12)


def test_decay_applies_to_injected_state_at_position_zero(rng):
    # k = 1 closed form: y_0 = (a_0 S_init + dt_0 x_0 B_0^T) C_0 + D x_0
    S0, x, Bm, Cm, dt, a, Dskip = _case(rng, 1, 2, 3, 4, 1)
    y, _ = O.scan_sequential(S0, x, Bm, Cm, dt, a, Dskip)
    for h in range(2):
        ref = (a[0, h] * S0[h] + np.outer(dt[0, h] * x[0, h], Bm[0, 0])) @ Cm[0, 0] + Dskip[h] * x[0, h]
        np.testing.assert_allclose(y[0, h], ref, rtol=1e-12)


def test_restart_invariant(rng):
    S0, x, Bm, Cm, dt, a, Dskip = _case(rng, 8, 4, 4, 4, 2)
    y, _ = O.scan_sequential(S0, x, Bm, Cm, dt, a, Dskip)
    for j in (1, 3, 7):
        _, S_mid = O.scan_sequential(S0, x[:j], Bm[:j], Cm[:j], dt[:j], a[:j], Dskip)
        y_tail, _ = O.scan_sequential(S_mid, x[j:], Bm[j:], Cm[j:], dt[j:], a[j:], Dskip)
        np.testing.assert_allclose(y_tail, y[j:], rtol=1e-12)


def test_superposition(rng):
    S0, x, Bm, Cm, dt, a, Dskip = _case(rng, 5, 4, 4, 4, 2)
    y, _ = O.scan_sequential(S0, x, Bm, Cm, dt, a, Dskip)
    y_state, _ = O.scan_sequential(S0, np.zeros_like(x), Bm, Cm, dt, a, Dskip)
    y_input, _ = O.scan_sequential(np.zeros_like(S0), x, Bm, Cm, dt, a, Dskip)
    np.testing.assert_allclose(y, y_state + y_input, rtol=1e-11, atol=1e-12)


def test_geometric_closed_form():
    # constant a, dt, x, B: S_k = a^k S_0 + dt x B^T (1 - a^k) / (1 - a)
    k, H, P, N = 7, 1, 2, 3
    S0 = np.arange(6, dtype=float).reshape(1, 2, 3)
    xv, Bv = np.array([0.5, -1.5]), np.array([1.0, 2.0, -1.0])
    x, Bm = np.tile(xv, (k, 1, 1)), np.tile(Bv, (k, 1, 1))
    Cm = np.zeros((k, 1, N))
    a0, dt0 = 0.8, 0.05
    _, S_fin = O.scan_sequential(S0, x, Bm, Cm, np.full((k, 1), dt0), np.full((k, 1), a0), np.zeros(1))
    ref = a0 ** k * S0[0] + dt0 * np.outer(xv, Bv) * (1 - a0 ** k) / (1 - a0)
    np.testing.assert_allclose(S_fin[0], ref, rtol=1e-12)


def test_c_zero_leaves_skip_only(rng):
    S0, x, Bm, Cm, dt, a, Dskip = _case(rng, 4, 4, 4, 4, 2)
    y, _ = O.scan_sequential(S0, x, Bm, np.zeros_like(Cm), dt, a, Dskip)
    np.testing.assert_allclose(y, Dskip[None, :, None] * x, rtol=1e-12)
