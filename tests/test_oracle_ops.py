"""Pins for the oracle's elementary ops: brute force, closed forms, invariants, Table 1."""
import math
import os

import numpy as np
import pytest

from oracle import hspec_oracle as O

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def test_widen_bf16_bits():
    # 1.0 = 0x3F80, -2.5 = 0xC020, smallest bf16 step above 1 = 0x3F81 = 1 + 2^-7
    bits = np.array([0x3F80, 0xC020, 0x3F81, 0x0000], dtype=np.uint16)
    assert O.widen(bits).tolist() == [1.0, -2.5, 1.0 + 2.0 ** -7, 0.0]


def test_gemm_triple_loop(rng):
    x = rng.standard_normal((3, 5))
    W = rng.standard_normal((4, 5))
    ref = [[sum(x[m, c] * W[n, c] for c in range(5)) for n in range(4)] for m in range(3)]
    np.testing.assert_allclose(O.gemm(x, W), np.array(ref), rtol=1e-13)
    # piecewise widening of W must not change anything
    np.testing.assert_array_equal(O.gemm(x, W, rows_per_piece=3), O.gemm(x, W))
    # a transposed operand would give a shape error or a different value
    assert O.gemm(x, W).shape == (3, 4)


def test_gemm_bf16_bits():
    W = np.array([[0x3F80, 0x4000], [0xBF80, 0x3F00]], dtype=np.uint16)   # [[1,2],[-1,.5]]
    x = np.array([[3.0, 4.0]])
    assert O.gemm(x, W).tolist() == [[11.0, -1.0]]


def test_rmsnorm_properties(rng):
    v = rng.standard_normal((4, 32))
    y = O.rmsnorm(v, np.ones(32), 0.0)
    np.testing.assert_allclose(np.sqrt(np.mean(y * y, axis=-1)), 1.0, rtol=1e-12)
    np.testing.assert_allclose(O.rmsnorm(7.5 * v, np.ones(32), 0.0), y, rtol=1e-12)
    w = rng.standard_normal(32)
    np.testing.assert_allclose(O.rmsnorm(v, w, 0.0), y * w, rtol=1e-12)
    # eps enters under the root, next to the mean square
    one = np.array([[3.0, 4.0]])
    np.testing.assert_allclose(O.rmsnorm(one, np.ones(2), 0.5), one / math.sqrt(12.5 + 0.5))


def test_silu_softplus_closed_forms():
    assert O.silu(np.array(0.0)) == 0.0
    np.testing.assert_allclose(O.silu(np.array([1.0, -1.0])), [1 / (1 + math.exp(-1)), -1 / (1 + math.exp(1))])
    np.testing.assert_allclose(O.softplus(np.array(0.0)), math.log(2.0))
    assert O.softplus(np.array(50.0)) == 50.0
    np.testing.assert_allclose(O.softplus(np.array(-30.0)), math.exp(-30.0), rtol=1e-10)
    np.testing.assert_allclose(O.softplus(np.array(20.0)), 20.0 + math.log1p(math.exp(-20.0)), rtol=1e-12)
    # softplus(x) - softplus(-x) = x
    x = np.linspace(-5, 5, 11)
    np.testing.assert_allclose(O.softplus(x) - O.softplus(-x), x, atol=1e-12)


def test_discretise_ranges():
    dt, a = O.discretise(np.zeros((1, 2)), np.array([0.0, 1.0]), np.array([0.0, math.log(2.0)]))
    np.testing.assert_allclose(dt[0], [math.log(2.0), math.log1p(math.e)])
    np.testing.assert_allclose(a[0], [math.exp(-math.log(2.0)), math.exp(-2.0 * math.log1p(math.e))])
    assert np.all((a > 0) & (a < 1))


def test_conv_silu_brute_force(rng):
    k, C, dc = 6, 3, 4
    raw, w, b = rng.standard_normal((k, C)), rng.standard_normal((C, dc)), rng.standard_normal(C)
    out = O.conv_silu(raw, w, b)
    for i in range(k):
        for c in range(C):
            acc = b[c]
            for j in range(dc):
                src = i - 3 + j
                acc += w[c, j] * (raw[src, c] if src >= 0 else 0.0)
            assert out[i, c] == pytest.approx(acc / (1 + math.exp(-acc)), rel=1e-12)
    # the LAST tap multiplies the current row; the first row sees only that tap
    np.testing.assert_allclose(out[0], O.silu(b + w[:, 3] * raw[0]), rtol=1e-12)
    # causality: changing a later row does not change earlier outputs
    raw2 = raw.copy()
    raw2[4] += 1.0
    np.testing.assert_array_equal(O.conv_silu(raw2, w, b)[:4], out[:4])


def test_rope_properties(rng):
    dh = 16
    v = rng.standard_normal((3, dh))
    np.testing.assert_array_equal(O.rope(v, 0, 1e4), v)
    for pos in (1, 17, 4097):
        np.testing.assert_allclose(np.linalg.norm(O.rope(v, pos, 1e4), axis=-1), np.linalg.norm(v, axis=-1), rtol=1e-12)
    # <R(p) q, R(s) k> depends only on p - s (small positions: fp32 angle rounding is negligible)
    q, k = rng.standard_normal(dh), rng.standard_normal(dh)
    d1 = O.rope(q, 9, 1e4) @ O.rope(k, 4, 1e4)
    d2 = O.rope(q, 25, 1e4) @ O.rope(k, 20, 1e4)
    assert d1 == pytest.approx(d2, abs=1e-5)
    # explicit pair (j, j + dh/2), frequency theta^(-2j/dh): rotate e_1 at position 1
    e = np.zeros(dh)
    e[1] = 1.0
    ang = float(np.float32(10000.0 ** (-2.0 / dh)))
    r = O.rope(e, 1, 1e4)
    assert r[1] == pytest.approx(math.cos(ang)) and r[1 + dh // 2] == pytest.approx(math.sin(ang))
    assert np.count_nonzero(r) == 2


def test_rope_angle_is_one_float32_product():
    # at a large position the float32 product differs measurably from the float64 one;
    # the oracle must use the float32 angle (the recipe the GPU follows)
    dh, theta, pos = 128, 1.0e6, 32799
    inv = np.float32(theta ** (-2.0 * 1 / dh))
    ang32 = float(np.float32(pos) * inv)
    e = np.zeros(dh)
    e[1] = 1.0
    r = O.rope(e, pos, theta)
    assert r[1] == pytest.approx(math.cos(ang32), abs=1e-12)
    assert r[1 + dh // 2] == pytest.approx(math.sin(ang32), abs=1e-12)


def test_argmax_margin_sort_and_ties(rng):
    logits = rng.standard_normal((5, 37))
    ids, margin = O.argmax_margin(logits)
    order = np.argsort(-logits, axis=-1, kind="stable")
    np.testing.assert_array_equal(ids, order[:, 0])
    np.testing.assert_allclose(margin, logits[np.arange(5), order[:, 0]] - logits[np.arange(5), order[:, 1]])
    tied = np.zeros((1, 9))
    tied[0, [6, 2, 4]] = 3.0
    ids, margin = O.argmax_margin(tied)
    assert ids[0] == 2 and margin[0] == 0.0


def _read_table1():
    rows = []
    with open(os.path.join(GOLDEN, "table1_kv_bytes.txt")) as f:
        for line in f:
            if line.strip() and not line.startswith("#"):
                name, t, d, inc = line.split()
                rows.append((name, int(t), int(d), float(inc)))
    return rows


def test_table1_kv_accounting():
    rows = _read_table1()
    # printed increase = (target + draft) / target of the printed sizes
    for name, t, d, inc in rows:
        assert round((t + d) / t, 3) == pytest.approx(inc, abs=5e-4), name
    # 20 KiB for a five-layer drafter with the target's 8 KV heads x 128: 4 KiB per layer
    assert O.kv_bytes_per_token(5, 8, 128, 2) == 20 * 1024
    assert O.kv_bytes_per_token(1, 8, 128, 2) == 4 * 1024
    # publicly documented target shapes reproduce the target column
    assert O.kv_bytes_per_token(36, 8, 128, 2) == 144 * 1024     # Qwen3-4B / Qwen3-8B: 36 layers
    assert O.kv_bytes_per_token(32, 8, 128, 2) == 128 * 1024     # Llama3.1-8B: 32 layers
    # what in-place reuse avoids for a batch: sum of contexts x per-token bytes
    assert O.drafter_kv_bytes_avoided([100, 28], 2, 8, 128) == 128 * 8 * 1024
