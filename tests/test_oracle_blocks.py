"""Scalar-loop pins for the oracle's three sub-blocks and for their composition into the step.

Everything on the brute-force side is written with Python floats, `math` and explicit index loops over plain
nested lists: no numpy broadcasting, no call into `oracle/`.  Each brute force takes the documented layout as
literal index arithmetic (which rows of a fused projection are which, where the norm sits, which position a row
is rotated at), so a slip in the oracle's slicing, ordering or offsets shows up as a mismatch.  Every pin is
paired with a sensitivity check: the same brute force with ONE deliberate mistake (SiLU on the wrong half,
position off by one, norm after the rotation, a permuted split, ...) must disagree with the oracle, which shows
that the comparison can tell the two apart on these inputs.

Layouts pinned here (Sec. 3.3.1, Sec. 3.3.2 "Positional alignment", App. B.1):
  MLP        w_gate_up rows = gate (first F) | up (last F); out = (SiLU(gate) * up) W_down^T
  attention  wqkv rows = q (Hq*dh) | k (Hkv*dh) | v (Hkv*dh); per-head RMSNorm of q and of the block's k BEFORE
             the rotation; block row i rotated at position ctx_len + i with pairs (j, j + dh/2) and angle
             pos * theta^(-2j/dh); query head hq reads KV head hq // (Hq/Hkv); one softmax over the visible
             prefix keys and block keys j <= i; window W keeps 0 <= pos_q - pos_k < W
  Mamba      in_proj rows = z (Di) | xBC (Di + 2GN) | dt (H or dt_rank); xBC after conv + SiLU = x [H,P] |
             B [G,N] | C [G,N]; y * SiLU(z) then RMSNorm over all Di channels; decay applied to S_init at
             position 0
  step       X += Mamba(norm(X)); X += Attn(norm(X)); X += MLP(norm(X)) per layer, final norm, LM head
"""
import math

import numpy as np
import pytest
import torch

import synth
from oracle import hspec_oracle as O
from conftest import to_np, weights_np

MINI = dict(D=8, n_fuse=1, r=8, L=2, has_attn=[1, 1], kv_slot=[0, 1], n_slots=2, Di=16, P=4, N=4, G=2,
            d_conv=4, dt_rank=0, Hq=4, Hkv=2, dh=8, rope_theta=1.0e4, window=0, qk_norm=1, F=16, V=11,
            rms_eps=1e-6, page_size=16, name="mini", B=1, k=5, ctx=("const", 0, 0))


def _bf16_to_float(bits):
    """uint16 bf16 pattern -> Python float (scalar bit manipulation, independent of the oracle's `widen`)."""
    import struct
    return struct.unpack("<f", struct.pack("<I", int(bits) << 16))[0]


def _lists(a):
    """numpy array (bf16 bit patterns or floats) -> nested Python lists of floats."""
    a = np.asarray(a)
    if a.dtype == np.uint16:
        flat = [_bf16_to_float(v) for v in a.ravel().tolist()]
        return np.array(flat, dtype=np.float64).reshape(a.shape).tolist()
    return a.astype(np.float64).tolist()


def _setup(ctx_lens, scale=8.0, **over):
    cfg = synth.derived(dict(MINI, **over))
    w = synth.make_weights(cfg)
    w = {k: (v.float() * scale).to(v.dtype) if v.dtype == torch.bfloat16 else v for k, v in w.items()}
    batch = synth.make_request_batch(cfg, ctx_lens=ctx_lens, extra_pages=2)
    return cfg, weights_np(w), batch


def _sub(w, l, block):
    p = f"layers.{l}.{block}."
    return {n[len(p):]: t for n, t in w.items() if n.startswith(p)}


# --------------------------------------------------------------------------- scalar building blocks


def _dot(a, b):
    s = 0.0
    for x, y in zip(a, b):
        s += x * y
    return s


def _linear(rows, W):
    """rows [M][K], W [N][K] -> [M][N], bias-free."""
    return [[_dot(r, wrow) for wrow in W] for r in rows]


def _silu(v):
    return v / (1.0 + math.exp(-v))


def _rmsnorm(v, g, eps):
    ms = 0.0
    for x in v:
        ms += x * x
    inv = 1.0 / math.sqrt(ms / len(v) + eps)
    return [x * inv * gi for x, gi in zip(v, g)]


def _rotate(v, pos, theta):
    dh = len(v)
    half = dh // 2
    out = [0.0] * dh
    for j in range(half):
        ang = pos * theta ** (-2.0 * j / dh)
        c, s = math.cos(ang), math.sin(ang)
        out[j] = v[j] * c - v[j + half] * s
        out[j + half] = v[j + half] * c + v[j] * s
    return out


# --------------------------------------------------------------------------- MLP


def _bf_mlp(u, w_gate_up, w_down, mistake=None):
    F = len(w_gate_up) // 2
    out = []
    for row in u:
        h = []
        for f in range(F):
            gate = _dot(row, w_gate_up[f])          # first F rows
            up = _dot(row, w_gate_up[F + f])        # last F rows
            if mistake == "silu_on_up":
                h.append(gate * _silu(up))
            elif mistake == "interleaved":
                h.append(_silu(_dot(row, w_gate_up[2 * f])) * _dot(row, w_gate_up[2 * f + 1]))
            else:
                h.append(_silu(gate) * up)
        out.append([_dot(h, w_down[d]) for d in range(len(w_down))])
    return out


def test_mlp_block_matches_scalar_loops():
    cfg, w, _ = _setup([3])
    sub = _sub(w, 0, "mlp")
    rng = np.random.default_rng(5)
    u = rng.standard_normal((3, cfg["D"]))
    got = O.mlp_block(u, sub)
    ref = _bf_mlp(u.tolist(), _lists(sub["w_gate_up"]), _lists(sub["w_down"]))
    np.testing.assert_allclose(got, np.array(ref), rtol=1e-11, atol=1e-13)
    for mistake in ("silu_on_up", "interleaved"):
        bad = np.array(_bf_mlp(u.tolist(), _lists(sub["w_gate_up"]), _lists(sub["w_down"]), mistake))
        assert np.max(np.abs(bad - got)) > 1e-2 * np.sqrt(np.mean(got ** 2)), mistake


# --------------------------------------------------------------------------- attention block


def _bf_attention_block(u, sub, cfg, k_pool, v_pool, page_row, ctx_len, mistake=None):
    """k_pool/v_pool: nested lists [page][slot][Hkv][dh] of floats."""
    k = len(u)
    Hq, Hkv, dh, ps = cfg["Hq"], cfg["Hkv"], cfg["dh"], cfg["page_size"]
    rep = Hq // Hkv
    theta, eps, W = cfg["rope_theta"], cfg["rms_eps"], cfg["window"]
    wqkv, wo = _lists(sub["wqkv"]), _lists(sub["wo"])
    qn, kn = _lists(sub["q_norm"]), _lists(sub["k_norm"])
    off = 1 if mistake == "pos_plus_one" else 0
    q = [[None] * Hq for _ in range(k)]
    kb = [[None] * Hkv for _ in range(k)]
    vb = [[None] * Hkv for _ in range(k)]
    for i in range(k):
        qkv = [_dot(u[i], row) for row in wqkv]
        for h in range(Hq):
            v = qkv[h * dh:(h + 1) * dh]
            if mistake == "norm_after_rope":
                v = _rmsnorm(_rotate(v, ctx_len + i, theta), qn, eps) if cfg["qk_norm"] else v
            else:
                v = _rmsnorm(v, qn, eps) if cfg["qk_norm"] else v
                v = _rotate(v, ctx_len + i + off, theta)
            q[i][h] = v
        for h in range(Hkv):
            base_k = Hq * dh + h * dh
            base_v = (Hq + Hkv) * dh + h * dh
            if mistake == "v_before_k":
                base_k, base_v = base_v, base_k
            v = qkv[base_k:base_k + dh]
            if mistake == "norm_after_rope":
                v = _rmsnorm(_rotate(v, ctx_len + i, theta), kn, eps) if cfg["qk_norm"] else v
            else:
                v = _rmsnorm(v, kn, eps) if cfg["qk_norm"] else v
                v = _rotate(v, ctx_len + i + off, theta)
            kb[i][h] = v
            vb[i][h] = qkv[base_v:base_v + dh]
    out = []
    for i in range(k):
        o_row = []
        pos_q = ctx_len + i
        for hq in range(Hq):
            h = hq // rep if mistake != "head_interleave" else hq % Hkv
            keys, vals = [], []
            for p in range(ctx_len):
                if W > 0 and not (0 <= pos_q - p < W):
                    continue
                pg = int(page_row[p // ps])
                keys.append(k_pool[pg][p % ps][h])          # as stored: no rotation applied here
                vals.append(v_pool[pg][p % ps][h])
            for j in range(i + 1):
                if W > 0 and not (0 <= pos_q - (ctx_len + j) < W):
                    continue
                keys.append(kb[j][h])
                vals.append(vb[j][h])
            s = [_dot(q[i][hq], key) / math.sqrt(dh) for key in keys]
            m = max(s)
            e = [math.exp(x - m) for x in s]
            tot = sum(e)
            o = [0.0] * dh
            for pw, val in zip(e, vals):
                for d in range(dh):
                    o[d] += pw / tot * val[d]
            o_row.extend(o)
        out.append([_dot(o_row, wo[d]) for d in range(len(wo))])
    return out, q, kb


@pytest.mark.parametrize("ctx,window,Hkv,qk_norm", [(21, 0, 2, 1), (0, 0, 2, 1), (37, 7, 1, 1), (16, 0, 4, 0),
                                                    (19, 3, 2, 1)])
def test_attention_block_matches_scalar_loops(ctx, window, Hkv, qk_norm):
    cfg, w, batch = _setup([ctx], window=window, Hkv=Hkv, qk_norm=qk_norm)
    sub = _sub(w, 1, "attn")
    rng = np.random.default_rng(11)
    u = rng.standard_normal((4, cfg["D"]))
    kp, vp = to_np(batch["k_pools"][1]), to_np(batch["v_pools"][1])
    page_row = to_np(batch["page_table"])[0]
    want = {}
    got = O.attention_block(u, sub, cfg, kp, vp, page_row, ctx, want=want)
    ref, q_ref, kb_ref = _bf_attention_block(u.tolist(), sub, cfg, _lists(kp), _lists(vp), page_row, ctx)
    # the oracle rounds inverse frequency and angle to float32 (its stated recipe); the brute force keeps float64
    np.testing.assert_allclose(got, np.array(ref), rtol=1e-5, atol=1e-6 * max(1, ctx))
    # the rotated q and block keys themselves: position of row i is ctx + i, norm first.  The oracle rounds the
    # inverse frequency and the angle to float32 (its stated recipe), so these agree to ~1e-6 of a radian * pos.
    np.testing.assert_allclose(want["q"], np.array(q_ref), atol=2e-5 * max(1, ctx))
    np.testing.assert_allclose(want["kb"], np.array(kb_ref), atol=2e-5 * max(1, ctx))


def test_attention_block_pin_is_sensitive_to_each_layout_mistake():
    ctx = 21
    cfg, w, batch = _setup([ctx])
    sub = _sub(w, 1, "attn")
    # norm gains far from one, so that norm-then-rotate and rotate-then-norm differ visibly
    g = np.linspace(0.3, 2.0, cfg["dh"]).astype(np.float32)
    sub = dict(sub, q_norm=g, k_norm=g[::-1].copy())
    rng = np.random.default_rng(12)
    u = rng.standard_normal((4, cfg["D"]))
    kp, vp = to_np(batch["k_pools"][1]), to_np(batch["v_pools"][1])
    page_row = to_np(batch["page_table"])[0]
    got = O.attention_block(u, sub, cfg, kp, vp, page_row, ctx)
    ok, _, _ = _bf_attention_block(u.tolist(), sub, cfg, _lists(kp), _lists(vp), page_row, ctx)
    np.testing.assert_allclose(got, np.array(ok), rtol=1e-5, atol=1e-5)
    rms = np.sqrt(np.mean(got ** 2))
    for mistake in ("pos_plus_one", "norm_after_rope", "v_before_k", "head_interleave"):
        bad, _, _ = _bf_attention_block(u.tolist(), sub, cfg, _lists(kp), _lists(vp), page_row, ctx, mistake)
        assert np.max(np.abs(np.array(bad) - got)) > 1e-2 * rms, mistake


def test_block_row_i_is_rotated_at_ctx_plus_i_with_explicit_angles():
    """q.l / kb.l kept by the whole step equal the normed projections rotated by explicit cos/sin of
    (ctx + i) * theta^(-2j/dh) (Sec. 3.3.2: the block continues the prefix's positions)."""
    ctx = 40
    cfg, w, batch = _setup([ctx])
    out = O.draft_block(cfg, w, [to_np(t) for t in batch["k_pools"]], [to_np(t) for t in batch["v_pools"]],
                        to_np(batch["page_table"]), batch["ctx_lens_host"], to_np(batch["last_hidden"]),
                        to_np(batch["last_token"]), 3, keep_intermediates=True)
    inter = out["intermediates"][0]
    l = 0
    sub = _sub(w, l, "attn")
    X = inter[f"x_after_mamba.{l}"]
    g_attn = _lists(w[f"layers.{l}.attn.norm"])
    wqkv = _lists(sub["wqkv"])
    qn, kn = _lists(sub["q_norm"]), _lists(sub["k_norm"])
    dh, Hq, half = cfg["dh"], cfg["Hq"], cfg["dh"] // 2
    for i in range(3):
        un = _rmsnorm(X[i].tolist(), g_attn, cfg["rms_eps"])
        qkv = [_dot(un, row) for row in wqkv]
        for (name, head, base, gain) in (("q", 3, 3 * dh, qn), ("kb", 1, Hq * dh + dh, kn)):
            v = _rmsnorm(qkv[base:base + dh], gain, cfg["rms_eps"])
            for j in range(half):
                ang = (ctx + i) * cfg["rope_theta"] ** (-2.0 * j / dh)
                lo = v[j] * math.cos(ang) - v[j + half] * math.sin(ang)
                hi = v[j + half] * math.cos(ang) + v[j] * math.sin(ang)
                assert inter[f"{name}.{l}"][i, head, j] == pytest.approx(lo, abs=1e-4)
                assert inter[f"{name}.{l}"][i, head, j + half] == pytest.approx(hi, abs=1e-4)
                # ... and NOT at ctx + i + 1 or at i alone (first frequency: one radian per position)
                if j == 0:
                    for wrong in (ctx + i + 1, i):
                        lo_w = v[0] * math.cos(wrong) - v[half] * math.sin(wrong)
                        assert abs(inter[f"{name}.{l}"][i, head, 0] - lo_w) > 1e-3


# --------------------------------------------------------------------------- Mamba mixer


def _bf_mamba(u, S_init, sub, cfg, mistake=None):
    k = len(u)
    Di, H, P, N, G, dc = cfg["Di"], cfg["H"], cfg["P"], cfg["N"], cfg["G"], cfg["d_conv"]
    d_xBC = Di + 2 * G * N
    in_proj, out_proj = _lists(sub["in_proj"]), _lists(sub["out_proj"])
    conv_w, conv_b = _lists(sub["conv_w"]), _lists(sub["conv_b"])
    dt_bias, A_log, Dskip, gn = _lists(sub["dt_bias"]), _lists(sub["A_log"]), _lists(sub["Dskip"]), _lists(sub["gnorm"])
    proj = _linear(u, in_proj)
    if mistake == "xBC_first":          # rows read as xBC | z | dt
        z = [row[d_xBC:d_xBC + Di] for row in proj]
        raw = [row[:d_xBC] for row in proj]
    else:                               # rows are z | xBC | dt
        z = [row[:Di] for row in proj]
        raw = [row[Di:Di + d_xBC] for row in proj]
    dt_raw = [row[Di + d_xBC:] for row in proj]
    if cfg["dt_rank"] > 0:
        dt_raw = _linear(dt_raw, _lists(sub["dt_up"]))
    xBC = [[0.0] * d_xBC for _ in range(k)]
    for i in range(k):
        for c in range(d_xBC):
            acc = conv_b[c]
            for j in range(dc):
                src = i - (dc - 1) + j          # last tap multiplies the current row; rows before the block are zero
                if src >= 0:
                    acc += conv_w[c][j] * raw[src][c]
            xBC[i][c] = _silu(acc)
    S = [[[S_init[h][p][n] for n in range(N)] for p in range(P)] for h in range(H)]
    y = [[0.0] * Di for _ in range(k)]
    for i in range(k):
        for h in range(H):
            g = h // (H // G)
            v = dt_raw[i][h] + dt_bias[h]
            dt = v if v > 20.0 else math.log1p(math.exp(v))
            a = math.exp(-dt * math.exp(A_log[h]))
            if mistake == "C_before_B":
                Bv = xBC[i][Di + G * N + g * N: Di + G * N + (g + 1) * N]
                Cv = xBC[i][Di + g * N: Di + (g + 1) * N]
            else:
                Bv = xBC[i][Di + g * N: Di + (g + 1) * N]
                Cv = xBC[i][Di + G * N + g * N: Di + G * N + (g + 1) * N]
            for p in range(P):
                xv = xBC[i][h * P + p]
                acc = 0.0
                for n in range(N):
                    prev = S[h][p][n]
                    if not (mistake == "no_decay_at_0" and i == 0):
                        prev = a * prev
                    S[h][p][n] = prev + dt * xv * Bv[n]
                    acc += S[h][p][n] * Cv[n]
                y[i][h * P + p] = acc + Dskip[h] * xv
    out = []
    for i in range(k):
        if mistake == "norm_then_gate":
            yn = [a_ * _silu(zz) for a_, zz in zip(_rmsnorm(y[i], gn, cfg["rms_eps"]), z[i])]
        elif mistake == "per_head_norm":
            yn = []
            for h in range(H):
                seg = [y[i][c] * _silu(z[i][c]) for c in range(h * P, (h + 1) * P)]
                yn.extend(_rmsnorm(seg, gn[h * P:(h + 1) * P], cfg["rms_eps"]))
        else:
            yn = _rmsnorm([yy * _silu(zz) for yy, zz in zip(y[i], z[i])], gn, cfg["rms_eps"])
        out.append([_dot(yn, out_proj[d]) for d in range(len(out_proj))])
    return out


@pytest.mark.parametrize("over", [dict(), dict(G=1), dict(dt_rank=2), dict(N=1, G=4)])
def test_mamba_mixer_matches_scalar_loops(over):
    cfg, w, _ = _setup([3], **over)
    sub = _sub(w, 0, "mamba")
    rng = np.random.default_rng(21)
    u = rng.standard_normal((5, cfg["D"]))
    S0 = rng.standard_normal((cfg["H"], cfg["P"], cfg["N"]))
    got = O.mamba_mixer(u, S0, sub, cfg)
    ref = _bf_mamba(u.tolist(), S0.tolist(), sub, cfg)
    np.testing.assert_allclose(got, np.array(ref), rtol=1e-9, atol=1e-11)


def test_mamba_mixer_pin_is_sensitive_to_each_layout_mistake():
    cfg, w, _ = _setup([3])
    sub = _sub(w, 0, "mamba")
    sub = dict(sub, gnorm=np.linspace(0.3, 2.0, cfg["Di"]).astype(np.float32))
    rng = np.random.default_rng(22)
    u = rng.standard_normal((5, cfg["D"]))
    S0 = rng.standard_normal((cfg["H"], cfg["P"], cfg["N"]))
    got = O.mamba_mixer(u, S0, sub, cfg)
    rms = np.sqrt(np.mean(got ** 2))
    np.testing.assert_allclose(got, np.array(_bf_mamba(u.tolist(), S0.tolist(), sub, cfg)), rtol=1e-9, atol=1e-11)
    for mistake in ("xBC_first", "C_before_B", "no_decay_at_0", "norm_then_gate", "per_head_norm"):
        bad = np.array(_bf_mamba(u.tolist(), S0.tolist(), sub, cfg, mistake))
        assert np.max(np.abs(bad - got)) > 1e-2 * rms, mistake


# --------------------------------------------------------------------------- composition of the step


def _bf_step(cfg, w, batch, b, k, mistake=None):
    D, eps = cfg["D"], cfg["rms_eps"]
    h = _lists(to_np(batch["last_hidden"])[b])
    f = [_dot(h, row) for row in _lists(w["proj_r"])]                 # nothing between the two projections
    s = [_dot(f, row) for row in _lists(w["proj_ds"])]
    H, P, N = cfg["H"], cfg["P"], cfg["N"]
    S_init = [[[s[(hh * P + p) * N + n] for n in range(N)] for p in range(P)] for hh in range(H)]
    embed = _lists(w["embed"])
    X = [list(embed[int(batch["last_token"][b])])] + [list(embed[cfg["mask_id"]]) for _ in range(k - 1)]
    ctx = int(batch["ctx_lens_host"][b])
    page_row = to_np(batch["page_table"])[b]

    def add(X, delta):
        return [[x + d for x, d in zip(xr, dr)] for xr, dr in zip(X, delta)]

    def normed(X, gain):
        g = _lists(gain)
        return [_rmsnorm(row, g, eps) for row in X]

    for l in range(cfg["L"]):
        blocks = ["mamba", "attn", "mlp"] if mistake != "attn_first" else ["attn", "mamba", "mlp"]
        for blk in blocks:
            if blk == "attn" and not cfg["has_attn"][l]:
                continue
            u = normed(X, w[f"layers.{l}.{blk}.norm"]) if mistake != "post_norm" else X
            if blk == "mamba":
                delta = _bf_mamba(u, S_init, _sub(w, l, "mamba"), cfg)
            elif blk == "attn":
                slot = cfg["kv_slot"][l]
                delta, _, _ = _bf_attention_block(u, _sub(w, l, "attn"), cfg,
                                                  _lists(to_np(batch["k_pools"][slot])),
                                                  _lists(to_np(batch["v_pools"][slot])), page_row, ctx)
            else:
                delta = _bf_mlp(u, _lists(w[f"layers.{l}.mlp.w_gate_up"]), _lists(w[f"layers.{l}.mlp.w_down"]))
            if mistake == "post_norm":
                delta = normed(delta, w[f"layers.{l}.{blk}.norm"])
            X = add(X, delta)
    xf = normed(X, w["final_norm"])
    logits = _linear(xf, _lists(w["lm_head"]))
    ids = []
    for row in logits:
        best = 0
        for v in range(1, len(row)):
            if row[v] > row[best]:
                best = v
        ids.append(best)
    return X, logits, ids


@pytest.mark.parametrize("ctxs,over", [([21, 0], dict()), ([33], dict(has_attn=[1, 0], kv_slot=[0, -1], n_slots=1)),
                                       ([18], dict(window=6, dt_rank=2))])
def test_draft_block_composition_matches_scalar_loops(ctxs, over):
    cfg, w, batch = _setup(ctxs, **over)
    k = 4
    out = O.draft_block(cfg, w, [to_np(t) for t in batch["k_pools"]], [to_np(t) for t in batch["v_pools"]],
                        to_np(batch["page_table"]), batch["ctx_lens_host"], to_np(batch["last_hidden"]),
                        to_np(batch["last_token"]), k)
    for b in range(len(ctxs)):
        X, logits, ids = _bf_step(cfg, w, batch, b, k)
        # the oracle's float32 angle recipe is the only intended difference: ~1e-6 relative on rotated values
        np.testing.assert_allclose(out["hidden"][b], np.array(X), rtol=1e-4, atol=1e-4)
        np.testing.assert_allclose(out["logits"][b], np.array(logits), rtol=1e-4, atol=1e-4)
        sure = out["margin"][b] > 1e-3
        assert np.array_equal(out["draft_ids"][b][sure], np.array(ids)[sure])


def test_composition_pin_is_sensitive_to_block_order_and_norm_placement():
    cfg, w, batch = _setup([21])
    k = 4
    out = O.draft_block(cfg, w, [to_np(t) for t in batch["k_pools"]], [to_np(t) for t in batch["v_pools"]],
                        to_np(batch["page_table"]), batch["ctx_lens_host"], to_np(batch["last_hidden"]),
                        to_np(batch["last_token"]), k)
    rms = np.sqrt(np.mean(out["hidden"][0] ** 2))
    for mistake in ("attn_first", "post_norm"):
        X, _, _ = _bf_step(cfg, w, batch, 0, k, mistake)
        assert np.max(np.abs(np.array(X) - out["hidden"][0])) > 1e-2 * rms, mistake
