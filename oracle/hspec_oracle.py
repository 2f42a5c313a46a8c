"""CPU oracle for the H-Spec block-parallel draft step.  TEST INFRASTRUCTURE ONLY.

A plain, slow, obviously-correct numpy restatement of what one drafter forward
pass computes (paper Sec. 3.3 and App. B.1), written from the definitions:
no blocking, no fusion, no reordering.  It shares no code with the CUDA
library and must never be imported by the product path; only the tests, the
smoke check and the benchmark's CPU-baseline leg call it.

Arithmetic: `dtype` (float64 by default; float32 for the full-size workloads,
where a float64 copy of the weights would not fit in host memory).  Storage
values arrive already rounded to what the GPU stores (bf16 for matrices, KV
and the last hidden state); nothing is rounded in between.

What pins each function (tests/test_oracle_*.py):
  gemm                  pure-Python triple loop
  rmsnorm/silu/softplus closed forms, limits, scale invariance
  conv_silu             pure-Python loops, zero left context
  scan_sequential       == scan_quadratic (two independent derivations), zero
                        initial state == plain recurrence, restart invariant,
                        superposition, geometric closed form, C = 0
  rope                  identity at position 0, norm, relative-position law
  attention_*           paged == contiguous, brute-force enumeration, two-part
                        online-softmax merge, mean-of-V, shift/permutation
                        invariance, window, NaN-poisoned slots
  argmax_margin         full sort, constructed ties
  kv_bytes_per_token    Table 1 of the paper (tests/golden/table1_kv_bytes.txt)
  mlp_block, attention_block, mamba_mixer
                        scalar index loops over nested lists that spell out the
                        documented layouts (gate | up; q | k | v, norm before the
                        rotation, row i at position ctx_len + i; z | xBC | dt,
                        x | B | C, gate then norm over all Di), each with planted
                        mistakes that must disagree
  draft_block           the same scalar loops composed into the whole step;
                        request independence, page-permutation invariance,
                        causal k-prefix property, ablation special cases.
                        The scalar loops pin the code to the layouts and the
                        order stated here.  That order itself (which sub-blocks,
                        pre-norm placement, Mamba-2 mixer internals) is a reading
                        of a paper that prints no worked forward pass:
                        **parity unpinned** with respect to the paper for the
                        composition.
"""
import numpy as np

from .accept_oracle import markov_head

# --------------------------------------------------------------------------- storage helpers


def widen(a, dtype=np.float64):
    """Return `a` as `dtype`.  uint16 arrays are bf16 bit patterns."""
    a = np.asarray(a)
    if a.dtype == np.uint16:
        return (a.astype(np.uint32) << 16).view(np.float32).astype(dtype, copy=False)
    return a.astype(dtype, copy=False)


# --------------------------------------------------------------------------- elementary ops


def gemm(x, W, dtype=np.float64, rows_per_piece=1 << 16):
    """y = x W^T for x [M, K], W [N, K] (every linear layer of the drafter is bias-free).

    W may be stored as bf16 bits; it is widened in pieces of whole output rows so
    a multi-GB matrix never needs a full-precision copy.  Every output element is
    still one full-length dot product.
    """
    x = widen(x, dtype)
    W = np.asarray(W)
    n_out = W.shape[0]
    y = np.empty(x.shape[:-1] + (n_out,), dtype=dtype)
    for lo in range(0, n_out, rows_per_piece):
        hi = min(n_out, lo + rows_per_piece)
        y[..., lo:hi] = x @ widen(W[lo:hi], dtype).T
    return y


def rmsnorm(v, w, eps):
    """RMSNorm(v; w) = v / sqrt(mean(v^2) + eps) * w over the last axis."""
    ms = np.mean(v * v, axis=-1, keepdims=True)
    return v / np.sqrt(ms + eps) * w


def silu(v):
    return v / (1.0 + np.exp(-v))


def softplus(v):
    """log(1 + exp(v)), taken as v itself for v > 20."""
    v = np.asarray(v)
    safe = np.minimum(v, 20.0)
    return np.where(v > 20.0, v, np.log1p(np.exp(safe)))


def conv_silu(raw, w, b):
    """Causal depthwise convolution over the block positions followed by SiLU.

    raw [k, C], w [C, d_conv], b [C].  out[i, c] = SiLU(b_c + sum_j w[c, j] *
    raw[i - (d_conv-1) + j, c]) with rows before the block taken as zero (only the
    SSM state is injected from the target context, Sec. 3.3.1).
    """
    k, C = raw.shape
    d_conv = w.shape[1]
    out = np.empty_like(raw)
    for i in range(k):
        acc = np.array(b, dtype=raw.dtype, copy=True)
        for j in range(d_conv):
            src = i - (d_conv - 1) + j
            if src >= 0:
                acc = acc + w[:, j] * raw[src]
        out[i] = silu(acc)
    return out


def discretise(dt_raw, dt_bias, A_log):
    """dt = softplus(dt_raw + dt_bias); a = exp(dt * A), A = -exp(A_log)  (per head)."""
    dt = softplus(dt_raw + dt_bias)
    a = np.exp(dt * (-np.exp(A_log)))
    return dt, a


# --------------------------------------------------------------------------- selective scan


def scan_sequential(S_init, x, Bm, Cm, dt, a, Dskip):
    """The recurrence of Sec. 3.3.1 taken one position at a time from the injected state.

    S_init [H, P, N]; x [k, H, P]; Bm, Cm [k, G, N]; dt, a [k, H]; Dskip [H].
    S_i = a_i S_{i-1} + (dt_i x_i) (outer) B_i   with S_{-1} = S_init,
    y_i = S_i C_i + Dskip x_i.  Head h reads group h // (H / G).
    Returns y [k, H, P] and the final state.
    """
    k, H, P = x.shape
    G = Bm.shape[1]
    hpg = H // G
    S = np.array(S_init, dtype=x.dtype, copy=True)
    y = np.empty_like(x)
    for i in range(k):
        for h in range(H):
            g = h // hpg
            S[h] = a[i, h] * S[h] + (dt[i, h] * x[i, h])[:, None] * Bm[i, g][None, :]
            y[i, h] = S[h] @ Cm[i, g] + Dskip[h] * x[i, h]
    return y, S


def scan_quadratic(S_init, x, Bm, Cm, dt, a, Dskip):
    """The same map written as the unrolled sum (the 'dual' form of the linear recurrence):

    y_t = sum_{s<=t} (prod_{s<r<=t} a_r) dt_s (C_t . B_s) x_s
          + (prod_{r<=t} a_r) S_init C_t + Dskip x_t.
    Products of the decays are formed directly, not through logs.
    """
    k, H, P = x.shape
    G = Bm.shape[1]
    hpg = H // G
    y = np.zeros_like(x)
    for h in range(H):
        g = h // hpg
        for t in range(k):
            acc = Dskip[h] * x[t, h]
            decay0 = 1.0
            for r in range(t + 1):
                decay0 = decay0 * a[r, h]
            acc = acc + decay0 * (S_init[h] @ Cm[t, g])
            for s in range(t + 1):
                decay = 1.0
                for r in range(s + 1, t + 1):
                    decay = decay * a[r, h]
                acc = acc + decay * dt[s, h] * np.dot(Cm[t, g], Bm[s, g]) * x[s, h]
            y[t, h] = acc
    return y


# --------------------------------------------------------------------------- attention


def rope(v, pos, theta):
    """Rotate-half RoPE of v [..., dh] at integer position `pos` (Sec. 3.3.2: the block
    continues the target prefix's positions with the target's theta).

    Pairs (j, j + dh/2).  The inverse frequencies are formed in float64 and rounded to
    float32; the angle is ONE float32 product float32(pos) * inv_freq; cos/sin of that
    float32 angle are then taken accurately.  (This fixes the rounding recipe: at
    positions near 32768 a float32 angle carries ~4e-3 rad of rounding.)
    """
    dh = v.shape[-1]
    half = dh // 2
    j = np.arange(half, dtype=np.float64)
    inv_freq = (float(theta) ** (-2.0 * j / dh)).astype(np.float32)
    ang = (np.float32(pos) * inv_freq).astype(np.float64)
    c, s = np.cos(ang).astype(v.dtype), np.sin(ang).astype(v.dtype)
    v1, v2 = v[..., :half], v[..., half:]
    return np.concatenate([v1 * c - v2 * s, v2 * c + v1 * s], axis=-1)


def gather_kv(pool, page_row, ctx_len):
    """Contiguous copy [ctx_len, Hkv, dh] of one request's prefix from a paged pool
    [num_pages, page, Hkv, dh]: token p lives at pool[page_row[p // page], p % page].
    Pure data movement: the storage dtype is preserved."""
    pool = np.asarray(pool)
    page = pool.shape[1]
    out = np.empty((ctx_len,) + pool.shape[2:], dtype=pool.dtype)
    for p in range(ctx_len):
        out[p] = pool[int(page_row[p // page]), p % page]
    return out


def attention_contiguous(q, Kp, Vp, kb, vb, window=0, scale=None, dtype=np.float64):
    """Block-query GQA attention over a contiguous target prefix plus the block itself.

    q [k, Hq, dh] (already normed + rotated); Kp, Vp [ctx, Hkv, dh] as stored by the target
    (keys already rotated); kb, vb [k, Hkv, dh] the block's own keys (rotated) and values.
    Row i sits at position ctx + i and sees prefix positions p < ctx and block rows j <= i;
    with window W > 0 only keys with 0 <= pos_q - pos_k < W.  One softmax over the union,
    scale 1/sqrt(dh), query head hq reads KV head hq // (Hq / Hkv).  Masked keys are
    excluded by SELECTION, so garbage (NaN) in invisible slots cannot leak.
    """
    k, Hq, dh = q.shape
    ctx = Kp.shape[0]
    Hkv = kb.shape[1]
    rep = Hq // Hkv
    scale = 1.0 / np.sqrt(dh) if scale is None else scale
    o = np.empty((k, Hq, dh), dtype=dtype)
    for h in range(Hkv):
        Kh, Vh = widen(Kp[:, h], dtype), widen(Vp[:, h], dtype)
        kbh, vbh = widen(kb[:, h], dtype), widen(vb[:, h], dtype)
        for i in range(k):
            pos_q = ctx + i
            lo = 0 if window <= 0 else max(0, pos_q - window + 1)   # first visible position
            p_lo = min(lo, ctx)                                      # first visible prefix key
            j_lo = max(0, lo - ctx)                                  # first visible block key
            n_pre = ctx - p_lo
            for hq in range(h * rep, (h + 1) * rep):
                qv = widen(q[i, hq], dtype)
                # scores over the union: visible prefix keys, then visible block keys j <= i
                s = np.concatenate([Kh[p_lo:] @ qv, kbh[j_lo:i + 1] @ qv]) * scale
                e = np.exp(s - np.max(s))
                p = (e / np.sum(e.astype(np.float64))).astype(dtype)
                o[i, hq] = p[:n_pre] @ Vh[p_lo:] + p[n_pre:] @ vbh[j_lo:i + 1]
    return o


def attention_paged(q, k_pool, v_pool, page_row, ctx_len, kb, vb, window=0, scale=None, dtype=np.float64):
    """Same as attention_contiguous with the prefix read in place from the target's paged
    pools through the request's page-table row (Sec. 3.3.2, in-place target-KV reuse)."""
    Kp = gather_kv(k_pool, page_row, ctx_len)
    Vp = gather_kv(v_pool, page_row, ctx_len)
    return attention_contiguous(q, Kp, Vp, kb, vb, window=window, scale=scale, dtype=dtype)


# --------------------------------------------------------------------------- heads


def argmax_margin(logits):
    """Per row: lowest index attaining the maximum, and the gap to the runner-up value."""
    logits = np.asarray(logits)
    ids = np.empty(logits.shape[0], dtype=np.int32)
    margin = np.empty(logits.shape[0], dtype=logits.dtype)
    for i in range(logits.shape[0]):
        row = logits[i]
        top = np.max(row)
        idx = int(np.nonzero(row == top)[0][0])
        ids[i] = idx
        rest = np.delete(row, idx)
        margin[i] = top - np.max(rest) if rest.size else np.inf
    return ids, margin


def kv_bytes_per_token(n_layers, n_kv_heads, head_dim, bytes_per_elem=2):
    """Bytes of K and V one token adds to a cache of n_layers attention layers (Table 1)."""
    return 2 * n_layers * n_kv_heads * head_dim * bytes_per_elem


def drafter_kv_bytes_avoided(ctx_lens, n_layers, n_kv_heads, head_dim, bytes_per_elem=2):
    """Bytes a drafter-side KV cache holding every context token would occupy; the method
    keeps none (Sec. 3.2), so this is what in-place reuse saves."""
    return int(sum(ctx_lens)) * kv_bytes_per_token(n_layers, n_kv_heads, head_dim, bytes_per_elem)


# --------------------------------------------------------------------------- sub-blocks


def state_init(h, W_r, W_dS, H, P, N, dtype=np.float64):
    """S_init = reshape(Proj_dS(Proj_r(concat h)), [H, P, N])  (Sec. 3.3.1, App. B.1).
    Two bias-free linear maps with nothing in between; h [n_fuse * D]."""
    f = gemm(widen(h, dtype)[None, :], W_r, dtype)
    s = gemm(f, W_dS, dtype)[0]
    return s.reshape(H, P, N), f[0]


def mamba_mixer(u, S_init, w, cfg, dtype=np.float64, scan=scan_sequential):
    """Mamba-2 mixer over the k block rows u [k, D], started from the injected state.

    in_proj rows are z | xBC | dt; xBC = x [H, P] | B [G, N] | C [G, N] after conv + SiLU;
    gated RMSNorm over the full inner width; bias-free out projection.
    """
    k = u.shape[0]
    Di, H, P, N, G = cfg["Di"], cfg["H"], cfg["P"], cfg["N"], cfg["G"]
    proj = gemm(u, w["in_proj"], dtype)
    z = proj[:, :Di]
    raw = proj[:, Di:Di + cfg["d_xBC"]]
    dt_raw = proj[:, Di + cfg["d_xBC"]:]
    if cfg["dt_rank"] > 0:
        dt_raw = gemm(dt_raw, w["dt_up"], dtype)
    xBC = conv_silu(raw, widen(w["conv_w"], dtype), widen(w["conv_b"], dtype))
    x = xBC[:, :Di].reshape(k, H, P)
    Bm = xBC[:, Di:Di + G * N].reshape(k, G, N)
    Cm = xBC[:, Di + G * N:].reshape(k, G, N)
    dt, a = discretise(dt_raw, widen(w["dt_bias"], dtype), widen(w["A_log"], dtype))
    out = scan(S_init, x, Bm, Cm, dt, a, widen(w["Dskip"], dtype))
    y = out[0] if isinstance(out, tuple) else out
    gated = y.reshape(k, Di) * silu(z)
    yn = rmsnorm(gated, widen(w["gnorm"], dtype), cfg["rms_eps"])
    return gemm(yn, w["out_proj"], dtype)


def attention_block(u, w, cfg, k_pool, v_pool, page_row, ctx_len, dtype=np.float64, want=None):
    """Attention sub-block on the normed rows u [k, D]: q/k/v projections, per-head RMSNorm
    of q and the block's k, RoPE at positions ctx_len + i, attention over the target's
    pages (as stored) plus the causal block, output projection."""
    k = u.shape[0]
    Hq, Hkv, dh = cfg["Hq"], cfg["Hkv"], cfg["dh"]
    qkv = gemm(u, w["wqkv"], dtype)
    q = qkv[:, :Hq * dh].reshape(k, Hq, dh)
    kb = qkv[:, Hq * dh:(Hq + Hkv) * dh].reshape(k, Hkv, dh)
    vb = qkv[:, (Hq + Hkv) * dh:].reshape(k, Hkv, dh)
    if cfg["qk_norm"]:
        q = rmsnorm(q, widen(w["q_norm"], dtype), cfg["rms_eps"])
        kb = rmsnorm(kb, widen(w["k_norm"], dtype), cfg["rms_eps"])
    q = np.stack([rope(q[i], ctx_len + i, cfg["rope_theta"]) for i in range(k)])
    kb = np.stack([rope(kb[i], ctx_len + i, cfg["rope_theta"]) for i in range(k)])
    o = attention_paged(q, k_pool, v_pool, page_row, ctx_len, kb, vb, window=cfg["window"], dtype=dtype)
    if want is not None:
        want["q"], want["kb"], want["vb"], want["attn_o"] = q, kb, vb, o
    return gemm(o.reshape(k, Hq * dh), w["wo"], dtype)


def mlp_block(u, w, dtype=np.float64):
    """SwiGLU MLP: (SiLU(u Wg^T) * (u Wu^T)) Wd^T; w_gate_up rows are gate | up."""
    gu = gemm(u, w["w_gate_up"], dtype)
    F = gu.shape[1] // 2
    return gemm(silu(gu[:, :F]) * gu[:, F:], w["w_down"], dtype)


# --------------------------------------------------------------------------- the whole step


def draft_block(cfg, weights, k_pools, v_pools, page_table, ctx_lens, last_hidden, last_token, k,
                dtype=np.float64, requests=None, keep_intermediates=False, scan=scan_sequential):
    """One block-parallel draft step for the chosen requests (default: all).

    Per request b (requests are independent):
      S_init from the last-position hidden state (computed once, shared by all layers);
      block rows X[0] = E[last_token], X[i>0] = E[mask] (no positional embedding);
      for each layer: X += Mamba(RMSNorm(X)); X += Attn(RMSNorm(X)) if the layer has
      attention (target KV of slot kv_slot[l]); X += MLP(RMSNorm(X));
      logits = RMSNorm(X) W_lm^T; draft ids = argmax (lowest index on ties), translated through
      `vocab_map` when the drafter predicts over a pruned vocabulary (the LM head then holds only those rows).
      When `markov_in` / `markov_out` are among the weights the logits first go through the causal-correction
      head (accept_oracle.markov_head), and `logits` / `margin` are the corrected ones.
    Returns dict: draft_ids [n, k], logits [n, k, V], hidden [n, k, D], margin [n, k],
    s_init [n, H, P, N] and, if asked, per-request intermediates.
    """
    B = len(ctx_lens)
    requests = list(range(B)) if requests is None else list(requests)
    D = cfg["D"]
    V = int(np.asarray(weights["lm_head"]).shape[0])      # the target vocabulary, or a pruned drafter vocabulary
    eps = cfg["rms_eps"]
    out = dict(draft_ids=np.empty((len(requests), k), np.int32),
               logits=np.empty((len(requests), k, V), dtype),
               hidden=np.empty((len(requests), k, D), dtype),
               margin=np.empty((len(requests), k), dtype),
               s_init=np.empty((len(requests), cfg["H"], cfg["P"], cfg["N"]), dtype),
               intermediates=[])
    for n, b in enumerate(requests):
        inter = {}
        S_init, f = state_init(last_hidden[b], weights["proj_r"], weights["proj_ds"],
                               cfg["H"], cfg["P"], cfg["N"], dtype)
        X = np.empty((k, D), dtype)
        X[0] = widen(np.asarray(weights["embed"])[int(last_token[b])], dtype)
        for i in range(1, k):
            X[i] = widen(np.asarray(weights["embed"])[cfg["mask_id"]], dtype)
        for l in range(cfg["L"]):
            X = X + mamba_mixer(rmsnorm(X, widen(weights[f"layers.{l}.mamba.norm"], dtype), eps),
                                S_init, _sub(weights, l, "mamba"), cfg, dtype, scan)
            if keep_intermediates:
                inter[f"x_after_mamba.{l}"] = X.copy()
            if cfg["has_attn"][l]:
                slot = cfg["kv_slot"][l]
                want = {} if keep_intermediates else None
                X = X + attention_block(rmsnorm(X, widen(weights[f"layers.{l}.attn.norm"], dtype), eps),
                                        _sub(weights, l, "attn"), cfg, k_pools[slot], v_pools[slot],
                                        page_table[b], int(ctx_lens[b]), dtype, want)
                if keep_intermediates:
                    inter[f"x_after_attn.{l}"] = X.copy()
                    for kk, vv in want.items():
                        inter[f"{kk}.{l}"] = vv
            X = X + mlp_block(rmsnorm(X, widen(weights[f"layers.{l}.mlp.norm"], dtype), eps),
                              _sub(weights, l, "mlp"), dtype)
            if keep_intermediates:
                inter[f"x_after_mlp.{l}"] = X.copy()
        logits = gemm(rmsnorm(X, widen(weights["final_norm"], dtype), eps), weights["lm_head"], dtype)
        if "markov_in" in weights:        # causal correction after the backbone (Sec. 3.3.3): sequential over positions
            ids, logits, margin = markov_head(logits[None], weights["markov_in"], weights["markov_out"],
                                              [int(last_token[b])], id_map=weights.get("vocab_map"), dtype=dtype)
            ids, logits, margin = ids[0], logits[0], margin[0]
        else:
            ids, margin = argmax_margin(logits)
        if "vocab_map" in weights:        # pruned drafter vocabulary: LM-head row index -> target token id
            ids = np.asarray(weights["vocab_map"])[ids].astype(np.int32)
        out["draft_ids"][n], out["logits"][n], out["hidden"][n] = ids, logits, X
        out["margin"][n], out["s_init"][n] = margin, S_init
        out["intermediates"].append(inter)
    return out


def _sub(weights, l, block):
    """Tensors of one sub-block of layer l, keyed by their short names."""
    p = f"layers.{l}.{block}."
    return {name[len(p):]: t for name, t in weights.items() if name.startswith(p)}
