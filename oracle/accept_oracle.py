"""CPU oracle for the steps next to the draft block.  TEST INFRASTRUCTURE ONLY.

Plain numpy / Python restatements, written from the definitions; shares no code
with the CUDA library and is never imported by the product path.

  token_probs     softmax probability of one chosen token per row: the draft
                  probability P_D(t_i) that the acceptance rule of App. A divides by.
  accept_lengths  the acceptance rule of App. A: draft t_i is accepted if every
                  earlier draft was and min(1, P_T / P_D) >= alpha_i; returns how
                  many leading drafts are accepted (the iteration then emits that
                  many tokens plus one target token).  The uniforms alpha are an
                  input, so both sides of a parity test see the same draws.  The
                  comparison is taken in float32 (the kernel's precision) because
                  it decides an integer.
  markov_head     the causal correction of Sec. 3.3.3: a first-order dependency
                  between adjacent draft positions, applied to the logits, of rank
                  r_m (256 in App. B.1).  The paper names the mechanism and its
                  rank and prints no formula; the READING taken here is a low-rank
                  bigram table: logits'_i = logits_i + W_out (W_in[prev_i]), with
                  prev_0 the last verified token and prev_i the token chosen at
                  position i - 1 from the adjusted logits, positions strictly in
                  order.  **parity unpinned** with respect to the paper (no worked
                  example, no formula); the arithmetic of the reading itself is
                  pinned as listed below.

  kv_inject_rows  the comparison drafters' KV injection (Sec. 2.2 "KV injection in block
                  drafting"), kept as a measured counter-example to the bytes H-Spec avoids:
                  per new position, projected key rows get the per-head RMSNorm (optional)
                  and rotate-half RoPE at that position, value rows are taken as they are,
                  and both are written into a drafter-side paged KV cache (scatter_kv).
                  The projection in front of it is an ordinary bias-free linear map.

What pins each function (tests/test_oracle_accept.py):
  token_probs     rows sum to one over all tokens, uniform logits, shift
                  invariance, two-token closed form (logistic)
  accept_lengths  pure-Python loop, alpha = 0 accepts all, P_T >= P_D accepts all,
                  alpha above the first ratio rejects all, prefix property, the
                  expected accepted length of the closed form sum_j prod_{i<=j} r_i
                  by Monte Carlo
  markov_head     dense bigram table + Python loops on tiny sizes, W_out = 0 is the
                  plain arg-max, a constructed chain (table forces t -> t + 1), and
                  locality (a change at position j cannot alter positions < j)
  kv_inject_rows / scatter_kv
                  scatter then gather (hspec_oracle.gather_kv) returns the rows, rows not
                  addressed keep their bits, position 0 leaves keys unrotated, the norm of
                  a key row is preserved by the rotation, relative-position law
                  <RoPE(a, p), RoPE(b, p + d)> independent of p
"""
import numpy as np


def token_probs(logits, ids, dtype=np.float64):
    """p[m] = softmax(logits[m])[ids[m]] for logits [M, V], ids [M]."""
    z = np.asarray(logits).astype(dtype)
    ids = np.asarray(ids).astype(np.int64)
    zmax = z.max(axis=-1, keepdims=True)
    e = np.exp(z - zmax)
    return e[np.arange(z.shape[0]), ids] / e.sum(axis=-1)


def accept_lengths(p_target, p_draft, alpha):
    """App. A: n[b] = number of leading positions i with min(1, P_T/P_D) >= alpha, for arrays [B, k].

    All three arrays are taken as float32 and the ratio, the minimum and the comparison are float32
    operations (IEEE division), so a float32 kernel reaches the same integers.
    """
    pt = np.asarray(p_target, dtype=np.float32)
    pd = np.asarray(p_draft, dtype=np.float32)
    al = np.asarray(alpha, dtype=np.float32)
    with np.errstate(divide="ignore", invalid="ignore"):
        ratio = pt / pd                      # P_D = 0 with P_T > 0 gives +inf: accepted; 0 / 0 gives NaN: rejected
    ok = np.minimum(np.float32(1.0), ratio) >= al
    ok &= ~np.isnan(ratio)
    B, k = ok.shape
    n = np.zeros(B, dtype=np.int32)
    for b in range(B):
        i = 0
        while i < k and ok[b, i]:
            i += 1
        n[b] = i
    return n


def markov_head(logits, W_in, W_out, last_token, id_map=None, dtype=np.float64):
    """Sequential first-order correction of block logits (the reading stated in the module header).

    logits [B, k, Vd]; W_in [V, r] (one row per possible PREVIOUS token, target vocabulary);
    W_out [Vd, r] (one row per draft-vocabulary token); last_token [B] (target ids);
    id_map [Vd] maps a draft-vocabulary index to its target id (None: identity).
    Returns (ids [B, k] draft-vocabulary indices, adjusted logits [B, k, Vd], margin [B, k]
    = top-1 minus top-2 of the adjusted logits).  Ties go to the lowest index.
    """
    z = np.asarray(logits).astype(dtype)
    Wi = np.asarray(W_in)
    Wo = np.asarray(W_out)
    if Wi.dtype == np.uint16:
        Wi = (Wi.astype(np.uint32) << 16).view(np.float32)
    if Wo.dtype == np.uint16:
        Wo = (Wo.astype(np.uint32) << 16).view(np.float32)
    Wi = Wi.astype(dtype)
    Wo = Wo.astype(dtype)
    B, k, Vd = z.shape
    ids = np.zeros((B, k), dtype=np.int64)
    adj = np.empty_like(z)
    margin = np.empty((B, k), dtype=dtype)
    for b in range(B):
        prev = int(last_token[b])
        for i in range(k):
            row = z[b, i] + Wo @ Wi[prev]
            adj[b, i] = row
            t = int(np.argmax(row))              # numpy returns the first (lowest) index of the maximum
            ids[b, i] = t
            if Vd > 1:
                top2 = np.partition(row, Vd - 2)[Vd - 2:]
                margin[b, i] = top2[1] - top2[0]
            else:
                margin[b, i] = np.inf
            prev = t if id_map is None else int(id_map[t])
    return ids, adj, margin


def kv_inject_rows(kv, k_norm_w, pos, theta, eps=1e-6, k_norm=True, dtype=np.float64):
    """Key / value rows of T new positions as a KV-injecting drafter would cache them.

    kv [T, 2, Hkv, dh] (projected keys | values); k_norm_w [dh]; pos [T] absolute positions.
    Keys: optional per-head RMSNorm over dh, then rotate-half RoPE at pos (pairs (j, j + dh/2),
    inv_freq = theta^(-2j/dh) rounded to float32, angle = ONE float32 product float(pos) * inv_freq);
    values unchanged.  Returns (K [T, Hkv, dh], V [T, Hkv, dh]) in `dtype`.
    """
    kv = np.asarray(kv).astype(dtype)
    T, _, Hkv, dh = kv.shape
    half = dh // 2
    K = kv[:, 0].copy()
    V = kv[:, 1].copy()
    if k_norm:
        K = K / np.sqrt(np.mean(K * K, axis=-1, keepdims=True) + eps) * np.asarray(k_norm_w).astype(dtype)
    inv_freq = (np.float64(theta) ** (-2.0 * np.arange(half, dtype=np.float64) / dh)).astype(np.float32)
    out = np.empty_like(K)
    for t in range(T):
        ang = (np.float32(pos[t]) * inv_freq).astype(np.float32).astype(np.float64)
        cs, sn = np.cos(ang), np.sin(ang)
        a, b = K[t, :, :half], K[t, :, half:]
        out[t, :, :half] = a * cs - b * sn
        out[t, :, half:] = b * cs + a * sn
    return out, V


def scatter_kv(pool, page_row, pos, rows):
    """Inverse of a paged gather: pool[page_row[p // page], p % page] = rows[i] for p = pos[i].
    pool [num_pages, page, Hkv, dh] is modified in place; pure data movement."""
    page = pool.shape[1]
    for i, p in enumerate(pos):
        pool[int(page_row[int(p) // page]), int(p) % page] = rows[i]
    return pool
