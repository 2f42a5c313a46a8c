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
