"""Seeded generators for weights, target KV pools, page tables and step inputs.

Everything is drawn with torch generators (CPU or CUDA) from seeds derived
from one base seed, rounded once to bf16 where the storage type is bf16, and
the SAME tensors are handed to the CUDA library and to the CPU oracle.  No
arithmetic of the method lives here.

Value recipe (weights ~ N(0, 0.02), K/V and last hidden ~ N(0, 1),
A = -exp(U[0, 2]), dt bias such that softplus(dt_bias) lies in [1e-3, 1e-1]):
  * every matrix (linear layers, embedding, LM head): N(0, 0.02), bf16
  * norm gains: 1 + N(0, 0.02), fp32
  * depthwise-conv taps U(-1/2, 1/2), conv bias N(0, 0.02), fp32
  * A_log ~ U[0, 2]; dt_bias = softplus^-1(exp(U[ln 1e-3, ln 1e-1])); D skip = 1
  * target K/V pools N(0, 1) bf16 (K is taken as already rotated);
    unused tail slots of the last page of a request can be NaN-poisoned
  * physical page ids: a random permutation over a pool sized to the sum of
    the requests' page counts
"""
import math
import zlib

import torch

BASE_SEED = 260924197


def tensor_seed(name, base=BASE_SEED):
    """Stable per-tensor seed: base + CRC32 of the tensor's name."""
    return (base + zlib.crc32(name.encode())) % (2 ** 63 - 1)


def _gen(device, seed):
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return g


def _normal(shape, std, name, device, dtype, mean=0.0):
    g = _gen(device, tensor_seed(name))
    n = 1
    for s in shape:
        n *= s
    # draw in fp32 in slabs so a multi-GB matrix never needs a full fp32 copy
    out = torch.empty(shape, dtype=dtype, device=device)
    flat = out.view(-1)
    slab = 1 << 26
    for lo in range(0, n, slab):
        hi = min(n, lo + slab)
        t = torch.randn(hi - lo, generator=g, device=device, dtype=torch.float32)
        flat[lo:hi] = (t * std + mean).to(dtype)
    return out


def _uniform(shape, lo, hi, name, device):
    g = _gen(device, tensor_seed(name))
    return torch.rand(shape, generator=g, device=device, dtype=torch.float32) * (hi - lo) + lo


def weight_shapes(cfg):
    """name -> (shape, kind) for every tensor of the drafter.

    kind: 'mat' (bf16 matrix), 'gain', 'conv_w', 'conv_b', 'A_log', 'dt_bias', 'Dskip'
    (all fp32 vectors).  Matrices are stored [out_features, in_features].
    """
    D, L = cfg["D"], cfg["L"]
    sh = {
        "embed": ((cfg["V"], D), "mat"),
        "proj_r": ((cfg["r"], cfg["n_fuse"] * D), "mat"),
        "proj_ds": ((cfg["d_S"], cfg["r"]), "mat"),
        "final_norm": ((D,), "gain"),
        "lm_head": ((cfg.get("V_draft", 0) or cfg["V"], D), "mat"),
    }
    if cfg.get("V_draft", 0):
        sh["vocab_map"] = ((cfg["V_draft"],), "vocab_map")   # drafter row -> target token id (pruned vocabulary)
    if cfg.get("markov_rank", 0):
        rm = cfg["markov_rank"]
        sh["markov_in"] = ((cfg["V"], rm), "markov")                                   # one row per previous token
        sh["markov_out"] = ((cfg.get("V_draft", 0) or cfg["V"], rm), "markov")         # one row per drafter-vocabulary row
    for l in range(L):
        p = f"layers.{l}."
        sh[p + "mamba.norm"] = ((D,), "gain")
        sh[p + "mamba.in_proj"] = ((cfg["d_in_proj"], D), "mat")   # rows: z | xBC | dt
        if cfg["dt_rank"] > 0:
            sh[p + "mamba.dt_up"] = ((cfg["H"], cfg["dt_rank"]), "mat")
        sh[p + "mamba.conv_w"] = ((cfg["d_xBC"], cfg["d_conv"]), "conv_w")
        sh[p + "mamba.conv_b"] = ((cfg["d_xBC"],), "conv_b")
        sh[p + "mamba.dt_bias"] = ((cfg["H"],), "dt_bias")
        sh[p + "mamba.A_log"] = ((cfg["H"],), "A_log")
        sh[p + "mamba.Dskip"] = ((cfg["H"],), "Dskip")
        sh[p + "mamba.gnorm"] = ((cfg["Di"],), "gain")
        sh[p + "mamba.out_proj"] = ((D, cfg["Di"]), "mat")
        if cfg["has_attn"][l]:
            sh[p + "attn.norm"] = ((D,), "gain")
            sh[p + "attn.wqkv"] = ((cfg["d_qkv"], D), "mat")        # rows: q | k | v
            sh[p + "attn.q_norm"] = ((cfg["dh"],), "gain")
            sh[p + "attn.k_norm"] = ((cfg["dh"],), "gain")
            sh[p + "attn.wo"] = ((D, cfg["Hq"] * cfg["dh"]), "mat")
        sh[p + "mlp.norm"] = ((D,), "gain")
        sh[p + "mlp.w_gate_up"] = ((2 * cfg["F"], D), "mat")       # rows: gate | up
        sh[p + "mlp.w_down"] = ((D, cfg["F"]), "mat")
    return sh


def make_weights(cfg, device="cpu", only=None):
    """All drafter tensors: dict name -> torch tensor (bf16 matrices, fp32 vectors)."""
    out = {}
    for name, (shape, kind) in weight_shapes(cfg).items():
        if only is not None and name not in only:
            continue
        if kind == "mat":
            t = _normal(shape, 0.02, name, device, torch.bfloat16)
        elif kind == "markov":
            # factor entries sized so that the rank-r table has entries of about half a logit
            t = _normal(shape, (0.25 / shape[1]) ** 0.25, name, device, torch.bfloat16)
        elif kind == "gain":
            t = _normal(shape, 0.02, name, device, torch.float32, mean=1.0)
        elif kind == "conv_w":
            t = _uniform(shape, -0.5, 0.5, name, device)
        elif kind == "conv_b":
            t = _normal(shape, 0.02, name, device, torch.float32)
        elif kind == "A_log":
            t = _uniform(shape, 0.0, 2.0, name, device)
        elif kind == "dt_bias":
            dt = torch.exp(_uniform(shape, math.log(1e-3), math.log(1e-1), name, device).double())
            t = (dt + torch.log(-torch.expm1(-dt))).float()      # inverse softplus
        elif kind == "vocab_map":
            # a seeded random subset of the target vocabulary, ascending (the real list is "most frequent tokens in
            # the training corpus", which is not available here)
            g = _gen("cpu", tensor_seed(name))
            t = torch.sort(torch.randperm(cfg["V"], generator=g)[:shape[0]])[0].to(torch.int32).to(device)
        elif kind == "Dskip":
            t = torch.ones(shape, dtype=torch.float32, device=device)
        else:
            raise ValueError(kind)
        out[name] = t
    return out


def make_ctx_lens(cfg, B=None, seed_offset=2):
    """Per-request context lengths (python ints) from the config's distribution."""
    B = cfg["B"] if B is None else B
    kind, lo, hi = cfg["ctx"]
    g = _gen("cpu", BASE_SEED + seed_offset)
    if kind == "const":
        return [int(lo)] * B
    u = torch.rand(B, generator=g, dtype=torch.float64)
    if kind == "uniform":
        v = torch.floor(lo + u * (hi - lo + 1))
    elif kind == "loguniform":
        v = torch.floor(torch.exp(math.log(lo) + u * (math.log(hi) - math.log(lo))))
    else:
        raise ValueError(kind)
    return [int(min(max(x, lo), hi)) for x in v.tolist()]


def make_request_batch(cfg, ctx_lens=None, device="cpu", poison_tail=False,
                       extra_pages=0, kv_std=1.0, seed_offset=0):
    """Step inputs and the target's paged KV cache for one batch of requests.

    Returns a dict with
      page_table [B, max_pages] int32 (entries past ceil(ctx/page) hold -1 and
        must never be read), ctx_lens [B] int32, last_hidden [B, n_fuse*D] bf16,
      last_token [B] int32, k_pools/v_pools: lists (one per KV slot) of
        [num_pages, page, Hkv, dh] bf16, num_pages, max_pages.
    """
    B = len(ctx_lens) if ctx_lens is not None else cfg["B"]
    if ctx_lens is None:
        ctx_lens = make_ctx_lens(cfg, B)
    ps = cfg["page_size"]
    n_pages_req = [(c + ps - 1) // ps for c in ctx_lens]
    num_pages = max(1, sum(n_pages_req) + extra_pages)
    max_pages = max(1, max(n_pages_req))
    g = _gen("cpu", BASE_SEED + 3 + seed_offset)
    perm = torch.randperm(num_pages, generator=g, dtype=torch.int64)
    page_table = torch.full((B, max_pages), -1, dtype=torch.int32)
    at = 0
    for b, n in enumerate(n_pages_req):
        page_table[b, :n] = perm[at:at + n].to(torch.int32)
        at += n
    k_pools, v_pools = [], []
    shape = (num_pages, ps, cfg["Hkv"], cfg["dh"])
    for s in range(cfg["n_slots"]):
        k_pools.append(_normal(shape, kv_std, f"kv.{s}.k.{seed_offset}", device, torch.bfloat16))
        v_pools.append(_normal(shape, kv_std, f"kv.{s}.v.{seed_offset}", device, torch.bfloat16))
    if poison_tail:
        for b, c in enumerate(ctx_lens):
            if c % ps:
                pg = int(page_table[b, n_pages_req[b] - 1])
                for s in range(cfg["n_slots"]):
                    k_pools[s][pg, c % ps:] = float("nan")
                    v_pools[s][pg, c % ps:] = float("nan")
        for s in range(cfg["n_slots"]):          # pages no request maps are garbage too
            for pg in perm[at:].tolist():
                k_pools[s][pg] = float("nan")
                v_pools[s][pg] = float("nan")
    last_hidden = _normal((B, cfg["n_fuse"] * cfg["D"]), 1.0, f"last_hidden.{seed_offset}",
                          device, torch.bfloat16)
    gt = _gen("cpu", BASE_SEED + 1 + seed_offset)
    last_token = torch.randint(0, cfg["V"], (B,), generator=gt, dtype=torch.int64).to(torch.int32)
    return dict(
        page_table=page_table.to(device), ctx_lens=torch.tensor(ctx_lens, dtype=torch.int32, device=device),
        ctx_lens_host=list(ctx_lens), last_hidden=last_hidden, last_token=last_token.to(device),
        k_pools=k_pools, v_pools=v_pools, num_pages=num_pages, max_pages=max_pages,
    )
