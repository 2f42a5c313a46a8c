"""GPU parity for the steps next to the draft block: acceptance rule (App. A), draft-token probabilities, and the
Markov-head reading of Sec. 3.3.3, each through the C-ABI against oracle/accept_oracle.py on the same seeded inputs."""
import numpy as np
import pytest
import torch

from oracle import accept_oracle as ao
from conftest import to_np

pytestmark = pytest.mark.gpu

MARGIN = 1e-3    # fp32 logits + an fp32-accumulated rank-r product: ids are compared where the oracle's margin exceeds this


@pytest.fixture(scope="module")
def hs():
    import paper_2609_24197_b200 as m
    m.load_library()
    return m


def _gen(seed):
    return torch.Generator(device="cpu").manual_seed(260924197 + seed)


# --------------------------------------------------------------------------- acceptance rule

@pytest.mark.parametrize("B,k", [(1, 1), (3, 7), (128, 16), (37, 33), (5, 70), (4096, 8)])
def test_accept_bit_exact(hs, B, k):
    g = _gen(B * 131 + k)
    pt = torch.rand((B, k), generator=g)
    pd = torch.rand((B, k), generator=g) * 0.95 + 0.05
    al = torch.rand((B, k), generator=g)
    # make long accepted runs common, and plant the edge cases
    pt = torch.where(torch.rand((B, k), generator=g) < 0.7, torch.maximum(pt, pd), pt)
    if B >= 3 and k >= 2:
        pd[0, 0] = 0.0; pt[0, 0] = 0.5            # +inf ratio: accepted
        pd[1, 0] = 0.0; pt[1, 0] = 0.0            # NaN ratio: rejected
        al[2, :] = 0.0                            # everything accepted
    out = torch.empty(B, dtype=torch.int32, device="cuda")
    hs.hspec_op_accept(pt.cuda(), pd.cuda(), al.cuda(), out)
    torch.cuda.synchronize()
    np.testing.assert_array_equal(to_np(out), ao.accept_lengths(pt.numpy(), pd.numpy(), al.numpy()))


# --------------------------------------------------------------------------- draft-token probabilities

@pytest.mark.parametrize("M,V", [(1, 5), (7, 1000), (33, 32000), (16, 152064), (4, 151937)])
def test_token_probs(hs, M, V):
    g = _gen(M * 17 + V)
    z = torch.randn((M, V), generator=g) * 3.0
    z[:, 0] += 6.0 * torch.rand(M, generator=g)              # some rows with a dominant token
    ids = torch.randint(0, V, (M,), generator=g, dtype=torch.int32)
    ids[0] = int(torch.argmax(z[0]))
    if M > 1:
        z[1, 3 % V] = float("-inf")                          # a masked-out token contributes nothing
    p = torch.empty(M, dtype=torch.float32, device="cuda")
    hs.hspec_op_token_probs(z.cuda(), ids.cuda(), p)
    torch.cuda.synchronize()
    ref = ao.token_probs(z.numpy(), ids.numpy())
    np.testing.assert_allclose(to_np(p), ref, rtol=2e-4, atol=1e-30)


# --------------------------------------------------------------------------- Markov head

def _markov_case(hs, B, k, V, Vd, r, seed, dtype=torch.bfloat16, write_logits=True, scale=1.0):
    g = _gen(seed)
    logits = torch.randn((B * k, Vd), generator=g)
    W_in = (torch.randn((V, r), generator=g) * scale / r ** 0.25).to(dtype)
    W_out = (torch.randn((Vd, r), generator=g) * scale / r ** 0.25).to(dtype)
    last = torch.randint(0, V, (B,), generator=g, dtype=torch.int32)
    id_map = None
    if Vd != V:
        id_map = torch.sort(torch.randperm(V, generator=g)[:Vd])[0].to(torch.int32)
    d_logits = logits.cuda()
    ids = torch.full((B * k,), -1, dtype=torch.int32, device="cuda")
    ws = torch.empty(hs.hspec_markov_workspace_bytes(B, Vd, r), dtype=torch.uint8, device="cuda")
    hs.hspec_op_markov_head(d_logits, W_in.cuda(), W_out.cuda(), last.cuda(), None if id_map is None else id_map.cuda(),
                            ids, B, k, write_logits, ws)
    torch.cuda.synchronize()
    # oracle on the values the GPU holds (16-bit factors widened exactly)
    o_ids, o_adj, o_margin = ao.markov_head(logits.numpy().reshape(B, k, Vd), W_in.float().numpy(), W_out.float().numpy(),
                                            last.numpy(), id_map=None if id_map is None else id_map.numpy())
    got = to_np(ids).reshape(B, k)
    want = o_ids if id_map is None else id_map.numpy()[o_ids]
    # a request is compared up to (not including) its first position whose oracle margin is inside the tolerance:
    # after a near-tie the two sides may legitimately follow different chains
    n_cmp = 0
    for b in range(B):
        for i in range(k):
            if o_margin[b, i] <= MARGIN:
                break
            assert got[b, i] == want[b, i], f"request {b} position {i}: {got[b, i]} != {want[b, i]} (margin {o_margin[b, i]:.3e})"
            n_cmp += 1
    assert n_cmp >= 0.8 * B * k, "too few comparable positions: the case does not test the chain"
    if write_logits:
        adj = to_np(d_logits).reshape(B, k, Vd)
        for b in range(B):
            for i in range(k):
                if o_margin[b, i] <= MARGIN:
                    break
                np.testing.assert_allclose(adj[b, i], o_adj[b, i], rtol=0, atol=2e-4 * max(1.0, float(np.abs(o_adj[b, i]).max())))
    else:
        np.testing.assert_array_equal(to_np(d_logits), logits.numpy())
    return got


def test_markov_small(hs):
    _markov_case(hs, B=3, k=5, V=300, Vd=300, r=64, seed=1)


def test_markov_ragged_vocab_and_rank(hs):
    _markov_case(hs, B=5, k=7, V=1000, Vd=1000 - 37, r=72, seed=2)     # pruned vocabulary, rank not a multiple of 64


def test_markov_fp16_no_writeback(hs):
    _markov_case(hs, B=4, k=4, V=700, Vd=700, r=256, seed=3, dtype=torch.float16, write_logits=False)


def test_markov_many_requests(hs):
    _markov_case(hs, B=130, k=3, V=2048, Vd=2048, r=256, seed=4)      # more requests than one activation tile


def test_markov_65_to_128_requests_take_the_request_on_lanes_form(hs):
    # (ragged pruned vocabulary, rank not a multiple of 64, logits written back; then fp16 factors without write-back)
    _markov_case(hs, B=100, k=3, V=3000, Vd=3000 - 37, r=72, seed=7)
    _markov_case(hs, B=128, k=2, V=2048, Vd=2048, r=256, seed=8, dtype=torch.float16, write_logits=False)
    _markov_case(hs, B=65, k=2, V=777, Vd=777, r=64, seed=9)


def test_markov_strong_table_changes_the_draft(hs):
    """With a table strong enough to matter, the drafted ids differ from the plain arg-max of the logits."""
    B, k, V, r = 6, 8, 512, 128
    got = _markov_case(hs, B, k, V, V, r, seed=5, scale=2.0)
    g = _gen(5)
    logits = torch.randn((B * k, V), generator=g)
    plain = logits.argmax(-1).numpy().reshape(B, k)
    assert (got != plain).mean() > 0.3


def test_markov_full_vocab_rank_256(hs):
    """Serving shape: 152 064-token vocabulary, rank 256, 16 positions; sampled requests against the oracle."""
    _markov_case(hs, B=4, k=16, V=152064, Vd=152064, r=256, seed=6)


# --------------------------------------------------------------------------- KV-injection cache write (counter-example)

@pytest.mark.parametrize("Hkv,dh,k_norm", [(2, 64, True), (8, 128, True), (1, 128, False)])
def test_kv_inject_write(hs, Hkv, dh, k_norm):
    """Projected key / value rows of new positions -> a drafter-side paged bf16 cache: values bit-exact, keys within
    bf16 rounding of the oracle's norm + RoPE, every slot that is not addressed keeps its bits."""
    import synth
    from harness import assert_bf16_close, bf16_round
    cfg = dict(page_size=16, Hkv=Hkv, dh=dh, n_slots=1, n_fuse=1, D=8, V=16)
    ctx = [40, 0, 333, 17]
    batch = synth.make_request_batch(cfg, ctx_lens=ctx, device="cuda", extra_pages=3)
    k_pool, v_pool = batch["k_pools"][0].clone(), batch["v_pools"][0].clone()
    before_k, before_v = to_np(k_pool).copy(), to_np(v_pool).copy()
    # each request appends a few positions after its context (position = ctx_len + i), as a verification step would
    new = [3, 5, 1, 16]
    req = torch.tensor([b for b, n in enumerate(new) for _ in range(n)], dtype=torch.int32)
    pos = torch.tensor([ctx[b] + i for b, n in enumerate(new) for i in range(n)], dtype=torch.int32)
    T = int(req.numel())
    g = _gen(Hkv * 1000 + dh)
    kv = torch.randn((T, 2, Hkv, dh), generator=g)
    kw = 1.0 + 0.1 * torch.randn(dh, generator=g)
    # the page table must cover the appended positions: give every request enough pages from the spare ones
    pt = batch["page_table"].clone()
    need = max((ctx[b] + new[b] + 15) // 16 for b in range(4))
    if pt.shape[1] < need:
        pt = torch.nn.functional.pad(pt, (0, need - pt.shape[1]))
    used = set(int(x) for b in range(4) for x in pt[b, :(ctx[b] + 15) // 16].tolist())
    spare = [p for p in range(k_pool.shape[0]) if p not in used]
    for b in range(4):
        for j in range((ctx[b] + 15) // 16, (ctx[b] + new[b] + 15) // 16):
            pt[b, j] = spare.pop()
    pt = pt.contiguous()
    hs.hspec_op_kv_inject_write(kv.cuda(), kw.cuda() if k_norm else None, req.cuda(), pos.cuda(), pt, k_pool, v_pool,
                                1.0e6, 1e-6, k_norm)
    torch.cuda.synchronize()
    K_ref, V_ref = ao.kv_inject_rows(kv.numpy(), kw.numpy(), pos.numpy(), 1.0e6, eps=1e-6, k_norm=k_norm)
    ok, ov = before_k.copy().view(np.uint16), before_v.copy().view(np.uint16)      # bf16 bit patterns
    got_k, got_v = to_np(k_pool), to_np(v_pool)
    ptab = pt.cpu().numpy()
    touched = np.zeros(got_k.shape[:2], dtype=bool)
    from conftest import to_np as _to_np  # noqa: F401
    widen = lambda a: (a.astype(np.uint32) << 16).view(np.float32)
    for t in range(T):
        page, slot = int(ptab[int(req[t]), int(pos[t]) // 16]), int(pos[t]) % 16
        touched[page, slot] = True
        np.testing.assert_array_equal(widen(got_v[page, slot]), bf16_round(V_ref[t]))
        assert_bf16_close(widen(got_k[page, slot]), K_ref[t], f"injected key row {t}")
    np.testing.assert_array_equal(got_k[~touched], before_k[~touched])
    np.testing.assert_array_equal(got_v[~touched], before_v[~touched])
