"""Parity of the whole draft step (hspec_draft_block) against the oracle, plus the properties that hold
at any size: request independence, page-permutation invariance (bit-exact), causal k-prefix, determinism."""
import numpy as np
import pytest
import torch

import synth
from harness import check_step, cuda_setup, oracle_step, assert_close, MARGIN

pytestmark = pytest.mark.gpu

MID = dict(D=512, n_fuse=2, r=512, L=2, has_attn=[1, 1], kv_slot=[1, 0], n_slots=2, Di=1024, P=64, N=128, G=4,
           d_conv=4, dt_rank=0, Hq=8, Hkv=2, dh=128, rope_theta=1.0e6, window=0, qk_norm=1, F=1536, V=2000,
           rms_eps=1e-6, page_size=16, name="mid", B=5, k=16, ctx=("uniform", 0, 3000))


@pytest.fixture(scope="module", autouse=True)
def _built():
    from paper_2609_24197_b200 import build
    build.build()


def test_tiny_config_full_parity():
    cfg = synth.get_config("tiny")
    drafter, w, batch = cuda_setup(cfg)
    r = check_step(cfg, drafter, w, batch, cfg["k"], what="tiny")
    assert r["ids_compared"] >= 4
    drafter.close()


@pytest.mark.parametrize("k", [1, 5, 16, 32])
def test_mid_config_ragged_contexts(k):
    cfg = synth.derived(dict(MID, k=k))
    drafter, w, batch = cuda_setup(cfg, ctx_lens=[0, 1, 17, 1000, 2999], max_k=32)
    check_step(cfg, drafter, w, batch, k, what=f"mid k={k}")
    drafter.close()


def test_mid_config_window_and_attentionless_layer():
    cfg = synth.derived(dict(MID, window=256, has_attn=[1, 0], kv_slot=[1, -1], B=3))
    drafter, w, batch = cuda_setup(cfg, ctx_lens=[100, 255, 700])
    check_step(cfg, drafter, w, batch, 7, what="mid window")
    drafter.close()


TOL_BF16 = 5e-2    # bf16 tensor-core operands: 8 significant bits on every GEMM input (fp16 mode: 11 bits, bar 2e-2)


@pytest.mark.parametrize("over", [dict(), dict(markov_rank=64, V_draft=700), dict(window=256, has_attn=[1, 0], kv_slot=[1, -1])])
def test_mid_config_bf16_operand_mode(over):
    """act_bf16 = 1: the GEMMs run bf16 x bf16 on the caller's own matrices (borrowed, no library copy) and every
    activation the library feeds to a GEMM is bf16.  Same step, same oracle; the bound is the looser one that 8-bit
    operands allow, and the measured error is printed so the two modes can be compared."""
    cfg = synth.derived(dict(MID, act_bf16=1, **over))
    drafter, w, batch = cuda_setup(cfg, ctx_lens=[0, 1, 17, 1000, 2999], max_k=32)
    r16 = check_step(cfg, drafter, w, batch, 16, what="mid bf16 operands", tol=TOL_BF16)
    drafter.close()
    cfg_h = synth.derived(dict(MID, **over))
    d_h, _, _ = cuda_setup(cfg_h, ctx_lens=[0, 1, 17, 1000, 2999], max_k=32, weights=w)
    rh = check_step(cfg_h, d_h, w, batch, 16, what="mid fp16 operands")
    d_h.close()
    print("bf16 operands:", r16, "fp16 operands:", rh)
    assert r16["ids_compared"] > 0 and rh["err_logits"] <= r16["err_logits"] * 1.5


def test_properties_bit_exact():
    cfg = synth.derived(dict(MID))
    drafter, w, batch = cuda_setup(cfg, ctx_lens=[33, 700, 16, 2100])
    k = 8
    mc = 2100

    def run(bt, kk=k):
        ids, logits, _ = drafter.draft(bt, kk, want_logits=True, max_ctx=mc)
        torch.cuda.synchronize()
        return ids.clone(), logits.clone()
    ids0, lg0 = run(batch)
    ids1, lg1 = run(batch)
    assert torch.equal(lg0, lg1) and torch.equal(ids0, ids1)                     # deterministic
    # page permutation: any physical placement with the table updated gives identical bits
    n = batch["num_pages"]
    perm = torch.randperm(n, generator=torch.Generator().manual_seed(11)).cuda()
    inv = torch.empty_like(perm)
    inv[perm] = torch.arange(n, device="cuda")
    pt = batch["page_table"].clone()
    valid = pt >= 0
    pt[valid] = perm[pt[valid].long()].to(torch.int32)
    moved = dict(batch, page_table=pt, k_pools=[t[inv] for t in batch["k_pools"]], v_pools=[t[inv] for t in batch["v_pools"]])
    ids2, lg2 = run(moved)
    assert torch.equal(lg0, lg2) and torch.equal(ids0, ids2)
    # the KV pools are never written
    kp_before = [t.clone() for t in batch["k_pools"]]
    run(batch)
    for a, b in zip(kp_before, batch["k_pools"]):
        assert torch.equal(a.view(torch.int16), b.view(torch.int16))
    # causal over block positions: the first j rows of a k-step are a j-step (same kernels, other launch shapes)
    ids3, lg3 = run(batch, 3)
    ref = lg0[:, :3].cpu().numpy()
    assert_close(lg3.cpu().numpy(), ref, "k-prefix", tol=5e-3)
    drafter.close()


def test_request_independence_across_batch_sizes():
    cfg = synth.derived(dict(MID))
    w = synth.make_weights(cfg, device="cuda")
    ctxs = [500, 40, 1300]
    d3, _, batch3 = cuda_setup(cfg, ctx_lens=ctxs, weights=w)
    _, lg3, _ = d3.draft(batch3, 6, want_logits=True, max_ctx=1300)
    torch.cuda.synchronize()
    # request 1 alone, with its own pages
    one = dict(batch3, ctx_lens=batch3["ctx_lens"][1:2].contiguous(), page_table=batch3["page_table"][1:2].contiguous(),
               last_hidden=batch3["last_hidden"][1:2].contiguous(), last_token=batch3["last_token"][1:2].contiguous(),
               ctx_lens_host=[40])
    _, lg1, _ = d3.draft(one, 6, want_logits=True, max_ctx=1300)
    torch.cuda.synchronize()
    assert_close(lg1[0].cpu().numpy(), lg3[1].cpu().numpy(), "request independence", tol=5e-3)
    d3.close()


def _full_size(name, n_check, **over):
    """The workload at its full size, in the launch configuration bench.py times, compared with the oracle on `n_check`
    sampled requests (requests are independent, so each is a complete comparison): the longest, the shortest and the
    median context, then seeded random ones.  The shortest is a request whose visible context is a single chunk
    (finished inside the attention kernel, no partials), the longest has the most chunks."""
    cfg = synth.get_config(name, **over)
    drafter, w, batch = cuda_setup(cfg, poison_tail=False, extra_pages=0)
    B = cfg["B"]
    order = np.argsort(batch["ctx_lens_host"])
    pick = [int(order[-1]), int(order[0]), int(order[B // 2])]
    rnd = np.random.default_rng(synth.BASE_SEED + 17).permutation(B).tolist()
    pick = list(dict.fromkeys(pick + [int(b) for b in rnd]))[:max(1, min(n_check, B))]
    r = check_step(cfg, drafter, w, batch, cfg["k"], requests=sorted(pick), dtype=np.float32, what=name)
    st = drafter.stats()
    assert st["rc"] == 0, st
    print(name, "requests", sorted(pick), "contexts", [batch["ctx_lens_host"][b] for b in sorted(pick)], r)
    drafter.close()
    del w, batch
    torch.cuda.empty_cache()
    return r


def test_latency_8b_full_size():
    _full_size("latency_8b", 1)


def test_serving_8b_full_size_sampled_requests():
    _full_size("serving_8b", 8)


def test_conc128_32b_full_size_sampled_requests():
    _full_size("conc128_32b", 8)


def test_serving_8b_and_conc128_32b_with_the_2048_token_window():
    # the paper's sliding window (App. B.1) on the two serving workloads: the variant bench.py reports beside the
    # full-context headline
    _full_size("serving_8b", 2, window=2048)
    _full_size("conc128_32b", 2, window=2048)


def test_paper_shape_drafter_sampled_requests():
    # the paper's own drafter shape (App. B.1): 48 Mamba heads x 64 with state = groups = conv = 4, five fused target
    # layers, three attention layers + one Mamba-MLP layer, 2048-token window
    _full_size("paper_8b", 3)


def test_sweep_cells_8b_sampled_requests():
    # cells of the concurrency x block-size sweep: 64 query rows per KV head at k = 16, 32 at k = 8, and at k = 32 the
    # only shape that runs two 128-row tiles per KV head at full size
    _full_size("sweep_8b_B128_k8", 2)
    _full_size("sweep_8b_B256_k16", 8)
    _full_size("sweep_8b_B128_k32", 5)


def test_mid_config_pruned_drafter_vocabulary():
    cfg = synth.derived(dict(MID, V_draft=700, B=2))
    drafter, w, batch = cuda_setup(cfg, ctx_lens=[300, 41])
    r = check_step(cfg, drafter, w, batch, 9, what="mid pruned vocab")
    assert r["ids_compared"] > 0
    drafter.close()


@pytest.mark.parametrize("over", [dict(markov_rank=64), dict(markov_rank=72, V_draft=700), dict(markov_rank=256, k=1)])
def test_mid_config_markov_head(over):
    """Causal-correction head behind the LM head (Sec. 3.3.3): the step's ids and corrected logits follow the oracle's
    sequential rule; with a pruned vocabulary the predecessor is looked up by its target id."""
    cfg = synth.derived(dict(MID, B=3, **over))
    k = cfg["k"] if "k" in over else 11
    drafter, w, batch = cuda_setup(cfg, ctx_lens=[300, 41, 1500])
    r = check_step(cfg, drafter, w, batch, k, what=f"mid markov {over}")
    assert r["ids_compared"] > 0
    # the head changes the draft: ids differ from the plain arg-max of the uncorrected logits somewhere
    if k > 1:
        plain = dict(w)
        del plain["markov_in"], plain["markov_out"]
        cfg0 = synth.derived(dict(cfg, markov_rank=0))
        d0, _, _ = cuda_setup(cfg0, ctx_lens=[300, 41, 1500], weights=plain)
        ids0 = d0.draft(batch, k)[0]
        ids1 = drafter.draft(batch, k)[0]
        torch.cuda.synchronize()
        assert (ids0 != ids1).any()
        d0.close()
    drafter.close()


def test_conc128_32b_markov_full_size_sampled_requests():
    _full_size("conc128_32b_markov", 2)


def test_bounded_wait_gives_up_and_reports_without_killing_the_context():
    # failure detection without a GPU fault: a wait nobody satisfies runs out, the kernel records a status code and
    # returns; the host sees HSPEC_ERR_TIMEOUT, clears it, and the same handle then drafts correctly
    import paper_2609_24197_b200 as hs
    cfg = synth.get_config("tiny")
    drafter, w, batch = cuda_setup(cfg)
    ids0, _, _ = drafter.draft(batch, cfg["k"])
    torch.cuda.synchronize()
    assert drafter.stats()["device_status"] == 0
    hs.hspec_debug_wait_selftest(drafter.handle, 50)
    st = drafter.stats()
    assert st["rc"] == -7 and st["device_status"] == 0x1FF            # HSPEC_ERR_TIMEOUT, the self-test's code
    hs.hspec_clear_status(drafter.handle)
    assert drafter.stats()["device_status"] == 0
    ids1, _, _ = drafter.draft(batch, cfg["k"])
    torch.cuda.synchronize()
    assert torch.equal(ids0, ids1) and drafter.stats()["device_status"] == 0
    drafter.close()


def test_step_is_capturable_in_a_cuda_graph_and_replays_bit_exactly():
    """hspec_draft_block only enqueues work on the caller's stream (no host synchronisation, no allocation), so a
    serving loop can capture it once and replay it; the replay reads the CURRENT contents of the input buffers."""
    cfg = synth.derived(dict(MID, B=3))
    drafter, w, batch = cuda_setup(cfg, ctx_lens=[300, 41, 1500])
    k = 9
    ids_direct = drafter.draft(batch, k)[0].clone()
    torch.cuda.synchronize()
    side = torch.cuda.Stream()
    with torch.cuda.stream(side):
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=side):
            ids_graph = drafter.draft(batch, k)[0]
    torch.cuda.synchronize()
    ids_graph.fill_(-1)
    graph.replay()
    torch.cuda.synchronize()
    assert torch.equal(ids_graph, ids_direct)
    # new inputs in the same buffers: the replay follows them
    batch["last_token"].copy_((batch["last_token"] + 7) % cfg["V"])
    batch["last_hidden"].copy_(batch["last_hidden"].flip(0))
    graph.replay()
    torch.cuda.synchronize()
    ids_new = drafter.draft(batch, k)[0]
    torch.cuda.synchronize()
    assert torch.equal(ids_graph, ids_new)
    assert not torch.equal(ids_new, ids_direct)
    assert drafter.stats()["device_status"] == 0
    drafter.close()


def test_smaller_batch_than_planned_fits_the_workspace():
    """The scratch layout depends on the step's own (B, k) (context chunking and K-slices change at thresholds), so the
    size reported for (max_batch, max_k) must cover every smaller step too: 73 requests on a handle made for 128,
    with contexts long enough that the two batch sizes cut them into different chunk lengths."""
    cfg = synth.derived(dict(MID, Hq=8, Hkv=8, B=73))
    ctx = [4200 + 13 * b for b in range(73)]
    drafter, w, batch = cuda_setup(cfg, ctx_lens=ctx, max_batch=128, max_k=16, poison_tail=False, extra_pages=0)
    r = check_step(cfg, drafter, w, batch, 16, requests=[0, 72], what="B=73 of 128")
    assert r["ids_compared"] > 0
    drafter.close()
