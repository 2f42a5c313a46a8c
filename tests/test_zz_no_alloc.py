"""The allocation-free LM-head + arg-max entry point gives the same result as the workspace-based one.

It exists for hosts that cannot allocate device memory while drafting (an engine whose KV-cache pool owns all free HBM,
a latency-critical loop, a plug-in without an allocator): its scratch is a fixed array inside the library.  This file is
collected last on purpose, so a run that stops at the first failure has already run every other test.
"""
import numpy as np
import pytest
import torch

from oracle import hspec_oracle as O

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def hs():
    import paper_2609_24197_b200 as m
    from paper_2609_24197_b200 import build
    build.build()
    m.load_library()
    return m


def _inputs(M, V, K, seed):
    g = torch.Generator(device="cuda").manual_seed(seed)
    x = torch.randn((M, K), generator=g, device="cuda").to(torch.float16)
    W = (torch.randn((V, K), generator=g, device="cuda") * 0.05).to(torch.float16)
    return x, W


@pytest.mark.parametrize("M,V,K", [(16, 1000, 256), (300, 20000, 128), (512, 4096, 64)])
def test_noalloc_matches_workspace_variant_twice_in_a_row(hs, M, V, K):
    for call in range(2):                                  # the second call reuses whatever the first left in the array
        x, W = _inputs(M, V, K, 100 + call)
        ids_ref = torch.full((M,), -1, dtype=torch.int32, device="cuda")
        logits_ref = torch.empty((M, V), dtype=torch.float32, device="cuda")
        ws = torch.empty(hs.hspec_gemm_workspace_bytes(M, V, K), dtype=torch.uint8, device="cuda")
        hs.hspec_op_lm_head_argmax(x, W, ids_ref, logits_ref, ws)
        ids = torch.full((M,), -2, dtype=torch.int32, device="cuda")
        logits = torch.empty((M, V), dtype=torch.float32, device="cuda")
        hs.hspec_op_lm_head_argmax_noalloc(x, W, ids, logits)
        torch.cuda.synchronize()
        assert torch.equal(ids, ids_ref), f"call {call}"
        ref = logits_ref.cpu().numpy().astype(np.float64)
        err = np.max(np.abs(logits.cpu().numpy() - ref)) / np.sqrt(np.mean(ref * ref))
        assert err <= 2e-2, f"call {call}: {err:.2e}"     # same kernels, same order: in practice identical bits
        assert torch.equal(logits, logits_ref)
        # ids only, no logits materialised
        ids2 = torch.full((M,), -3, dtype=torch.int32, device="cuda")
        hs.hspec_op_lm_head_argmax_noalloc(x, W, ids2)
        torch.cuda.synchronize()
        assert torch.equal(ids2, ids_ref)


@pytest.mark.parametrize("M,V,K", [(16, 1000, 256), (300, 20000, 128), (512, 4096, 64)])
def test_noalloc_matches_the_oracle_and_allocates_nothing(hs, M, V, K):
    """Against the definition (oracle GEMM + lowest-index arg-max), with a planted exact tie, on two calls in a row;
    and the 'allocates nothing' claim itself: free device memory and torch's allocator are unchanged across a call
    made after the first one (the first call on a device resolves the built-in array's address)."""
    x, W = _inputs(M, V, K, 300)
    W[V - 3] = W[5]                      # rows 5 and V-3 tie exactly: the lower index must win
    x[0] = W[5] * 40
    ids = torch.full((M,), -2, dtype=torch.int32, device="cuda")
    logits = torch.empty((M, V), dtype=torch.float32, device="cuda")
    hs.hspec_op_device_status(clear=True)
    hs.hspec_op_lm_head_argmax_noalloc(x, W, ids, logits)            # first call on this device (if none came before)
    torch.cuda.synchronize()
    ref = O.gemm(x.double().cpu().numpy(), W.double().cpu().numpy())
    ref_ids, margin = O.argmax_margin(ref)
    sure = margin > 1e-3
    for call in range(2):
        ids.fill_(-2)
        logits.fill_(float("nan"))
        free0, alloc0 = torch.cuda.mem_get_info()[0], torch.cuda.memory_allocated()
        hs.hspec_op_lm_head_argmax_noalloc(x, W, ids, logits)
        torch.cuda.synchronize()
        assert torch.cuda.mem_get_info()[0] == free0 and torch.cuda.memory_allocated() == alloc0, f"call {call} allocated"
        lg = logits.cpu().numpy()
        err = np.max(np.abs(lg - ref)) / np.sqrt(np.mean(ref * ref))
        assert err <= 1e-4, f"call {call}: {err:.2e}"
        got = ids.cpu().numpy()
        np.testing.assert_array_equal(got, np.argmax(lg, axis=-1))
        np.testing.assert_array_equal(got[sure], ref_ids[sure])
        assert got[0] == 5 and lg[0, 5] == lg[0, V - 3]
    st = hs.hspec_op_device_status(clear=True)           # a bounded wait that gave up inside the call would show here
    assert st["rc"] == 0 and st["device_status"] == 0, st


def test_noalloc_rejects_sizes_beyond_the_built_in_scratch(hs):
    x, W = _inputs(513, 256, 64, 7)
    ids = torch.empty((513,), dtype=torch.int32, device="cuda")
    with pytest.raises(hs.HSpecError, match="at most 512 rows"):
        hs.hspec_op_lm_head_argmax_noalloc(x, W, ids)
