"""Shared glue for the GPU parity tests: seeded inputs -> CUDA library and -> CPU oracle."""
import numpy as np
import torch

import synth
from oracle import hspec_oracle as O
from conftest import to_np

TOL = 2e-2      # max-abs error relative to the RMS of the reference tensor (bf16 operands, fp32 accumulation)
MARGIN = 1e-2   # draft ids are compared only where the oracle's top-1 margin exceeds this


def rel_err(got, ref):
    ref = np.asarray(ref, dtype=np.float64)
    got = np.asarray(got, dtype=np.float64)
    rms = float(np.sqrt(np.mean(ref * ref)))
    return float(np.max(np.abs(got - ref))) / max(rms, 1e-30)


def assert_close(got, ref, what, tol=TOL):
    assert np.isfinite(np.asarray(got, dtype=np.float64)).all(), f"{what}: non-finite output"
    e = rel_err(got, ref)
    assert e <= tol, f"{what}: max-abs error {e:.3e} of the reference RMS exceeds {tol:.1e}"
    return e


def rms_err(got, ref):
    ref = np.asarray(ref, dtype=np.float64)
    got = np.asarray(got, dtype=np.float64)
    return float(np.sqrt(np.mean((got - ref) ** 2))) / max(float(np.sqrt(np.mean(ref * ref))), 1e-30)


def assert_bf16_close(got, ref, what, ulps=2, floor=1e-3):
    """For an op whose OUTPUT is stored in bf16: every element within `ulps` bf16 steps (2^-8 relative each) of the
    reference, plus `floor` x RMS for elements that cancel to near zero."""
    ref = np.asarray(ref, dtype=np.float64)
    got = np.asarray(got, dtype=np.float64)
    assert np.isfinite(got).all(), f"{what}: non-finite output"
    rms = float(np.sqrt(np.mean(ref * ref)))
    bound = ulps * 2.0 ** -8 * np.abs(ref) + floor * rms
    bad = np.abs(got - ref) > bound
    assert not bad.any(), f"{what}: {int(bad.sum())} elements off by more than {ulps} bf16 steps; worst " \
                          f"{float(np.max(np.abs(got - ref) / bound)):.2f}x the bound"


def bf16_round(a):
    """float array -> values representable in bf16 (as float32), via torch's round-to-nearest-even."""
    return torch.from_numpy(np.asarray(a, dtype=np.float32)).to(torch.bfloat16).float().numpy()


def oracle_step(cfg, weights, batch, k, requests=None, dtype=np.float64, **kw):
    w = {n: to_np(t) for n, t in weights.items()}
    return O.draft_block(cfg, w, [to_np(t) for t in batch["k_pools"]], [to_np(t) for t in batch["v_pools"]],
                         to_np(batch["page_table"]), batch["ctx_lens_host"], to_np(batch["last_hidden"]),
                         to_np(batch["last_token"]), k, dtype=dtype, requests=requests, **kw)


def check_step(cfg, drafter, weights, batch, k, requests=None, dtype=np.float64, what="step", tol=TOL):
    """Run the CUDA step for the whole batch and the oracle for `requests`; compare."""
    ids, logits, hidden = drafter.draft(batch, k, want_logits=True, want_hidden=True,
                                        max_ctx=max(batch["ctx_lens_host"] + [1]))
    torch.cuda.synchronize()
    st = drafter.stats()
    assert st["device_status"] == 0, f"device status {st['device_status']:#x}"
    B = len(batch["ctx_lens_host"])
    requests = list(range(B)) if requests is None else list(requests)
    ref = oracle_step(cfg, weights, batch, k, requests, dtype)
    ids, logits, hidden = ids.cpu().numpy(), logits.cpu().numpy(), hidden.cpu().numpy()
    # the fused arg-max must agree with the library's own logits exactly (lowest index on ties)
    own = np.argmax(logits, axis=-1).astype(np.int32)
    if "vocab_map" in weights:
        own = weights["vocab_map"].cpu().numpy()[own]
    np.testing.assert_array_equal(ids, own)
    e_h = assert_close(hidden[requests], ref["hidden"], what + " hidden", tol)
    sure = ref["margin"] > MARGIN
    if "markov_in" in weights:
        # the correction at position i depends on the token chosen at i - 1: after a near-tie the two sides may
        # follow different chains, so a request is compared up to and including its first unsure position only
        chain_ok = np.ones_like(sure)
        chain_ok[:, 1:] = np.cumprod(sure[:, :-1], axis=1).astype(bool)
        assert sure.shape[1] == 1 or chain_ok[:, 1:].any(), what + ": no chained position is comparable"
        e_l = assert_close(logits[requests][chain_ok], ref["logits"][chain_ok], what + " logits", tol)
        sure &= chain_ok
    else:
        e_l = assert_close(logits[requests], ref["logits"], what + " logits", tol)
    assert np.array_equal(ids[requests][sure], ref["draft_ids"][sure]), what + " draft ids differ above the margin"
    return dict(err_hidden=e_h, err_logits=e_l, ids_compared=int(sure.sum()), ids_total=int(sure.size))


def cuda_setup(cfg, ctx_lens=None, poison_tail=True, extra_pages=2, max_batch=None, max_k=None, weights=None):
    import paper_2609_24197_b200 as hs
    weights = weights if weights is not None else synth.make_weights(cfg, device="cuda")
    batch = synth.make_request_batch(cfg, ctx_lens=ctx_lens, device="cuda", poison_tail=poison_tail,
                                     extra_pages=extra_pages)
    B = len(batch["ctx_lens_host"])
    drafter = hs.Drafter(cfg, weights, max_batch or B, max_k or cfg["k"], max(batch["ctx_lens_host"] + [1]))
    return drafter, weights, batch
