"""Error behaviour of the boundary on a GPU: every documented failure is reported through a status code, and none
of them faults the device (bad inputs are caught by checks, never followed as addresses)."""
import numpy as np
import pytest
import torch

import synth
from harness import check_step, cuda_setup, oracle_step, assert_close

pytestmark = pytest.mark.gpu

MID = dict(D=512, n_fuse=2, r=512, L=2, has_attn=[1, 1], kv_slot=[1, 0], n_slots=2, Di=1024, P=64, N=128, G=4,
           d_conv=4, dt_rank=0, Hq=8, Hkv=2, dh=128, rope_theta=1.0e6, window=0, qk_norm=1, F=1536, V=2000,
           rms_eps=1e-6, page_size=16, name="mid", B=3, k=8, ctx=("uniform", 0, 3000))


@pytest.fixture(scope="module")
def hs():
    import paper_2609_24197_b200 as m
    from paper_2609_24197_b200 import build
    build.build()
    m.load_library()
    return m


def _draft(hs, drafter, batch, k, **over):
    B = batch["ctx_lens"].shape[0]
    ids = torch.full((B, k), -1, dtype=torch.int32, device="cuda")
    a = dict(page_table=batch["page_table"], ctx_lens=batch["ctx_lens"], last_hidden=batch["last_hidden"],
             last_token=batch["last_token"], workspace=drafter.workspace)
    a.update(over)
    hs.hspec_draft_block(drafter.handle, a["page_table"], a["ctx_lens"], a["last_hidden"], a["last_token"], k,
                         batch["k_pools"], batch["v_pools"], a["workspace"], ids, max_ctx=max(batch["ctx_lens_host"]))
    torch.cuda.synchronize()
    return ids


def _bad_table(batch):
    pt = batch["page_table"].clone()
    pt[0, 2] = batch["num_pages"] + 3        # request 0, a full page inside a full key tile
    pt[2, 0] = -4                            # request 2, a negative id
    return pt


def test_debug_validation_rejects_a_bad_page_table_before_anything_is_enqueued(hs, monkeypatch):
    monkeypatch.setenv("HSPEC_DEBUG", "1")                  # read when the handle is created
    cfg = synth.derived(dict(MID))
    drafter, w, batch = cuda_setup(cfg, ctx_lens=[700, 41, 300])
    good = _draft(hs, drafter, batch, 8)
    before = drafter.stats()["kernel_launches"]
    with pytest.raises(hs.HSpecError, match=r"\(-5\).*page id out of range"):
        _draft(hs, drafter, batch, 8, page_table=_bad_table(batch))
    cl = batch["ctx_lens"].clone()
    cl[1] = -1
    with pytest.raises(hs.HSpecError, match=r"\(-1\).*ctx_lens out of range"):
        _draft(hs, drafter, batch, 8, ctx_lens=cl)
    st = drafter.stats()
    assert st["kernel_launches"] == before and st["rc"] == 0          # the check returned on the host: no launch
    assert torch.equal(_draft(hs, drafter, batch, 8), good)
    drafter.close()


def test_without_validation_a_bad_page_id_is_counted_and_read_as_zeros(hs, monkeypatch):
    monkeypatch.delenv("HSPEC_DEBUG", raising=False)
    cfg = synth.derived(dict(MID))
    drafter, w, batch = cuda_setup(cfg, ctx_lens=[700, 41, 300])
    good = _draft(hs, drafter, batch, 8)
    assert drafter.stats()["rc"] == 0
    ids = _draft(hs, drafter, batch, 8, page_table=_bad_table(batch))
    st = drafter.stats()
    assert st["rc"] == -5 and st["bad_inputs"] >= 2 and st["device_status"] == 0, st
    assert torch.equal(ids[1], good[1])                      # the request with clean pages is unaffected
    hs.hspec_clear_status(drafter.handle)
    assert torch.equal(_draft(hs, drafter, batch, 8), good) and drafter.stats()["rc"] == 0
    drafter.close()


def test_workspace_too_small_missing_tensor_and_range_checks(hs):
    cfg = synth.derived(dict(MID))
    drafter, w, batch = cuda_setup(cfg, ctx_lens=[700, 41, 300])
    before = drafter.stats()["kernel_launches"]
    with pytest.raises(hs.HSpecError, match=r"\(-4\).*workspace needs"):
        _draft(hs, drafter, batch, 8, workspace=drafter.workspace[:1024 * 1024])
    with pytest.raises(hs.HSpecError, match=r"\(-1\).*B or k out of range"):
        _draft(hs, drafter, batch, 9)                        # the handle was made for k <= 8
    with pytest.raises(hs.HSpecError, match=r"\(-1\).*1024-byte aligned"):
        _draft(hs, drafter, batch, 8, workspace=drafter.workspace[16:])
    assert drafter.stats()["kernel_launches"] == before
    drafter.close()
    # one tensor withheld: the step refuses to run and names it
    part = {n: t for n, t in w.items() if n != "layers.1.mlp.w_down"}
    d2 = hs.Drafter(cfg, part, 3, 8, 700)
    with pytest.raises(hs.HSpecError, match=r"\(-3\).*layers\.1\.mlp\.w_down"):
        _draft(hs, d2, batch, 8)
    hs.hspec_load_weights(d2.handle, {"layers.1.mlp.w_down": w["layers.1.mlp.w_down"]})
    _draft(hs, d2, batch, 8)
    assert d2.stats()["rc"] == 0
    d2.close()


def test_large_hidden_channels_inside_the_fp16_range_keep_parity_and_beyond_it_are_flagged(hs):
    """Target hidden states carry outlier channels.  Up to fp16's 65504 they go through unchanged (parity with the
    oracle holds); beyond it the library clamps at the store instead of producing inf, counts the event, and
    hspec_get_stats returns HSPEC_ERR_F16_RANGE: a flag, not a fault, and never a silent NaN."""
    cfg = synth.derived(dict(MID))
    drafter, w, batch = cuda_setup(cfg, ctx_lens=[700, 41, 300])
    lh = batch["last_hidden"].clone()
    lh[0, 5], lh[1, 100], lh[2, 900] = 1.0e4, -2.0e4, 6.0e4
    big = dict(batch, last_hidden=lh)
    r = check_step(cfg, drafter, w, big, 8, what="outlier channels in range")
    assert drafter.stats()["rc"] == 0 and r["ids_compared"] > 0
    lh2 = batch["last_hidden"].clone()
    lh2[1, 7] = 1.0e5
    ids = _draft(hs, drafter, batch, 8, last_hidden=lh2)
    st = drafter.stats()
    assert st["rc"] == -8 and st["f16_range_events"] >= 1 and st["device_status"] == 0, st
    assert (ids >= 0).all() and (ids < cfg["V"]).all()
    hs.hspec_clear_status(drafter.handle)
    _draft(hs, drafter, batch, 8)
    assert drafter.stats()["rc"] == 0
    drafter.close()


def test_peaked_target_keys_in_a_whole_step(hs):
    """The whole step on a cache whose keys grow along the context (x1 at position 0 to x3 at the end): the attention
    rows' maxima climb by more than 2^8 over the context, the tensor-core kernel's lazy reference maximum moves, and
    the step still matches the oracle.  (The ramp is kept at x3 because the step hands q and the block's k to the
    tensor cores as bf16, like the cache they meet: a score s carries an absolute error of about 2^-9 |s|, so with
    keys twelve times larger the rounding of q alone moves the hidden state by 5e-2 of its RMS - measured on the
    oracle by rounding its q - which is a property of bf16 attention, not of the kernel.  The attention op's own
    test uses x12 and planted peaks with the same bf16 q on both sides.)"""
    cfg = synth.derived(dict(MID, B=3, k=16))
    drafter, w, batch = cuda_setup(cfg, ctx_lens=[4099, 700, 9000], poison_tail=False)
    pt = batch["page_table"].cpu()
    for kp in batch["k_pools"]:
        for b, ctx in enumerate(batch["ctx_lens_host"]):
            pos = torch.arange(ctx)
            pages, slots = pt[b, pos // 16].long().cuda(), (pos % 16).cuda()
            factor = (1.0 + 2.0 * pos.float() / (ctx - 1)).cuda()
            kp[pages, slots] = (kp[pages, slots].float() * factor[:, None, None]).to(torch.bfloat16)
    hs.hspec_clear_status(drafter.handle)
    check_step(cfg, drafter, w, batch, 16, what="peaked keys")
    st = drafter.stats()
    assert st["rc"] == 0 and st["attn_rescales"] > 0, st
    drafter.close()
