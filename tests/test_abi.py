"""The C-ABI library loads on a CPU-only box and exports every symbol include/hspec.h declares."""
import ctypes
import os
import re

import pytest

import paper_2609_24197_b200 as hs
from paper_2609_24197_b200 import build as hbuild

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    hbuild.build()
    return hs.load_library()


def _declared():
    text = open(os.path.join(ROOT, "include", "hspec.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(hspec_[a-z0-9_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = _declared()
    assert "hspec_draft_block" in names and "hspec_op_attention" in names
    for n in names:
        assert hasattr(lib, n), n
    assert sorted(hs.EXPORTS) == names


def test_init_validates_config_without_a_gpu(lib):
    import synth
    cfg = hs.make_config(synth.get_config("tiny"), max_batch=2, max_k=8, max_pages_per_req=16)
    h = hs.hspec_init(cfg)
    assert hs.hspec_workspace_bytes(cfg) > 0
    hs.hspec_destroy(h)
    bad = hs.make_config(synth.get_config("tiny", dh=48), max_batch=2, max_k=8, max_pages_per_req=16)
    with pytest.raises(hs.HSpecError, match="head dim"):
        hs.hspec_init(bad)
    with pytest.raises(hs.HSpecError):
        hs.hspec_init(hs.make_config(synth.get_config("tiny"), max_batch=1, max_k=64, max_pages_per_req=1))


def test_workspace_grows_with_batch(lib):
    import synth
    base = synth.get_config("latency_8b")
    small = hs.hspec_workspace_bytes(hs.make_config(base, 1, 16, 128))
    large = hs.hspec_workspace_bytes(hs.make_config(base, 32, 16, 512))
    assert 0 < small < large


def test_no_cpu_path(lib):
    import torch
    if torch.cuda.is_available():
        pytest.skip("CPU-only check")
    import synth
    cfg = synth.get_config("tiny")
    with pytest.raises(hs.HSpecError, match="no CUDA device"):
        hs.Drafter(cfg, {}, 1, 8, 256)


def test_markov_config_and_workspace_without_a_gpu(lib):
    """markov_rank is validated at init, enlarges the step's workspace (fp32 logits of the block + the per-position
    scratch), and the stand-alone op reports its scratch size."""
    import synth
    plain = synth.get_config("tiny")
    with_head = synth.get_config("tiny", markov_rank=64)
    w0 = hs.hspec_workspace_bytes(hs.make_config(plain, 2, 8, 16))
    w1 = hs.hspec_workspace_bytes(hs.make_config(with_head, 2, 8, 16))
    assert w1 >= w0 + 2 * 8 * plain["V"] * 4
    with pytest.raises(hs.HSpecError, match="markov_rank"):
        hs.hspec_init(hs.make_config(synth.get_config("tiny", markov_rank=12), 2, 8, 16))
    B, Vd, r = 3, 1000, 64
    need = hs.hspec_markov_workspace_bytes(B, Vd, r)
    tiles = (Vd + 127) // 128
    assert need >= B * r * 2 + 2 * tiles * B * 4
    assert hs.hspec_markov_workspace_bytes(0, Vd, r) == 0


def test_new_entry_points_reject_bad_arguments_without_touching_the_gpu(lib):
    """Argument checks come first: NULL pointers and bad sizes are refused with HSPEC_ERR_INVALID_ARG (-1 .. small
    negative codes), never passed to a kernel."""
    null = ctypes.c_void_p(None)
    assert lib.hspec_op_accept(null, null, null, null, 4, 4, null) < 0
    assert lib.hspec_op_token_probs(null, 10, null, null, 1, 10, null) < 0
    assert lib.hspec_op_markov_head(null, 10, null, null, hs.HSPEC_F16, null, null, null, 1, 1, 10, 64, 0, null, 0, null) < 0
    msg = lib.hspec_last_error(None)
    assert msg and b"hspec_op_markov_head" in msg
