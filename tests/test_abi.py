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
