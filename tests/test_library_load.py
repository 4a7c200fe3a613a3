"""CPU-side checks of the CUDA library: it builds for sm_100a, loads without a GPU, exports every entry point that
include/ta.h declares, and its pure-host helpers behave. No kernel is launched here."""
import ctypes as C
import os
import re

import pytest

import paper_2604_11288_b200 as ta
from paper_2604_11288_b200 import build as ta_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    ta_build.build()
    return ta.binding.lib()


def _declared():
    text = open(os.path.join(ROOT, "include", "ta.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(ta_[a-z_0-9]+)\s*\(", text)))


def test_exports_every_declared_symbol(lib):
    names = _declared()
    assert {"ta_sponsor_mask", "ta_score", "ta_select_topk", "ta_compact_kv", "ta_compress"} <= set(names)
    for n in names:
        assert hasattr(lib, n), n


def test_policy_presets(lib):
    p = ta.ta_policy_default(ta.TA_PRESET_THEOREM, 16)
    assert (p.n_sink, p.n_recent, p.k_protected) == (1, 4, -1)
    assert (round(p.alpha, 3), round(p.beta, 3), round(p.gamma, 3), round(p.delta, 3), round(p.lambda_, 3)) == \
        (1.0, 0.5, 0.3, 0.2, 0.1)
    assert round(p.voucher_decay, 3) == 0.8 and round(p.budget_decay, 3) == 0.9
    p = ta.ta_policy_default(ta.TA_PRESET_SEC33, 16)
    assert (p.n_sink, p.n_recent, p.k_protected) == (1, 2, 4)  # K=16 -> 12 + 4
    p = ta.ta_policy_default(ta.TA_PRESET_AUDIT, 16)
    assert (p.n_sink, p.n_recent, p.k_protected) == (4, 6, 6)
    with pytest.raises(ta.TAError):
        ta.ta_policy_default(9, 16)


def test_scratch_size_and_validation(lib):
    p = ta.ta_policy_default(0, 16)
    b = ta.make_batch(32, 1, 4096, 4096, 4096)
    scored = ta.ta_scratch_bytes(b, 32, 8, 128, 16, p)
    assert scored >= 32 * 8 * 4096 * 4  # the fused utilities
    p.mode = ta.TA_MODE_FAST
    assert ta.ta_scratch_bytes(b, 32, 8, 128, 16, p) < scored
    bad = ta.make_batch(1, 2, 100, 100, 150)  # total != B * n
    with pytest.raises(ta.TAError) as e:
        ta.ta_scratch_bytes(bad, 32, 8, 128, 16, p)
    assert e.value.status == ta.TA_ERR_INVALID_ARG
    assert "invalid" in ta.status_string(ta.TA_ERR_INVALID_ARG)


def test_no_device_is_an_error_not_a_crash(lib):
    import torch
    if torch.cuda.is_available():
        pytest.skip("a device is present")
    h = C.c_void_p()
    assert lib.ta_ctx_create(0, 1024, C.byref(h)) != ta.TA_OK
    assert not h.value


def test_missing_library_fails_loudly(monkeypatch, tmp_path):
    monkeypatch.setattr(ta.binding, "_lib", None)
    monkeypatch.setattr(ta.binding, "LIB_PATH", str(tmp_path / "libta.so"))
    with pytest.raises(FileNotFoundError):
        ta.binding.lib()
