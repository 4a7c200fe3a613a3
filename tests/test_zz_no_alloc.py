"""ta_select_topk_static is the selection step for callers that cannot allocate GPU memory (code living inside a
serving process whose pool owns the device, plugins under a fixed memory budget, loops that cannot afford
cudaMalloc's synchronisation). It needs no context: its working memory is a fixed array inside the library.

The check: through the C ABI, its indices and counts must equal those of the regular ta_select_topk bit for bit, on
two calls in a row that share the built-in array (a larger scored batch, then a smaller fast-mode batch, so that
stale contents of the first call would show in the second), and an oversized problem must be refused.
This file sorts last on purpose: a run that stops at the first failure has then already run every other test."""
import ctypes as C

import numpy as np
import pytest
import torch

import paper_2604_11288_b200 as ta
from ta_testlib import Gpu, oracle_policy
from test_gpu_steps import _workload

pytestmark = pytest.mark.gpu


def _both(w, pol, K, L, seed):
    g = Gpu(w, pol, K, L)
    try:
        flags, V, u0 = g.sponsor_mask()
        A = P = None
        if not pol.fast:
            gen = torch.Generator().manual_seed(seed)
            A = ((torch.rand((L, w.Hkv, w.total), generator=gen) * 32).round() / 32).cuda()  # with exact ties
            P = (torch.rand((L, w.Hkv, w.total), generator=gen) * 0.1).cuda()
        idx_ref, cnt_ref = g.select(flags, V, u0, A, P)
        idx = torch.full_like(idx_ref, -9)
        cnt = torch.full_like(cnt_ref, -9)
        ta.ta_select_topk_static(g.p, g.batch, w.Hkv, K, flags, V, u0, A, P, idx, cnt, g.stream)
        torch.cuda.synchronize()
        assert g.poll() == ta.TA_OK
        assert torch.equal(cnt, cnt_ref)
        assert torch.equal(idx, idx_ref)
        assert int(cnt_ref.min()) >= 0 and int(cnt_ref.max()) <= K
    finally:
        g.close()


def test_static_select_matches_regular_on_two_calls_in_a_row():
    w1 = _workload([3000, 9000, 700, 0, 41], [[5, 6, 7], [9]], seed=21, Hq=4, Hkv=2)
    _both(w1, oracle_policy(48, "THEOREM"), 48, 2, 1)
    w2 = _workload([1200, 64, 5], [[1, 2], [3]], [6, 20], alphabet=6, seed=22, Hq=4, Hkv=2)
    _both(w2, oracle_policy(16, "SEC33", fast=True, vocab_size=6), 16, 3, 2)
    _both(w1, oracle_policy(48, "THEOREM"), 48, 2, 3)


def test_static_select_rejects_oversized_problem():
    p = ta.ta_policy_default(ta.TA_PRESET_THEOREM, 16)
    p.mode = ta.TA_MODE_FAST
    n = 5 << 20  # more tokens than the built-in array has bytes
    b = ta.make_batch(1, 8, n // 8, n // 8, n)
    dummy = torch.zeros(16, dtype=torch.int32, device="cuda")
    st = ta.binding.lib().ta_select_topk_static(C.byref(p), C.byref(b), 1, 16, dummy.data_ptr(), dummy.data_ptr(),
                                                dummy.data_ptr(), None, None, dummy.data_ptr(), dummy.data_ptr(),
                                                None)
    assert st == ta.TA_ERR_SCRATCH_TOO_SMALL
