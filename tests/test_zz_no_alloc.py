"""ta_select_topk_static is the selection step for callers that cannot allocate GPU memory (code living inside a
serving process whose pool owns the device, plugins under a fixed memory budget, loops that cannot afford
cudaMalloc's synchronisation). It needs no context: its working memory is a fixed array inside the library.

The check: through the C ABI, its indices and counts must equal those of the regular ta_select_topk bit for bit, and
those of the CPU oracle's selection on the same utilities, on two calls in a row that share the built-in array (a
larger scored batch, then a smaller fast-mode batch, so that stale contents of the first call would show in the
second); an oversized problem must be refused; and a sequence whose offsets point outside the token arrays must come
back empty without a write behind the outputs (there is no context whose status could report it).
This file sorts last on purpose: a run that stops at the first failure has then already run every other test."""
import ctypes as C

import numpy as np
import pytest
import torch

import oracle
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
        # and against the oracle's selection on the same fp32 utilities (exact: the scores are inputs here)
        Vh, u0h, ih, ch = V.cpu().numpy(), u0.cpu().numpy(), idx.cpu().numpy(), cnt.cpu().numpy()
        Ah = None if A is None else A.cpu().numpy()
        Ph = None if P is None else P.cpu().numpy()
        for l in range(L):
            for b in range(w.B):
                o, e = int(w.cu[b]), int(w.cu[b + 1])
                for h in range(w.Hkv):
                    u = u0h[o:e] if pol.fast else oracle.utility(pol.alpha, pol.delta, Ah[l, h, o:e], Ph[l, h, o:e],
                                                                 u0h[o:e])
                    io, co = oracle.select(Vh[o:e], u, K, pol.n_sink, pol.n_recent, pol.k_protected)
                    assert int(ch[l, b, h]) == int(co), f"count l{l} b{b} h{h}"
                    np.testing.assert_array_equal(ih[l, b, h], io, err_msg=f"l{l} b{b} h{h}")
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


def test_static_select_rejects_sequences_outside_the_token_arrays():
    w = _workload([300, 200, 100], [[4, 5]], seed=23, Hq=4, Hkv=2)
    K, L, guard = 8, 2, 3
    pol = oracle_policy(K, "THEOREM")
    g = Gpu(w, pol, K, L)
    try:
        flags, V, u0 = g.sponsor_mask()
        A = torch.rand((L, w.Hkv, w.total), device="cuda")
        bad_cu = torch.tensor([0, 300, 500, 1300], dtype=torch.int32, device="cuda")  # ends 700 tokens too far
        batch = ta.make_batch(L, 3, 0, 1024, w.total, bad_cu)
        idx = torch.full((L + guard, 3, w.Hkv, K), -9, dtype=torch.int32, device="cuda")
        cnt = torch.full((L + guard, 3, w.Hkv), -9, dtype=torch.int32, device="cuda")
        ta.ta_select_topk_static(g.p, batch, w.Hkv, K, flags, V, u0, A, None, idx, cnt, g.stream)
        torch.cuda.synchronize()
        assert (idx[L:] == -9).all() and (cnt[L:] == -9).all()
        assert (cnt[:L, 2] == 0).all() and (idx[:L, 2] == -1).all()
        assert (cnt[:L, :2] == K).all()
        # a regular call afterwards still matches (the shared array holds nothing stale that matters)
        idx2 = torch.full((L, 3, w.Hkv, K), -9, dtype=torch.int32, device="cuda")
        cnt2 = torch.full((L, 3, w.Hkv), -9, dtype=torch.int32, device="cuda")
        ta.ta_select_topk_static(g.p, g.batch, w.Hkv, K, flags, V, u0, A, None, idx2, cnt2, g.stream)
        idx_ref, cnt_ref = g.select(flags, V, u0, A, None)
        torch.cuda.synchronize()
        assert torch.equal(idx2, idx_ref) and torch.equal(cnt2, cnt_ref)
    finally:
        g.close()
