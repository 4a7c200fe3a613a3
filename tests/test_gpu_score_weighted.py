"""GPU parity of the weighted attention term alpha*A + delta*P (ta_score_weighted, the form the fused path uses)
against the CPU oracle, element by element; the time-out path of the bounded device waits; and device-side rejection of
sequence offsets that point outside the token arrays."""
import numpy as np
import pytest
import torch

import oracle
import paper_2604_11288_b200 as ta
import ta_workloads as tw
from ta_testlib import SCORE_ATOL, SCORE_RTOL, Gpu, bf16_bits, oracle_policy, unit_kv
from test_gpu_steps import _workload

pytestmark = pytest.mark.gpu


def _weighted_case(lengths, Hq, Hkv, W, seed=0, layers=1, cluster=0, edit=None, guard=0, **pol_kw):
    w = _workload(lengths, [[1, 2]], seed=seed, Hq=Hq, Hkv=Hkv, W=W)
    w.n_layers = layers
    pol = oracle_policy(4, W=W, **pol_kw)
    Qh, Kh, _ = tw.make_qkv(w, range(layers))
    if edit is not None:
        edit(w, Qh, Kh)
    g = Gpu(w, pol, 4, layers)
    try:
        if cluster:
            ta.ta_ctx_set_score_cluster(g.ctx, cluster)
        Qd, Kd = Qh.cuda(), Kh.cuda()
        u = torch.full((layers + guard, w.Hkv, w.total), float("nan"), dtype=torch.float32, device="cuda")
        ta.ta_score_weighted(g.ctx, g.p, g.batch, w.Hq, w.Hkv, w.d, ta.view(Qd), ta.view(Kd, not w.uniform), None, u,
                             g.stream)
        torch.cuda.synchronize()
        assert g.poll() == ta.TA_OK
        if guard:
            assert torch.isnan(u[layers:]).all(), "wrote behind its output"
        u = u.cpu().numpy()
        G = Hq // Hkv
        for l in range(layers):
            for b in range(w.B):
                o, e = int(w.cu[b]), int(w.cu[b + 1])
                for h in range(Hkv):
                    A, P = oracle.attention(bf16_bits(Qh[l, b, h * G:(h + 1) * G]), unit_kv(w, Kh, l, b, h), e - o,
                                            scale=pol.softmax_scale, causal=pol.causal, rho=pol.pension_rho)
                    want = pol.alpha * A.astype(np.float64) + pol.delta * P.astype(np.float64)
                    # each term within the tolerance of the attention terms (a weighted sum of two such terms)
                    tol = (abs(pol.alpha) + abs(pol.delta)) * SCORE_ATOL + SCORE_RTOL * (
                        abs(pol.alpha) * np.abs(A) + abs(pol.delta) * np.abs(P))
                    err = np.abs(u[l, h, o:e].astype(np.float64) - want)
                    bad = np.nonzero(~(err <= tol))[0]
                    assert bad.size == 0, (f"l{l} b{b} h{h} n{e - o}: {bad.size} outside tolerance, first {bad[:6]}, "
                                           f"got {u[l, h, o:e][bad[:6]]}, want {want[bad[:6]]}")
    finally:
        g.close()


def test_weighted_one_row_block_ragged():
    _weighted_case([1000, 128, 129, 4096 + 37], 8, 2, 32)


def test_weighted_two_row_blocks():
    _weighted_case([700, 2500, 64, 65], 8, 2, 64, seed=1)


def test_weighted_general_windows_and_padding_rows():
    _weighted_case([777, 130], 4, 1, 24, seed=2)      # 96 rows
    _weighted_case([1500, 200], 4, 1, 48, seed=3)     # 192 rows: the second group of a pair has 64 live rows
    _weighted_case([300, 5, 1, 0, 31], 2, 2, 8, seed=4)  # 8 rows; sequences shorter than the window


def test_weighted_many_units_several_rounds_and_guard():
    _weighted_case([300], 32, 8, 32, seed=5, layers=20, guard=8)
    _weighted_case([260, 140], 8, 2, 64, seed=6, layers=90, guard=4)


@pytest.mark.parametrize("cluster", [1, 2, 4, 8])
@pytest.mark.parametrize("W", [32, 64])
def test_weighted_cluster_sizes(cluster, W):
    _weighted_case([8192 - 77, 1300], 4, 1, W, seed=7, cluster=cluster)


@pytest.mark.parametrize("W", [32, 64])
def test_weighted_scores_far_from_the_first_keys(W):
    # keys that score about 98 bits above the rest, early, late and inside the masked tail; a row whose first keys
    # score far below everything else (the polynomial exponentials clamp at 2^126 and 2^-126)
    def edit(w, Qh, Kh):
        G = w.Hq // w.Hkv
        q = Qh[0, 0, 1, W - 1].float()
        for j in (40, 700, 1290):
            Kh[0, 0, j] = (6.0 * q).to(torch.bfloat16)
        q2 = Qh[0, 0, G + 2, W - 3].float()
        Kh[0, 1, 0:16] = (-6.0 * q2).to(torch.bfloat16)
        q3 = Qh[0, 1, 0, 5].float()
        Kh[0, 0, int(w.cu[2]) - W + 2] = (6.0 * q3).to(torch.bfloat16)

    _weighted_case([1300, 300], 8, 2, W, seed=8, edit=edit)


def test_weighted_non_causal_custom_scale_and_weights():
    _weighted_case([900, 333], 4, 1, 32, seed=9, causal=0, softmax_scale=0.05, alpha=0.3, delta=2.5)
    _weighted_case([900], 8, 2, 64, seed=10, alpha=1.0, delta=0.0)


def test_weighted_with_a_negative_row_weight_takes_the_general_form():
    # alpha + delta*w_t is negative for the latest window rows: the weights cannot go into the exponents
    _weighted_case([1100, 90], 8, 2, 32, seed=11, alpha=0.02, delta=-1.0)
    _weighted_case([600], 8, 2, 64, seed=12, alpha=0.02, delta=-1.0)


def test_weighted_equals_separate_terms():
    w = _workload([2000, 450], [[1, 2]], seed=13, Hq=8, Hkv=2, W=32)
    pol = oracle_policy(4, W=32)
    Qh, Kh, _ = tw.make_qkv(w, [0])
    g = Gpu(w, pol, 4, 1)
    try:
        Qd, Kd = Qh.cuda(), Kh.cuda()
        A, P = g.score(Qd, Kd)
        u = torch.empty_like(A)
        ta.ta_score_weighted(g.ctx, g.p, g.batch, w.Hq, w.Hkv, w.d, ta.view(Qd), ta.view(Kd, True), None, u, g.stream)
        torch.cuda.synchronize()
        assert g.poll() == ta.TA_OK
        want = pol.alpha * A.double() + pol.delta * P.double()
        assert torch.allclose(u.double(), want, rtol=2e-4, atol=2e-6)
    finally:
        g.close()


def test_bounded_wait_runs_out_and_the_context_stays_usable():
    w = _workload([500], [[1, 2]], seed=14, Hq=8, Hkv=2, W=32)
    pol = oracle_policy(4, W=32)
    g = Gpu(w, pol, 4, 1)
    try:
        outcome = torch.zeros(1, dtype=torch.int32, device="cuda")
        ta.ta_ctx_selftest_wait(g.ctx, 1_000_000, outcome, g.stream)  # 1 ms
        torch.cuda.synchronize()
        assert int(outcome.item()) == 4, "the kernel did not reach its end, or a wait on a dead barrier succeeded"
        assert g.poll() == ta.TA_ERR_TIMEOUT
        assert g.poll() == ta.TA_OK
        # the same context scores correctly afterwards
        Qh, Kh, _ = tw.make_qkv(w, [0])
        A, P = g.score(Qh.cuda(), Kh.cuda())
        torch.cuda.synchronize()
        assert g.poll() == ta.TA_OK
        Ao, Po = oracle.attention(bf16_bits(Qh[0, 0, 0:4]), unit_kv(w, Kh, 0, 0, 0), 500, scale=0.0, causal=1,
                                  rho=pol.pension_rho)
        np.testing.assert_allclose(A[0, 0].cpu().numpy(), Ao, rtol=SCORE_RTOL, atol=SCORE_ATOL)
        with pytest.raises(ta.TAError):
            ta.ta_ctx_selftest_wait(g.ctx, 0, outcome, g.stream)
        with pytest.raises(ta.TAError):
            ta.ta_ctx_selftest_wait(g.ctx, 5_000_000_000, outcome, g.stream)
    finally:
        g.close()


def test_sequence_offsets_outside_the_token_arrays_are_rejected_on_the_device():
    # cu_seqlens is device data: the host cannot see that the last sequence ends 700 tokens past total_tokens
    w = _workload([300, 200, 100], [[4, 5]], seed=15, Hq=8, Hkv=2, W=32)
    K = 8
    pol = oracle_policy(K, W=32)
    Qh, Kh, Vh = tw.make_qkv(w, [0])
    g = Gpu(w, pol, K, 1)
    try:
        bad_cu = torch.tensor([0, 300, 500, 1300], dtype=torch.int32, device="cuda")
        batch = ta.make_batch(1, 3, 0, 1024, w.total, bad_cu)
        guard = 4
        idx = torch.full((1 + guard, 3, w.Hkv, K), -7, dtype=torch.int32, device="cuda")
        cnt = torch.full((1 + guard, 3, w.Hkv), -7, dtype=torch.int32, device="cuda")
        ko = torch.full((1 + guard, 3, w.Hkv, K, w.d), 1.0, dtype=torch.bfloat16, device="cuda")
        vo = torch.full_like(ko, 1.0)
        Qd, Kd, Vd = Qh.cuda(), Kh.cuda(), Vh.cuda()
        ta.ta_compress(g.ctx, g.pats, g.p, batch, w.Hq, w.Hkv, w.d, K, g.ids, ta.view(Qd), ta.view(Kd, True),
                       ta.view(Vd, True), 0, ko, vo, idx, cnt, g.stream)
        torch.cuda.synchronize()
        assert g.poll() == ta.TA_ERR_DEVICE_BOUNDS
        assert g.poll() == ta.TA_OK
        assert (idx[1:] == -7).all() and (cnt[1:] == -7).all() and (ko[1:] == 1.0).all() and (vo[1:] == 1.0).all()
        c = cnt[0].cpu().numpy()
        assert (c[2] == 0).all() and (idx[0, 2] == -1).all(), "the rejected sequence must come back empty"
        assert (c[0] == K).all() and (c[1] == K).all()
    finally:
        g.close()
