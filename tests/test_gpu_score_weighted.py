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


@pytest.mark.parametrize("preset", ["THEOREM", "SEC33"])
def test_head_sharded_allheads_selection(preset):
    # A layer whose 4 KV heads (8 query heads) live on two shards: each shard sums its own heads' weighted attention,
    # a plain fp32 add stands in for the all-reduce between the two calls, and each shard then selects and gathers
    # its own heads. Every head of both shards must retain what the oracle's all-heads selection retains.
    from paper_2604_11288_b200 import sharding
    from ta_testlib import assert_selection_matches, oracle_patterns
    w = _workload([1500, 20, 700, 9, 2300], [[4, 5], [9]], seed=41, Hq=8, Hkv=4, W=16)
    K, L, shards = 12, 2, 2
    pol = oracle_policy(K, preset, W=16)
    Qh, Kh, Vh = tw.make_qkv(w, range(L))
    Qd, Kd, Vd = Qh.cuda(), Kh.cuda(), Vh.cuda()
    g = Gpu(w, pol, K, L)
    try:
        part, views = [], []
        for r in range(shards):
            (k0, k1), (q0, q1) = sharding.head_shard(w.Hq, w.Hkv, r, shards)
            Qs, Ks, Vs = Qd[:, :, q0:q1], Kd[:, k0:k1], Vd[:, k0:k1]   # strided views of the shard's heads
            views.append((k0, k1, q0, q1, Qs, Ks, Vs))
            u = torch.full((L, w.total), float("nan"), dtype=torch.float32, device="cuda")
            ta.ta_score_headsum(g.ctx, g.p, g.batch, q1 - q0, k1 - k0, w.d, ta.view(Qs), ta.view(Ks, True), u, g.stream)
            part.append(u)
        u_all = part[0] + part[1]  # the caller's all-reduce
        idx = torch.full((L, w.B, w.Hkv, K), -7, dtype=torch.int32, device="cuda")
        cnt = torch.full((L, w.B, w.Hkv), -7, dtype=torch.int32, device="cuda")
        ko = torch.full((L, w.B, w.Hkv, K, w.d), 1.0, dtype=torch.bfloat16, device="cuda")
        vo = torch.full_like(ko, 1.0)
        for (k0, k1, q0, q1, Qs, Ks, Vs) in views:
            n_h = k1 - k0
            i_s = torch.full((L, w.B, n_h, K), -7, dtype=torch.int32, device="cuda")
            c_s = torch.full((L, w.B, n_h), -7, dtype=torch.int32, device="cuda")
            ko_s = torch.full((L, w.B, n_h, K, w.d), 1.0, dtype=torch.bfloat16, device="cuda")
            vo_s = torch.full_like(ko_s, 1.0)
            ta.ta_compress_from_headsum(g.ctx, g.pats, g.p, g.batch, n_h, w.d, K, g.ids, u_all, ta.view(Ks, True),
                                        ta.view(Vs, True), 0, ko_s, vo_s, i_s, c_s, g.stream)
            idx[:, :, k0:k1], cnt[:, :, k0:k1], ko[:, :, k0:k1], vo[:, :, k0:k1] = i_s, c_s, ko_s, vo_s
        torch.cuda.synchronize()
        assert g.poll() == ta.TA_OK
        idx, cnt = idx.cpu().numpy(), cnt.cpu().numpy()
        f_o, V_o, u0_o = oracle.sponsor_mask(w.ids, w.cu, oracle_patterns(w), pol)
        exact = 0
        for l in range(L):
            for b in range(w.B):
                o, e = int(w.cu[b]), int(w.cu[b + 1])
                Kb = np.stack([unit_kv(w, Kh, l, b, h) for h in range(w.Hkv)])
                A, P = oracle.attention_allheads(bf16_bits(Qh[l, b]), Kb, e - o, rho=pol.pension_rho)
                u = oracle.utility(pol.alpha, pol.delta, A, P, u0_o[o:e])
                io, co = oracle.select(V_o[o:e], u, K, pol.n_sink, pol.n_recent, pol.k_protected)
                exact += bool(assert_selection_matches(idx[l, b, 0], cnt[l, b, 0], io, co, u, f"l{l} b{b}"))
                for h in range(w.Hkv):
                    np.testing.assert_array_equal(idx[l, b, h], idx[l, b, 0])
                    assert cnt[l, b, h] == cnt[l, b, 0]
                    c = int(cnt[l, b, h])
                    np.testing.assert_array_equal(bf16_bits(ko[l, b, h]),
                                                  oracle.compact(unit_kv(w, Kh, l, b, h), idx[l, b, h], c, K))
                    np.testing.assert_array_equal(bf16_bits(vo[l, b, h]),
                                                  oracle.compact(unit_kv(w, Vh, l, b, h), idx[l, b, h], c, K))
        assert exact >= L * w.B - 1
        # and the same retained sets as the single-GPU all-heads call
        i1, c1, _, _ = g.compress_allheads(Qd, Kd, Vd)
        torch.cuda.synchronize()
        same = (i1.cpu().numpy() == idx).all(axis=-1).mean()
        assert same >= 0.9 and (c1.cpu().numpy() == cnt).all()
    finally:
        g.close()


def test_epoch_reuse_notices_a_changed_policy():
    # same non-zero epoch, scored call then fast call then another preset: nothing stale may be reused
    from ta_testlib import assert_selection_matches, gpu_policy, oracle_patterns, oracle_unit
    w = _workload([900, 300], [[4, 5]], seed=16, Hq=8, Hkv=2, W=32)
    K = 10
    Qh, Kh, Vh = tw.make_qkv(w, [0])
    Qd, Kd, Vd = Qh.cuda(), Kh.cuda(), Vh.cuda()
    g = Gpu(w, oracle_policy(K, "THEOREM", W=32), K, 1)
    try:
        for pol in (oracle_policy(K, "THEOREM", W=32), oracle_policy(K, "THEOREM", W=32, fast=True),
                    oracle_policy(K, "SEC33", W=32, fast=True), oracle_policy(K, "SEC33", W=32)):
            g.pol, g.p = pol, gpu_policy(pol)
            idx, cnt, ko, vo = g.compress(Qd, Kd, Vd, epoch=77)
            torch.cuda.synchronize()
            assert g.poll() == ta.TA_OK
            idx, cnt = idx.cpu().numpy(), cnt.cpu().numpy()
            f_o, V_o, u0_o = oracle.sponsor_mask(w.ids, w.cu, oracle_patterns(w), pol)
            for b in range(w.B):
                for h in range(w.Hkv):
                    A, P, u, io, co = oracle_unit(w, pol, K, Qh, Kh, 0, b, h, V_o, u0_o)
                    assert_selection_matches(idx[0, b, h], cnt[0, b, h], io, co, u, f"fast={pol.fast} b{b} h{h}")
    finally:
        g.close()


@pytest.mark.parametrize("W", [1, 5, 33, 63])
def test_weighted_odd_windows(W):
    # windows that are not a multiple of 8: G*W rows that end inside a 16-row group of the accumulator
    _weighted_case([700, 40, 3], 4, 1, W, seed=20 + W)
    _weighted_case([1400], 8, 2, W, seed=40 + W)


def _lse_rows(w, Qh, Kh, L):
    """Natural-log softmax normalisers of every window row (what a prefill attention kernel leaves behind), fp64."""
    G = w.Hq // w.Hkv
    lse = torch.zeros((L, w.B, w.Hq, w.W), dtype=torch.float64)
    for l in range(L):
        for b in range(w.B):
            o, e = int(w.cu[b]), int(w.cu[b + 1])
            n = e - o
            if n == 0:
                continue
            for h in range(w.Hq):
                k = Kh[l, h // G, o:e].double()
                s = (Qh[l, b, h].double() @ k.T) / np.sqrt(128.0)
                pos = torch.arange(n - w.W, n).view(-1, 1)
                s = s.masked_fill(torch.arange(n).view(1, -1) > pos, float("-inf"))
                lse[l, b, h] = torch.where(pos.view(-1) >= 0, torch.logsumexp(s, -1), torch.zeros(w.W).double())
    return lse


@pytest.mark.parametrize("W", [32, 64])
def test_compress_with_supplied_normalisers_reads_the_keys_once(W):
    from ta_testlib import assert_selection_matches, oracle_patterns, oracle_unit
    w = _workload([1700, 90, 640], [[4, 5], [9]], seed=50 + W, Hq=8, Hkv=2, W=W)
    K, L = 24, 2
    pol = oracle_policy(K, "THEOREM", W=W)
    Qh, Kh, Vh = tw.make_qkv(w, range(L))
    lse = _lse_rows(w, Qh, Kh, L).float().cuda()
    g = Gpu(w, pol, K, L)
    try:
        Qd, Kd, Vd = Qh.cuda(), Kh.cuda(), Vh.cuda()
        idx = torch.full((L, w.B, w.Hkv, K), -7, dtype=torch.int32, device="cuda")
        cnt = torch.full((L, w.B, w.Hkv), -7, dtype=torch.int32, device="cuda")
        ko = torch.full((L, w.B, w.Hkv, K, w.d), 1.0, dtype=torch.bfloat16, device="cuda")
        vo = torch.full_like(ko, 1.0)
        ta.ta_compress_lse(g.ctx, g.pats, g.p, g.batch, w.Hq, w.Hkv, w.d, K, g.ids, ta.view(Qd), ta.view(Kd, True),
                           ta.view(Vd, True), lse, 0, ko, vo, idx, cnt, g.stream)
        torch.cuda.synchronize()
        assert g.poll() == ta.TA_OK
        idx, cnt = idx.cpu().numpy(), cnt.cpu().numpy()
        f_o, V_o, u0_o = oracle.sponsor_mask(w.ids, w.cu, oracle_patterns(w), pol)
        for l in range(L):
            for b in range(w.B):
                for h in range(w.Hkv):
                    A, P, u, io, co = oracle_unit(w, pol, K, Qh, Kh, l, b, h, V_o, u0_o)
                    assert_selection_matches(idx[l, b, h], cnt[l, b, h], io, co, u, f"l{l} b{b} h{h}")
                    c = int(cnt[l, b, h])
                    np.testing.assert_array_equal(bf16_bits(ko[l, b, h]),
                                                  oracle.compact(unit_kv(w, Kh, l, b, h), idx[l, b, h], c, K))
        with pytest.raises(ta.TAError):
            ta.ta_compress_lse(g.ctx, g.pats, g.p, g.batch, w.Hq, w.Hkv, w.d, K, g.ids, ta.view(Qd), ta.view(Kd, True),
                               ta.view(Vd, True), None, 0, ko, vo, idx, cnt, g.stream)
    finally:
        g.close()
