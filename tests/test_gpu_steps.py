"""GPU parity, step by step: each C-ABI entry point against the CPU oracle on the same seeded bytes, at sizes that
span several tiles and a ragged tail, plus the degenerate cases of the method."""
import numpy as np
import pytest
import torch

import oracle
import paper_2604_11288_b200 as ta
import ta_workloads as tw
from ta_testlib import (Gpu, assert_scores_close, assert_selection_matches, bf16_bits, oracle_patterns, oracle_policy,
                        oracle_unit, unit_kv)

pytestmark = pytest.mark.gpu


def _workload(lengths, pats, spans=None, budgets=None, alphabet=None, seed=0, Hq=8, Hkv=2, W=8, plant=True):
    """A packed batch with random ids; with a small alphabet the patterns occur by chance everywhere."""
    rng = np.random.default_rng(seed)
    lengths = np.asarray(lengths, np.int32)
    total = int(lengths.sum())
    hi = alphabet if alphabet else tw.VOCAB
    ids = rng.integers(0, hi, size=total).astype(np.int32)
    cu = np.zeros(len(lengths) + 1, np.int32)
    cu[1:] = np.cumsum(lengths)
    if plant and not alphabet:
        for b in range(len(lengths)):
            n = int(lengths[b])
            for _ in range(max(1, n // 300)):
                p = pats[int(rng.integers(0, len(pats)))]
                if n > len(p) + 2:
                    s = int(rng.integers(0, n - len(p)))
                    ids[cu[b] + s:cu[b] + s + len(p)] = p
    w = tw.Workload(name="t", seed=1234 + seed, n_layers=1, Hq=Hq, Hkv=Hkv, d=128, W=W, K_list=[], modes=[],
                    uniform=False, lengths=lengths, cu=cu, ids=ids, pattern_ids=[list(map(int, p)) for p in pats],
                    pattern_budget=budgets or [15.0] * len(pats), pattern_span=spans or [6] * len(pats), planted=[],
                    vocab=hi)
    return w


def _check_mask(w, pol):
    g = Gpu(w, pol, 4, 1)
    try:
        flags, V, u0 = g.sponsor_mask()
        assert g.poll() == ta.TA_OK
        f_o, V_o, u0_o = oracle.sponsor_mask(w.ids, w.cu, oracle_patterns(w), pol)
        np.testing.assert_array_equal(flags.cpu().numpy(), f_o)
        np.testing.assert_array_equal(V.cpu().numpy().view(np.uint32), V_o.view(np.uint32))
        np.testing.assert_array_equal(u0.cpu().numpy().view(np.uint32), u0_o.view(np.uint32))
        return f_o
    finally:
        g.close()


@pytest.mark.parametrize("seed", range(4))
def test_mask_small_alphabet_bit_exact(seed):
    rng = np.random.default_rng(seed)
    pats = [list(rng.integers(0, 4, size=int(rng.integers(1, 9)))) for _ in range(int(rng.integers(1, 12)))]
    spans = [int(rng.integers(1, 65)) for _ in pats]
    buds = [float(rng.integers(1, 30)) for _ in pats]
    lengths = [1, 2, 511, 512, 513, 1700, 0, 37]
    w = _workload(lengths, pats, spans, buds, alphabet=4, seed=seed)
    pol = oracle_policy(4, vocab_size=4, age_steps=seed)
    f = _check_mask(w, pol)
    assert (f & 4).any() and (f & 2).any()


def test_mask_many_patterns_and_vocab():
    rng = np.random.default_rng(9)
    pats = [list(rng.integers(0, tw.VOCAB, size=int(rng.integers(1, 4)))) for _ in range(256)]
    w = _workload([5000, 3000, 9000], pats, [int(rng.integers(1, 33)) for _ in pats], seed=9)
    _check_mask(w, oracle_policy(4, vocab_size=tw.VOCAB))


def test_mask_no_patterns_and_bad_token_id():
    w = _workload([700], [[1, 2]], seed=3)
    w.pattern_ids, w.pattern_budget, w.pattern_span = [], [], []
    f = _check_mask(w, oracle_policy(4))
    assert not f.any()
    # an id outside the vocabulary is reported through the context, and nothing faults
    w2 = _workload([700], [[1, 2]], seed=3)
    w2.ids[123] = tw.VOCAB + 5
    g = Gpu(w2, oracle_policy(4), 4, 1)
    try:
        g.sponsor_mask()
        assert g.poll() == ta.TA_ERR_DEVICE_BOUNDS
        assert g.poll() == ta.TA_OK  # cleared
    finally:
        g.close()


@pytest.mark.parametrize("rank,threshold,budget,span", [(False, 0.5, 15.0, 6), (True, 0.3, 1.0, 6), (True, 0.3, 15.0, 64)])
def test_mask_from_detector_confidences_bit_exact(rank, threshold, budget, span):
    # Section 5.1: anchors from a learned detector's confidences (TA-Learned, TA-LearnRank), ragged batch with
    # sequences shorter than a span, spans that run into each other and across tile borders, NaN and exact-threshold
    # confidences; aged budgets
    lengths = [700, 3, 1, 0, 1500, 513, 64]
    w = _workload(lengths, [[1, 2]], seed=21)
    rng = np.random.default_rng(77)
    conf = rng.random(w.total).astype(np.float32)
    conf[rng.random(w.total) < 0.9] *= 0.25          # most tokens well below either threshold
    conf[rng.integers(0, w.total, 20)] = threshold   # equal is not above
    conf[rng.integers(0, w.total, 5)] = np.nan
    conf[508:516] = 0.97                             # a run of anchors across the first tile border
    pol = oracle_policy(8, age_steps=2)
    g = Gpu(w, pol, 8, 1)
    try:
        flags, V, u0 = g.sponsor_mask_conf(torch.from_numpy(conf).cuda(), threshold, budget, span, rank)
        torch.cuda.synchronize()
        assert g.poll() == ta.TA_OK
        f_o, V_o, u0_o = oracle.sponsor_mask_conf(w.ids, w.cu, conf, threshold, budget, span, rank, pol)
        np.testing.assert_array_equal(flags.cpu().numpy(), f_o)
        np.testing.assert_array_equal(V.cpu().numpy().view(np.uint32), V_o.view(np.uint32))
        np.testing.assert_array_equal(u0.cpu().numpy().view(np.uint32), u0_o.view(np.uint32))
        assert (f_o & ta.TA_FLAG_SPONSORED).any() and (f_o & ta.TA_FLAG_ANCHOR_END).sum() > 50
        # the outputs feed the unchanged selection step: fast-mode selection equals the oracle's
        polf = oracle_policy(8, fast=True, age_steps=2)
        g2 = Gpu(w, polf, 8, 1)
        try:
            idx, cnt = g2.select(flags, V, u0)
            torch.cuda.synchronize()
            idx, cnt = idx.cpu().numpy(), cnt.cpu().numpy()
            for b in range(w.B):
                o, e = int(w.cu[b]), int(w.cu[b + 1])
                io, co = oracle.select(V_o[o:e], u0_o[o:e], 8, polf.n_sink, polf.n_recent, polf.k_protected)
                assert cnt[0, b, 0] == co
                np.testing.assert_array_equal(idx[0, b, 0], io)
        finally:
            g2.close()
    finally:
        g.close()


@pytest.mark.parametrize("D,Cn,total", [(64, 1, 5), (2048, 8, 1000), (4096, 3, 333), (8192, 8, 40)])
def test_embedding_detector_matches_oracle(D, Cn, total):
    # Section 3.2, third detector: largest cosine similarity to the concept embeddings. Token counts that are not a
    # multiple of 16, a padded row stride, planted near-copies of concepts, a zero row and a NaN row.
    g = torch.Generator().manual_seed(100 + D + Cn)
    stride = D + 24
    buf = torch.randn(total, stride, generator=g).to(torch.bfloat16)
    concepts = torch.randn(Cn, D, generator=g).to(torch.bfloat16)
    for i in range(0, total, 7):
        buf[i, :D] = (concepts[i % Cn].float() * 2.0 + 0.05 * torch.randn(D, generator=g)).to(torch.bfloat16)
    if total > 3:
        buf[2, :D] = 0
        buf[3, 5] = float("nan")
    w = _workload([32], [[1, 2]], seed=1)
    gp = Gpu(w, oracle_policy(4), 4, 1)
    try:
        conf = torch.full((total,), -7.0, dtype=torch.float32, device="cuda")
        ta.ta_detect_embedding(gp.ctx, total, buf.cuda(), stride, D, concepts.cuda(), Cn, conf, gp.stream)
        torch.cuda.synchronize()
        assert gp.poll() == ta.TA_OK
        got = conf.cpu().numpy()
        want = oracle.embedding_confidence(bf16_bits(buf[:, :D]), bf16_bits(concepts))
        if total > 3:
            assert np.isnan(got[3]) and got[2] == 0.0
            got, want = np.delete(got, 3), np.delete(want, 3)
        # fp32 tensor-core accumulation (not rounded to nearest) of D bf16 products against double, values in [-1, 1]
        np.testing.assert_allclose(got, want, rtol=0, atol=2e-6 + 4e-9 * D)
        assert want.max() > 0.99
    finally:
        gp.close()


def _score_case(lengths, Hq, Hkv, W, causal=1, seed=0, layers=1, permute=False, scale=0.0, edit=None):
    w = _workload(lengths, [[1, 2]], seed=seed, Hq=Hq, Hkv=Hkv, W=W)
    w.n_layers = layers
    pol = oracle_policy(4, W=W, causal=causal, softmax_scale=scale)
    Qh, Kh, _ = tw.make_qkv(w, range(layers))
    if edit is not None:
        edit(w, Qh, Kh)
    g = Gpu(w, pol, 4, layers)
    try:
        Qd = Qh.cuda()
        if permute:  # token-major storage [L, total, Hkv, d] viewed as [L, Hkv, total, d]
            Kd = Kh.permute(0, 2, 1, 3).contiguous().cuda().permute(0, 2, 1, 3)
        else:
            Kd = Kh.cuda()
        A, P = g.score(Qd, Kd)
        torch.cuda.synchronize()
        assert g.poll() == ta.TA_OK
        A, P = A.cpu().numpy(), P.cpu().numpy()
        G = Hq // Hkv
        for l in range(layers):
            for b in range(w.B):
                o, e = int(w.cu[b]), int(w.cu[b + 1])
                for h in range(Hkv):
                    Ao, Po = oracle.attention(bf16_bits(Qh[l, b, h * G:(h + 1) * G]), unit_kv(w, Kh, l, b, h), e - o,
                                              scale=scale, causal=causal, rho=pol.pension_rho)
                    assert_scores_close(A[l, h, o:e], Ao, f"A l{l} b{b} h{h} n{e - o}")
                    assert_scores_close(P[l, h, o:e], Po, f"P l{l} b{b} h{h} n{e - o}")
        return w, pol, Qh, Kh, Qd, Kd, A, g
    except Exception:
        g.close()
        raise


def test_score_single_tile():
    *_, g = _score_case([100], 8, 2, 32)
    g.close()


def test_score_multi_tile_ragged_tail():
    *_, g = _score_case([1000, 128, 129, 4096 + 37], 8, 2, 32)
    g.close()


def test_score_window_64_two_row_blocks():
    *_, g = _score_case([700, 2500], 8, 2, 64)
    g.close()


def test_score_small_row_count_and_short_sequences():
    # G*W = 8 rows (padded to 128); sequences shorter than the window, of length 1, and empty
    *_, g = _score_case([5, 1, 0, 300, 31], 2, 2, 8)
    g.close()


def test_score_non_causal_and_custom_scale():
    *_, g = _score_case([900], 4, 1, 32, causal=0, scale=0.05)
    g.close()


def test_score_layers_and_strided_keys():
    *_, g = _score_case([1500, 260], 8, 2, 32, layers=3, permute=True)
    g.close()


def test_score_more_units_than_ctas_stays_inside_its_outputs():
    # 160 units of one tile-row each on a persistent grid of fewer CTAs: the grid walks the units in rounds, and the
    # positions of the last round that lie beyond the last unit must do nothing (guard layers behind A and P stay
    # untouched)
    L, guard = 20, 16
    w = _workload([300], [[1, 2]], seed=3, Hq=32, Hkv=8, W=32)
    w.n_layers = L
    pol = oracle_policy(4, W=32)
    Qh, Kh, _ = tw.make_qkv(w, range(L))
    g = Gpu(w, pol, 4, L)
    try:
        A = torch.full((L + guard, w.Hkv, w.total), float("nan"), dtype=torch.float32, device="cuda")
        P = torch.full_like(A, float("nan"))
        Qd, Kd = Qh.cuda(), Kh.cuda()  # held until the kernel has run: a view is only a pointer
        ta.ta_score(g.ctx, g.p, g.batch, w.Hq, w.Hkv, w.d, ta.view(Qd), ta.view(Kd, not w.uniform), None, A, P,
                    g.stream)
        torch.cuda.synchronize()
        assert g.poll() == ta.TA_OK
        assert torch.isnan(A[L:]).all() and torch.isnan(P[L:]).all()
        assert not torch.isnan(A[:L]).any() and not torch.isnan(P[:L]).any()
        G = w.Hq // w.Hkv
        for l in (0, 7, L - 1):
            for h in range(w.Hkv):
                Ao, Po = oracle.attention(bf16_bits(Qh[l, 0, h * G:(h + 1) * G]), unit_kv(w, Kh, l, 0, h), 300,
                                          scale=0.0, causal=1, rho=pol.pension_rho)
                assert_scores_close(A[l, h].cpu().numpy(), Ao, f"A l{l} h{h}")
                assert_scores_close(P[l, h].cpu().numpy(), Po, f"P l{l} h{h}")
    finally:
        g.close()


def test_score_cluster_sizes():
    # 16, 32 and 64 tiles: clusters of 4 and 8 CTAs per unit
    *_, g = _score_case([2048 + 5], 4, 1, 32)
    g.close()
    *_, g = _score_case([8192 - 77], 4, 1, 32, seed=2)
    g.close()


@pytest.mark.parametrize("W", [32, 64])
def test_score_scores_far_above_and_below_the_first_keys(W):
    # keys aligned with one query row score about 68 nats (98 in base 2) above the rest: the running normaliser of
    # that row must survive a jump far beyond anything the row's first keys suggested, early and late in the sequence;
    # and a row whose first 16 keys score far below the rest
    def edit(w, Qh, Kh):
        G = w.Hq // w.Hkv
        q = Qh[0, 0, 1, W - 1].float()           # query head 1 reads KV head 0; the last window row sees every key
        for j in (40, 700, 1290):
            Kh[0, 0, j] = (6.0 * q).to(torch.bfloat16)
        q2 = Qh[0, 0, G + 2, W - 3].float()      # KV head 1
        Kh[0, 1, 0:16] = (-6.0 * q2).to(torch.bfloat16)
        q3 = Qh[0, 1, 0, 5].float()              # second sequence: a spike in its last, masked tile
        Kh[0, 0, int(w.cu[2]) - W + 2] = (6.0 * q3).to(torch.bfloat16)

    *_, g = _score_case([1300, 300], 8, 2, W, seed=7, edit=edit)
    g.close()


@pytest.mark.parametrize("W", [32, 64])
def test_score_with_supplied_lse_matches_two_pass(W):
    w, pol, Qh, Kh, Qd, Kd, A2, g = _score_case([1300, 70], 8, 2, W, seed=5)
    try:
        # log-sum-exp of every window row, from a library softmax in fp64
        G = w.Hq // w.Hkv
        lse = torch.full((1, w.B, w.Hq, w.W), 0.0, dtype=torch.float64)
        for b in range(w.B):
            o, e = int(w.cu[b]), int(w.cu[b + 1])
            n = e - o
            for h in range(w.Hq):
                k = Kh[0, h // G, o:e].double()
                s = (Qh[0, b, h].double() @ k.T) / np.sqrt(128.0)
                pos = torch.arange(n - w.W, n).view(-1, 1)
                s = s.masked_fill(torch.arange(n).view(1, -1) > pos, float("-inf"))
                lse[0, b, h] = torch.where(pos.view(-1) >= 0, torch.logsumexp(s, -1), torch.zeros(w.W).double())
        A1, _ = g.score(Qd, Kd, lse=lse.float().cuda())
        torch.cuda.synchronize()
        assert g.poll() == ta.TA_OK
        A1 = A1.cpu().numpy()
        for h in range(w.Hkv):
            assert_scores_close(A1[0, h], A2[0, h], f"lse path h{h}")
    finally:
        g.close()


def _select_case(w, pol, K, L=1, u_parts=None):
    """Runs mask + (given A, P) select on the GPU and compares with the oracle unit by unit."""
    g = Gpu(w, pol, K, L)
    try:
        flags, V, u0 = g.sponsor_mask()
        A = P = None
        if not pol.fast:
            A, P = u_parts
        idx, cnt = g.select(flags, V, u0, A, P)
        torch.cuda.synchronize()
        assert g.poll() == ta.TA_OK
        idx, cnt = idx.cpu().numpy(), cnt.cpu().numpy()
        f_o, V_o, u0_o = oracle.sponsor_mask(w.ids, w.cu, oracle_patterns(w), pol)
        for l in range(L):
            for b in range(w.B):
                o, e = int(w.cu[b]), int(w.cu[b + 1])
                for h in range(w.Hkv):
                    if pol.fast:
                        u = u0_o[o:e]
                    else:
                        u = oracle.utility(pol.alpha, pol.delta, A[l, h, o:e].cpu().numpy(),
                                           P[l, h, o:e].cpu().numpy(), u0_o[o:e])
                    io, co = oracle.select(V_o[o:e], u, K, pol.n_sink, pol.n_recent, pol.k_protected)
                    assert cnt[l, b, h] == co
                    np.testing.assert_array_equal(idx[l, b, h], io, err_msg=f"l{l} b{b} h{h}")
        return idx, cnt
    finally:
        g.close()


@pytest.mark.parametrize("preset", ["THEOREM", "SEC33", "AUDIT"])
@pytest.mark.parametrize("K", [1, 5, 16, 300])
def test_select_fast_bit_exact(preset, K):
    pats = [[1, 2], [3], [2, 2, 1]]
    w = _workload([1, 3, 17, 600, 1025, 0, 2500], pats, [6, 3, 20], alphabet=6, seed=K)
    _select_case(w, oracle_policy(K, preset, fast=True, vocab_size=6), K)


@pytest.mark.parametrize("K", [16, 2048, 4096])
def test_select_scored_given_scores_bit_exact(K):
    # the same fp32 A and P go to both sides, so the selection must agree exactly, ties included
    w = _workload([3000, 40000, 700], [[5, 6, 7], [9]], seed=K, Hq=4, Hkv=2)
    L = 2
    gen = torch.Generator().manual_seed(K)
    A = torch.rand((L, w.Hkv, w.total), generator=gen).cuda()
    A = (A * 64).round() / 64  # many exact ties
    P = (torch.rand((L, w.Hkv, w.total), generator=gen) * 0.1).cuda()
    _select_case(w, oracle_policy(K, "THEOREM"), K, L, (A, P))


@pytest.mark.parametrize("K", [64, 2048])
def test_select_many_long_units_keys_in_registers_of_big_blocks(K):
    # 48 units of up to 32768 tokens: too many to split each over a cluster, so a block of 1024 threads holds a
    # unit's keys in registers; exact ties, a full-length unit, one just above the 512-thread limit and a short one
    w = _workload([32768, 16385, 20011, 900], [[5, 6, 7], [9]], seed=100 + K, Hq=4, Hkv=2)
    L = 6
    gen = torch.Generator().manual_seed(K)
    A = torch.rand((L, w.Hkv, w.total), generator=gen).cuda()
    A = (A * 128).round() / 128
    P = (torch.rand((L, w.Hkv, w.total), generator=gen) * 0.1).cuda()
    _select_case(w, oracle_policy(K, "THEOREM"), K, L, (A, P))


@pytest.mark.parametrize("lengths", [[100000, 65537, 70], [200000, 131073], [262144]])
def test_select_few_very_long_units_split_over_clusters_of_big_blocks(lengths):
    # few units beyond 65536 tokens: each is split over a cluster of 8 blocks of 1024 threads (16 keys per thread up
    # to 131072 tokens, 32 up to 262144); exact ties across the slices, slices that end inside the last block
    K = 4096
    w = _workload(lengths, [[5, 6, 7], [9]], seed=7 + len(lengths), Hq=2, Hkv=1)
    gen = torch.Generator().manual_seed(len(lengths))
    A = torch.rand((1, w.Hkv, w.total), generator=gen).cuda()
    A = (A * 512).round() / 512
    P = (torch.rand((1, w.Hkv, w.total), generator=gen) * 0.1).cuda()
    P = (P * 256).round() / 256
    _select_case(w, oracle_policy(K, "THEOREM"), K, 1, (A, P))
    _select_case(w, oracle_policy(K, "THEOREM", fast=True), K)


@pytest.mark.parametrize("lengths,L", [([200000], 1), ([32768, 20000, 9000, 700], 6)])
def test_select_three_distinct_utilities_keep_every_pass_crowded(lengths, L):
    # utilities that take three values only (no recency, anchor or frequency term): a third of the keys stays a
    # candidate through every radix pass, so the passes over all keys, the passes of a split unit beyond the second
    # and the tie rule (lowest position first) all run; one unit split over a cluster, and 48 units of one block each
    K = 4096
    w = _workload(lengths, [[5, 6, 7], [9]], seed=31 + L, Hq=4, Hkv=2)
    gen = torch.Generator().manual_seed(L)
    A = (torch.randint(1, 4, (L, w.Hkv, w.total), generator=gen).float() / 4).cuda()
    P = torch.zeros((L, w.Hkv, w.total)).cuda()
    _select_case(w, oracle_policy(K, "THEOREM", beta=0.0, gamma=0.0, lam=0.0), K, L, (A, P))


def test_select_sponsored_overflow_and_precedence():
    # far more sponsored tokens than protected slots: nearest-to-anchor first, earlier anchors win ties
    w = _workload([5000], [[1]], [12], alphabet=40, seed=4)
    idx, cnt = _select_case(w, oracle_policy(32, "THEOREM", fast=True, vocab_size=40), 32)
    assert cnt[0, 0, 0] == 32


def test_compact_strided_and_zero_fill():
    w = _workload([300, 50, 0, 1000], [[1, 2]], seed=8, Hq=4, Hkv=2)
    K = 64
    pol = oracle_policy(K, fast=True)
    _, Kh, Vh = tw.make_qkv(w, [0, 1], need_q=False)
    g = Gpu(w, pol, K, 2)
    try:
        Kd = Kh.permute(0, 2, 1, 3).contiguous().cuda().permute(0, 2, 1, 3)  # token-major storage
        Vd = Vh.cuda()
        flags, V, u0 = g.sponsor_mask()
        idx, cnt = g.select(flags, V, u0)
        ko, vo = g.compact(Kd, Vd, idx, cnt)
        torch.cuda.synchronize()
        assert g.poll() == ta.TA_OK
        idx, cnt = idx.cpu().numpy(), cnt.cpu().numpy()
        for l in range(2):
            for b in range(w.B):
                for h in range(w.Hkv):
                    want_k = oracle.compact(unit_kv(w, Kh, l, b, h), idx[l, b, h], int(cnt[l, b, h]), K)
                    want_v = oracle.compact(unit_kv(w, Vh, l, b, h), idx[l, b, h], int(cnt[l, b, h]), K)
                    np.testing.assert_array_equal(bf16_bits(ko[l, b, h]), want_k)
                    np.testing.assert_array_equal(bf16_bits(vo[l, b, h]), want_v)
        assert cnt[0, 1, 0] == 50 and cnt[0, 2, 0] == 0
    finally:
        g.close()


@pytest.mark.parametrize("fast,K", [(False, 24), (True, 24), (False, 12)])
def test_compress_equals_steps_and_oracle(fast, K):
    # K = 12 in scored mode: the selection kernel gathers the rows itself (also for the sequence shorter than K)
    w = _workload([900, 2100, 64, 10], [[4, 5], [6]], seed=12, Hq=8, Hkv=2, W=32)
    L = 2
    pol = oracle_policy(K, "THEOREM", fast=fast, W=32)
    Qh, Kh, Vh = tw.make_qkv(w, range(L))
    g = Gpu(w, pol, K, L)
    try:
        Qd, Kd, Vd = Qh.cuda(), Kh.cuda(), Vh.cuda()
        idx, cnt, ko, vo = g.compress(Qd, Kd, Vd, epoch=7)
        idx2, cnt2, ko2, vo2 = g.compress(Qd, Kd, Vd, epoch=7)  # reuses the per-sequence results
        torch.cuda.synchronize()
        assert g.poll() == ta.TA_OK
        assert torch.equal(idx, idx2) and torch.equal(cnt, cnt2) and torch.equal(ko, ko2) and torch.equal(vo, vo2)
        idx, cnt = idx.cpu().numpy(), cnt.cpu().numpy()
        f_o, V_o, u0_o = oracle.sponsor_mask(w.ids, w.cu, oracle_patterns(w), pol)
        exact = 0
        for l in range(L):
            for b in range(w.B):
                for h in range(w.Hkv):
                    A, P, u, io, co = oracle_unit(w, pol, K, Qh, Kh, l, b, h, V_o, u0_o)
                    same = assert_selection_matches(idx[l, b, h], cnt[l, b, h], io, co, u, f"l{l} b{b} h{h}")
                    exact += same
                    if fast:
                        assert same
                    sel, c = idx[l, b, h], int(cnt[l, b, h])
                    np.testing.assert_array_equal(bf16_bits(ko[l, b, h]), oracle.compact(unit_kv(w, Kh, l, b, h), sel, c, K))
                    np.testing.assert_array_equal(bf16_bits(vo[l, b, h]), oracle.compact(unit_kv(w, Vh, l, b, h), sel, c, K))
        assert exact >= 0.9 * L * w.B * w.Hkv
    finally:
        g.close()


@pytest.mark.parametrize("with_second", [False, True])
def test_compress_with_external_scores_bit_exact(with_second):
    # Section 4.5: sponsorship on top of another method's importance score. Here the provider is a SnapKV-style
    # max-pooled attention mass (computed on the host) and, optionally, a second arbitrary term weighted by delta.
    w = _workload([1200, 300, 40, 2600], [[4, 5], [9]], seed=31, Hq=8, Hkv=2, W=32)
    K, L = 24, 2
    pol = oracle_policy(K, "SEC33", W=32)
    Qh, Kh, Vh = tw.make_qkv(w, range(L))
    rng = np.random.default_rng(3)
    G = w.Hq // w.Hkv
    score = np.zeros((L, w.Hkv, w.total), np.float32)
    for l in range(L):
        for b in range(w.B):
            o, e = int(w.cu[b]), int(w.cu[b + 1])
            for h in range(w.Hkv):
                A, _ = oracle.attention(bf16_bits(Qh[l, b, h * G:(h + 1) * G]), unit_kv(w, Kh, l, b, h), e - o)
                pad = np.pad(A, 3, constant_values=-np.inf)
                score[l, h, o:e] = np.max(np.stack([pad[k:k + e - o] for k in range(7)]), axis=0)
    score2 = rng.standard_normal(score.shape).astype(np.float32) if with_second else None
    g = Gpu(w, pol, K, L)
    try:
        s2 = None if score2 is None else torch.from_numpy(score2).cuda()
        idx, cnt, ko, vo = g.compress_scores(torch.from_numpy(score).cuda(), s2, Kh.cuda(), Vh.cuda())
        torch.cuda.synchronize()
        assert g.poll() == ta.TA_OK
        idx, cnt = idx.cpu().numpy(), cnt.cpu().numpy()
        f_o, V_o, u0_o = oracle.sponsor_mask(w.ids, w.cu, oracle_patterns(w), pol)
        for l in range(L):
            for b in range(w.B):
                o, e = int(w.cu[b]), int(w.cu[b + 1])
                for h in range(w.Hkv):
                    u = oracle.utility(pol.alpha, pol.delta, score[l, h, o:e],
                                       None if score2 is None else score2[l, h, o:e], u0_o[o:e])
                    io, co = oracle.select(V_o[o:e], u, K, pol.n_sink, pol.n_recent, pol.k_protected)
                    assert cnt[l, b, h] == co
                    np.testing.assert_array_equal(idx[l, b, h], io, err_msg=f"l{l} b{b} h{h}")
                    np.testing.assert_array_equal(bf16_bits(ko[l, b, h]), oracle.compact(unit_kv(w, Kh, l, b, h), io, co, K))
                    np.testing.assert_array_equal(bf16_bits(vo[l, b, h]), oracle.compact(unit_kv(w, Vh, l, b, h), io, co, K))
    finally:
        g.close()


def test_compress_with_budgets_per_layer_and_head_bit_exact():
    # Section 4.5 with a provider that sets its own budget per layer (pyramid) and per head: every unit must come out
    # as if the whole call had used that unit's budget (sinks, recents and protected pool sized from it)
    w = _workload([1500, 90, 12, 700], [[4, 5], [9]], seed=33, Hq=8, Hkv=2, W=32)
    L, K_max = 3, 40
    budgets = np.array([[40, 24], [24, 9], [16, 40]], np.int32)  # 5 distinct values; 9 and 16 < a short sequence's n
    pol = oracle_policy(K_max, "THEOREM", W=32)
    Qh, Kh, Vh = tw.make_qkv(w, range(L))
    rng = np.random.default_rng(4)
    score = rng.random((L, w.Hkv, w.total)).astype(np.float32)
    score[:, :, ::7] = 0.5  # ties
    g = Gpu(w, pol, K_max, L, n_budget_classes=5)
    try:
        idx, cnt, ko, vo = g.compress_scores_budgets(budgets, torch.from_numpy(score).cuda(), None, Kh.cuda(), Vh.cuda())
        torch.cuda.synchronize()
        assert g.poll() == ta.TA_OK
        idx, cnt = idx.cpu().numpy(), cnt.cpu().numpy()
        f_o, V_o, u0_o = oracle.sponsor_mask(w.ids, w.cu, oracle_patterns(w), pol)
        for l in range(L):
            for b in range(w.B):
                o, e = int(w.cu[b]), int(w.cu[b + 1])
                for h in range(w.Hkv):
                    Ku = int(budgets[l, h])
                    u = oracle.utility(pol.alpha, pol.delta, score[l, h, o:e], None, u0_o[o:e])
                    io, co = oracle.select(V_o[o:e], u, Ku, pol.n_sink, pol.n_recent, pol.k_protected)
                    assert cnt[l, b, h] == co == min(Ku, e - o)
                    np.testing.assert_array_equal(idx[l, b, h, :Ku], io, err_msg=f"l{l} b{b} h{h}")
                    assert (idx[l, b, h, Ku:] == -1).all()
                    for out, src in ((ko, Kh), (vo, Vh)):
                        got = bf16_bits(out[l, b, h])
                        np.testing.assert_array_equal(got[:Ku], oracle.compact(unit_kv(w, src, l, b, h), io, co, Ku))
                        assert not got[Ku:].any()
        # the same call twice, and after a call of another entry point on the same context: same result
        idx2, cnt2, ko2, vo2 = g.compress_scores_budgets(budgets, torch.from_numpy(score).cuda(), None, Kh.cuda(), Vh.cuda())
        torch.cuda.synchronize()
        assert np.array_equal(idx2.cpu().numpy(), idx) and torch.equal(ko2, ko) and torch.equal(vo2, vo)
        # argument checks on the host
        bad = budgets.copy()
        bad[0, 0] = K_max + 1
        with pytest.raises(ta.TAError) as ei:
            g.compress_scores_budgets(bad, torch.from_numpy(score).cuda(), None, Kh.cuda(), Vh.cuda())
        assert ei.value.status == ta.TA_ERR_INVALID_ARG
        small = Gpu(w, pol, K_max, L)  # scratch without room for budget classes
        try:
            with pytest.raises(ta.TAError) as ei:
                small.compress_scores_budgets(budgets, torch.from_numpy(score).cuda(), None, Kh.cuda(), Vh.cuda())
            assert ei.value.status == ta.TA_ERR_SCRATCH_TOO_SMALL
        finally:
            small.close()
    finally:
        g.close()


def test_compress_budgets_with_own_attention_scores():
    # budgets per (layer, head) with TA's own attention terms: every unit as the one-budget path with K = its budget
    w = _workload([1100, 200, 2300], [[4, 5], [9]], seed=35, Hq=8, Hkv=2, W=32)
    L, K_max = 2, 48
    budgets = np.array([[48, 12], [20, 48]], np.int32)
    pol = oracle_policy(K_max, "THEOREM", W=32)
    Qh, Kh, Vh = tw.make_qkv(w, range(L))
    g = Gpu(w, pol, K_max, L, n_budget_classes=3)
    try:
        idx, cnt, ko, vo = g.compress_budgets(budgets, Qh.cuda(), Kh.cuda(), Vh.cuda())
        torch.cuda.synchronize()
        assert g.poll() == ta.TA_OK
        idx, cnt = idx.cpu().numpy(), cnt.cpu().numpy()
        f_o, V_o, u0_o = oracle.sponsor_mask(w.ids, w.cu, oracle_patterns(w), pol)
        exact = 0
        for l in range(L):
            for b in range(w.B):
                for h in range(w.Hkv):
                    Ku = int(budgets[l, h])
                    A, P, u, io, co = oracle_unit(w, pol, Ku, Qh, Kh, l, b, h, V_o, u0_o)
                    exact += assert_selection_matches(idx[l, b, h, :Ku], cnt[l, b, h], io, co, u, f"l{l} b{b} h{h}")
                    assert (idx[l, b, h, Ku:] == -1).all()
                    sel, c = idx[l, b, h, :Ku], int(cnt[l, b, h])
                    for out, src in ((ko, Kh), (vo, Vh)):
                        got = bf16_bits(out[l, b, h])
                        np.testing.assert_array_equal(got[:Ku], oracle.compact(unit_kv(w, src, l, b, h), sel, c, Ku))
                        assert not got[Ku:].any()
        assert exact >= 0.9 * L * w.B * w.Hkv
    finally:
        g.close()


@pytest.mark.parametrize("preset", ["THEOREM", "SEC33"])
def test_compress_allheads_shared_selection(preset):
    # Eq. 1's A_i summed over all query heads of the layer: one retained set per (layer, sequence), the same for every
    # KV head; ragged batch, two layers, a sequence shorter than the window and one shorter than the budget
    w = _workload([1500, 20, 700, 9], [[4, 5], [9]], seed=41, Hq=8, Hkv=4, W=16)
    K, L = 12, 2
    pol = oracle_policy(K, preset, W=16)
    Qh, Kh, Vh = tw.make_qkv(w, range(L))
    g = Gpu(w, pol, K, L)
    try:
        idx, cnt, ko, vo = g.compress_allheads(Qh.cuda(), Kh.cuda(), Vh.cuda())
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
                    np.testing.assert_array_equal(bf16_bits(ko[l, b, h]), oracle.compact(unit_kv(w, Kh, l, b, h), idx[l, b, h], c, K))
                    np.testing.assert_array_equal(bf16_bits(vo[l, b, h]), oracle.compact(unit_kv(w, Vh, l, b, h), idx[l, b, h], c, K))
        assert exact >= L * w.B - 1
    finally:
        g.close()


def test_host_argument_checks():
    w = _workload([300], [[1, 2]], seed=1)
    pol = oracle_policy(8, fast=True)
    g = Gpu(w, pol, 8, 1)
    try:
        _, Kh, Vh = tw.make_qkv(w, [0], need_q=False)
        Kd, Vd = Kh.cuda(), Vh.cuda()
        idx = torch.zeros((1, 1, 2, 8), dtype=torch.int32, device="cuda")
        cnt = torch.zeros((1, 1, 2), dtype=torch.int32, device="cuda")
        out = torch.zeros((1, 1, 2, 8, 128), dtype=torch.bfloat16, device="cuda")
        L = ta.binding.lib()
        import ctypes as C
        vk, vv = ta.view(Kd, True), ta.view(Vd, True)
        call = lambda d, K, vk=vk: L.ta_compact_kv(g.ctx, C.byref(g.batch), 2, d, K, vk, vv, idx.data_ptr(),
                                                   cnt.data_ptr(), out.data_ptr(), out.data_ptr(), None)
        assert call(64, 8) == ta.TA_ERR_UNSUPPORTED
        assert call(128, 5000) == ta.TA_ERR_UNSUPPORTED
        assert call(128, 0) == ta.TA_ERR_INVALID_ARG
        bad = ta.ta_bf16_view(vk.ptr + 2, vk.stride_l, vk.stride_b, vk.stride_h, vk.stride_n)
        assert call(128, 8, bad) == ta.TA_ERR_ALIGNMENT
        small = ta.ta_ctx_create(0, 1024)
        st = L.ta_sponsor_mask(small, g.pats, C.byref(g.p), C.byref(g.batch), g.ids.data_ptr(), idx.data_ptr(),
                               idx.data_ptr(), idx.data_ptr(), None)
        assert st == ta.TA_ERR_SCRATCH_TOO_SMALL
        ta.ta_ctx_destroy(small)
        assert g.poll() == ta.TA_OK
    finally:
        g.close()


def test_host_argument_checks_of_the_widened_entry_points():
    import ctypes as C
    w = _workload([300], [[1, 2]], seed=1)
    g = Gpu(w, oracle_policy(8), 8, 1)
    gf = Gpu(w, oracle_policy(8, fast=True), 8, 1)
    try:
        L = ta.binding.lib()
        t = w.total
        buf = torch.zeros(max(t, 64) * 64, dtype=torch.float32, device="cuda")
        p = buf.data_ptr()
        conf = lambda thr, bud, span: L.ta_sponsor_mask_conf(g.ctx, C.byref(g.p), C.byref(g.batch), g.ids.data_ptr(), p,
                                                            C.c_float(thr), C.c_float(bud), span, 0, p, p, p, None)
        assert conf(0.5, 15.0, 0) == ta.TA_ERR_INVALID_ARG
        assert conf(0.5, 15.0, 65) == ta.TA_ERR_UNSUPPORTED
        assert conf(float("nan"), 15.0, 6) == ta.TA_ERR_INVALID_ARG
        assert conf(0.5, 15.0, 6) == ta.TA_OK
        # caller-supplied scores and the shared selection are scored-mode entry points
        _, Kh, Vh = tw.make_qkv(w, [0], need_q=False)
        Kd, Vd = Kh.cuda(), Vh.cuda()
        vk, vv = ta.view(Kd, True), ta.view(Vd, True)
        args = (g.ids.data_ptr(), p, None, vk, vv, 0, p, p, p, p, None)
        assert L.ta_compress_scores(gf.ctx, gf.pats, C.byref(gf.p), C.byref(gf.batch), 2, 128, 8, *args) == ta.TA_ERR_INVALID_ARG
        assert L.ta_compress_scores(g.ctx, g.pats, C.byref(g.p), C.byref(g.batch), 2, 128, 8, g.ids.data_ptr(), None,
                                    None, vk, vv, 0, p, p, p, p, None) == ta.TA_ERR_INVALID_ARG
        assert L.ta_compress_allheads(gf.ctx, gf.pats, C.byref(gf.p), C.byref(gf.batch), 8, 2, 128, 8,
                                      g.ids.data_ptr(), vk, vk, vv, 0, p, p, p, p, None) == ta.TA_ERR_INVALID_ARG
        # embedding detector: width, concept count, alignment
        det = lambda D, Cn, ptr=p, stride=None: L.ta_detect_embedding(g.ctx, 10, ptr, D if stride is None else stride,
                                                                      D, p, Cn, p, None)
        assert det(48, 2) == ta.TA_ERR_UNSUPPORTED          # not a multiple of 32
        assert det(16384, 2) == ta.TA_ERR_UNSUPPORTED
        assert det(64, 9) == ta.TA_ERR_UNSUPPORTED
        assert det(64, 0) == ta.TA_ERR_INVALID_ARG
        assert det(64, 2, p + 2) == ta.TA_ERR_ALIGNMENT
        assert det(64, 2, p, 60) == ta.TA_ERR_INVALID_ARG   # stride shorter than a row
        # decode step: state description and scratch
        st = ta.ta_stream()
        st.n_layers, st.batch, st.Hkv, st.K, st.cache_len = 1, 1, 2, 8, 0
        for k in ("pos", "slot", "tok", "A", "P", "V", "S", "next_slot", "n_seen", "hist", "tok_ring", "anc_B", "anc_L"):
            setattr(st, k, p)
        step = lambda: L.ta_stream_step(g.ctx, g.pats, C.byref(g.p), C.byref(st), p, p, p, None)
        st.cache_len = 9
        assert step() == ta.TA_ERR_INVALID_ARG
        st.cache_len, st.K = 0, 5000
        assert step() == ta.TA_ERR_UNSUPPORTED
        st.K, st.hist = 8, None
        assert step() == ta.TA_ERR_INVALID_ARG
        st.hist = p
        small = ta.ta_ctx_create(0, 64)
        assert L.ta_stream_step(small, g.pats, C.byref(g.p), C.byref(st), p, p, p, None) == ta.TA_ERR_SCRATCH_TOO_SMALL
        ta.ta_ctx_destroy(small)
        assert st.cache_len == 0  # refused calls leave the state description alone
        torch.cuda.synchronize()
        assert g.poll() == ta.TA_OK
    finally:
        g.close()
        gf.close()


@pytest.mark.parametrize("fast", [False, True])
@pytest.mark.parametrize("pinned", [True, False])
def test_compress_host_matches_device_path(fast, pinned):
    """The host-buffer entry point (staged copies; pinned caches gathered in place) gives the device path's result."""
    w = tw.config1(n=1500, Hq=8, Hkv=2)  # uniform batch of one sequence
    K, L = 16, 2
    pol = oracle_policy(K, "THEOREM", fast=fast, W=w.W)
    Qh, Kh, Vh = tw.make_qkv(w, range(L))
    g = Gpu(w, pol, K, L)
    try:
        idx, cnt, ko, vo = g.compress(Qh.cuda(), Kh.cuda(), Vh.cuda())
        torch.cuda.synchronize()
        pin = (lambda t: t.pin_memory()) if pinned else (lambda t: t)
        ids_h = pin(torch.from_numpy(w.ids))
        q_h, k_h, v_h = pin(Qh.contiguous()), pin(Kh.contiguous()), pin(Vh.contiguous())
        ko_h, vo_h = pin(torch.zeros(ko.shape, dtype=torch.bfloat16)), pin(torch.zeros(vo.shape, dtype=torch.bfloat16))
        idx_h, cnt_h = pin(torch.zeros(idx.shape, dtype=torch.int32)), pin(torch.zeros(cnt.shape, dtype=torch.int32))
        hb = ta.make_batch(L, w.B, int(w.lengths[0]), w.max_n, w.total, None)
        nbytes = ta.ta_compress_host_workspace_bytes(hb, w.Hq, w.Hkv, w.d, K, g.p)
        ws = torch.empty(nbytes + 256, dtype=torch.uint8, device="cuda")
        ws_ptr = (ws.data_ptr() + 255) // 256 * 256
        ta.ta_compress_host(g.ctx, g.pats, g.p, hb, w.Hq, w.Hkv, w.d, K, ids_h, None if fast else q_h, k_h, v_h, ko_h,
                            vo_h, idx_h, cnt_h, ws_ptr, nbytes, g.stream)
        torch.cuda.synchronize()
        assert g.poll() == ta.TA_OK
        assert torch.equal(idx_h, idx.cpu()) and torch.equal(cnt_h, cnt.cpu())
        assert torch.equal(ko_h.view(torch.int16), ko.cpu().view(torch.int16))
        assert torch.equal(vo_h.view(torch.int16), vo.cpu().view(torch.int16))
    finally:
        g.close()


def test_fused_path_is_deterministic():
    """Three runs on the same inputs give bit-identical indices and caches (no atomics on the data path decide
    anything: histograms are integer, ties break by position)."""
    w = _workload([2500, 700, 4100], [[4, 5], [6]], seed=31, Hq=8, Hkv=2, W=32)
    K, L = 40, 2
    pol = oracle_policy(K, "THEOREM", W=32)
    Qh, Kh, Vh = tw.make_qkv(w, range(L))
    g = Gpu(w, pol, K, L)
    try:
        Qd, Kd, Vd = Qh.cuda(), Kh.cuda(), Vh.cuda()
        ref = None
        for _ in range(3):
            out = g.compress(Qd, Kd, Vd)
            torch.cuda.synchronize()
            if ref is None:
                ref = out
            else:
                for a, b in zip(ref, out):
                    assert torch.equal(a.view(torch.int16) if a.dtype == torch.bfloat16 else a,
                                       b.view(torch.int16) if b.dtype == torch.bfloat16 else b)
        assert g.poll() == ta.TA_OK
    finally:
        g.close()


def test_score_general_window_sizes():
    # windows that do not divide 32 use per-element pension weights: 96 rows (one row block) and 192 rows (two)
    *_, g = _score_case([777, 130], 4, 1, 24, seed=7)
    g.close()
    *_, g = _score_case([1500], 4, 1, 48, seed=8)
    g.close()


def test_score_without_pension_output():
    w, pol, Qh, Kh, Qd, Kd, A_ref, g = _score_case([900, 260], 8, 2, 32, seed=9)
    try:
        A, P = g.score(Qd, Kd, want_P=False)
        torch.cuda.synchronize()
        assert P is None and g.poll() == ta.TA_OK
        np.testing.assert_allclose(A.cpu().numpy(), A_ref, rtol=1e-5, atol=1e-7)
    finally:
        g.close()


def test_compress_with_zero_pension_weight():
    # delta = 0: the fused kernel skips the pension sums altogether
    w = _workload([1200, 300], [[4, 5]], seed=14, Hq=8, Hkv=2, W=32)
    K = 20
    pol = oracle_policy(K, "SEC33", W=32, delta=0.0)
    Qh, Kh, Vh = tw.make_qkv(w, [0])
    g = Gpu(w, pol, K, 1)
    try:
        idx, cnt, ko, vo = g.compress(Qh.cuda(), Kh.cuda(), Vh.cuda())
        torch.cuda.synchronize()
        assert g.poll() == ta.TA_OK
        idx, cnt = idx.cpu().numpy(), cnt.cpu().numpy()
        f_o, V_o, u0_o = oracle.sponsor_mask(w.ids, w.cu, oracle_patterns(w), pol)
        for b in range(w.B):
            for h in range(w.Hkv):
                A, P, u, io, co = oracle_unit(w, pol, K, Qh, Kh, 0, b, h, V_o, u0_o)
                assert_selection_matches(idx[0, b, h], cnt[0, b, h], io, co, u, f"b{b} h{h}")
    finally:
        g.close()
