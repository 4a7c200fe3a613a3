"""Pins the CPU oracle to things other than itself: values printed in the paper, closed forms, invariants,
library routines on special cases, and exhaustive search on tiny inputs. No GPU involved."""
import itertools
import os
import re

import numpy as np
import pytest
import torch

import oracle

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _rows(name):
    out = []
    with open(os.path.join(GOLD, name)) as f:
        for line in f:
            line = line.strip()
            if line and not line.startswith("#"):
                out.append(line.split())
    return out


def bf16_bits(x: torch.Tensor) -> np.ndarray:
    return x.to(torch.bfloat16).contiguous().view(torch.int16).numpy().view(np.uint16)


# ------------------------------------------------------------------------------------------------ vouchers (Eq. 2)
def test_voucher_closed_form_and_printed_value():
    ids = np.array([1, 2, 3, 4, 5, 6, 7, 8, 9, 10], np.int32)
    pats = oracle.Patterns([[2]])
    atok, aend, Be, Le = oracle.anchors(ids, pats)
    V = oracle.vouchers(aend, Be, Le)
    assert V[0] == 0 and V[1] == 0  # the anchor itself is not sponsored: i < j
    for k, exact, printed in _rows("voucher_b15_l6.txt"):
        k = int(k)
        assert V[1 + k] == pytest.approx(float(exact), rel=2e-7)
        if printed != "-":
            assert round(float(V[1 + k]), 1) == float(printed)
    assert V[8] == 0 and V[9] == 0  # j <= i + L


def test_voucher_overlap_adds_and_clips_at_end():
    # anchors (id 2) at positions 1 and 4, L = 6, n = 9: position j gets 15*0.8^(j-1) [j<=7] + 15*0.8^(j-4) [j>4]
    ids = np.array([0, 2, 0, 0, 2, 0, 0, 0, 0], np.int32)
    atok, aend, Be, Le = oracle.anchors(ids, oracle.Patterns([[2]]))
    V = oracle.vouchers(aend, Be, Le)
    for j in range(9):
        want = 0.0
        if 1 < j <= 7:
            want += 15 * 0.8 ** (j - 1)
        if 4 < j <= 10:
            want += 15 * 0.8 ** (j - 4)
        assert V[j] == pytest.approx(want, rel=1e-6, abs=1e-12)
    # the second span would run to position 10 but the sequence stops at 8: nothing is written past the end
    assert V.shape[0] == 9


def test_voucher_budget_decay_and_custom_span():
    ids = np.array([0, 2, 0, 0, 0, 0], np.int32)
    pats = oracle.Patterns([[2]], budget=[10.0], span=[3])
    atok, aend, Be, Le = oracle.anchors(ids, pats, budget_decay=0.9, age_steps=2)
    assert Be[1] == pytest.approx(10 * 0.81, rel=1e-6)  # B^(t+1) = 0.9 B^(t)  (Section 3.2)
    V = oracle.vouchers(aend, Be, Le)
    np.testing.assert_allclose(V, [0, 0, 8.1 * 0.8, 8.1 * 0.64, 8.1 * 0.512, 0], rtol=1e-6)


# ------------------------------------------------------------------------------------------------ matcher
def _regex_matches(ids, pats):
    """All pattern occurrences found with the standard library's regex engine on a string encoding."""
    s = "".join(chr(ord("a") + int(t)) for t in ids)
    out = []
    for p, pat in enumerate(pats):
        ps = "".join(chr(ord("a") + int(t)) for t in pat)
        for m in re.finditer("(?=" + re.escape(ps) + ")", s):
            out.append((p, m.start(), m.start() + len(pat) - 1))
    return out


@pytest.mark.parametrize("seed", range(8))
def test_matcher_against_regex_search(seed):
    rng = np.random.default_rng(seed)
    n = int(rng.integers(1, 60))
    ids = rng.integers(0, 4, size=n).astype(np.int32)
    pats = [list(rng.integers(0, 4, size=int(rng.integers(1, 5)))) for _ in range(int(rng.integers(1, 5)))]
    spans = [int(rng.integers(1, 8)) for _ in pats]
    buds = [float(rng.integers(1, 20)) for _ in pats]
    atok, aend, Be, Le = oracle.anchors(ids, oracle.Patterns(pats, buds, spans))
    want_tok = np.zeros(n, np.uint8)
    ends = {}
    for p, s, e in _regex_matches(ids, pats):
        want_tok[s:e + 1] = 1
        ends.setdefault(e, []).append(p)
    np.testing.assert_array_equal(atok, want_tok)
    for e in range(n):
        if e in ends:
            # longest pattern wins, then the lowest index
            best = sorted(ends[e], key=lambda p: (-len(pats[p]), p))[0]
            assert aend[e] == 1 and Le[e] == spans[best] and Be[e] == buds[best]
        else:
            assert aend[e] == 0 and Le[e] == 0 and Be[e] == 0


def test_matcher_prefix_decoy_and_sequence_boundary():
    pats = oracle.Patterns([[5, 6, 7]])
    # decoy: proper prefix 5 6 followed by a different id -> no anchor, no S flag
    atok, aend, _, _ = oracle.anchors(np.array([1, 5, 6, 9, 5, 6, 7, 1], np.int32), pats)
    np.testing.assert_array_equal(atok, [0, 0, 0, 0, 1, 1, 1, 0])
    np.testing.assert_array_equal(aend, [0, 0, 0, 0, 0, 0, 1, 0])
    # a pattern straddling two sequences of a packed batch must not match
    ids = np.array([1, 5, 6, 7, 1, 1], np.int32)
    cu = np.array([0, 3, 6], np.int32)
    flags, V, u0 = oracle.sponsor_mask(ids, cu, pats, oracle.Policy(vocab_size=16))
    assert flags.sum() == 0 and V.sum() == 0


# ------------------------------------------------------------------------------------------------ utility (Eq. 1, 3)
def test_utility_hand_example():
    rows = _rows("utility_example.txt")
    ids = np.array([int(r[1]) for r in rows], np.int32)
    A = np.array([float(r[2]) for r in rows], np.float32)
    P = np.array([float(r[3]) for r in rows], np.float32)
    u0_want = np.array([float(r[4]) for r in rows])
    u_want = np.array([float(r[5]) for r in rows])
    pats = oracle.Patterns([[9]], budget=[15.0], span=[2])
    atok, aend, Be, Le = oracle.anchors(ids, pats)
    V = oracle.vouchers(aend, Be, Le)
    u0 = oracle.static_utility(ids, atok, V)
    np.testing.assert_allclose(u0, u0_want, atol=2e-6)
    u = oracle.utility(1.0, 0.2, A, P, u0)
    np.testing.assert_allclose(u, u_want, atol=2e-6)
    # TA-Fast (Eq. 3) is Eq. 1 with alpha = delta = 0, exactly
    np.testing.assert_array_equal(oracle.utility(0.0, 0.0, A, P, u0), u0)
    # the histogram route counts the same occurrences
    np.testing.assert_array_equal(oracle.static_utility(ids, atok, V, vocab=16), u0)


def test_static_utility_hist_equals_direct_count():
    rng = np.random.default_rng(3)
    ids = rng.integers(0, 50, size=500).astype(np.int32)
    atok, aend, Be, Le = oracle.anchors(ids, oracle.Patterns([[7, 8], [3]]))
    V = oracle.vouchers(aend, Be, Le)
    np.testing.assert_array_equal(oracle.static_utility(ids, atok, V), oracle.static_utility(ids, atok, V, vocab=50))


# ------------------------------------------------------------------------------------------------ attention terms
def _torch_attention(Q, K, n, causal, rho, scale=None):
    """Column sums of a library softmax in fp64. Q [G,W,d], K [n,d] float64 tensors."""
    G, W, d = Q.shape
    Wp = min(W, n)
    scale = scale or 1.0 / np.sqrt(d)
    Qv = Q[:, W - Wp:, :]
    s = torch.einsum("gtc,ic->gti", Qv, K) * scale
    pos = torch.arange(n - Wp, n).view(1, Wp, 1)
    if causal:
        s = s.masked_fill(torch.arange(n).view(1, 1, n) > pos, float("-inf"))
    a = torch.softmax(s, dim=-1)
    w = (1 - rho) * rho ** torch.arange(Wp - 1, -1, -1, dtype=torch.float64)
    return a.sum((0, 1)), (a * w.view(1, Wp, 1)).sum((0, 1))


@pytest.mark.parametrize("G,W,n,causal", [(1, 1, 17, 1), (4, 8, 50, 1), (4, 8, 50, 0), (2, 16, 5, 1), (3, 5, 33, 1)])
def test_attention_against_library_softmax(G, W, n, causal):
    torch.manual_seed(G * 100 + W + n)
    d = 16
    Q = torch.randn(G, W, d).to(torch.bfloat16)
    K = torch.randn(n, d).to(torch.bfloat16)
    A, P = oracle.attention(bf16_bits(Q), bf16_bits(K), n, causal=causal, rho=0.9)
    Aw, Pw = _torch_attention(Q.double(), K.double(), n, causal, 0.9)
    np.testing.assert_allclose(A, Aw.numpy(), rtol=1e-6, atol=1e-9)
    np.testing.assert_allclose(P, Pw.numpy(), rtol=1e-6, atol=1e-9)
    Wp = min(W, n)
    assert A.sum() == pytest.approx(G * Wp, rel=1e-6)  # every softmax row sums to one
    assert P.sum() == pytest.approx(G * (1 - 0.9 ** Wp), rel=1e-6)


def test_attention_equal_keys_and_causal_zeros():
    n, W, d = 12, 4, 8
    Q = torch.randn(1, W, d).to(torch.bfloat16)
    K = torch.ones(n, d).to(torch.bfloat16)
    A, P = oracle.attention(bf16_bits(Q), bf16_bits(K), n, causal=1, rho=0.5)
    # row t sits at position q = n-W+t and spreads its mass evenly over q+1 keys
    want = np.zeros(n)
    for t in range(W):
        q = n - W + t
        want[: q + 1] += 1.0 / (q + 1)
    np.testing.assert_allclose(A, want, rtol=1e-6)
    # the last key is visible to the last row only
    assert A[n - 1] == pytest.approx(1.0 / n, rel=1e-6)


def test_attention_rho_zero_is_last_row():
    torch.manual_seed(5)
    n, W, d = 20, 6, 8
    Q = torch.randn(2, W, d).to(torch.bfloat16)
    K = torch.randn(n, d).to(torch.bfloat16)
    _, P = oracle.attention(bf16_bits(Q), bf16_bits(K), n, causal=1, rho=0.0)
    s = (Q[:, -1, :].double() @ K.double().T) / np.sqrt(d)
    want = torch.softmax(s, -1).sum(0)
    np.testing.assert_allclose(P, want.numpy(), rtol=1e-6)


# ------------------------------------------------------------------------------------------------ selection
def _exhaustive(V, u, K, n_sink, n_recent, k_prot):
    """Section 3.3 by exhaustive search: the protected pool is the subset of sponsored candidates of its size
    with the largest voucher sum; the main pool the subset of the rest with the largest utility sum."""
    n = len(u)
    K_eff = min(K, n)
    if K_eff == n:
        return list(range(n))
    p = K_eff - n_sink - n_recent if k_prot < 0 else k_prot
    p = max(0, min(p, K_eff))
    K_main = K_eff - p
    order = list(range(min(n_sink, n))) + [n - 1 - r for r in range(min(n_recent, n))]
    mand = []
    for i in order:
        if i not in mand and len(mand) < K_main:
            mand.append(i)
    cand = [i for i in range(n) if i not in mand and V[i] > 0]
    take = min(p, len(cand))
    prot = max(itertools.combinations(cand, take), key=lambda s: sum(float(V[i]) for i in s)) if take else ()
    rest = [i for i in range(n) if i not in mand and i not in prot]
    r = K_eff - len(mand) - len(prot)
    main = max(itertools.combinations(rest, r), key=lambda s: sum(float(u[i]) for i in s)) if r else ()
    return sorted(set(mand) | set(prot) | set(main))


@pytest.mark.parametrize("seed", range(12))
def test_select_exhaustive_small(seed):
    rng = np.random.default_rng(100 + seed)
    n = int(rng.integers(3, 12))
    u = rng.permutation(n).astype(np.float32) + rng.random(n).astype(np.float32) * 0.5  # distinct
    V = np.zeros(n, np.float32)
    spons = rng.random(n) < 0.4
    V[spons] = (rng.permutation(n)[spons] + 1).astype(np.float32)  # distinct positive
    u = u + V
    n_sink, n_recent = int(rng.integers(0, 3)), int(rng.integers(0, 4))
    for k_prot in (-1, 0, 2):
        for K in range(1, n + 2):
            idx, cnt = oracle.select(V, u, K, n_sink, n_recent, k_prot)
            want = _exhaustive(V, u, K, n_sink, n_recent, k_prot)
            assert cnt == min(K, n) == len(want)  # exactly K tokens are retained (Section 3.3)
            assert list(idx[:cnt]) == want
            assert all(idx[cnt:] == -1)


def test_select_reduces_to_plain_topk_without_anchors():
    # Algorithm 1 step 8: S <- top-K(u). With no sponsored token and no mandatory slots the partition is inert.
    rng = np.random.default_rng(7)
    n = 500
    u = rng.standard_normal(n).astype(np.float32)
    V = np.zeros(n, np.float32)
    for K in (1, 16, 499, 500, 700):
        for k_prot in (-1, 0, 5):
            idx, cnt = oracle.select(V, u, K, 0, 0, k_prot)
            want = np.sort(torch.topk(torch.from_numpy(u), min(K, n)).indices.numpy())
            np.testing.assert_array_equal(idx[:cnt], want)


def test_select_ties_prefer_lower_position():
    u = np.array([1, 5, 5, 5, 0, 5], np.float32)
    V = np.zeros(6, np.float32)
    idx, cnt = oracle.select(V, u, 2, 0, 0, 0)
    assert list(idx[:cnt]) == [1, 2]
    V = np.array([0, 3, 3, 0, 3, 0], np.float32)
    idx, cnt = oracle.select(V, np.zeros(6, np.float32), 2, 0, 0, 2)
    assert list(idx[:cnt]) == [1, 2]


def _one_anchor_case(n, anchor_end, L, unsponsored_u):
    ids = np.arange(100, 100 + n).astype(np.int32)
    ids[anchor_end] = 7
    pats = oracle.Patterns([[7]], span=[L])
    atok, aend, Be, Le = oracle.anchors(ids, pats)
    V = oracle.vouchers(aend, Be, Le)
    u = np.where(V > 0, V, np.float32(unsponsored_u)).astype(np.float32)
    return V, u


def test_theorem2_span_retained_regardless_of_attention():
    # Theorem 2: K >= 1 + W + L with K_p >= L keeps [i+1, i+L] whatever the attention scores are.
    n, e, L, W = 300, 120, 6, 4
    V, u = _one_anchor_case(n, e, L, 1e6)  # every unsponsored token out-scores the span
    for K in (1 + W + L, 16, 40):
        idx, cnt = oracle.select(V, u, K, 1, W, -1)
        assert set(range(e + 1, e + L + 1)) <= set(idx[:cnt])
        assert 0 in idx[:cnt] and set(range(n - W, n)) <= set(idx[:cnt])
    # one slot short: exactly one span token (the farthest, smallest voucher) is lost
    idx, cnt = oracle.select(V, u, W + L, 1, W, -1)
    assert set(range(e + 1, e + L + 1)) - set(idx[:cnt]) == {e + L}


def test_minimum_budget_corollary():
    # K* = 1 + W + l; W = 4, l = 10: K* = 15 (value fully sponsored when L = l).
    n, e, L, W = 400, 200, 10, 4
    V, u = _one_anchor_case(n, e, L, 1e6)
    idx, cnt = oracle.select(V, u, 15, 1, W, -1)
    assert set(range(e + 1, e + 11)) <= set(idx[:cnt])
    idx, cnt = oracle.select(V, u, 14, 1, W, -1)
    assert len(set(range(e + 1, e + 11)) - set(idx[:cnt])) == 1


@pytest.mark.parametrize("K,m,fits", [(16, 1, False), (16, 5, False), (64, 4, True), (64, 10, False), (19, 1, True)])
def test_theorem4_decoy_tolerance(K, m, fits):
    # m decoys + 1 true anchor, spans of L = 6: all kept iff K >= 1 + W + (m+1) L; K_p = K - 1 - W.
    L, W, n = 6, 4, 600
    ids = np.arange(100, 100 + n).astype(np.int32)
    ends = [20 + 30 * j for j in range(m + 1)]
    for e in ends:
        ids[e] = 7
    atok, aend, Be, Le = oracle.anchors(ids, oracle.Patterns([[7]]))
    V = oracle.vouchers(aend, Be, Le)
    u = np.where(V > 0, V, np.float32(1e6)).astype(np.float32)
    idx, cnt = oracle.select(V, u, K, 1, W, -1)
    spons = {e + k for e in ends for k in range(1, L + 1)}
    kept = spons & set(idx[:cnt])
    assert (K >= 1 + W + (m + 1) * L) == fits
    if fits:
        assert kept == spons
    else:
        assert len(kept) == K - 1 - W  # the protected pool overflows: K_p of them survive


def test_worked_credential_example():
    g = {r[0]: [int(x) for x in r[1:]] for r in _rows("credential_example.txt")}
    n, K, e = g["n"][0], g["K"][0], g["anchor_end"][0]
    rng = np.random.default_rng(11)
    ids = rng.integers(1000, 32000, size=n).astype(np.int32)
    anchor = [11, 12, 13]
    ids[e - 2:e + 1] = anchor
    ids[e + 1:e + 1 + g["value_len"][0]] = np.arange(500, 500 + g["value_len"][0])
    pol = oracle.preset("AUDIT", K, fast=1)
    cu = np.array([0, n], np.int32)
    flags, V, u0 = oracle.sponsor_mask(ids, cu, oracle.Patterns([anchor]), pol)
    sponsored = np.nonzero(flags & 4)[0]
    assert list(sponsored) == list(range(g["value_first"][0], g["value_first"][0] + g["span"][0]))
    idx, cnt = oracle.select(V, u0, K, pol.n_sink, pol.n_recent, pol.k_protected)
    assert list(idx[:cnt]) == g["ta_fast_retained"]
    # the sponsored span survives under every partition the paper states
    for name in ("THEOREM", "SEC33", "AUDIT"):
        p = oracle.preset(name, K)
        idx, cnt = oracle.select(V, u0, K, p.n_sink, p.n_recent, p.k_protected)
        assert set(sponsored) <= set(idx[:cnt])
        assert cnt == K
    # a window-only policy (no patterns; 4 sinks + last 12) cannot reach the needle
    flags0, V0, u00 = oracle.sponsor_mask(ids, cu, oracle.Patterns([]), pol)
    idx, cnt = oracle.select(V0, np.zeros(n, np.float32), K, 4, 12, 0)
    assert list(idx[:cnt]) == g["window_only_retained"]
    assert not (set(range(g["value_first"][0], g["value_first"][0] + g["value_len"][0])) & set(idx[:cnt]))


def test_select_keep_all_and_degenerate_sizes():
    u = np.array([3, 1, 2], np.float32)
    V = np.array([0, 5, 0], np.float32)
    for K in (3, 4, 100):
        idx, cnt = oracle.select(V, u, K, 1, 4, -1)
        assert cnt == 3 and list(idx[:3]) == [0, 1, 2] and all(idx[3:] == -1)
    # n smaller than sinks + recents: the mandatory list is truncated in priority order
    idx, cnt = oracle.select(np.zeros(5, np.float32), np.arange(5, dtype=np.float32), 2, 4, 6, 0)
    assert list(idx[:cnt]) == [0, 1]


# ------------------------------------------------------------------------------------------------ compaction
def test_compact_is_index_select():
    rng = np.random.default_rng(2)
    src = rng.integers(0, 65536, size=(40, 2 * 16), dtype=np.uint16)[:, :16]  # strided rows
    idx = np.array([0, 3, 17, 39, -1, -1], np.int32)
    out = oracle.compact(src, idx, 4, 6)
    np.testing.assert_array_equal(out[:4], src[idx[:4]])
    assert not out[4:].any()


def test_compress_layer_matches_step_by_step():
    """The chained per-layer routine (used for timing and full-size parity) equals the individually pinned steps."""
    import ta_workloads as tw
    w = tw.config5(B=3, n_lo=40, n_hi=90, n_layers=1, K=12, decoys_per_seq=2, Hq=4, Hkv=2, W=8)
    Q, K, V = tw.make_qkv(w, [0])
    pats = oracle.Patterns(w.pattern_ids, w.pattern_budget, w.pattern_span)
    pol = oracle.preset("THEOREM", 12, obs_window=w.W)
    Qb, Kb, Vb = bf16_bits(Q[0]), bf16_bits(K[0]), bf16_bits(V[0])
    idx, cnt, ko, vo, _ = oracle.compress_layer(w.ids, w.cu, False, w.Hq, w.Hkv, w.d, 12, pats, pol, Qb, Kb, Vb)
    flags, Vv, u0 = oracle.sponsor_mask(w.ids, w.cu, pats, pol)
    G = w.Hq // w.Hkv
    for b in range(w.B):
        o, e = int(w.cu[b]), int(w.cu[b + 1])
        for g in range(w.Hkv):
            A, P = oracle.attention(Qb[b, g * G:(g + 1) * G], Kb[g, o:e], e - o, rho=pol.pension_rho)
            u = oracle.utility(pol.alpha, pol.delta, A, P, u0[o:e])
            i2, c2 = oracle.select(Vv[o:e], u, 12, pol.n_sink, pol.n_recent, pol.k_protected)
            np.testing.assert_array_equal(idx[b, g], i2)
            assert cnt[b, g] == c2
            np.testing.assert_array_equal(ko[b, g], oracle.compact(Kb[g, o:e], i2, c2, 12))
            np.testing.assert_array_equal(vo[b, g], oracle.compact(Vb[g, o:e], i2, c2, 12))


# ------------------------------------------------------------------------- learned-detector anchors (Section 5.1)
def test_conf_anchors_rank_mode_closed_form():
    # TA-LearnRank: V_j = sum_i f_i 0.8^(j-i) 1[f_i > 0.3, i < j <= i+L]; two anchors, one below the threshold
    conf = np.array([0.0, 0.9, 0.2, 0.0, 0.6, 0.3, 0.0, 0.0, 0.0, 0.0, 0.0, 0.0], np.float32)
    L = 6
    atok, aend, Be, Le = oracle.anchors_conf(conf, 0.3, 1.0, L, True)
    assert aend.tolist() == [0, 1, 0, 0, 1, 0, 0, 0, 0, 0, 0, 0]  # 0.2 and exactly 0.3 are not above 0.3
    assert (atok == aend).all()
    V = oracle.vouchers(aend, Be, Le)
    f1, f4 = float(np.float32(0.9)), float(np.float32(0.6))
    for j in range(12):
        want = 0.0
        if 1 < j <= 1 + L:
            want += f1 * 0.8 ** (j - 1)
        if 4 < j <= 4 + L:
            want += f4 * 0.8 ** (j - 4)
        assert V[j] == pytest.approx(want, rel=1e-6, abs=1e-12)
    # "higher-confidence anchors receive more protection": right after each anchor the ratio is the confidence ratio
    assert V[2] / 0.8 == pytest.approx(f1, rel=1e-6)


def test_conf_anchors_fixed_budget_equals_one_token_pattern():
    # TA-Learned with the indicator of a token id as "confidence" is the pattern detector with that one-token pattern
    rng = np.random.default_rng(5)
    ids = rng.integers(0, 4, 200).astype(np.int32)
    conf = (ids == 2).astype(np.float32)
    for age in (0, 3):
        a1 = oracle.anchors_conf(conf, 0.5, 15.0, 6, False, age_steps=age)
        a2 = oracle.anchors(ids, oracle.Patterns([[2]]), age_steps=age)
        for x, y in zip(a1, a2):
            np.testing.assert_array_equal(x, y)
    # rank mode with confidence 1 everywhere an anchor is: budget * 1 = budget
    a3 = oracle.anchors_conf(conf, 0.3, 15.0, 6, True)
    np.testing.assert_array_equal(a3[2], oracle.anchors(ids, oracle.Patterns([[2]]))[2])


def test_conf_anchors_nan_and_budget_age():
    conf = np.array([np.nan, 0.8, 1.0], np.float32)
    atok, aend, Be, Le = oracle.anchors_conf(conf, 0.5, 2.0, 4, True, budget_decay=0.9, age_steps=2)
    assert aend.tolist() == [0, 1, 1] and Le.tolist() == [0, 4, 4]
    assert Be[1] == pytest.approx(2.0 * 0.8 * 0.81, rel=1e-6) and Be[2] == pytest.approx(2.0 * 0.81, rel=1e-6)


# ------------------------------------------------------------------------------- attention summed over all heads
def test_attention_allheads_is_sum_over_kv_heads_and_normalised():
    g = torch.Generator().manual_seed(11)
    Hq, Hkv, W, d, n = 8, 2, 5, 16, 37
    Q = bf16_bits(torch.randn(Hq, W, d, generator=g))
    K = bf16_bits(torch.randn(Hkv, n, d, generator=g))
    A, P = oracle.attention_allheads(Q, K, n, rho=0.7)
    G = Hq // Hkv
    As = np.zeros(n)
    Ps = np.zeros(n)
    for h in range(Hkv):
        a, p = oracle.attention(Q[h * G:(h + 1) * G], K[h], n, rho=0.7)
        As += a
        Ps += p
    np.testing.assert_allclose(A, As, rtol=1e-6, atol=1e-9)
    np.testing.assert_allclose(P, Ps, rtol=1e-6, atol=1e-9)
    assert A.sum() == pytest.approx(Hq * W, rel=1e-6)          # every softmax row sums to one
    assert P.sum() == pytest.approx(Hq * (1 - 0.7 ** W), rel=1e-6)
    # one KV head: the per-group routine
    A1, P1 = oracle.attention_allheads(Q[:G], K[:1], n, rho=0.7)
    a, p = oracle.attention(Q[:G], K[0], n, rho=0.7)
    np.testing.assert_array_equal(A1, a)
    np.testing.assert_array_equal(P1, p)


# ------------------------------------------------------------------ Algorithm 1 in the decode loop (streaming oracle)
from oracle.ta_stream_oracle import StreamOracle  # noqa: E402


def _uniform_attn(units, t):
    return [{p: 1.0 / (len(un.pos) + 1) for p in un.pos + [t]} for un in units]


def test_stream_vouchers_closed_form():
    # anchor (id 2) at position 3; B = 15, L = 6: the token arriving k steps later gets 15*(0.9*0.8)^k, and every
    # later step multiplies it by 0.9 (Algorithm 1 step 10)
    so = StreamOracle(oracle.Patterns([[2]]), oracle.Policy(), K=64, n_units=1)
    ids = [7, 7, 7, 2] + [5] * 10
    for t, x in enumerate(ids):
        so.step(x, _uniform_attn(so.units, t))
    n = len(ids)
    V = so.units[0].V
    for j in range(n):
        k = j - 3
        want = 15.0 * (0.72 ** k) * 0.9 ** (n - j) if 1 <= k <= 6 else 0.0
        assert float(V[j]) == pytest.approx(want, rel=2e-6, abs=1e-12), j
    assert so.units[0].S == [0, 0, 0, 1] + [0] * 10


def test_stream_without_decay_matches_one_shot_oracle():
    # budget_decay = 1 and K >= n: after the last token the streamed vouchers, anchor flags and attention-free utility
    # are the one-shot oracle's, bit for bit (multi-token patterns, overlapping spans, a prefix-only decoy)
    rng = np.random.default_rng(9)
    ids = rng.integers(0, 5, 120).astype(np.int32)
    pats = oracle.Patterns([[1, 2], [3], [4, 1, 2]], budget=[15.0, 4.0, 9.0], span=[6, 3, 8])
    pol = oracle.Policy(budget_decay=1.0, vocab_size=8)
    so = StreamOracle(pats, pol, K=1000, n_units=1)
    for t, x in enumerate(ids):
        assert so.step(int(x), _uniform_attn(so.units, t)) == [-1]
    cu = np.array([0, len(ids)], np.int32)
    flags, V, u0 = oracle.sponsor_mask(ids, cu, pats, pol)
    np.testing.assert_array_equal(np.array(so.units[0].V, np.float32).view(np.uint32), V.view(np.uint32))
    np.testing.assert_array_equal(np.array(so.units[0].S, np.uint8), flags & 1)
    np.testing.assert_array_equal(so.static_utility(0).view(np.uint32), u0.view(np.uint32))


def test_stream_attention_only_evicts_least_accumulated():
    # no patterns, alpha = 1 and every other weight 0, no mandatory or protected slots: each step drops the cached
    # token with the least accumulated attention (H2O-style), latest position among equals
    rng = np.random.default_rng(4)
    pol = oracle.Policy(alpha=1.0, beta=0.0, gamma=0.0, delta=0.0, lam=0.0, n_sink=0, n_recent=0, k_protected=0)
    K = 6
    so = StreamOracle(oracle.Patterns([]), pol, K=K, n_units=2)
    acc = [dict(), dict()]
    for t in range(40):
        attn = []
        for u in range(2):
            ps = so.units[u].pos + [t]
            a = rng.random(len(ps)).astype(np.float32)
            a[rng.integers(0, len(ps))] = a[0]  # some exact ties
            attn.append({p: float(x) for p, x in zip(ps, a)})
        ev = so.step(int(rng.integers(0, 50)), attn)
        for u in range(2):
            for p, x in attn[u].items():
                acc[u][p] = np.float32(acc[u].get(p, np.float32(0)) + np.float32(x))
            if len(acc[u]) > K:
                lo = min(acc[u].values())
                want = max(p for p, x in acc[u].items() if x == lo)
                assert ev[u] == want
                del acc[u][want]
            else:
                assert ev[u] == -1
            assert sorted(acc[u]) == so.units[u].pos


def test_stream_sponsored_span_survives_adversarial_attention():
    # Theorem 2 in the streaming setting: budget 1 + W + L with W = 4 recents; the six tokens after the anchor are
    # never evicted while their (decaying) vouchers exceed the largest competing utility, whatever the attention says
    pol = oracle.Policy()  # 1 sink, 4 recent, protected = the rest
    L, K = 6, 1 + 4 + 6
    so = StreamOracle(oracle.Patterns([[2]]), pol, K=K, n_units=1)
    ids = [9] * 20 + [2] + [30 + i for i in range(6)] + [9] * 6
    for t, x in enumerate(ids):
        un = so.units[0]
        attn = {p: (0.0 if 21 <= p <= 26 else 1.0) for p in un.pos + [t]}  # the value tokens get no attention at all
        so.step(x, [attn])
        if t >= 26:
            assert set(range(21, 27)) <= set(so.units[0].pos), t
    assert len(so.units[0].pos) == K


# ----------------------------------------------------------------- embedding-based detector (Section 3.2, variant 3)
def test_embedding_confidence_special_cases():
    g = torch.Generator().manual_seed(2)
    a = torch.randn(3, 64, generator=g).to(torch.bfloat16)
    e = torch.stack([a[0], -a[1], 4.0 * a[2], torch.zeros(64).to(torch.bfloat16),
                     torch.cat([torch.ones(32), torch.zeros(32)]).to(torch.bfloat16)])
    conf = oracle.embedding_confidence(bf16_bits(e), bf16_bits(a))
    assert conf[0] == pytest.approx(1.0, abs=1e-6)          # identical to concept 0
    assert conf[2] == pytest.approx(1.0, abs=1e-6)          # concept 2 times a power of two (exact in bf16)
    assert conf[3] == 0.0                                   # zero vector
    # -a[1]: similarity -1 with concept 1; the maximum is over the other two concepts, against a library routine
    ref = torch.nn.functional.cosine_similarity(e[1].double()[None], a.double(), dim=-1).max().item()
    assert conf[1] == pytest.approx(ref, abs=1e-6) and conf[1] < 1.0
    # orthogonal halves
    c2 = torch.cat([torch.zeros(32), torch.ones(32)]).to(torch.bfloat16)[None]
    assert oracle.embedding_confidence(bf16_bits(e[4:5]), bf16_bits(c2))[0] == 0.0
    assert oracle.embedding_confidence(bf16_bits(e[4:5]), bf16_bits(-e[4:5]))[0] == pytest.approx(-1.0, abs=1e-6)
