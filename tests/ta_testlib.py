"""Shared helpers of the GPU parity tests: run the CUDA library through its C ABI binding, run the CPU oracle on
the same bytes, compare. Nothing here computes any part of the method."""
from __future__ import annotations

import numpy as np
import torch

import oracle
import paper_2604_11288_b200 as ta

SCORE_RTOL, SCORE_ATOL = 1e-3, 1e-5  # tolerance of the attention terms, fp32


def bf16_bits(x: torch.Tensor) -> np.ndarray:
    return x.detach().cpu().contiguous().view(torch.int16).numpy().view(np.uint16)


def oracle_policy(K, preset="THEOREM", fast=False, W=32, **kw) -> oracle.Policy:
    return oracle.preset(preset, K, fast=1 if fast else 0, obs_window=W, **kw)


def gpu_policy(pol: oracle.Policy) -> ta.ta_policy:
    p = ta.ta_policy()
    p.alpha, p.beta, p.gamma, p.delta, p.lambda_ = pol.alpha, pol.beta, pol.gamma, pol.delta, pol.lam
    p.voucher_decay, p.budget_decay, p.age_steps = pol.voucher_decay, pol.budget_decay, pol.age_steps
    p.n_sink, p.n_recent, p.k_protected = pol.n_sink, pol.n_recent, pol.k_protected
    p.obs_window, p.pension_rho, p.softmax_scale = pol.obs_window, pol.pension_rho, pol.softmax_scale
    p.causal, p.mode, p.vocab_size = pol.causal, (ta.TA_MODE_FAST if pol.fast else ta.TA_MODE_SCORED), pol.vocab_size
    return p


class Gpu:
    """Owns a context, a pattern set and the device copies of one workload's per-sequence inputs."""

    def __init__(self, w, pol: oracle.Policy, K, n_layers, device="cuda:0", n_budget_classes=0):
        self.w, self.pol, self.K, self.L = w, pol, K, n_layers
        self.dev = torch.device(device)
        self.p = gpu_policy(pol)
        self.ids = torch.from_numpy(w.ids).to(self.dev)
        self.cu = None if w.uniform else torch.from_numpy(w.cu).to(self.dev)
        n_uni = int(w.lengths[0]) if w.uniform else 0
        self.batch = ta.make_batch(n_layers, w.B, n_uni, w.max_n, w.total, self.cu)
        need = ta.ta_scratch_bytes(self.batch, w.Hq, w.Hkv, w.d, K, self.p)
        if n_budget_classes:
            need = max(need, ta.ta_scratch_bytes_budgets(self.batch, w.Hkv, K, self.p, n_budget_classes))
        self.ctx = ta.ta_ctx_create(self.dev.index or 0, need)
        self.pats = ta.ta_patterns_create(self.ctx, w.pattern_ids, w.pattern_budget, w.pattern_span)
        self.stream = torch.cuda.current_stream(self.dev).cuda_stream

    def close(self):
        ta.ta_patterns_destroy(self.pats)
        ta.ta_ctx_destroy(self.ctx)

    def poll(self):
        return ta.ta_ctx_poll(self.ctx)

    def sponsor_mask(self):
        t = self.w.total
        flags = torch.empty(t, dtype=torch.uint8, device=self.dev)
        V = torch.empty(t, dtype=torch.float32, device=self.dev)
        u0 = torch.empty(t, dtype=torch.float32, device=self.dev)
        ta.ta_sponsor_mask(self.ctx, self.pats, self.p, self.batch, self.ids, flags, V, u0, self.stream)
        return flags, V, u0

    def sponsor_mask_conf(self, conf, threshold, budget, span, rank):
        t = self.w.total
        flags = torch.empty(t, dtype=torch.uint8, device=self.dev)
        V = torch.empty(t, dtype=torch.float32, device=self.dev)
        u0 = torch.empty(t, dtype=torch.float32, device=self.dev)
        ta.ta_sponsor_mask_conf(self.ctx, self.p, self.batch, self.ids, conf, threshold, budget, span, rank, flags, V,
                                u0, self.stream)
        return flags, V, u0

    def score(self, Q, K, lse=None, want_P=True):
        w = self.w
        A = torch.full((self.L, w.Hkv, w.total), float("nan"), dtype=torch.float32, device=self.dev)
        P = torch.full_like(A, float("nan")) if want_P else None
        ta.ta_score(self.ctx, self.p, self.batch, w.Hq, w.Hkv, w.d, ta.view(Q), ta.view(K, not w.uniform), lse, A, P,
                    self.stream)
        return A, P

    def select(self, flags, V, u0, A=None, P=None):
        w = self.w
        idx = torch.full((self.L, w.B, w.Hkv, self.K), -7, dtype=torch.int32, device=self.dev)
        cnt = torch.full((self.L, w.B, w.Hkv), -7, dtype=torch.int32, device=self.dev)
        ta.ta_select_topk(self.ctx, self.p, self.batch, w.Hkv, self.K, flags, V, u0, A, P, idx, cnt, self.stream)
        return idx, cnt

    def compact(self, Kc, Vc, idx, cnt):
        w = self.w
        ko = torch.full((self.L, w.B, w.Hkv, self.K, w.d), 1.0, dtype=torch.bfloat16, device=self.dev)
        vo = torch.full_like(ko, 1.0)
        rag = not w.uniform
        ta.ta_compact_kv(self.ctx, self.batch, w.Hkv, w.d, self.K, ta.view(Kc, rag), ta.view(Vc, rag), idx, cnt, ko, vo,
                         self.stream)
        return ko, vo

    def compress_allheads(self, Q, Kc, Vc, epoch=0):
        w = self.w
        idx = torch.full((self.L, w.B, w.Hkv, self.K), -7, dtype=torch.int32, device=self.dev)
        cnt = torch.full((self.L, w.B, w.Hkv), -7, dtype=torch.int32, device=self.dev)
        ko = torch.full((self.L, w.B, w.Hkv, self.K, w.d), 1.0, dtype=torch.bfloat16, device=self.dev)
        vo = torch.full_like(ko, 1.0)
        rag = not w.uniform
        ta.ta_compress_allheads(self.ctx, self.pats, self.p, self.batch, w.Hq, w.Hkv, w.d, self.K, self.ids, ta.view(Q),
                                ta.view(Kc, rag), ta.view(Vc, rag), epoch, ko, vo, idx, cnt, self.stream)
        return idx, cnt, ko, vo

    def compress_scores(self, score, score2, Kc, Vc, epoch=0):
        w = self.w
        idx = torch.full((self.L, w.B, w.Hkv, self.K), -7, dtype=torch.int32, device=self.dev)
        cnt = torch.full((self.L, w.B, w.Hkv), -7, dtype=torch.int32, device=self.dev)
        ko = torch.full((self.L, w.B, w.Hkv, self.K, w.d), 1.0, dtype=torch.bfloat16, device=self.dev)
        vo = torch.full_like(ko, 1.0)
        rag = not w.uniform
        ta.ta_compress_scores(self.ctx, self.pats, self.p, self.batch, w.Hkv, w.d, self.K, self.ids, score, score2,
                              ta.view(Kc, rag), ta.view(Vc, rag), epoch, ko, vo, idx, cnt, self.stream)
        return idx, cnt, ko, vo

    def compress_scores_budgets(self, budgets, score, score2, Kc, Vc):
        w = self.w
        idx = torch.full((self.L, w.B, w.Hkv, self.K), -7, dtype=torch.int32, device=self.dev)
        cnt = torch.full((self.L, w.B, w.Hkv), -7, dtype=torch.int32, device=self.dev)
        ko = torch.full((self.L, w.B, w.Hkv, self.K, w.d), 1.0, dtype=torch.bfloat16, device=self.dev)
        vo = torch.full_like(ko, 1.0)
        rag = not w.uniform
        ta.ta_compress_scores_budgets(self.ctx, self.pats, self.p, self.batch, w.Hkv, w.d, self.K, budgets, self.ids,
                                      score, score2, ta.view(Kc, rag), ta.view(Vc, rag), ko, vo, idx, cnt, self.stream)
        return idx, cnt, ko, vo

    def compress_budgets(self, budgets, Q, Kc, Vc):
        w = self.w
        idx = torch.full((self.L, w.B, w.Hkv, self.K), -7, dtype=torch.int32, device=self.dev)
        cnt = torch.full((self.L, w.B, w.Hkv), -7, dtype=torch.int32, device=self.dev)
        ko = torch.full((self.L, w.B, w.Hkv, self.K, w.d), 1.0, dtype=torch.bfloat16, device=self.dev)
        vo = torch.full_like(ko, 1.0)
        rag = not w.uniform
        ta.ta_compress_budgets(self.ctx, self.pats, self.p, self.batch, w.Hq, w.Hkv, w.d, self.K, budgets, self.ids,
                               ta.view(Q), ta.view(Kc, rag), ta.view(Vc, rag), ko, vo, idx, cnt, self.stream)
        return idx, cnt, ko, vo

    def compress(self, Q, Kc, Vc, epoch=0):
        w = self.w
        idx = torch.full((self.L, w.B, w.Hkv, self.K), -7, dtype=torch.int32, device=self.dev)
        cnt = torch.full((self.L, w.B, w.Hkv), -7, dtype=torch.int32, device=self.dev)
        ko = torch.full((self.L, w.B, w.Hkv, self.K, w.d), 1.0, dtype=torch.bfloat16, device=self.dev)
        vo = torch.full_like(ko, 1.0)
        rag = not w.uniform
        ta.ta_compress(self.ctx, self.pats, self.p, self.batch, w.Hq, w.Hkv, w.d, self.K, self.ids, ta.view(Q),
                       ta.view(Kc, rag), ta.view(Vc, rag), epoch, ko, vo, idx, cnt, self.stream)
        return idx, cnt, ko, vo


def oracle_patterns(w) -> oracle.Patterns:
    return oracle.Patterns(w.pattern_ids, w.pattern_budget, w.pattern_span)


def unit_kv(w, T, l, b, g):
    """Rows of sequence b, head g of layer slot l as a uint16 array [n, d] (a view: no copy)."""
    if w.uniform:
        return bf16_bits(T[l, b, g])
    o, e = int(w.cu[b]), int(w.cu[b + 1])
    return bf16_bits(T[l, g, o:e])


def oracle_unit(w, pol, K, Qh, Kh, l, b, g, V, u0):
    """Oracle A, P, u, idx, count for one unit. Qh/Kh are host torch tensors (bf16)."""
    G = w.Hq // w.Hkv
    o, e = int(w.cu[b]), int(w.cu[b + 1])
    n = e - o
    if pol.fast:
        A = P = None
        u = u0[o:e].copy()
    else:
        A, P = oracle.attention(bf16_bits(Qh[l, b, g * G:(g + 1) * G]), unit_kv(w, Kh, l, b, g), n,
                                scale=pol.softmax_scale, causal=pol.causal, rho=pol.pension_rho)
        u = oracle.utility(pol.alpha, pol.delta, A, P, u0[o:e])
    idx, cnt = oracle.select(V[o:e], u, K, pol.n_sink, pol.n_recent, pol.k_protected)
    return A, P, u, idx, cnt


def assert_scores_close(got, want, what):
    got = np.asarray(got, np.float64)
    want = np.asarray(want, np.float64)
    err = np.abs(got - want)
    tol = SCORE_ATOL + SCORE_RTOL * np.abs(want)
    bad = np.nonzero(~(err <= tol))[0]
    assert bad.size == 0, (f"{what}: {bad.size}/{got.size} outside 1e-3 rel / 1e-5 abs; first {bad[:8]}, "
                           f"got {got[bad[:8]]}, want {want[bad[:8]]}, worst ratio {np.nanmax(err / tol):.3g}")


def assert_selection_matches(idx_gpu, cnt_gpu, idx_ora, cnt_ora, u_ora, what):
    """Bit-exact, except that tokens whose oracle utilities are within the score tolerance of the budget boundary
    may be swapped. Returns True when the two index lists are identical."""
    assert int(cnt_gpu) == int(cnt_ora), f"{what}: count {int(cnt_gpu)} != {int(cnt_ora)}"
    g = np.asarray(idx_gpu)
    o = np.asarray(idx_ora)
    c = int(cnt_ora)
    assert (g[c:] == -1).all(), f"{what}: padding is not -1"
    if (g[:c] == o[:c]).all():
        return True
    assert (np.diff(g[:c]) > 0).all(), f"{what}: indices not strictly ascending"
    only_o = np.setdiff1d(o[:c], g[:c])
    only_g = np.setdiff1d(g[:c], o[:c])
    assert only_o.size == only_g.size
    tau = float(u_ora[only_o].min())
    eps = SCORE_ATOL + SCORE_RTOL * abs(tau)
    gap = float(u_ora[only_o].max() - u_ora[only_g].min())
    assert gap <= 2 * eps, (f"{what}: selection differs outside the tolerance band: oracle-only {only_o[:8]} "
                            f"(u {u_ora[only_o][:8]}), gpu-only {only_g[:8]} (u {u_ora[only_g][:8]}), gap {gap:.3g}")
    return False
