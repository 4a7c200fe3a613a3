"""TEST INFRASTRUCTURE — not part of the product.

Plain statement of Algorithm 1 ("Transactional Attention: per-step retention") run in the decode loop: one new token
per step, a cache of at most K tokens per unit after every step. Written from the paper's text (Section 3.1, Section
3.2, Eq. 1, Eq. 2, Algorithm 1, Section 3.3); slow on purpose (Python lists, numpy float32 scalars, one rounding per
operation, no fused multiply-add). The per-unit selection is the one-shot oracle's routine (ora_select), the anchor
test is the one-shot oracle's (ora_anchors) on the trailing token ids.

Readings taken where the paper is silent:
  * Algorithm 1 step 1 detects anchors "in the KV-cache"; here an anchor is detected once, when the token that
    completes a pattern arrives, on the full stream of token ids (an evicted prefix of a pattern still counts: the
    ids were seen), and it keeps sponsoring even if its own cache entry is evicted later.
  * "When anchor x_i is detected, it sponsors the next L tokens": token j's voucher is fixed when j arrives,
    V_j = sum over anchors i with i < j <= i + L_i of B_i^(now) * decay^(j-i), nearest anchor first, where the budget
    has decayed once per step since detection (Algorithm 1 step 10), i.e. B_i^(now) = B_i * budget_decay^(j-i).
    From then on "decay budgets" multiplies every allocated voucher by budget_decay at the end of each step
    (all contributions to V_j decay by the same factor, so decaying the sum is decaying the budgets).
  * A_i accumulates the attention mass the unit's query heads put on token i at every step it is cached
    (Appendix A Definition 1); P_i is the exponential moving average of the same per-step mass,
    P <- rho*P + (1-rho)*a, zero for a token that just arrived plus its first sample.
  * R_i = (i0+1)/n and F_i = (occurrences of the token's id so far)/n with n = tokens seen so far, evicted ones included.
  * S_i = 1 on every token of a completed match that is still cached (set when the match completes).
  * While a unit holds at most K tokens nothing is evicted. Otherwise the retained set is the budget partition of
    Section 3.3 applied to the K+1 cached tokens in position order (sinks = earliest cached, recents = latest).

Pinned by (tests/test_oracle_pins.py): closed forms of the vouchers, B*(0.9*0.8)^k at arrival and *0.9 per later step;
with budget_decay = 1 and K >= n the state after the last token equals the one-shot oracle's vouchers, flags and
attention-free utility bit for bit; with no patterns and only alpha != 0 every step evicts the cached token of least
accumulated attention (exhaustive check); a sponsored span outlives adversarial attention while its vouchers dominate.
"""
from __future__ import annotations

import numpy as np

from . import ta_oracle as one_shot

F32 = np.float32
MAX_PATTERN_LEN = 8


class Unit:
    """One (layer, sequence, KV head): the cached tokens in position order."""

    def __init__(self):
        self.pos, self.A, self.P, self.V, self.S = [], [], [], [], []


class StreamOracle:
    def __init__(self, pats: one_shot.Patterns, pol: one_shot.Policy, K: int, n_units: int):
        self.pats, self.pol, self.K = pats, pol, K
        self.ids = []        # every token id seen so far
        self.anchors = {}    # position -> (budget at detection, span)
        self.units = [Unit() for _ in range(n_units)]

    # -- Algorithm 1 steps 1-6 for the newest token
    def _detect_and_voucher(self, x):
        pol = self.pol
        t = len(self.ids)
        self.ids.append(int(x))
        lo = max(0, t + 1 - MAX_PATTERN_LEN)
        window = np.array(self.ids[lo:], np.int32)
        atok, aend, Be, Le = one_shot.anchors(window, self.pats, pol.budget_decay, 0)
        if aend[-1]:
            self.anchors[t] = (F32(Be[-1]), int(Le[-1]))
        # positions of the window that belong to a match completed by this token
        match_len = 0
        for p in self.pats.ids:
            if len(p) <= len(window) and list(window[len(window) - len(p):]) == list(p):
                match_len = max(match_len, len(p))
        flagged = set(range(t - match_len + 1, t + 1))
        # voucher of the new token: nearest anchor first
        bd, vd = F32(pol.budget_decay), F32(pol.voucher_decay)
        Lmax = max([0] + [L for (_, L) in self.anchors.values()])
        v = F32(0.0)
        w = F32(1.0)
        for k in range(1, Lmax + 1):
            w = F32(w * vd)
            i = t - k
            if i in self.anchors and k <= self.anchors[i][1]:
                Bk = self.anchors[i][0]
                for _ in range(k):
                    Bk = F32(Bk * bd)
                v = F32(v + F32(Bk * w))
        return t, v, flagged

    def step(self, x, attn_by_pos):
        """x: the new token id. attn_by_pos[u]: dict position -> attention mass of this step's query on that cached
        token (the new token included), for every unit u. Returns the evicted position per unit (-1: none)."""
        pol, K = self.pol, self.K
        t, v_new, flagged = self._detect_and_voucher(x)
        n = t + 1
        rho = F32(pol.pension_rho)
        omr = F32(F32(1.0) - rho)
        counts = {}
        for i in self.ids:
            counts[i] = counts.get(i, 0) + 1
        evicted = []
        for u, un in enumerate(self.units):
            un.pos.append(t)
            un.A.append(F32(0.0))
            un.P.append(F32(0.0))
            un.V.append(v_new)
            un.S.append(0)
            m = len(un.pos)
            for r in range(m):
                a = F32(attn_by_pos[u][un.pos[r]])
                un.A[r] = F32(un.A[r] + a)
                un.P[r] = F32(F32(rho * un.P[r]) + F32(omr * a))
                if un.pos[r] in flagged:
                    un.S[r] = 1
            drop = -1
            if m > K:
                u0 = np.zeros(m, F32)
                for r in range(m):
                    R = F32(F32(un.pos[r] + 1) / F32(n))
                    Ff = F32(F32(counts[self.ids[un.pos[r]]]) / F32(n))
                    t0 = F32(F32(F32(pol.beta) * R) + F32(F32(pol.gamma) * F32(un.S[r])))
                    t1 = F32(t0 - F32(F32(pol.lam) * Ff))
                    u0[r] = F32(t1 + un.V[r])
                util = one_shot.utility(pol.alpha, pol.delta, np.array(un.A, F32), np.array(un.P, F32), u0)
                idx, cnt = one_shot.select(np.array(un.V, F32), util, K, pol.n_sink, pol.n_recent, pol.k_protected)
                keep = set(int(i) for i in idx[:cnt])
                gone = [r for r in range(m) if r not in keep]
                assert len(gone) == 1
                drop = un.pos[gone[0]]
                for lst in (un.pos, un.A, un.P, un.V, un.S):
                    del lst[gone[0]]
            bd = F32(pol.budget_decay)
            un.V = [F32(vv * bd) for vv in un.V]
            evicted.append(drop)
        return evicted

    def static_utility(self, u):
        """(beta*R + gamma*S - lambda*F) + V of unit u's cached tokens as of now (for the pins)."""
        pol, un = self.pol, self.units[u]
        n = len(self.ids)
        out = np.zeros(len(un.pos), F32)
        for r in range(len(un.pos)):
            c = sum(1 for i in self.ids if i == self.ids[un.pos[r]])
            R = F32(F32(un.pos[r] + 1) / F32(n))
            Ff = F32(F32(c) / F32(n))
            t0 = F32(F32(F32(pol.beta) * R) + F32(F32(pol.gamma) * F32(un.S[r])))
            t1 = F32(t0 - F32(F32(pol.lam) * Ff))
            out[r] = F32(t1 + un.V[r])
        return out
