"""GPU parity of ta_stream_step (Algorithm 1 run once per decode step) against the streaming CPU oracle: the same
token stream and the same per-step attention masses go to both; evicted positions and the whole per-unit state must
agree bit for bit after every step."""
import ctypes as C

import numpy as np
import pytest
import torch

import oracle
import paper_2604_11288_b200 as ta
from oracle.ta_stream_oracle import StreamOracle
from ta_testlib import gpu_policy

pytestmark = pytest.mark.gpu


class GpuStream:
    def __init__(self, pats: oracle.Patterns, pol: oracle.Policy, K, L, B, Hkv, dev="cuda:0"):
        self.dev = torch.device(dev)
        self.p = gpu_policy(pol)
        self.U, self.C, self.B = L * B * Hkv, K + 1, B
        z = lambda shape, dt: torch.zeros(shape, dtype=dt, device=self.dev)
        self.t = dict(pos=z((self.U, self.C), torch.int32), slot=z((self.U, self.C), torch.int32),
                      tok=z((self.U, self.C), torch.int32), A=z((self.U, self.C), torch.float32),
                      P=z((self.U, self.C), torch.float32), V=z((self.U, self.C), torch.float32),
                      S=z((self.U, self.C), torch.uint8), next_slot=z((self.U,), torch.int32),
                      n_seen=z((B,), torch.int32), hist=z((B, pol.vocab_size), torch.int32),
                      tok_ring=z((B, 8), torch.int32), anc_B=z((B, 64), torch.float32), anc_L=z((B, 64), torch.int32))
        st = ta.ta_stream()
        st.n_layers, st.batch, st.Hkv, st.K, st.cache_len = L, B, Hkv, K, 0
        for k, v in self.t.items():
            setattr(st, k, v.data_ptr())
        self.st = st
        self.ctx = ta.ta_ctx_create(0, ta.ta_stream_scratch_bytes(st))
        self.pats = ta.ta_patterns_create(self.ctx, pats.ids, pats.budget, pats.span)
        self.evicted = torch.full((self.U,), -9, dtype=torch.int32, device=self.dev)
        self.stream = torch.cuda.current_stream(self.dev).cuda_stream

    def step(self, new_ids, attn_rows):
        ta.ta_stream_step(self.ctx, self.pats, self.p, self.st, torch.from_numpy(new_ids).to(self.dev),
                          torch.from_numpy(attn_rows).to(self.dev), self.evicted, self.stream)
        torch.cuda.synchronize()
        return self.evicted.cpu().numpy()

    def close(self):
        ta.ta_patterns_destroy(self.pats)
        ta.ta_ctx_destroy(self.ctx)


def _run(K, L, B, Hkv, steps, pats, pol, seed, check_every=1):
    rng = np.random.default_rng(seed)
    g = GpuStream(pats, pol, K, L, B, Hkv)
    U, Cc = g.U, g.C
    ora = [StreamOracle(pats, pol, K, L * Hkv) for _ in range(B)]  # units of sequence b: (l, g) -> l*Hkv + g
    unit_of = lambda l, b, h: (l * B + b) * Hkv + h
    # host mirror of which cache row holds which position (what a caller's attention kernel would know)
    row_of = [dict() for _ in range(U)]
    next_row = np.zeros(U, np.int64)
    alphabet = 12
    plant = [p for p in pats.ids]
    try:
        queue = [[] for _ in range(B)]
        for t in range(steps):
            new_ids = np.zeros(B, np.int32)
            for b in range(B):
                if not queue[b] and plant and rng.random() < 0.08:
                    queue[b] = list(plant[int(rng.integers(0, len(plant)))])
                new_ids[b] = queue[b].pop(0) if queue[b] else int(rng.integers(0, alphabet))
            attn_rows = np.zeros((U, Cc), np.float32)
            attn_pos = [[None] * (L * Hkv) for _ in range(B)]
            for l in range(L):
                for b in range(B):
                    for h in range(Hkv):
                        u = unit_of(l, b, h)
                        row_of[u][t] = int(next_row[u])
                        ps = sorted(row_of[u])
                        a = rng.random(len(ps)).astype(np.float32)
                        a /= a.sum()
                        if rng.random() < 0.3:
                            a[:] = a[0]  # ties
                        d = {}
                        for p, x in zip(ps, a):
                            attn_rows[u, row_of[u][p]] = x
                            d[p] = float(x)
                        attn_pos[b][l * Hkv + h] = d
            ev = g.step(new_ids, attn_rows)
            for b in range(B):
                ev_o = ora[b].step(int(new_ids[b]), attn_pos[b])
                for l in range(L):
                    for h in range(Hkv):
                        u = unit_of(l, b, h)
                        assert ev[u] == ev_o[l * Hkv + h], f"step {t} unit {u}"
                        if ev[u] >= 0:
                            next_row[u] = row_of[u].pop(int(ev[u]))
                        else:
                            next_row[u] = len(row_of[u])
            assert g.st.cache_len == min(t + 1, K)
            if t % check_every == 0 or t == steps - 1:
                n = g.st.cache_len
                S = {k: v.cpu().numpy() for k, v in g.t.items()}
                np.testing.assert_array_equal(S["next_slot"], next_row.astype(np.int32))
                for b in range(B):
                    for l in range(L):
                        for h in range(Hkv):
                            u, un = unit_of(l, b, h), ora[b].units[l * Hkv + h]
                            np.testing.assert_array_equal(S["pos"][u, :n], np.array(un.pos, np.int32))
                            np.testing.assert_array_equal(S["S"][u, :n], np.array(un.S, np.uint8))
                            for name, ref in (("A", un.A), ("P", un.P), ("V", un.V)):
                                np.testing.assert_array_equal(S[name][u, :n].view(np.uint32),
                                                              np.array(ref, np.float32).view(np.uint32),
                                                              err_msg=f"{name} step {t} unit {u}")
                            np.testing.assert_array_equal(S["slot"][u, :n],
                                                          np.array([row_of[u][p] for p in un.pos], np.int32))
                            np.testing.assert_array_equal(S["tok"][u, :n],
                                                          np.array([ora[b].ids[p] for p in un.pos], np.int32))
        assert ta.ta_ctx_poll(g.ctx) == ta.TA_OK
    finally:
        g.close()


def test_stream_small_budget_all_presets():
    pats = oracle.Patterns([[1, 2], [3], [4, 1, 2]], budget=[15.0, 4.0, 9.0], span=[6, 3, 8])
    for preset in ("THEOREM", "SEC33", "AUDIT"):
        pol = oracle.preset(preset, 16, vocab_size=64)
        _run(K=16, L=2, B=2, Hkv=2, steps=90, pats=pats, pol=pol, seed=1)


def test_stream_budget_larger_than_a_block():
    # K + 1 = 301 entries per unit: the ordered state is shifted in two 256-entry chunks
    pats = oracle.Patterns([[5, 6]], budget=[15.0], span=[40])
    pol = oracle.preset("THEOREM", 300, vocab_size=64)
    _run(K=300, L=1, B=1, Hkv=2, steps=380, pats=pats, pol=pol, seed=2, check_every=37)


def test_stream_no_patterns_tiny_budget():
    pol = oracle.preset("SEC33", 1, vocab_size=64)
    _run(K=1, L=1, B=3, Hkv=1, steps=12, pats=oracle.Patterns([]), pol=pol, seed=3)
