"""GPU parity of the fused ta_compress call on seeded random shapes: head counts, window sizes, uniform and ragged
batches (empty, one-token and tile-boundary lengths included), layer counts beyond one round of the persistent score
grid, budgets from 1 to more than a sequence holds, both presets, scored and fast mode. Every output is allocated with
guard layers behind it, which must come back untouched."""
import numpy as np
import pytest
import torch

import oracle
import paper_2604_11288_b200 as ta
import ta_workloads as tw
from ta_testlib import (Gpu, assert_selection_matches, bf16_bits, oracle_patterns, oracle_policy, oracle_unit, unit_kv)
from test_gpu_steps import _workload

pytestmark = pytest.mark.gpu
GUARD = 3


def _draw(rng):
    Hkv = int(rng.choice([1, 2, 4, 8]))
    W = int(rng.choice([8, 16, 24, 32, 48, 64]))
    G = int(rng.choice([g for g in (1, 2, 4, 8) if g * W <= 256]))
    B = int(rng.integers(1, 5))
    if rng.random() < 0.3:
        lengths = [int(rng.integers(1, 2500))] * B
    else:
        special = [0, 1, 5, 40, 127, 128, 129, 300, 1000, 2100, 2600]
        lengths = [int(rng.choice(special)) if rng.random() < 0.5 else int(rng.integers(1, 3000)) for _ in range(B)]
    if sum(lengths) == 0:
        lengths[0] = 17
    L = int(rng.integers(1, 4))
    if rng.random() < 0.15:  # many short units: the score grid walks them in more than one round
        L = int(rng.integers(20, 40))
        lengths = [min(x, 400) for x in lengths]
    K = int(rng.choice([1, 2, 5, 12, 16, 24, 64, 100, 300]))
    return dict(Hq=Hkv * G, Hkv=Hkv, W=W, lengths=lengths, L=L, K=K, preset=str(rng.choice(["THEOREM", "SEC33"])),
                fast=bool(rng.random() < 0.25), seed=int(rng.integers(1, 1000)))


@pytest.mark.parametrize("seed", [11, 12])
def test_compress_random_shapes(seed):
    rng = np.random.default_rng(seed)
    for case in range(20):
        c = _draw(rng)
        what = f"seed {seed} case {case}: {c}"
        L, K, fast = c["L"], c["K"], c["fast"]
        w = _workload(c["lengths"], [[4, 5], [6], [7, 8, 9]], seed=c["seed"], Hq=c["Hq"], Hkv=c["Hkv"], W=c["W"])
        w.n_layers = L
        pol = oracle_policy(K, c["preset"], fast=fast, W=c["W"])
        Qh, Kh, Vh = tw.make_qkv(w, range(L))
        g = Gpu(w, pol, K, L)
        try:
            Qd, Kd, Vd = Qh.cuda(), Kh.cuda(), Vh.cuda()  # held until the call has run: a view is only a pointer
            idx = torch.full((L + GUARD, w.B, w.Hkv, K), -7, dtype=torch.int32, device=g.dev)
            cnt = torch.full((L + GUARD, w.B, w.Hkv), -7, dtype=torch.int32, device=g.dev)
            ko = torch.full((L + GUARD, w.B, w.Hkv, K, w.d), 1.0, dtype=torch.bfloat16, device=g.dev)
            vo = torch.full_like(ko, 1.0)
            rag = not w.uniform
            ta.ta_compress(g.ctx, g.pats, g.p, g.batch, w.Hq, w.Hkv, w.d, K, g.ids,
                           ta.view(None) if fast else ta.view(Qd), ta.view(Kd, rag), ta.view(Vd, rag), 0, ko, vo, idx,
                           cnt, g.stream)
            torch.cuda.synchronize()
            assert g.poll() == ta.TA_OK, what
            assert (idx[L:] == -7).all() and (cnt[L:] == -7).all() and (ko[L:] == 1.0).all() and (vo[L:] == 1.0).all(), what
            idx_h, cnt_h = idx[:L].cpu().numpy(), cnt[:L].cpu().numpy()
            f_o, V_o, u0_o = oracle.sponsor_mask(w.ids, w.cu, oracle_patterns(w), pol)
            for l in (range(L) if L <= 3 else (0, L - 1)):
                for b in range(w.B):
                    for h in range(w.Hkv):
                        A, P, u, io, co = oracle_unit(w, pol, K, Qh, Kh, l, b, h, V_o, u0_o)
                        same = assert_selection_matches(idx_h[l, b, h], cnt_h[l, b, h], io, co, u, f"{what} l{l} b{b} h{h}")
                        if fast:
                            assert same, what
                        sel, n_sel = idx_h[l, b, h], int(cnt_h[l, b, h])
                        np.testing.assert_array_equal(bf16_bits(ko[l, b, h]),
                                                      oracle.compact(unit_kv(w, Kh, l, b, h), sel, n_sel, K), err_msg=what)
                        np.testing.assert_array_equal(bf16_bits(vo[l, b, h]),
                                                      oracle.compact(unit_kv(w, Vh, l, b, h), sel, n_sel, K), err_msg=what)
        finally:
            g.close()
