"""Seeded synthetic inputs shaped like the paper's credential-retrieval workloads.

This module serves both the CUDA library's tests/benchmark and the CPU oracle. It only draws random numbers and
plants token-id sequences; it contains none of the method's arithmetic (no matching, scoring or selection).

The paper's workloads are prompts fed to Llama/Mistral models (a 4096-token needle-in-a-haystack prompt with the
credential at relative depth 0.1..0.9, tool-call conversations with 12-32 character credentials, decoy anchors).
Neither the models nor the prompts are available, so these generators stand in for them: token ids are uniform
over a 32000-entry vocabulary with anchor patterns and value spans planted at the stated depths, and Q/K/V are
N(0,1) values rounded to bf16.
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np
import torch

VOCAB = 32000
BASE_SEED = 0x11288 * 16


@dataclass
class Workload:
    name: str
    seed: int
    n_layers: int
    Hq: int
    Hkv: int
    d: int
    W: int
    K_list: list
    modes: list  # of "scored" / "fast"
    uniform: bool
    lengths: np.ndarray  # [B] int32
    cu: np.ndarray  # [B+1] int32
    ids: np.ndarray  # [total] int32, packed
    pattern_ids: list  # list of list[int]
    pattern_budget: list
    pattern_span: list
    planted: list  # (sequence, position of the anchor's last token, value length)
    decoys: list = field(default_factory=list)  # (sequence, position of the decoy's last token)
    vocab: int = VOCAB

    @property
    def B(self):
        return int(self.lengths.shape[0])

    @property
    def total(self):
        return int(self.cu[-1])

    @property
    def max_n(self):
        return int(self.lengths.max())


def _fresh_ids(rng, count, exclude):
    """`count` distinct ids not in `exclude`."""
    out = []
    seen = set(exclude)
    while len(out) < count:
        t = int(rng.integers(0, VOCAB))
        if t not in seen:
            seen.add(t)
            out.append(t)
    return out


def _make_patterns(rng, lens):
    used = set()
    pats = []
    for ln in lens:
        p = _fresh_ids(rng, ln, used)
        used.update(p)
        pats.append(p)
    return pats, used


def _filler(rng, total, pattern_tokens):
    return rng.integers(0, VOCAB, size=total, dtype=np.int64).astype(np.int32)


def _plant(ids, start, pattern, value):
    seq = list(pattern) + list(value)
    ids[start:start + len(seq)] = np.array(seq, np.int32)
    return start + len(pattern) - 1  # position of the anchor's last token


def _finish(name, idx, n_layers, W, K_list, modes, uniform, lengths, ids, pats, budget, span, planted, decoys=(),
            Hq=32, Hkv=8, d=128):
    lengths = np.asarray(lengths, np.int32)
    cu = np.zeros(lengths.shape[0] + 1, np.int32)
    cu[1:] = np.cumsum(lengths)
    return Workload(name=name, seed=BASE_SEED + idx, n_layers=n_layers, Hq=Hq, Hkv=Hkv, d=d, W=W, K_list=list(K_list),
                    modes=list(modes), uniform=uniform, lengths=lengths, cu=cu, ids=ids, pattern_ids=pats,
                    pattern_budget=list(budget), pattern_span=list(span), planted=list(planted), decoys=list(decoys))


def config1(n=4096, K=16, Hq=32, Hkv=8, W=32):
    """One layer, one 4096-token sequence, one 3-id anchor pattern planted four times (each followed by 8 value
    ids) with the anchor's last token at relative depth 0.1/0.3/0.5/0.9; K = 16; scored TA."""
    rng = np.random.default_rng(BASE_SEED + 1)
    pats, used = _make_patterns(rng, [3])
    ids = _filler(rng, n, used)
    planted = []
    for depth in (0.1, 0.3, 0.5, 0.9):
        e = int(depth * n)
        val = _fresh_ids(rng, 8, used)
        _plant(ids, e - 2, pats[0], val)
        planted.append((0, e, 8))
    return _finish("c1", 1, 1, W, [K], ["scored"], True, [n], ids, pats, [15.0], [6], planted, Hq=Hq, Hkv=Hkv)


def config2(n=4096, n_layers=32, K_list=(16, 32, 64, 128, 256, 1024), Hq=32, Hkv=8, W=32):
    """32 layers, one 4096-token sequence, a single 3-id anchor followed by 16 value ids at depth 0.5; budget
    sweep; scored TA and TA-Fast."""
    rng = np.random.default_rng(BASE_SEED + 2)
    pats, used = _make_patterns(rng, [3])
    ids = _filler(rng, n, used)
    e = int(0.5 * n)
    _plant(ids, e - 2, pats[0], _fresh_ids(rng, 16, used))
    return _finish("c2", 2, n_layers, W, K_list, ["scored", "fast"], True, [n], ids, pats, [15.0], [6], [(0, e, 16)],
                   Hq=Hq, Hkv=Hkv)


def _plant_many(rng, ids, base, n, pats, used, count, vlen_lo, vlen_hi, seq, planted):
    """Plant `count` non-overlapping (pattern + value) spans at uniform random depths inside [base, base+n)."""
    slot = n // count
    for s in range(count):
        p = int(rng.integers(0, len(pats)))
        vlen = int(rng.integers(vlen_lo, vlen_hi + 1))
        need = len(pats[p]) + vlen
        if slot <= need + 1:
            continue
        start = s * slot + int(rng.integers(0, slot - need))
        e = _plant(ids, base + start, pats[p], _fresh_ids(rng, vlen, used))
        planted.append((seq, e - base, vlen))


def config3(B=16, n=32768, n_layers=32, K=2048, plants=64, Hq=32, Hkv=8, W=64):
    """32 layers, 16 sequences of 32768 tokens, 8 distinct patterns of 1-3 ids, 64 planted spans per sequence with
    value lengths 4-24 at uniform random depths; K = 2048; observation window 64; scored TA."""
    rng = np.random.default_rng(BASE_SEED + 3)
    pats, used = _make_patterns(rng, [1, 1, 2, 2, 2, 3, 3, 3])
    ids = _filler(rng, B * n, used)
    planted = []
    for b in range(B):
        _plant_many(rng, ids, b * n, n, pats, used, plants, 4, 24, b, planted)
    return _finish("c3", 3, n_layers, W, [K], ["scored"], True, [n] * B, ids, pats, [15.0] * 8, [6] * 8, planted,
                   Hq=Hq, Hkv=Hkv)


def config4(B=4, n=131072, n_layers=32, K=4096, plants=512, Hkv=8):
    """TA-Fast only: 4 sequences of 131072 tokens, 8 patterns whose spans are 8-32 tokens, 512 planted anchors per
    sequence of which about a quarter overlap the previous anchor's span and about a quarter abut it; K = 4096."""
    rng = np.random.default_rng(BASE_SEED + 4)
    spans = [8, 12, 16, 20, 24, 28, 32, 32]
    pats, used = _make_patterns(rng, [2, 2, 2, 2, 3, 3, 3, 3])
    ids = _filler(rng, B * n, used)
    planted = []
    slot = n // plants
    for b in range(B):
        prev_end, prev_span = None, None
        for s in range(plants):
            p = int(rng.integers(0, len(pats)))
            kind = int(rng.integers(0, 4))  # 0: overlap the previous span, 1: abut it, 2-3: free placement
            lp = len(pats[p])
            if prev_end is not None and kind == 0 and prev_span > lp + 1:
                start = prev_end + 1 + int(rng.integers(0, prev_span - lp))  # anchor inside the previous span
            elif prev_end is not None and kind == 1:
                start = prev_end + prev_span + 1 - (lp - 1) - 1  # this span starts where the previous one stops
                start = max(start, prev_end + 1)
            else:
                lo = s * slot
                if prev_end is not None:
                    lo = max(lo, prev_end + prev_span + 2)
                start = lo + int(rng.integers(0, max(1, slot // 4)))
            if start + lp + spans[p] >= n:
                break
            e = _plant(ids, b * n + start, pats[p], _fresh_ids(rng, spans[p], used)) - b * n
            planted.append((b, e, spans[p]))
            prev_end, prev_span = e, spans[p]
    return _finish("c4", 4, n_layers, 32, [K], ["fast"], True, [n] * B, ids, pats, [15.0] * 8, spans, planted,
                   Hq=32, Hkv=Hkv)


def config5(B=64, n_lo=2048, n_hi=16384, n_layers=32, K=64, decoys_per_seq=32, Hq=32, Hkv=8, W=32):
    """Ragged agentic batch: 64 sequences with lengths uniform in [2048, 16384], 4 patterns of 2-3 ids, 1-8
    planted credential-style spans per sequence (value lengths 6-40) and 32 decoys per sequence that repeat a
    pattern's proper prefix followed by an id that breaks the match; K = 64; scored TA."""
    rng = np.random.default_rng(BASE_SEED + 5)
    pats, used = _make_patterns(rng, [2, 2, 3, 3])
    lengths = rng.integers(n_lo, n_hi + 1, size=B).astype(np.int32)
    cu = np.zeros(B + 1, np.int64)
    cu[1:] = np.cumsum(lengths)
    ids = _filler(rng, int(cu[-1]), used)
    planted, decoys = [], []
    for b in range(B):
        n = int(lengths[b])
        base = int(cu[b])
        count = int(rng.integers(1, 9))
        _plant_many(rng, ids, base, n, pats, used, count, 6, 40, b, planted)
        occupied = np.zeros(n, bool)
        for (sb, e, vl) in planted:
            if sb == b:
                occupied[max(0, e - 3):min(n, e + vl + 2)] = True
        placed = 0
        while placed < decoys_per_seq:
            p = int(rng.integers(0, len(pats)))
            plen = int(rng.integers(1, len(pats[p])))  # proper prefix
            pos = int(rng.integers(1, n - plen - 2))
            if occupied[pos - 1:pos + plen + 2].any():
                continue
            breaker = _fresh_ids(rng, 1, used)[0]
            ids[base + pos:base + pos + plen] = np.array(pats[p][:plen], np.int32)
            ids[base + pos + plen] = breaker
            occupied[pos - 1:pos + plen + 2] = True
            decoys.append((b, pos + plen - 1))
            placed += 1
    return _finish("c5", 5, n_layers, W, [K], ["scored"], False, lengths, ids, pats, [15.0] * 4, [6] * 4, planted,
                   decoys, Hq=Hq, Hkv=Hkv)


CONFIGS = {"c1": config1, "c2": config2, "c3": config3, "c4": config4, "c5": config5}


def make_qkv(w: Workload, layers, device="cpu", need_q=True, need_kv=True):
    """Q_obs [L,B,Hq,W,d], K and V [L,B,Hkv,n,d] (uniform) or [L,Hkv,total,d] (ragged), bf16 ~ N(0,1).

    `layers` is a list of layer indices; each layer's tensors come from their own seeded stream, so any subset of
    layers can be drawn independently and reproducibly. Values drawn on different devices differ; a test draws once
    and hands the same bytes to both sides.
    """
    layers = list(layers)
    L = len(layers)
    kv_shape = (w.B, w.Hkv, int(w.lengths[0]), w.d) if w.uniform else (w.Hkv, w.total, w.d)
    # the outputs are allocated once and filled layer by layer (no second copy of a 30 GB cache while stacking)
    Q = torch.empty((L, w.B, w.Hq, w.W, w.d), dtype=torch.bfloat16, device=device) if need_q else None
    K = torch.empty((L,) + kv_shape, dtype=torch.bfloat16, device=device) if need_kv else None
    V = torch.empty((L,) + kv_shape, dtype=torch.bfloat16, device=device) if need_kv else None
    for i, l in enumerate(layers):
        g = torch.Generator(device=device)
        g.manual_seed(w.seed * 1000 + l)
        if need_q:
            Q[i].copy_(torch.randn((w.B, w.Hq, w.W, w.d), generator=g, device=device, dtype=torch.float32))
        if need_kv:
            torch.randn(kv_shape, generator=g, device=device, dtype=torch.bfloat16, out=K[i])
            torch.randn(kv_shape, generator=g, device=device, dtype=torch.bfloat16, out=V[i])
    return Q, K, V
