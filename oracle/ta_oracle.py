"""TEST INFRASTRUCTURE: ctypes access to the CPU oracle (oracle/ta_oracle.cpp).

Thin marshalling only; every step of the method is in the C++ file, each function citing the passage of the
paper it follows. `build_oracle()` compiles the shared object with g++ (no CUDA involved).
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from dataclasses import dataclass, field

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "ta_oracle.cpp")
_LIB = os.path.join(_HERE, "libta_oracle.so")
_lib = None


def build_oracle(force: bool = False) -> str:
    """Compile oracle/ta_oracle.cpp -> oracle/libta_oracle.so (skipped when up to date)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["g++", "-O2", "-std=c++17", "-fopenmp", "-ffp-contract=off", "-shared", "-fPIC", _SRC, "-o", _LIB]
        subprocess.run(cmd, check=True)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        build_oracle()
        _lib = C.CDLL(_LIB)
    return _lib


def _p(a, t):
    return a.ctypes.data_as(C.POINTER(t))


@dataclass
class Patterns:
    """A pattern set P (Section 3.2): token-id sequences with per-pattern sponsor budget B and span L."""

    ids: list  # list of lists of int
    budget: list = None  # default 15 (Eq. 2)
    span: list = None  # default 6 (Eq. 2)

    def __post_init__(self):
        if self.budget is None:
            self.budget = [15.0] * len(self.ids)
        if self.span is None:
            self.span = [6] * len(self.ids)

    def flat(self):
        off = np.zeros(len(self.ids) + 1, np.int32)
        for p, s in enumerate(self.ids):
            off[p + 1] = off[p] + len(s)
        flat = np.array([t for s in self.ids for t in s] or [0], np.int32)
        return flat, off, np.array(self.budget or [0], np.float32), np.array(self.span or [0], np.int32)


@dataclass
class Policy:
    """Hyper-parameters of Eq. 1 / Eq. 2 / Section 3.3 with the paper's defaults."""

    alpha: float = 1.0
    beta: float = 0.5
    gamma: float = 0.3
    delta: float = 0.2
    lam: float = 0.1
    voucher_decay: float = 0.8
    budget_decay: float = 0.9
    age_steps: int = 0
    n_sink: int = 1
    n_recent: int = 4
    k_protected: int = -1
    obs_window: int = 32
    pension_rho: float = 0.9
    softmax_scale: float = 0.0
    causal: int = 1
    fast: int = 0
    vocab_size: int = 32000


def preset(name: str, K: int, **kw) -> Policy:
    """The three budget partitions the paper states (Theorems 2-4; Section 3.3; the baseline-audit table)."""
    if name == "THEOREM":
        return Policy(n_sink=1, n_recent=4, k_protected=-1, **kw)
    if name == "SEC33":
        return Policy(n_sink=1, n_recent=2, k_protected=K // 4, **kw)
    if name == "AUDIT":
        return Policy(n_sink=4, n_recent=6, k_protected=6, **kw)
    raise ValueError(name)


def num_threads() -> int:
    return int(_load().ora_num_threads())


def anchors(ids: np.ndarray, pats: Patterns, budget_decay=0.9, age_steps=0):
    lib = _load()
    ids = np.ascontiguousarray(ids, np.int32)
    n = ids.shape[0]
    flat, off, bud, span = pats.flat()
    atok = np.zeros(n, np.uint8)
    aend = np.zeros(n, np.uint8)
    Be = np.zeros(n, np.float32)
    Le = np.zeros(n, np.int32)
    lib.ora_anchors(C.c_int(n), _p(ids, C.c_int32), C.c_int(len(pats.ids)), _p(flat, C.c_int32), _p(off, C.c_int32),
                    _p(bud, C.c_float), _p(span, C.c_int32), C.c_float(budget_decay), C.c_int(age_steps),
                    _p(atok, C.c_uint8), _p(aend, C.c_uint8), _p(Be, C.c_float), _p(Le, C.c_int32))
    return atok, aend, Be, Le


def anchors_conf(conf: np.ndarray, threshold, budget, span, rank, budget_decay=0.9, age_steps=0):
    """Anchors from a detector's per-token confidence (Section 5.1): same outputs as anchors()."""
    lib = _load()
    conf = np.ascontiguousarray(conf, np.float32)
    n = conf.shape[0]
    atok = np.zeros(n, np.uint8)
    aend = np.zeros(n, np.uint8)
    Be = np.zeros(n, np.float32)
    Le = np.zeros(n, np.int32)
    lib.ora_anchors_conf(C.c_int(n), _p(conf, C.c_float), C.c_float(threshold), C.c_float(budget), C.c_int(span),
                         C.c_int(1 if rank else 0), C.c_float(budget_decay), C.c_int(age_steps), _p(atok, C.c_uint8),
                         _p(aend, C.c_uint8), _p(Be, C.c_float), _p(Le, C.c_int32))
    return atok, aend, Be, Le


def embedding_confidence(emb: np.ndarray, concepts: np.ndarray):
    """Embedding-based anchor detector (Section 3.2 "Anchor detection", instantiation 3): the confidence of token i is
    the largest cosine similarity between its input embedding and the anchor-concept embeddings. emb uint16 (bf16
    bits) [n, D], concepts uint16 [C, D]; evaluated in double, rounded to fp32; a zero vector has similarity 0.
    Pinned by: identical vectors -> 1, opposite -> -1, orthogonal -> 0, scale invariance."""
    def dec(a):
        return (a.astype(np.uint32) << 16).view(np.float32).astype(np.float64)
    e, c = dec(np.ascontiguousarray(emb)), dec(np.ascontiguousarray(concepts))
    ne = np.sqrt((e * e).sum(-1))
    nc = np.sqrt((c * c).sum(-1))
    dots = e @ c.T
    den = ne[:, None] * nc[None, :]
    cos = np.where(den > 0, dots / np.where(den > 0, den, 1.0), 0.0)
    return cos.max(-1).astype(np.float32)


def vouchers(aend, Be, Le, voucher_decay=0.8):
    lib = _load()
    n = aend.shape[0]
    V = np.zeros(n, np.float32)
    lib.ora_vouchers(C.c_int(n), _p(aend, C.c_uint8), _p(Be, C.c_float), _p(Le, C.c_int32), C.c_float(voucher_decay),
                     _p(V, C.c_float))
    return V


def static_utility(ids, atok, V, beta=0.5, gamma=0.3, lam=0.1, vocab=None):
    lib = _load()
    ids = np.ascontiguousarray(ids, np.int32)
    n = ids.shape[0]
    u0 = np.zeros(n, np.float32)
    if vocab is None:
        lib.ora_static_utility(C.c_int(n), _p(ids, C.c_int32), _p(atok, C.c_uint8), _p(V, C.c_float), C.c_float(beta),
                               C.c_float(gamma), C.c_float(lam), _p(u0, C.c_float))
    else:
        lib.ora_static_utility_hist(C.c_int(n), _p(ids, C.c_int32), C.c_int(vocab), _p(atok, C.c_uint8),
                                    _p(V, C.c_float), C.c_float(beta), C.c_float(gamma), C.c_float(lam),
                                    _p(u0, C.c_float))
    return u0


def sponsor_mask(ids, cu, pats: Patterns, pol: Policy):
    """Per-token flags (bit0 S, bit1 anchor end, bit2 sponsored), vouchers and attention-free utility for a packed
    batch described by cu (B+1 offsets)."""
    total = int(cu[-1])
    flags = np.zeros(total, np.uint8)
    V = np.zeros(total, np.float32)
    u0 = np.zeros(total, np.float32)
    for b in range(len(cu) - 1):
        o, e = int(cu[b]), int(cu[b + 1])
        atok, aend, Be, Le = anchors(ids[o:e], pats, pol.budget_decay, pol.age_steps)
        v = vouchers(aend, Be, Le, pol.voucher_decay)
        V[o:e] = v
        u0[o:e] = static_utility(ids[o:e], atok, v, pol.beta, pol.gamma, pol.lam, vocab=pol.vocab_size)
        flags[o:e] = atok | (aend << 1) | ((v > 0).astype(np.uint8) << 2)
    return flags, V, u0


def sponsor_mask_conf(ids, cu, conf, threshold, budget, span, rank, pol: Policy):
    """sponsor_mask() with the anchors taken from a detector's confidences instead of token-id patterns."""
    total = int(cu[-1])
    flags = np.zeros(total, np.uint8)
    V = np.zeros(total, np.float32)
    u0 = np.zeros(total, np.float32)
    for b in range(len(cu) - 1):
        o, e = int(cu[b]), int(cu[b + 1])
        atok, aend, Be, Le = anchors_conf(conf[o:e], threshold, budget, span, rank, pol.budget_decay, pol.age_steps)
        v = vouchers(aend, Be, Le, pol.voucher_decay)
        V[o:e] = v
        u0[o:e] = static_utility(ids[o:e], atok, v, pol.beta, pol.gamma, pol.lam, vocab=pol.vocab_size)
        flags[o:e] = atok | (aend << 1) | ((v > 0).astype(np.uint8) << 2)
    return flags, V, u0


def attention(Q: np.ndarray, K: np.ndarray, n: int, scale=0.0, causal=1, rho=0.9):
    """Q: uint16 (bf16 bits) [G, W, d]; K: uint16 [n, d] (any row stride). Returns A, P float32 [n]."""
    lib = _load()
    assert Q.dtype == np.uint16 and K.dtype == np.uint16
    Q = np.ascontiguousarray(Q)
    G, W, d = Q.shape
    if n == 0:
        return np.zeros(0, np.float32), np.zeros(0, np.float32)
    assert K.strides[1] == 2
    A = np.zeros(n, np.float32)
    P = np.zeros(n, np.float32)
    lib.ora_attention(C.c_int(n), C.c_int(G), C.c_int(W), C.c_int(d), _p(Q, C.c_uint16), C.c_int64(W * d),
                      C.c_int64(d), _p(K, C.c_uint16), C.c_int64(K.strides[0] // 2), C.c_double(scale),
                      C.c_int(causal), C.c_double(rho), _p(A, C.c_float), _p(P, C.c_float))
    return A, P


def attention_allheads(Q: np.ndarray, K: np.ndarray, n: int, scale=0.0, causal=1, rho=0.9):
    """Q: uint16 [Hq, W, d]; K: uint16 [Hkv, n, d] (contiguous). A, P float32 [n] summed over all query heads."""
    lib = _load()
    assert Q.dtype == np.uint16 and K.dtype == np.uint16
    Q = np.ascontiguousarray(Q)
    K = np.ascontiguousarray(K)
    Hq, W, d = Q.shape
    Hkv = K.shape[0]
    if n == 0:
        return np.zeros(0, np.float32), np.zeros(0, np.float32)
    A = np.zeros(n, np.float32)
    P = np.zeros(n, np.float32)
    lib.ora_attention_allheads(C.c_int(n), C.c_int(Hq), C.c_int(Hkv), C.c_int(W), C.c_int(d), _p(Q, C.c_uint16),
                               C.c_int64(W * d), C.c_int64(d), _p(K, C.c_uint16), C.c_int64(K.shape[1] * d),
                               C.c_int64(d), C.c_double(scale), C.c_int(causal), C.c_double(rho), _p(A, C.c_float),
                               _p(P, C.c_float))
    return A, P


def utility(alpha, delta, A, P, u0):
    lib = _load()
    n = u0.shape[0]
    u = np.zeros(n, np.float32)
    A = np.ascontiguousarray(A, np.float32)
    P = None if P is None else np.ascontiguousarray(P, np.float32)
    u0 = np.ascontiguousarray(u0, np.float32)
    lib.ora_utility(C.c_int(n), C.c_float(alpha), C.c_float(delta), _p(A, C.c_float),
                    C.POINTER(C.c_float)() if P is None else _p(P, C.c_float),
                    _p(u0, C.c_float), _p(u, C.c_float))
    return u


def select(V, u, K, n_sink=1, n_recent=4, k_protected=-1):
    lib = _load()
    V = np.ascontiguousarray(V, np.float32)
    u = np.ascontiguousarray(u, np.float32)
    n = u.shape[0]
    idx = np.full(max(K, 1), -1, np.int32)
    cnt = C.c_int32(0)
    lib.ora_select(C.c_int(n), C.c_int(K), C.c_int(n_sink), C.c_int(n_recent), C.c_int(k_protected), _p(V, C.c_float),
                   _p(u, C.c_float), _p(idx, C.c_int32), C.byref(cnt))
    return idx[:K], int(cnt.value)


def compact(src: np.ndarray, idx: np.ndarray, count: int, K: int):
    """src: uint16 [n, d] (row stride arbitrary); returns uint16 [K, d]."""
    lib = _load()
    d = src.shape[1]
    dst = np.empty((K, d), np.uint16)
    idx = np.ascontiguousarray(idx, np.int32)
    lib.ora_compact(C.c_int(d), C.c_int(K), _p(src, C.c_uint16), C.c_int64(src.strides[0] // 2), _p(idx, C.c_int32),
                    C.c_int(count), _p(dst, C.c_uint16))
    return dst


def compress_layer(ids, cu, uniform, Hq, Hkv, d, K, pats: Patterns, pol: Policy, Q, Kc, Vc):
    """Algorithm 1 for one layer. Q uint16 [B,Hq,W,d]; Kc, Vc uint16 [B,Hkv,n,d] (uniform) or [Hkv,total,d].
    Returns idx [B,Hkv,K], count [B,Hkv], k_out, v_out [B,Hkv,K,d] (uint16) and (seconds_seq, seconds_units)."""
    lib = _load()
    ids = np.ascontiguousarray(ids, np.int32)
    cu = np.ascontiguousarray(cu, np.int32)
    B = cu.shape[0] - 1
    flat, off, bud, span = pats.flat()
    idx = np.full((B, Hkv, K), -1, np.int32)
    cnt = np.zeros((B, Hkv), np.int32)
    ko = np.zeros((B, Hkv, K, d), np.uint16)
    vo = np.zeros((B, Hkv, K, d), np.uint16)
    sec = np.zeros(2, np.float64)
    if Q is None:
        Q = np.zeros(1, np.uint16)
    for a in (Q, Kc, Vc):
        assert a.dtype == np.uint16 and a.flags["C_CONTIGUOUS"]
    lib.ora_compress_layer(
        C.c_int(B), _p(cu, C.c_int32), C.c_int(1 if uniform else 0), C.c_int(Hq), C.c_int(Hkv), C.c_int(d),
        C.c_int(pol.obs_window), C.c_int(K), _p(ids, C.c_int32), C.c_int(pol.vocab_size), C.c_int(len(pats.ids)),
        _p(flat, C.c_int32), _p(off, C.c_int32), _p(bud, C.c_float), _p(span, C.c_int32), C.c_float(pol.alpha),
        C.c_float(pol.beta), C.c_float(pol.gamma), C.c_float(pol.delta), C.c_float(pol.lam),
        C.c_float(pol.voucher_decay), C.c_float(pol.budget_decay), C.c_int(pol.age_steps), C.c_int(pol.n_sink),
        C.c_int(pol.n_recent), C.c_int(pol.k_protected), C.c_double(pol.pension_rho), C.c_double(pol.softmax_scale),
        C.c_int(pol.causal), C.c_int(pol.fast), _p(Q, C.c_uint16), _p(Kc, C.c_uint16), _p(Vc, C.c_uint16),
        _p(idx, C.c_int32), _p(cnt, C.c_int32), _p(ko, C.c_uint16), _p(vo, C.c_uint16), _p(sec, C.c_double))
    return idx, cnt, ko, vo, (float(sec[0]), float(sec[1]))
