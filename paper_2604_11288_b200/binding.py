"""ctypes binding of libta.so: the same names and arguments as include/ta.h, marshalling only.

Every step of the method runs in the CUDA kernels behind these calls. There is no CPU path: if the shared library is
missing, loading raises. Tensors are passed as raw device (or, for ta_compress_host, host) addresses; torch is used
by callers only to own memory and streams.
"""
from __future__ import annotations

import ctypes as C
import os

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libta.so")

TA_OK = 0
TA_ERR_INVALID_ARG, TA_ERR_UNSUPPORTED, TA_ERR_ALIGNMENT, TA_ERR_SCRATCH_TOO_SMALL = 1, 2, 3, 4
TA_ERR_CUDA, TA_ERR_TIMEOUT, TA_ERR_DEVICE_BOUNDS = 5, 6, 7
TA_MODE_SCORED, TA_MODE_FAST = 0, 1
TA_FLAG_ANCHOR_TOKEN, TA_FLAG_ANCHOR_END, TA_FLAG_SPONSORED = 1, 2, 4
TA_PRESET_THEOREM, TA_PRESET_SEC33, TA_PRESET_AUDIT = 0, 1, 2


class ta_policy(C.Structure):
    _fields_ = [("alpha", C.c_float), ("beta", C.c_float), ("gamma", C.c_float), ("delta", C.c_float),
                ("lambda_", C.c_float), ("voucher_decay", C.c_float), ("budget_decay", C.c_float),
                ("age_steps", C.c_int32), ("n_sink", C.c_int32), ("n_recent", C.c_int32), ("k_protected", C.c_int32),
                ("obs_window", C.c_int32), ("pension_rho", C.c_float), ("softmax_scale", C.c_float),
                ("causal", C.c_int32), ("mode", C.c_int32), ("vocab_size", C.c_int32)]


class ta_batch(C.Structure):
    _fields_ = [("n_layers", C.c_int32), ("batch", C.c_int32), ("n_uniform", C.c_int32), ("max_n", C.c_int32),
                ("total_tokens", C.c_int64), ("cu_seqlens", C.c_void_p)]


class ta_bf16_view(C.Structure):
    _fields_ = [("ptr", C.c_void_p), ("stride_l", C.c_int64), ("stride_b", C.c_int64), ("stride_h", C.c_int64),
                ("stride_n", C.c_int64)]


class ta_stream(C.Structure):
    _fields_ = [("n_layers", C.c_int32), ("batch", C.c_int32), ("Hkv", C.c_int32), ("K", C.c_int32),
                ("cache_len", C.c_int32), ("pos", C.c_void_p), ("slot", C.c_void_p), ("tok", C.c_void_p),
                ("A", C.c_void_p), ("P", C.c_void_p), ("V", C.c_void_p), ("S", C.c_void_p), ("next_slot", C.c_void_p),
                ("n_seen", C.c_void_p), ("hist", C.c_void_p), ("tok_ring", C.c_void_p), ("anc_B", C.c_void_p),
                ("anc_L", C.c_void_p)]


class TAError(RuntimeError):
    def __init__(self, status, what):
        self.status = status
        super().__init__(f"{what}: {status_string(status)} (ta_status {status})")


_lib = None


def lib():
    """Loads libta.so (built in-tree by paper_2604_11288_b200.build). Raises if it is not there."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise FileNotFoundError(f"{LIB_PATH} is missing: run `python -m paper_2604_11288_b200.build` (there is no "
                                    "fallback path)")
        L = C.CDLL(LIB_PATH)
        vp, i32, u64, sz = C.c_void_p, C.c_int, C.c_uint64, C.c_size_t
        PP, PB = C.POINTER(ta_policy), C.POINTER(ta_batch)
        sigs = {
            "ta_policy_default": (i32, [i32, i32, PP]),
            "ta_ctx_create": (i32, [i32, sz, C.POINTER(vp)]),
            "ta_ctx_destroy": (None, [vp]),
            "ta_scratch_bytes": (i32, [PB, i32, i32, i32, i32, PP, C.POINTER(sz)]),
            "ta_ctx_poll": (i32, [vp]),
            "ta_ctx_last_cuda_error": (i32, [vp]),
            "ta_status_string": (C.c_char_p, [i32]),
            "ta_ctx_enable_timing": (i32, [vp, i32]),
            "ta_ctx_read_timing": (i32, [vp, C.POINTER(C.c_float)]),
            "ta_patterns_create": (i32, [vp, i32, vp, vp, vp, vp, C.POINTER(vp)]),
            "ta_patterns_destroy": (None, [vp]),
            "ta_sponsor_mask": (i32, [vp, vp, PP, PB, vp, vp, vp, vp, vp]),
            "ta_detect_embedding": (i32, [vp, C.c_int64, vp, C.c_int64, i32, vp, i32, vp, vp]),
            "ta_sponsor_mask_conf": (i32, [vp, PP, PB, vp, vp, C.c_float, C.c_float, i32, i32, vp, vp, vp, vp]),
            "ta_score": (i32, [vp, PP, PB, i32, i32, i32, ta_bf16_view, ta_bf16_view, vp, vp, vp, vp]),
            "ta_score_weighted": (i32, [vp, PP, PB, i32, i32, i32, ta_bf16_view, ta_bf16_view, vp, vp, vp]),
            "ta_ctx_set_wait_limit": (i32, [vp, u64]),
            "ta_ctx_set_score_cluster": (i32, [vp, i32]),
            "ta_ctx_selftest_wait": (i32, [vp, u64, vp, vp]),
            "ta_ctx_last_launch_info": (i32, [vp, C.POINTER(C.c_int32)]),
            "ta_select_topk": (i32, [vp, PP, PB, i32, i32, vp, vp, vp, vp, vp, vp, vp, vp]),
            "ta_select_topk_static": (i32, [PP, PB, i32, i32, vp, vp, vp, vp, vp, vp, vp, vp]),
            "ta_compact_kv": (i32, [vp, PB, i32, i32, i32, ta_bf16_view, ta_bf16_view, vp, vp, vp, vp, vp]),
            "ta_compress": (i32, [vp, vp, PP, PB, i32, i32, i32, i32, vp, ta_bf16_view, ta_bf16_view, ta_bf16_view,
                                  u64, vp, vp, vp, vp, vp]),
            "ta_compress_lse": (i32, [vp, vp, PP, PB, i32, i32, i32, i32, vp, ta_bf16_view, ta_bf16_view, ta_bf16_view, vp,
                                      u64, vp, vp, vp, vp, vp]),
            "ta_compress_allheads": (i32, [vp, vp, PP, PB, i32, i32, i32, i32, vp, ta_bf16_view, ta_bf16_view,
                                           ta_bf16_view, u64, vp, vp, vp, vp, vp]),
            "ta_score_headsum": (i32, [vp, PP, PB, i32, i32, i32, ta_bf16_view, ta_bf16_view, vp, vp]),
            "ta_compress_from_headsum": (i32, [vp, vp, PP, PB, i32, i32, i32, vp, vp, ta_bf16_view, ta_bf16_view, u64,
                                               vp, vp, vp, vp, vp]),
            "ta_compress_scores": (i32, [vp, vp, PP, PB, i32, i32, i32, vp, vp, vp, ta_bf16_view, ta_bf16_view, u64, vp,
                                         vp, vp, vp, vp]),
            "ta_scratch_bytes_budgets": (i32, [PB, i32, i32, PP, i32, C.POINTER(sz)]),
            "ta_compress_scores_budgets": (i32, [vp, vp, PP, PB, i32, i32, i32, vp, vp, vp, vp, ta_bf16_view,
                                                 ta_bf16_view, vp, vp, vp, vp, vp]),
            "ta_compress_budgets": (i32, [vp, vp, PP, PB, i32, i32, i32, i32, vp, vp, ta_bf16_view, ta_bf16_view,
                                          ta_bf16_view, vp, vp, vp, vp, vp]),
            "ta_stream_scratch_bytes": (i32, [C.POINTER(ta_stream), C.POINTER(sz)]),
            "ta_stream_step": (i32, [vp, vp, PP, C.POINTER(ta_stream), vp, vp, vp, vp]),
            "ta_compress_host_workspace_bytes": (i32, [PB, i32, i32, i32, i32, PP, C.POINTER(sz)]),
            "ta_compress_host": (i32, [vp, vp, PP, PB, i32, i32, i32, i32, vp, vp, vp, vp, vp, vp, vp, vp, vp, sz, vp]),
        }
        for name, (res, args) in sigs.items():
            fn = getattr(L, name)
            fn.restype = res
            fn.argtypes = args
        _lib = L
    return _lib


def status_string(status: int) -> str:
    return lib().ta_status_string(int(status)).decode()


def _check(status, what):
    if status != TA_OK:
        raise TAError(status, what)


def _ptr(t):
    """Address of a torch tensor / numpy array / int / None."""
    if t is None:
        return None
    if isinstance(t, int):
        return t
    if hasattr(t, "data_ptr"):
        return t.data_ptr()
    return t.ctypes.data


def view(t, ragged=False) -> ta_bf16_view:
    """ta_bf16_view of a bf16 tensor [L, B, H, n, d] (uniform) or [L, H, total, d] (ragged); strides in elements."""
    if t is None:
        return ta_bf16_view(None, 0, 0, 0, 0)
    s = t.stride()
    assert s[-1] == 1, "head_dim must be contiguous"
    if ragged:
        assert t.dim() == 4
        return ta_bf16_view(t.data_ptr(), s[0], 0, s[1], s[2])
    assert t.dim() == 5
    return ta_bf16_view(t.data_ptr(), s[0], s[1], s[2], s[3])


def ta_policy_default(preset: int, K: int) -> ta_policy:
    p = ta_policy()
    _check(lib().ta_policy_default(preset, K, C.byref(p)), "ta_policy_default")
    return p


def make_batch(n_layers, batch, n_uniform, max_n, total_tokens, cu_seqlens=None) -> ta_batch:
    return ta_batch(n_layers, batch, n_uniform, max_n, total_tokens, _ptr(cu_seqlens))


def ta_scratch_bytes(batch: ta_batch, Hq, Hkv, d, K, policy: ta_policy) -> int:
    out = C.c_size_t(0)
    _check(lib().ta_scratch_bytes(C.byref(batch), Hq, Hkv, d, K, C.byref(policy), C.byref(out)), "ta_scratch_bytes")
    return out.value


def ta_ctx_create(device: int, scratch_bytes: int):
    h = C.c_void_p()
    _check(lib().ta_ctx_create(device, scratch_bytes, C.byref(h)), "ta_ctx_create")
    return h


def ta_ctx_destroy(ctx):
    lib().ta_ctx_destroy(ctx)


def ta_ctx_poll(ctx) -> int:
    return lib().ta_ctx_poll(ctx)


def ta_ctx_enable_timing(ctx, enable: bool):
    _check(lib().ta_ctx_enable_timing(ctx, 1 if enable else 0), "ta_ctx_enable_timing")


def ta_ctx_read_timing(ctx):
    out = (C.c_float * 5)()
    _check(lib().ta_ctx_read_timing(ctx, out), "ta_ctx_read_timing")
    return list(out)


def ta_patterns_create(ctx, pattern_ids, budget=None, span=None):
    """pattern_ids: list of lists of token ids (host). Returns an opaque handle."""
    n = len(pattern_ids)
    flat = [int(t) for p in pattern_ids for t in p]
    off = [0]
    for p in pattern_ids:
        off.append(off[-1] + len(p))
    a_flat = (C.c_int32 * max(1, len(flat)))(*flat)
    a_off = (C.c_int32 * (n + 1))(*off)
    a_b = (C.c_float * max(1, n))(*[float(x) for x in budget]) if budget is not None else None
    a_s = (C.c_int32 * max(1, n))(*[int(x) for x in span]) if span is not None else None
    h = C.c_void_p()
    _check(lib().ta_patterns_create(ctx, n, C.cast(a_flat, C.c_void_p), C.cast(a_off, C.c_void_p),
                                    C.cast(a_b, C.c_void_p) if a_b is not None else None,
                                    C.cast(a_s, C.c_void_p) if a_s is not None else None, C.byref(h)),
           "ta_patterns_create")
    return h


def ta_patterns_destroy(pats):
    lib().ta_patterns_destroy(pats)


def ta_detect_embedding(ctx, total_tokens, emb, stride_tok, D, concepts, n_concepts, conf, stream=None):
    _check(lib().ta_detect_embedding(ctx, int(total_tokens), _ptr(emb), int(stride_tok), int(D), _ptr(concepts),
                                     int(n_concepts), _ptr(conf), stream), "ta_detect_embedding")


def ta_sponsor_mask_conf(ctx, policy, batch, token_ids, conf, threshold, budget, span, rank_by_confidence, flags,
                         voucher, u_static, stream=None):
    _check(lib().ta_sponsor_mask_conf(ctx, C.byref(policy), C.byref(batch), _ptr(token_ids), _ptr(conf),
                                      C.c_float(threshold), C.c_float(budget), int(span), int(rank_by_confidence),
                                      _ptr(flags), _ptr(voucher), _ptr(u_static), stream), "ta_sponsor_mask_conf")


def ta_sponsor_mask(ctx, pats, policy, batch, token_ids, flags, voucher, u_static, stream=None):
    _check(lib().ta_sponsor_mask(ctx, pats, C.byref(policy), C.byref(batch), _ptr(token_ids), _ptr(flags),
                                 _ptr(voucher), _ptr(u_static), stream), "ta_sponsor_mask")


def ta_score(ctx, policy, batch, Hq, Hkv, d, q_obs: ta_bf16_view, k: ta_bf16_view, lse_obs, A, P, stream=None):
    _check(lib().ta_score(ctx, C.byref(policy), C.byref(batch), Hq, Hkv, d, q_obs, k, _ptr(lse_obs), _ptr(A), _ptr(P),
                          stream), "ta_score")


def ta_score_weighted(ctx, policy, batch, Hq, Hkv, d, q_obs: ta_bf16_view, k: ta_bf16_view, lse_obs, u_att, stream=None):
    _check(lib().ta_score_weighted(ctx, C.byref(policy), C.byref(batch), Hq, Hkv, d, q_obs, k, _ptr(lse_obs),
                                   _ptr(u_att), stream), "ta_score_weighted")


def ta_ctx_set_wait_limit(ctx, nanoseconds: int):
    _check(lib().ta_ctx_set_wait_limit(ctx, int(nanoseconds)), "ta_ctx_set_wait_limit")


def ta_compress_lse(ctx, pats, policy, batch, Hq, Hkv, d, K, token_ids, q_obs: ta_bf16_view, k: ta_bf16_view,
                    v: ta_bf16_view, lse_obs, seq_epoch, k_out, v_out, idx, count, stream=None):
    _check(lib().ta_compress_lse(ctx, pats, C.byref(policy), C.byref(batch), Hq, Hkv, d, K, _ptr(token_ids), q_obs, k, v,
                                 _ptr(lse_obs), seq_epoch, _ptr(k_out), _ptr(v_out), _ptr(idx), _ptr(count), stream),
           "ta_compress_lse")


def ta_score_headsum(ctx, policy, batch, Hq, Hkv, d, q_obs: ta_bf16_view, k: ta_bf16_view, u_heads, stream=None):
    _check(lib().ta_score_headsum(ctx, C.byref(policy), C.byref(batch), Hq, Hkv, d, q_obs, k, _ptr(u_heads), stream),
           "ta_score_headsum")


def ta_compress_from_headsum(ctx, pats, policy, batch, Hkv, d, K, token_ids, u_heads, k: ta_bf16_view,
                             v: ta_bf16_view, seq_epoch, k_out, v_out, idx, count, stream=None):
    _check(lib().ta_compress_from_headsum(ctx, pats, C.byref(policy), C.byref(batch), Hkv, d, K, _ptr(token_ids),
                                          _ptr(u_heads), k, v, seq_epoch, _ptr(k_out), _ptr(v_out), _ptr(idx),
                                          _ptr(count), stream), "ta_compress_from_headsum")


def ta_ctx_last_launch_info(ctx):
    """(CTAs per unit of the score kernel, its clusters, selection gathered the rows itself, kernels enqueued)."""
    out = (C.c_int32 * 4)()
    _check(lib().ta_ctx_last_launch_info(ctx, out), "ta_ctx_last_launch_info")
    return list(out)


def ta_ctx_selftest_wait(ctx, limit_ns: int, outcome, stream=None):
    _check(lib().ta_ctx_selftest_wait(ctx, int(limit_ns), _ptr(outcome), stream), "ta_ctx_selftest_wait")


def ta_ctx_set_score_cluster(ctx, ctas_per_unit: int):
    _check(lib().ta_ctx_set_score_cluster(ctx, int(ctas_per_unit)), "ta_ctx_set_score_cluster")


def ta_select_topk(ctx, policy, batch, Hkv, K, flags, voucher, u_static, A, P, idx, count, stream=None):
    _check(lib().ta_select_topk(ctx, C.byref(policy), C.byref(batch), Hkv, K, _ptr(flags), _ptr(voucher),
                                _ptr(u_static), _ptr(A), _ptr(P), _ptr(idx), _ptr(count), stream), "ta_select_topk")


def ta_select_topk_static(policy, batch, Hkv, K, flags, voucher, u_static, A, P, idx, count, stream=None):
    """ta_select_topk for callers that may not allocate device memory: no context, working memory in a fixed
    array inside the library (see include/ta.h for the size limit and the sharing rules)."""
    _check(lib().ta_select_topk_static(C.byref(policy), C.byref(batch), Hkv, K, _ptr(flags), _ptr(voucher),
                                       _ptr(u_static), _ptr(A), _ptr(P), _ptr(idx), _ptr(count), stream),
           "ta_select_topk_static")


def ta_compact_kv(ctx, batch, Hkv, d, K, k: ta_bf16_view, v: ta_bf16_view, idx, count, k_out, v_out, stream=None):
    _check(lib().ta_compact_kv(ctx, C.byref(batch), Hkv, d, K, k, v, _ptr(idx), _ptr(count), _ptr(k_out), _ptr(v_out),
                               stream), "ta_compact_kv")


def ta_compress(ctx, pats, policy, batch, Hq, Hkv, d, K, token_ids, q_obs: ta_bf16_view, k: ta_bf16_view,
                v: ta_bf16_view, seq_epoch, k_out, v_out, idx, count, stream=None):
    _check(lib().ta_compress(ctx, pats, C.byref(policy), C.byref(batch), Hq, Hkv, d, K, _ptr(token_ids), q_obs, k, v,
                             int(seq_epoch), _ptr(k_out), _ptr(v_out), _ptr(idx), _ptr(count), stream), "ta_compress")


def ta_compress_allheads(ctx, pats, policy, batch, Hq, Hkv, d, K, token_ids, q_obs: ta_bf16_view, k: ta_bf16_view,
                         v: ta_bf16_view, seq_epoch, k_out, v_out, idx, count, stream=None):
    _check(lib().ta_compress_allheads(ctx, pats, C.byref(policy), C.byref(batch), Hq, Hkv, d, K, _ptr(token_ids), q_obs,
                                      k, v, int(seq_epoch), _ptr(k_out), _ptr(v_out), _ptr(idx), _ptr(count), stream),
           "ta_compress_allheads")


def ta_compress_scores(ctx, pats, policy, batch, Hkv, d, K, token_ids, score, score2, k: ta_bf16_view,
                       v: ta_bf16_view, seq_epoch, k_out, v_out, idx, count, stream=None):
    _check(lib().ta_compress_scores(ctx, pats, C.byref(policy), C.byref(batch), Hkv, d, K, _ptr(token_ids),
                                    _ptr(score), _ptr(score2), k, v, int(seq_epoch), _ptr(k_out), _ptr(v_out),
                                    _ptr(idx), _ptr(count), stream), "ta_compress_scores")


def ta_scratch_bytes_budgets(batch: ta_batch, Hkv, K_max, policy: ta_policy, n_budget_classes) -> int:
    out = C.c_size_t(0)
    _check(lib().ta_scratch_bytes_budgets(C.byref(batch), Hkv, K_max, C.byref(policy), n_budget_classes, C.byref(out)),
           "ta_scratch_bytes_budgets")
    return out.value


def ta_compress_scores_budgets(ctx, pats, policy, batch, Hkv, d, K_max, budgets, token_ids, score, score2,
                               k: ta_bf16_view, v: ta_bf16_view, k_out, v_out, idx, count, stream=None):
    """budgets: host int32 array [n_layers][Hkv] (numpy or a CPU tensor)."""
    _check(lib().ta_compress_scores_budgets(ctx, pats, C.byref(policy), C.byref(batch), Hkv, d, K_max, _ptr(budgets),
                                            _ptr(token_ids), _ptr(score), _ptr(score2), k, v, _ptr(k_out), _ptr(v_out),
                                            _ptr(idx), _ptr(count), stream), "ta_compress_scores_budgets")


def ta_compress_budgets(ctx, pats, policy, batch, Hq, Hkv, d, K_max, budgets, token_ids, q_obs: ta_bf16_view,
                        k: ta_bf16_view, v: ta_bf16_view, k_out, v_out, idx, count, stream=None):
    """budgets: host int32 array [n_layers][Hkv] (numpy or a CPU tensor)."""
    _check(lib().ta_compress_budgets(ctx, pats, C.byref(policy), C.byref(batch), Hq, Hkv, d, K_max, _ptr(budgets),
                                     _ptr(token_ids), q_obs, k, v, _ptr(k_out), _ptr(v_out), _ptr(idx), _ptr(count),
                                     stream), "ta_compress_budgets")


def ta_stream_scratch_bytes(st: ta_stream) -> int:
    out = C.c_size_t(0)
    _check(lib().ta_stream_scratch_bytes(C.byref(st), C.byref(out)), "ta_stream_scratch_bytes")
    return out.value


def ta_stream_step(ctx, pats, policy, st: ta_stream, new_ids, attn, evicted_pos, stream=None):
    _check(lib().ta_stream_step(ctx, pats, C.byref(policy), C.byref(st), _ptr(new_ids), _ptr(attn), _ptr(evicted_pos),
                                stream), "ta_stream_step")


def ta_compress_host_workspace_bytes(batch, Hq, Hkv, d, K, policy) -> int:
    out = C.c_size_t(0)
    _check(lib().ta_compress_host_workspace_bytes(C.byref(batch), Hq, Hkv, d, K, C.byref(policy), C.byref(out)),
           "ta_compress_host_workspace_bytes")
    return out.value


def ta_compress_host(ctx, pats, policy, batch, Hq, Hkv, d, K, token_ids, q_obs, k, v, k_out, v_out, idx, count,
                     workspace, workspace_bytes, stream=None):
    _check(lib().ta_compress_host(ctx, pats, C.byref(policy), C.byref(batch), Hq, Hkv, d, K, _ptr(token_ids),
                                  _ptr(q_obs), _ptr(k), _ptr(v), _ptr(k_out), _ptr(v_out), _ptr(idx), _ptr(count),
                                  _ptr(workspace), workspace_bytes, stream), "ta_compress_host")
