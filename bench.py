#!/usr/bin/env python
"""Benchmark of the Transactional Attention KV-cache compaction path on B200.

One step = one pass of the whole path (anchor mask, vouchers, attention-free utility, attention scores, budget-K
selection, K/V gather) over one batch of seeded synthetic input, through the library's C ABI: a single ta_compress
call covering all layers of the workload. The metric is context tokens compressed per second per layer, i.e.
(tokens in the batch) / (step time / layers). Prints ONE JSON line on rank 0.

The default workload is the largest configuration that fits one GPU at its full layer count: 32 layers x 16 sequences
x 32768 tokens, observation window 64, K = 2048, scored (69 GB of keys and values). The step time is the median of
--rounds timed regions of --steps calls each; the other configurations (single layer, the 4096-token budget sweep in
both modes, the attention-free 131072-token case, the ragged batch) are reported beside it at their full layer
counts, each with one unit checked against the CPU oracle.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--rounds R] [--workload c3] [--budget K] [--mode scored|fast]
  python bench.py --impl reference   # times the CPU oracle (the only baseline there is) on a bounded sample
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402
import torch  # noqa: E402

import ta_workloads as tw  # noqa: E402

METRIC = "context tokens compressed/sec per layer (all heads)"
UNIT = "tokens/s"


# ------------------------------------------------------------------------------------------------ helpers
def measured_peak_hbm():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        try:
            return float(json.load(open(p))["hbm_gbs"]), "measured"
        except Exception:
            pass
    return 6650.0, "fallback"


class ClockSampler:
    """Samples SM clock and throttle reasons with nvidia-smi while the timed region runs (read-only queries)."""
    Q = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index, self.proc, self.lines = index, None, []

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "20"], stdout=subprocess.PIPE,
                                         stderr=subprocess.DEVNULL, text=True)
            self.t = threading.Thread(target=self._read, daemon=True)
            self.t.start()
        except Exception:
            self.proc = None
        t0 = time.time()
        while self.proc and not self.lines and time.time() - t0 < 3.0:  # first sample before the timed region
            time.sleep(0.01)

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append((time.time(), line.strip()))

    def stop(self, t_lo=None, t_hi=None, note="timed region"):
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["unavailable"]}
        t0, have = time.time(), len(self.lines)
        while len(self.lines) < have + 2 and time.time() - t0 < 0.5:  # the region may be shorter than one interval
            time.sleep(0.01)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            pass
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for (ts, ln) in self.lines:
            if t_lo is not None and not (t_lo <= ts <= t_hi + 0.06):
                continue
            f = [x.strip() for x in ln.split(",")]
            if len(f) < 6:
                continue
            try:
                sm.append(float(f[0]))
                mx.append(float(f[1]))
            except ValueError:
                continue
            for nm, v in zip(names, f[2:6]):
                if v.lower().startswith("active"):
                    reasons.add(nm)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm), "window": note}


def recorded_traffic(workload, layers):
    """DRAM bytes per launch of the score kernel from the committed ncu capture, or None when the kernel source has
    changed since (the counters then no longer describe it) or the capture was for another workload. The capture is
    taken at a few layers per call (an ncu capture must stay small); the kernel's traffic is proportional to the
    layers it processes, so the per-layer figure is scaled to the launch timed here."""
    import hashlib
    try:
        rec = json.load(open(os.path.join(ROOT, "profiles", "score_kernel_traffic.json")))
        src = open(os.path.join(ROOT, "paper_2604_11288_b200", "csrc", "ta_score.cu"), "rb").read()
        if hashlib.sha256(src).hexdigest()[:16] != rec["source_sha256_16"]:
            return None
        if rec["workload"] != workload:
            return None
        return rec["dram_bytes_per_launch"] / rec["layers_per_call"] * layers
    except Exception:
        return None


def build_workload(name, budget):
    w = tw.CONFIGS[name]()
    K = budget if budget else w.K_list[0]
    return w, K


def algorithmic_bytes(w, L, K, fast):
    """Bytes the method itself must move for one step of L layers (what a perfect implementation reads + writes)."""
    total, B = w.total, w.B
    k_eff = int(sum(min(K, int(n)) for n in w.lengths))
    score = 0 if fast else L * (total * w.Hkv * w.d * 2 + B * w.Hq * w.W * w.d * 2)
    gather = L * 2 * 2 * w.Hkv * k_eff * w.d * 2          # K and V rows, read + write
    idx = L * w.Hkv * k_eff * 4
    per_seq = total * (4 + 1 + 4 + 4)                     # ids, flags, voucher, static utility: once per batch
    return {"score": score, "gather": gather + idx, "per_sequence": per_seq, "total": score + gather + idx + per_seq}


def score_kernel_bytes(w, L):
    """Algorithmic bytes of one launch of the scoring kernel: every key row once, the query window once, one fused
    fp32 utility written and one static utility read per (token, KV head)."""
    return L * (w.total * w.Hkv * (w.d * 2 + 4 + 4) + w.B * w.Hq * w.W * w.d * 2)


# ------------------------------------------------------------------------------------------------ CPU oracle legs
def oracle_leg(w, K, fast, budget_s=12.0, max_layers=512):
    """Times the CPU oracle (as it stands) on whole layers of the workload until about `budget_s` seconds are
    spent. Inputs are drawn on the CPU from the same generator family."""
    import oracle
    pats = oracle.Patterns(w.pattern_ids, w.pattern_budget, w.pattern_span)
    pol = oracle.preset("THEOREM", K, fast=1 if fast else 0, obs_window=w.W)
    sub, note = w, "all sequences"
    macs = float(w.total) * w.Hq * w.W * w.d  # multiply-adds of one layer's score matrix
    if macs > 2e10 and not fast:
        # a layer of this workload is minutes of CPU work: time a subset of sequences instead
        keep = max(1, int(w.B * 2e10 / macs))
        sub = subset_sequences(w, keep)
        note = f"first {keep} of {w.B} sequences"
    bits = lambda t: t.contiguous().view(torch.int16).numpy().view(np.uint16)
    layers, spent, t_units = 0, 0.0, 0.0
    while layers < max_layers and spent < budget_s:
        Q, Kc, Vc = tw.make_qkv(sub, [layers % w.n_layers], need_q=not fast)
        t0 = time.perf_counter()
        oracle.compress_layer(sub.ids, sub.cu, sub.uniform, sub.Hq, sub.Hkv, sub.d, K, pats, pol,
                              None if fast else bits(Q[0]), bits(Kc[0]), bits(Vc[0]))
        dt = time.perf_counter() - t0
        spent += dt
        layers += 1
    value = sub.total * layers / spent
    return {"value": value, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
            "sample": f"{layers} layer(s) of {w.name}, {note}, {spent:.1f} s"}, spent / layers


def subset_sequences(w, keep):
    import copy
    s = copy.copy(w)
    s.lengths = w.lengths[:keep].copy()
    s.cu = w.cu[:keep + 1].copy()
    s.ids = w.ids[:int(s.cu[-1])].copy()
    return s


# ------------------------------------------------------------------------------------------------ GPU leg
class Inputs:
    """Device copies of one workload at L layers per call; shared by runs with different budgets and modes."""

    def __init__(self, w, L, dev, need_q=True):
        import paper_2604_11288_b200 as ta
        self.w, self.L, self.dev = w, L, dev
        self.ids = torch.from_numpy(w.ids).to(dev)
        self.cu = None if w.uniform else torch.from_numpy(w.cu).to(dev)
        self.Q, self.Kc, self.Vc = tw.make_qkv(w, range(L), device=dev, need_q=need_q)
        self.rag = not w.uniform
        self.vq = ta.view(self.Q) if need_q else ta.view(None)
        self.vk, self.vv = ta.view(self.Kc, self.rag), ta.view(self.Vc, self.rag)


class Runner:
    score_cluster = 0  # --score-cluster: CTAs per unit in the score kernel (0: the library chooses)

    def __init__(self, inp, K, fast):
        import paper_2604_11288_b200 as ta
        w, L, dev = inp.w, inp.L, inp.dev
        self.ta, self.inp, self.w, self.K, self.L, self.fast, self.dev = ta, inp, w, K, L, fast, dev
        p = ta.ta_policy_default(ta.TA_PRESET_THEOREM, K)
        p.obs_window = w.W
        p.mode = ta.TA_MODE_FAST if fast else ta.TA_MODE_SCORED
        p.vocab_size = w.vocab
        self.p = p
        self.batch = ta.make_batch(L, w.B, int(w.lengths[0]) if w.uniform else 0, w.max_n, w.total, inp.cu)
        self.ctx = ta.ta_ctx_create(dev.index, ta.ta_scratch_bytes(self.batch, w.Hq, w.Hkv, w.d, K, p))
        self.pats = ta.ta_patterns_create(self.ctx, w.pattern_ids, w.pattern_budget, w.pattern_span)
        if Runner.score_cluster:
            ta.ta_ctx_set_score_cluster(self.ctx, Runner.score_cluster)
        self.idx = torch.empty((L, w.B, w.Hkv, K), dtype=torch.int32, device=dev)
        self.cnt = torch.empty((L, w.B, w.Hkv), dtype=torch.int32, device=dev)
        self.ko = torch.empty((L, w.B, w.Hkv, K, w.d), dtype=torch.bfloat16, device=dev)
        self.vo = torch.empty_like(self.ko)
        self.stream = torch.cuda.current_stream(dev).cuda_stream
        self.vq = inp.vq if not fast else ta.view(None)

    def step(self):
        w, i = self.w, self.inp
        self.ta.ta_compress(self.ctx, self.pats, self.p, self.batch, w.Hq, w.Hkv, w.d, self.K, i.ids, self.vq, i.vk,
                            i.vv, 0, self.ko, self.vo, self.idx, self.cnt, self.stream)

    def launch_info(self):
        cl, clusters, gathered, launches = self.ta.ta_ctx_last_launch_info(self.ctx)
        return {"score_ctas_per_unit": cl, "score_clusters": clusters, "gather_fused_into_select": bool(gathered),
                "kernels_per_step": launches}

    def close(self):
        self.ta.ta_patterns_destroy(self.pats)
        self.ta.ta_ctx_destroy(self.ctx)


def time_rounds(run, steps, warmup, rounds, barrier=None):
    """`rounds` timed regions of `steps` calls each (CUDA events on the launching stream, synchronised on both
    sides); returns the per-step milliseconds of every round."""
    for _ in range(warmup):
        run()
    out = []
    for _ in range(rounds):
        torch.cuda.synchronize()
        if barrier:
            barrier()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(steps):
            run()
        e1.record()
        torch.cuda.synchronize()
        if barrier:
            barrier()
        out.append(e0.elapsed_time(e1) / steps)
    return out


def kernel_breakdown(r, steps):
    """Per-stage device times of ta_compress from CUDA events recorded on the call's stream inside the library."""
    ta = r.ta
    ta.ta_ctx_enable_timing(r.ctx, True)
    acc = np.zeros(5)
    for _ in range(steps):
        r.step()
        acc += np.array(ta.ta_ctx_read_timing(r.ctx))
    ta.ta_ctx_enable_timing(r.ctx, False)
    return acc / steps


def selection_agrees(idx_gpu, cnt_gpu, idx_ora, cnt_ora, u_ora):
    """The rule of the parity tests: identical, except for swaps between tokens whose oracle utilities lie within
    the score tolerance (1e-3 relative, 1e-5 absolute) of the budget boundary."""
    c = int(cnt_ora)
    if int(cnt_gpu) != c or not (idx_gpu[c:] == -1).all():
        return False
    g, o = idx_gpu[:c], idx_ora[:c]
    if (g == o).all():
        return True
    if not (np.diff(g) > 0).all():
        return False
    only_o, only_g = np.setdiff1d(o, g), np.setdiff1d(g, o)
    if only_o.size != only_g.size:
        return False
    tau = float(u_ora[only_o].min())
    eps = 1e-5 + 1e-3 * abs(tau)
    return float(u_ora[only_o].max() - u_ora[only_g].min()) <= 2 * eps


def oracle_check(r):
    """Part of the CPU-oracle leg: recomputes ONE sampled unit (layer, sequence, KV head) of the workload on the host
    from the same bytes and compares the GPU's retained indices and compacted rows with it (outside any timed
    region). Returns (agrees, description)."""
    import oracle
    w, inp, K = r.w, r.inp, r.K
    l, b, g = r.L // 2, w.B - 1, w.Hkv // 2
    r.step()
    torch.cuda.synchronize()
    bits = lambda t: t.contiguous().cpu().view(torch.int16).numpy().view(np.uint16)
    pats = oracle.Patterns(w.pattern_ids, w.pattern_budget, w.pattern_span)
    pol = oracle.preset("THEOREM", K, fast=1 if r.fast else 0, obs_window=w.W)
    flags, V, u0 = oracle.sponsor_mask(w.ids, w.cu, pats, pol)
    o, e = int(w.cu[b]), int(w.cu[b + 1])
    n, G = e - o, w.Hq // w.Hkv
    k_unit = bits(inp.Kc[l, b, g] if w.uniform else inp.Kc[l, g, o:e])
    v_unit = bits(inp.Vc[l, b, g] if w.uniform else inp.Vc[l, g, o:e])
    if r.fast:
        u = u0[o:e].copy()
    else:
        A, P = oracle.attention(bits(inp.Q[l, b, g * G:(g + 1) * G]), k_unit, n, scale=pol.softmax_scale,
                                causal=pol.causal, rho=pol.pension_rho)
        u = oracle.utility(pol.alpha, pol.delta, A, P, u0[o:e])
    io, co = oracle.select(V[o:e], u, K, pol.n_sink, pol.n_recent, pol.k_protected)
    ig, cg = r.idx[l, b, g].cpu().numpy(), int(r.cnt[l, b, g].item())
    ok = selection_agrees(ig, cg, io, co, u)
    if ok:  # the compacted rows must be the rows the GPU's own indices name, bit for bit
        ok = bool((bits(r.ko[l, b, g]) == oracle.compact(k_unit, ig, cg, K)).all() and
                  (bits(r.vo[l, b, g]) == oracle.compact(v_unit, ig, cg, K)).all())
    return ok, f"unit (layer {l}, sequence {b}, KV head {g}), n={n}"


def host_memory_budget():
    """Bytes of pinned host memory the end-to-end leg may take: a quarter of what is available, at most 16 GB."""
    try:
        for line in open("/proc/meminfo"):
            if line.startswith("MemAvailable:"):
                return min(int(line.split()[1]) * 1024 // 4, 16 << 30)
    except Exception:
        pass
    return 4 << 30


def e2e_leg(w, K, fast, L, dev, steps, warmup):
    """The same metric through ta_compress_host: inputs start in pinned host memory, results end there. Uses as many
    layers per call as the host-memory budget allows (the metric is per layer)."""
    import paper_2604_11288_b200 as ta
    per_layer = 2 * w.Hkv * w.total * w.d * 2 + w.B * w.Hq * w.W * w.d * 2 + 2 * w.B * w.Hkv * K * w.d * 2
    Le = int(max(1, min(L, host_memory_budget() // per_layer)))
    inp = Inputs(w, Le, dev, need_q=not fast)
    r = Runner(inp, K, fast)
    try:
        r.step()
        torch.cuda.synchronize()
        pin = lambda t: torch.empty(t.shape, dtype=t.dtype, pin_memory=True).copy_(t)
        ids_h = torch.from_numpy(w.ids).pin_memory()
        q_h = pin(inp.Q) if not fast else None
        k_h, v_h = pin(inp.Kc), pin(inp.Vc)
        ko_h = torch.empty(r.ko.shape, dtype=torch.bfloat16).pin_memory()
        vo_h = torch.empty(r.vo.shape, dtype=torch.bfloat16).pin_memory()
        idx_h = torch.empty(r.idx.shape, dtype=torch.int32).pin_memory()
        cnt_h = torch.empty(r.cnt.shape, dtype=torch.int32).pin_memory()
        hb = ta.make_batch(Le, w.B, int(w.lengths[0]) if w.uniform else 0, w.max_n, w.total,
                           None if w.uniform else w.cu.ctypes.data)
        nbytes = ta.ta_compress_host_workspace_bytes(hb, w.Hq, w.Hkv, w.d, K, r.p)
        ws = torch.empty(nbytes + 256, dtype=torch.uint8, device=dev)
        ws_ptr = (ws.data_ptr() + 255) // 256 * 256

        def run():
            ta.ta_compress_host(r.ctx, r.pats, r.p, hb, w.Hq, w.Hkv, w.d, K, ids_h, q_h, k_h, v_h, ko_h, vo_h, idx_h,
                                cnt_h, ws_ptr, nbytes, r.stream)

        ms = float(np.median(time_rounds(run, steps, warmup, 3)))
        # V is pinned: only its retained rows cross the bus (read in place by the gather kernel); same for K in fast mode
        k_eff = int(sum(min(K, int(x)) for x in w.lengths)) * Le * w.Hkv
        row = w.d * 2
        h2d = ids_h.numel() * 4 + (q_h.numel() * 2 if q_h is not None else 0)
        h2d += (k_eff * row if fast else k_h.numel() * 2) + k_eff * row
        d2h = ko_h.numel() * 2 + vo_h.numel() * 2 + idx_h.numel() * 4 + cnt_h.numel() * 4
        same = bool((idx_h.to(dev) == r.idx).all()) and bool((ko_h.to(dev) == r.ko).all())
        return {"value": w.total * Le / (ms * 1e-3), "unit": UNIT, "h2d_bytes_per_step": h2d,
                "d2h_bytes_per_step": d2h, "ms_per_step": ms, "layers_per_call": Le,
                "matches_device_path": same}
    finally:
        r.close()
        del inp
        torch.cuda.empty_cache()


def measure(r, steps, warmup, rounds, barrier=None):
    """Times one runner: median / min / max over the rounds, per-stage times, roofline fractions."""
    w, L, K, fast = r.w, r.L, r.K, r.fast
    per_round = time_rounds(r.step, steps, warmup, rounds, barrier)
    ms = float(np.median(per_round))
    br = kernel_breakdown(r, max(3, min(steps, 10)))
    ab = algorithmic_bytes(w, L, K, fast)
    peak, how = measured_peak_hbm()
    out = {"workload": w.name, "layers_per_call": L, "K": K, "mode": "fast" if fast else "scored",
           "value": w.total * L / (ms * 1e-3), "unit": UNIT, "ms_per_step": ms,
           "ms_per_step_min": float(min(per_round)), "ms_per_step_max": float(max(per_round)), "rounds": rounds,
           "steps_per_round": steps,
           "stage_ms": {"mask": br[0], "score": br[1], "select": br[2], "compact": br[3]},
           "step_algorithmic_bytes": ab["total"], "step_hbm_frac": ab["total"] / (ms * 1e-3) / 1e9 / peak}
    out.update(r.launch_info())
    if not fast and br[1] > 0:
        out["score_hbm_frac"] = score_kernel_bytes(w, L) / (br[1] * 1e-3) / 1e9 / peak
        out["score_tflops"] = 2.0 * (w.Hq // w.Hkv) * w.W * w.d * w.total * w.Hkv * L / (br[1] * 1e-3) / 1e12
    if br[3] > 0 and not out["gather_fused_into_select"]:
        out["compact_hbm_frac"] = ab["gather"] / (br[3] * 1e-3) / 1e9 / peak
    return out, per_round


def measure_others(main_name, dev, steps, warmup):
    """The other configurations at their full layer counts (supplementary; never in place of the main line), each
    with one unit checked against the CPU oracle."""
    out = []
    plan = [("c1", None), ("c2", None), ("c3", None), ("c4", None), ("c5", None)]
    for name, _ in plan:
        if name == main_name:
            continue
        try:
            w = tw.CONFIGS[name]()
            L = w.n_layers
            only_fast = w.modes == ["fast"]
            inp = Inputs(w, L, dev, need_q=not only_fast)
            try:
                for mode in w.modes:
                    fast = mode == "fast"
                    for K in w.K_list:
                        r = Runner(inp, K, fast)
                        try:
                            m, _ = measure(r, steps, warmup, 3)
                            ok, what = oracle_check(r)
                            m["matches_oracle"] = ok
                            m["oracle_sample"] = what
                            if r.ta.ta_ctx_poll(r.ctx) != 0:
                                m["error"] = "device status"
                            out.append(m)
                        finally:
                            r.close()
            finally:
                del inp
                torch.cuda.empty_cache()
        except Exception as ex:  # supplementary only: never lose the main line
            out.append({"workload": name, "error": str(ex)[:200]})
    return out


def window_lse(inp, w, L):
    """Natural-log softmax normalisers [L][B][Hq][W] of the observation-window rows of a uniform batch, by torch on the
    device (what a prefill attention kernel would have left behind; input preparation, never timed)."""
    G, n, W = w.Hq // w.Hkv, int(w.lengths[0]), w.W
    lse = torch.empty((L, w.B, w.Hq, W), dtype=torch.float32, device=inp.dev)
    pos = torch.arange(n - W, n, device=inp.dev).view(1, -1, 1)
    key = torch.arange(n, device=inp.dev).view(1, 1, -1)
    for l in range(L):
        for b in range(w.B):
            k = inp.Kc[l, b].float().repeat_interleave(G, dim=0)           # [Hq, n, d]
            s = torch.bmm(inp.Q[l, b].float(), k.transpose(1, 2)) / float(np.sqrt(w.d))  # [Hq, W, n]
            s = s.masked_fill(key > pos, float("-inf"))
            lse[l, b] = torch.logsumexp(s, dim=-1)
    return lse


def measure_variants(dev, steps=10, warmup=3):
    """Timings of the entry points beyond the one-shot ta_compress, on synthetic inputs of the main workload's shape:
    selection shared by the heads of a layer, a caller-supplied score, detector-confidence anchors, and the per-step
    retention of the decode loop. Supplementary: reported next to the main line, never in place of it."""
    import paper_2604_11288_b200 as ta
    out = []
    peak, _ = measured_peak_hbm()
    w, K = build_workload("c2", 0)
    L = w.n_layers
    inp = Inputs(w, L, dev)
    r = Runner(inp, K, False)
    try:
        def allheads():
            ta.ta_compress_allheads(r.ctx, r.pats, r.p, r.batch, w.Hq, w.Hkv, w.d, K, inp.ids, r.vq, inp.vk, inp.vv, 0, r.ko,
                                    r.vo, r.idx, r.cnt, r.stream)
        ms = float(np.median(time_rounds(allheads, steps, warmup, 3)))
        out.append({"entry": "ta_compress_allheads", "workload": f"c2, {L} layers, K={K}", "ms_per_step": ms,
                    "value": w.total * L / (ms * 1e-3), "unit": UNIT})
        # the same step when the caller's prefill kernel has left the softmax normalisers of the window rows: one pass
        # over the keys. The normalisers are prepared here with torch (a stand-in for that kernel), outside the timing.
        lse = window_lse(inp, w, L)

        def with_lse():
            ta.ta_compress_lse(r.ctx, r.pats, r.p, r.batch, w.Hq, w.Hkv, w.d, K, inp.ids, r.vq, inp.vk, inp.vv, lse, 0,
                               r.ko, r.vo, r.idx, r.cnt, r.stream)
        ms = float(np.median(time_rounds(with_lse, steps, warmup, 3)))
        out.append({"entry": "ta_compress_lse", "workload": f"c2, {L} layers, K={K}, normalisers supplied",
                    "ms_per_step": ms, "value": w.total * L / (ms * 1e-3), "unit": UNIT})
        score = torch.rand((L, w.Hkv, w.total), dtype=torch.float32, device=dev)

        def scores():
            ta.ta_compress_scores(r.ctx, r.pats, r.p, r.batch, w.Hkv, w.d, K, inp.ids, score, None, inp.vk, inp.vv, 0, r.ko,
                                  r.vo, r.idx, r.cnt, r.stream)
        ms = float(np.median(time_rounds(scores, steps, warmup, 3)))
        out.append({"entry": "ta_compress_scores", "workload": f"c2, {L} layers, K={K}, scores resident",
                    "ms_per_step": ms, "value": w.total * L / (ms * 1e-3), "unit": UNIT})
    finally:
        r.close()
    # budgets per layer (a pyramid from 64 down to 16 tokens in 8 levels) on the same scores
    Kmax = 64
    rb = Runner(inp, Kmax, False)
    try:
        levels = np.linspace(64, 16, 8).round().astype(np.int32)
        budgets = np.repeat(levels[(np.arange(L) * 8) // L][:, None], w.Hkv, axis=1).astype(np.int32).copy()
        ctxb = ta.ta_ctx_create(dev.index, ta.ta_scratch_bytes_budgets(rb.batch, w.Hkv, Kmax, rb.p, 8))
        patsb = ta.ta_patterns_create(ctxb, w.pattern_ids, w.pattern_budget, w.pattern_span)
        score = torch.rand((L, w.Hkv, w.total), dtype=torch.float32, device=dev)

        def budgeted():
            ta.ta_compress_scores_budgets(ctxb, patsb, rb.p, rb.batch, w.Hkv, w.d, Kmax, budgets, inp.ids, score, None,
                                          inp.vk, inp.vv, rb.ko, rb.vo, rb.idx, rb.cnt, rb.stream)
        ms = float(np.median(time_rounds(budgeted, steps, warmup, 3)))
        out.append({"entry": "ta_compress_scores_budgets",
                    "workload": f"c2, {L} layers, budgets 64..16 by layer (8 levels), scores resident",
                    "ms_per_step": ms, "value": w.total * L / (ms * 1e-3), "unit": UNIT})
        ta.ta_patterns_destroy(patsb)
        ta.ta_ctx_destroy(ctxb)
    finally:
        rb.close()
    # detector-confidence anchors on the token stream of c4 (4 x 131072 tokens)
    w4, K4 = build_workload("c4", 0)
    inp4 = Inputs(w4, 1, dev, need_q=False)
    r4 = Runner(inp4, K4, True)
    try:
        conf = torch.rand(w4.total, dtype=torch.float32, device=dev) * 0.4
        conf[torch.randint(0, w4.total, (2048,), device=dev)] = 0.95
        flags = torch.empty(w4.total, dtype=torch.uint8, device=dev)
        V = torch.empty(w4.total, dtype=torch.float32, device=dev)
        u0 = torch.empty_like(V)

        def mask_conf():
            ta.ta_sponsor_mask_conf(r4.ctx, r4.p, r4.batch, inp4.ids, conf, 0.5, 15.0, 6, 0, flags, V, u0, r4.stream)
        ms = float(np.median(time_rounds(mask_conf, steps, warmup, 3)))
        bytes_ = w4.total * (4 + 4 + 1 + 4 + 4)  # ids, conf read; flags, voucher, static utility written
        out.append({"entry": "ta_sponsor_mask_conf", "workload": f"c4 token stream, {w4.total} tokens",
                    "ms_per_step": ms, "GBps": bytes_ / (ms * 1e-3) / 1e9, "hbm_frac": bytes_ / (ms * 1e-3) / 1e9 / peak,
                    "value": w4.total / (ms * 1e-3), "unit": "tokens/s"})
        # embedding detector on the same token stream: 2048-wide input embeddings, 8 anchor concepts
        D = 2048
        emb = torch.randn((w4.total, D), dtype=torch.float32, device=dev).to(torch.bfloat16)
        concepts = torch.randn((8, D), dtype=torch.float32, device=dev).to(torch.bfloat16)

        def detect():
            ta.ta_detect_embedding(r4.ctx, w4.total, emb, D, D, concepts, 8, conf, r4.stream)
        ms = float(np.median(time_rounds(detect, steps, warmup, 3)))
        bytes_ = w4.total * (D * 2 + 4)
        out.append({"entry": "ta_detect_embedding", "workload": f"{w4.total} tokens x {D} bf16, 8 concepts",
                    "ms_per_step": ms, "GBps": bytes_ / (ms * 1e-3) / 1e9, "hbm_frac": bytes_ / (ms * 1e-3) / 1e9 / peak,
                    "value": w4.total / (ms * 1e-3), "unit": "tokens/s"})
        del emb
    finally:
        r4.close()
    # decode loop: 32 layers x 16 sequences x 8 KV heads, K = 256 cached tokens per unit
    Ls, Bs, Hs, Ks, vocab = 32, 16, 8, 256, 32000
    U, C_ = Ls * Bs * Hs, Ks + 1
    z = lambda shape, dt: torch.zeros(shape, dtype=dt, device=dev)
    t = dict(pos=z((U, C_), torch.int32), slot=z((U, C_), torch.int32), tok=z((U, C_), torch.int32),
             A=z((U, C_), torch.float32), P=z((U, C_), torch.float32), V=z((U, C_), torch.float32),
             S=z((U, C_), torch.uint8), next_slot=z((U,), torch.int32), n_seen=z((Bs,), torch.int32),
             hist=z((Bs, vocab), torch.int32), tok_ring=z((Bs, 8), torch.int32), anc_B=z((Bs, 64), torch.float32),
             anc_L=z((Bs, 64), torch.int32))
    st = ta.ta_stream()
    st.n_layers, st.batch, st.Hkv, st.K, st.cache_len = Ls, Bs, Hs, Ks, 0
    for k, v in t.items():
        setattr(st, k, v.data_ptr())
    p = ta.ta_policy_default(ta.TA_PRESET_THEOREM, Ks)
    p.vocab_size = vocab
    ctx = ta.ta_ctx_create(dev.index, ta.ta_stream_scratch_bytes(st))
    pats = ta.ta_patterns_create(ctx, w.pattern_ids, w.pattern_budget, w.pattern_span)
    try:
        attn = torch.rand((U, C_), dtype=torch.float32, device=dev)
        ev = torch.empty((U,), dtype=torch.int32, device=dev)
        ids = torch.randint(0, vocab, (Ks + 64, Bs), dtype=torch.int32, device=dev)
        stream = torch.cuda.current_stream(dev).cuda_stream
        for i in range(Ks + 8):  # fill the caches, then a few evicting steps as warm-up
            ta.ta_stream_step(ctx, pats, p, st, ids[i], attn, ev, stream)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        n_timed = 40
        e0.record()
        for i in range(n_timed):
            ta.ta_stream_step(ctx, pats, p, st, ids[Ks + 8 + i], attn, ev, stream)
        e1.record()
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1) / n_timed
        state_bytes = U * C_ * (3 * 4 + 3 * 4 + 1) * 2 + U * C_ * 4  # ordered state read + written, attention read
        out.append({"entry": "ta_stream_step", "workload": f"{Ls} layers x {Bs} sequences x {Hs} KV heads, K={Ks}, "
                    "steady state (one eviction per unit and step)", "ms_per_step": ms, "kernels_per_step": 2,
                    "unit_steps_per_s": U / (ms * 1e-3), "state_GBps": state_bytes / (ms * 1e-3) / 1e9})
        if ta.ta_ctx_poll(ctx) != 0:
            out[-1]["error"] = "device status"
    finally:
        ta.ta_patterns_destroy(pats)
        ta.ta_ctx_destroy(ctx)
    torch.cuda.empty_cache()
    return out


# ------------------------------------------------------------------------------------------------ main
def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--rounds", type=int, default=5, help="timed regions of --steps calls; the median is reported")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="c3", choices=sorted(tw.CONFIGS))
    ap.add_argument("--budget", type=int, default=0, help="K (default: the workload's first budget)")
    ap.add_argument("--mode", default="", choices=["", "scored", "fast"])
    ap.add_argument("--layers", type=int, default=0, help="layers per call (default: the workload's layer count)")
    ap.add_argument("--no-extra", action="store_true", help="skip the other workloads and entry points")
    ap.add_argument("--no-other", action="store_true", help="skip the other workloads, keep the entry points")
    ap.add_argument("--score-cluster", type=int, default=0, help="tuning: CTAs per unit in the score kernel")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu", action="store_true")
    a = ap.parse_args()

    Runner.score_cluster = a.score_cluster
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    warmup = max(a.warmup, 3)
    rounds = max(a.rounds, 1)
    w, K = build_workload(a.workload, a.budget)
    fast = (a.mode or w.modes[0]) == "fast"
    L = a.layers or w.n_layers
    config = {"workload": f"{w.name}: {L} layers x {w.B} seq, n={'ragged ' if not w.uniform else ''}{w.max_n}, "
                          f"Hq={w.Hq} Hkv={w.Hkv} d={w.d}, W={w.W}, K={K}, {'TA-Fast' if fast else 'scored TA'}",
              "layers_per_call": L, "budget_K": K, "mode": "fast" if fast else "scored", "preset": "THEOREM",
              "l2": "inputs larger than L2 (every step streams all layers' keys)", "parallelism": f"replicas x{world}"}

    if a.impl == "reference":
        if rank != 0:
            return
        base, per_layer_s = oracle_leg(w, K, fast, budget_s=min(60.0, 4.0 * max(1, a.steps + warmup)))
        line = {"impl": "reference", "metric": METRIC, "value": base["value"], "unit": UNIT, "n_gpus": a.gpus,
                "steps": a.steps, "warmup": warmup, "ms_per_step": w.total * L / base["value"] * 1e3, "higher_is_better": True,
                "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic", "config": config,
                "cpu_baseline": base,
                "e2e": {"value": base["value"], "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
        print(json.dumps(line))
        return

    # the CPU leg runs before the first CUDA call of this process
    cpu = None
    if rank == 0 and world == 1 and not a.no_cpu:
        cpu, _ = oracle_leg(w, K, fast)

    dev = torch.device("cuda", local)
    torch.cuda.set_device(dev)
    barrier = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)
        barrier = dist.barrier
        w.seed += 7919 * rank  # every rank compacts its own batch (weak scaling, no exchange)

    inp = Inputs(w, L, dev, need_q=not fast)
    r = Runner(inp, K, fast)
    sampler = ClockSampler(local)
    sampler.start()
    t_lo = time.time()
    m, per_round = measure(r, a.steps, warmup, rounds, barrier)
    t_hi = time.time()
    note = "timed regions"
    if sum(1 for (ts, _) in sampler.lines if t_lo <= ts <= t_hi + 0.06) < 3:
        # the timed regions are shorter than a few sampling intervals: keep the same loop running, untimed, and
        # sample the clocks under that load
        note = "untimed continuation of the same loop (timed regions shorter than the sampling interval)"
        t_lo = time.time()
        while time.time() - t_lo < 0.5:
            for _ in range(20):
                r.step()
            torch.cuda.synchronize()
        t_hi = time.time()
    clocks = sampler.stop(t_lo, t_hi, note)
    status = r.ta.ta_ctx_poll(r.ctx)
    if status != 0:
        raise SystemExit(f"device reported {r.ta.status_string(status)}")
    ms = m["ms_per_step"]
    if world > 1:
        from paper_2604_11288_b200.sharding import max_over_ranks
        ms = max_over_ranks(ms, dev)
    value = world * w.total * L / (ms * 1e-3)

    if rank != 0:
        r.close()
        return

    peak, how = measured_peak_hbm()
    stage = m["stage_ms"]
    dom = "compact" if fast else "score"
    ab = algorithmic_bytes(w, L, K, fast)
    dom_bytes = ab["gather"] if fast else score_kernel_bytes(w, L)
    achieved = dom_bytes / (stage[dom] * 1e-3) / 1e9 if stage[dom] > 0 else 0.0
    roofline = {"kernel": "ta_compact_kernel" if fast else "ta_score_kernel", "bound": "hbm", "achieved": achieved,
                "peak": peak, "peak_source": f"of {how}", "unit": "GB/s", "frac": achieved / peak,
                "traffic": None if fast else recorded_traffic(w.name, L),
                "ms_per_launch": stage[dom], "stage_ms": stage,
                "step_algorithmic_bytes": ab["total"], "step_frac": ab["total"] / (ms * 1e-3) / 1e9 / peak}
    roofline.update(r.launch_info())
    if not fast:
        roofline["tensor_tflops"] = m.get("score_tflops")
        roofline["kernel_algorithmic_bytes"] = dom_bytes

    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": a.steps, "warmup": warmup,
            "ms_per_step": ms, "ms_per_step_min": m["ms_per_step_min"], "ms_per_step_max": m["ms_per_step_max"],
            "rounds": rounds, "ms_per_step_rounds": per_round, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic", "config": config, "clocks": clocks,
            "gpu_launches": m["kernels_per_step"] * a.steps * rounds, "roofline": roofline}
    if cpu:
        ok, what = oracle_check(r)
        cpu["matches_oracle"] = ok
        cpu["oracle_sample"] = what
        line["cpu_baseline"] = cpu
    r.close()
    del r, inp
    torch.cuda.empty_cache()
    if not a.no_e2e and world == 1:
        try:
            line["e2e"] = e2e_leg(w, K, fast, L, dev, max(2, min(a.steps, 3)), 3)
        except Exception as ex:
            line["e2e"] = {"error": str(ex)[:200]}
    if not a.no_extra and world == 1:
        if not a.no_other:
            line["other_workloads"] = measure_others(w.name, dev, max(3, min(a.steps, 5)), 3)
        try:
            line["variants"] = measure_variants(dev)
        except Exception as ex:
            line["variants"] = [{"error": str(ex)[:200]}]
    print(json.dumps(line))


if __name__ == "__main__":
    main()
