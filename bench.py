#!/usr/bin/env python
"""Benchmark of the HyQuant prefill hot path on B200.

One "step" = one pass of the whole path over one synthetic prefill batch:
hyq_select_vertical -> hyq_quantize_blocks (Q, K, V) -> hyq_hybrid_attention_prefill
(its pre-pass included).  The metric is effective TFLOPS = 4*D*causal_pairs / time.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config c2] [--impl reference]

Prints ONE JSON line (rank 0).  With --impl reference the CPU oracle is timed instead
(rank 0 only) on a bounded sample of the same workload.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2608_27875_b200 import workloads as wl  # noqa: E402

METRIC = "hybrid prefill attention effective TFLOPS"
# the arithmetic types the path computes in, per low-bit format of Q and K
DTYPE_NOTE = {wl.FMT_INT4: "int4 x int4 -> f32 scores (e4m3 MMA), fp16 P.V, bf16 full-precision tiles",
              wl.FMT_INT8: "int8 x int8 -> s32 scores, fp16 P.V, bf16 full-precision tiles",
              wl.FMT_FP8_E4M3: "e4m3 x e4m3 -> f32 scores, fp16 P.V, bf16 full-precision tiles"}
FORMAT_SETS = {"int8": (wl.FMT_INT8,) * 3, "fp8": (wl.FMT_FP8_E4M3,) * 3,
               "int4": (wl.FMT_INT4, wl.FMT_INT4, wl.FMT_FP8_E4M3)}
NOMINAL = {"bf16_tflops": 2250.0, "lowbit_tflops": 4500.0, "hbm_gbs": 8000.0}
FALLBACK = {"bf16_tflops": 1590.0, "hbm_gbs": 6650.0}
# dram__bytes_read.sum + dram__bytes_write.sum of one launch of the dominant kernel, from the ncu
# capture summarised under profiles/ (bytes per launch of the benchmark workload; None = no capture yet)
NCU_TRAFFIC_BYTES = {"c2": 733547008 + 503056896}
# decode_kernel on the c2 cache shape, captured at batch 4 (157.169 MB read + 3.803 MB written); traffic grows in
# proportion to the batch, so the bench scales it by B / 4
NCU_DECODE_TRAFFIC_BYTES_B4 = 157169152 + 3803392


def workload_config(w, world: int = 1, strong: bool = False) -> dict:
    """The `config` object of the JSON line: the same keys and values from both arms (hyq and reference)."""
    return {"workload": w.name, "B": w.B * (1 if strong else max(1, world)), "Hq": w.Hq, "Hkv": w.Hkv, "L": w.L, "D": w.D,
            "window": w.window, "k": w.k, "formats": list(w.fmts)}


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return {"bf16_tflops": float(d["bf16_tflops"]), "hbm_gbs": float(d["hbm_gbs"]), "source": "measured",
                "bf16_tflops_sustained": float(d.get("bf16_tflops_sustained", 0.0)) or None}
    return dict(FALLBACK, source="fallback")


def fp_pairs(w: wl.Workload, idx: np.ndarray) -> int:
    """Number of causal pairs scored in full precision: per head W*L - W(W-1)/2 window pairs plus,
    for each vertical key j, the L - j - W rows that see it outside their window."""
    L, W = w.L, min(w.window, w.L)
    win = W * L - W * (W - 1) // 2
    extra = np.maximum(0, L - idx.astype(np.int64) - W).sum()
    return int(idx.shape[0] * idx.shape[1] * win + extra)


def roofline_seconds(w, n_fp, p16, p8, bw_gbs):
    n_lq = w.causal_pairs - n_fp
    t_mma = 4 * w.D * n_fp / (p16 * 1e12) + 4 * w.D * n_lq / (p8 * 1e12)
    qb, kvb = w.B * w.Hq * w.L * w.D, w.B * w.Hkv * w.L * w.D
    code = lambda n, f: n // 2 if f == wl.FMT_INT4 else n   # noqa: E731
    bytes_min = 2 * qb + code(qb, w.q_fmt) + 2 * 2 * kvb + code(kvb, w.k_fmt) + code(kvb, w.v_fmt) + 4 * qb
    return max(t_mma, bytes_min / (bw_gbs * 1e9)), t_mma, bytes_min


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu, self.proc, self.lines = gpu_index, None, []

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                          "-lms", "100", "-i", str(self.gpu)], stdout=subprocess.PIPE, text=True)
            threading.Thread(target=lambda: self.lines.extend(self.proc.stdout), daemon=True).start()
        except Exception:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in self.lines:
            f = [x.strip() for x in ln.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1]))
                mx.append(float(f[2]))
            except ValueError:
                continue
            for n, v in zip(names, f[5:9]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


# ------------------------------------------------------------------------------------------------
def oracle_sample(w: wl.Workload, budget_s: float):
    """Times the CPU oracle on a bounded sample of the workload: one KV-head group (its g query
    heads), selection and quantization in full, attention on evenly spaced query rows chosen so
    that the whole call costs about `budget_s`.  Returns (seconds, pairs, description)."""
    import oracle
    w1 = w.scaled(B=1)
    Q, K, V = wl.make_inputs(w1, heads=[0])
    qb, kb, vb = wl.bits(Q), wl.bits(K), wl.bits(V)
    t0 = time.perf_counter()
    idx = oracle.select_vertical(qb, kb, w.window, w.k)
    qz = [oracle.quantize(x, f, 64) for x, f in zip((qb, kb, vb), w.fmts)]
    t_pre = time.perf_counter() - t0
    (qc, qs), (kc, ks), (vc, vs) = qz
    g = w.Hq // w.Hkv

    def run(rows):
        t = time.perf_counter()
        oracle.attention_rows(qb, kb, vb, qc, kc, vc, qs, ks, vs, w.fmts, idx, w.window, rows)
        return time.perf_counter() - t

    # grow the row sample until one call costs a good share of the budget (the per-call cost of
    # materialising the head's fp64 views makes a tiny pilot a poor predictor)
    n_rows, t_attn = 32, 0.0
    while True:
        rows = np.linspace(0, w.L - 1, n_rows).astype(np.int32)
        t_attn = run(rows)
        if t_attn >= 0.4 * budget_s or n_rows >= w.L:
            break
        n_rows = int(min(w.L, n_rows * min(8.0, max(1.5, 0.8 * budget_s / max(t_attn, 1e-3)))))
    pairs = g * int((rows.astype(np.int64) + 1).sum())
    desc = (f"1 of {w.B * w.Hkv} (batch, kv-head) groups ({g} query heads): selection + quantization in full "
            f"({t_pre:.2f} s), attention on {n_rows} evenly spaced query rows ({pairs:.3g} causal pairs, {t_attn:.2f} s); "
            f"TFLOPS = 4*D*pairs / attention seconds")
    return t_attn, pairs, desc, oracle.num_threads()


def run_reference(args, w):
    import oracle
    oracle.build()
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    n_steps = args.steps + args.warmup
    budget = max(2.0, min(20.0, 150.0 / n_steps))
    vals, desc, cores = [], "", 1
    for s in range(n_steps):
        t, pairs, desc, cores = oracle_sample(w, budget)
        if s >= args.warmup:
            vals.append((t, pairs))
    t_tot, p_tot = sum(v[0] for v in vals), sum(v[1] for v in vals)
    tflops = 4 * w.D * p_tot / t_tot / 1e12
    line = {
        "impl": "reference", "metric": METRIC, "value": tflops, "unit": "TFLOPS", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * t_tot / max(1, args.steps),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": workload_config(w, int(os.environ.get("WORLD_SIZE", "1")), getattr(args, "strong", False)),
        "cpu_baseline": {"value": tflops, "unit": "TFLOPS", "cores": cores, "kind": "oracle", "sample": desc},
        "e2e": {"value": tflops, "unit": "TFLOPS", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))



def launches_per_step(w) -> int:
    """Kernels of the library launched by one pass of the path: select 3, quantize 3, the attention pre-pass (bitmask,
    V to fp16; with vertical keys the gather and, for FP8 / INT4 scores, the vertical-line operand tiles; 2 INT4
    widenings when used) and the two launches of the attention kernel."""
    prepass = 1 + ((2 + (1 if w.q_fmt != wl.FMT_INT8 else 0)) if w.k > 0 else 0) + (2 if w.q_fmt == wl.FMT_INT4 else 0)
    attention = 2                                       # the second launch goes through the redo list (normally empty)
    return 3 + 3 + prepass + attention


def method_error_report(w, path, Q, K, V, n_random: int = 16):
    """Error of the METHOD against exact attention (all pairs in full precision), measured on the GPU's outputs: the
    hybrid operator as benchmarked, the same low-bit codes with neither vertical keys nor window (uniform low-bit) and
    with the window only.  Reference: the CPU oracle's exact attention (window >= L) on a row sample that touches
    every structural boundary, for one (batch, KV head) group per batch element.  Sum|err| / Sum|ref| and max-abs."""
    import oracle
    api = path.api
    outs = {"hybrid": path.out.clone()}
    for name, (k_on, win) in {"uniform_lowbit": (False, 0), "window_only": (False, w.window)}.items():
        outs[name] = api.hyq_hybrid_attention_prefill(path.Q, path.K, path.V, path.qc, path.kc, path.vc, path.qs, path.ks, path.vs,
                                                      w.fmts, path.idx if k_on else None, win)
    torch.cuda.synchronize()
    rows = wl.sample_rows(w.L, w.window, n_random=n_random, edge=2)
    g = w.Hq // w.Hkv
    num = {n: 0.0 for n in outs}
    mx = {n: 0.0 for n in outs}
    den = 0.0
    groups = []
    for b in range(w.B):
        kvh = b % w.Hkv
        hs = slice(kvh * g, (kvh + 1) * g)
        qb, kb, vb = wl.bits(Q[b:b + 1, hs]), wl.bits(K[b:b + 1, kvh:kvh + 1]), wl.bits(V[b:b + 1, kvh:kvh + 1])
        zc = lambda h, f: np.zeros((1, h, w.L, oracle.code_row_bytes(f, w.D)), dtype=np.uint8)   # noqa: E731
        zs = lambda h: np.zeros((1, h, -(-w.L // 64)), dtype=np.float32)                              # noqa: E731
        exact = oracle.attention_rows(qb, kb, vb, zc(g, w.q_fmt), zc(1, w.k_fmt), zc(1, w.v_fmt), zs(g), zs(1), zs(1),
                                      w.fmts, None, w.L, rows)          # window >= L: every pair in full precision
        den += float(np.abs(exact).sum())
        for n, o in outs.items():
            d = np.abs(o[b:b + 1, hs][:, :, torch.from_numpy(rows).long().to(o.device)].double().cpu().numpy() - exact)
            num[n] += float(d.sum())
            mx[n] = max(mx[n], float(d.max()))
        groups.append([b, kvh])
    rep = {f"{n}_vs_exact": {"sum_abs_err_over_sum_abs_ref": num[n] / den, "max_abs": mx[n]} for n in outs}
    rep["sample"] = (f"{len(rows)} rows (first/last, window edge, tile edges, {n_random} seeded random rows) of the {g} query "
                     f"heads of one KV head per batch element: (b, kv head) = {groups}; reference = CPU oracle, exact attention in fp64")
    return rep

# ------------------------------------------------------------------------------------------------
class DevicePath:
    """The hot path on device tensors with every buffer preallocated (nothing allocates per step)."""

    def __init__(self, w: wl.Workload, dev, out_dtype=torch.float32):
        from paper_2608_27875_b200 import api
        self.api, self.w, self.dev = api, w, dev
        B, Hq, Hkv, L, D = w.B, w.Hq, w.Hkv, w.L, w.D
        nb = -(-L // 64)
        e = lambda *s, dt=torch.uint8: torch.empty(*s, dtype=dt, device=dev)   # noqa: E731
        self.Q, self.K, self.V = e(B, Hq, L, D, dt=torch.bfloat16), e(B, Hkv, L, D, dt=torch.bfloat16), e(B, Hkv, L, D, dt=torch.bfloat16)
        self.idx = e(B, Hq, w.k, dt=torch.int32)
        self.sel_ws = e(max(16, api.hyq_select_vertical_workspace(B, Hq, Hkv, L, L, D, w.window, w.k)))
        self.qc, self.kc, self.vc = (e(B, h, L, api.code_row_bytes(f, D)) for h, f in zip((Hq, Hkv, Hkv), w.fmts))
        self.qs, self.ks, self.vs = (e(B, h, nb, dt=torch.float32) for h in (Hq, Hkv, Hkv))
        self.out = e(B, Hq, L, D, dt=out_dtype)
        self.status = torch.zeros(1, dtype=torch.int32, device=dev)
        self.args = api.make_attn_args(self.Q, self.K, self.V, self.qc, self.kc, self.vc, self.qs, self.ks, self.vs,
                                       w.fmts, self.idx, w.window, self.out, status_word=self.status)
        self.attn_ws = e(max(16, api.hyq_hybrid_attention_prefill_workspace(self.args)))
        self.args.workspace, self.args.workspace_bytes = self.attn_ws.data_ptr(), self.attn_ws.numel()
        self.ev = [torch.cuda.Event(enable_timing=True) for _ in range(4)]
        # events recorded by the library right around the attention kernel proper
        self.kev = [torch.cuda.Event(enable_timing=True) for _ in range(2)]
        for e_ in self.kev:
            e_.record()
        self.args.ev_kernel_start, self.args.ev_kernel_stop = (e_.cuda_event for e_ in self.kev)
        self.launches_per_step = launches_per_step(w)

    def load(self, Q, K, V):
        self.Q.copy_(Q, non_blocking=True)
        self.K.copy_(K, non_blocking=True)
        self.V.copy_(V, non_blocking=True)

    def step(self, timed: bool = False, kernel_events=None):
        """One pass of the path.  kernel_events: a pair of CUDA events that the library records around the attention
        kernel proper in this step (default: the path's own pair, overwritten every step)."""
        api, w = self.api, self.w
        k0, k1 = kernel_events if kernel_events is not None else self.kev
        self.args.ev_kernel_start, self.args.ev_kernel_stop = k0.cuda_event, k1.cuda_event
        if timed:
            self.ev[0].record()
        api.hyq_select_vertical(self.Q, self.K, w.window, w.k, workspace=self.sel_ws, out=self.idx)
        if timed:
            self.ev[1].record()
        api.hyq_quantize_blocks(self.Q, w.q_fmt, codes=self.qc, scales=self.qs)
        api.hyq_quantize_blocks(self.K, w.k_fmt, codes=self.kc, scales=self.ks)
        api.hyq_quantize_blocks(self.V, w.v_fmt, codes=self.vc, scales=self.vs)
        if timed:
            self.ev[2].record()
        import ctypes
        rc = api.lib().hyq_hybrid_attention_prefill(ctypes.byref(self.args), torch.cuda.current_stream().cuda_stream)
        if rc:
            raise api.HyqError(rc, "hyq_hybrid_attention_prefill")
        if timed:
            self.ev[3].record()


class PipelinedHostPath:
    """End to end from pinned host buffers with the (batch, KV head) units pipelined: the path has no exchange
    between units, so the H2D copy of unit u+1 and the D2H copy of unit u-1 overlap the kernels of unit u
    (three streams, two buffer slots; every unit goes through the same public calls as the whole batch)."""

    def __init__(self, w: wl.Workload, dev, out_dtype=torch.float32):
        self.w, self.g = w, w.Hq // w.Hkv
        wu = w.scaled(B=1, Hq=self.g, Hkv=1)
        self.slots = [DevicePath(wu, dev, out_dtype) for _ in range(2)]
        self.s_in, self.s_cmp, self.s_out = (torch.cuda.Stream(device=dev) for _ in range(3))
        self.in_done = [torch.cuda.Event() for _ in range(2)]
        self.cmp_done = [torch.cuda.Event() for _ in range(2)]
        self.out_done = [torch.cuda.Event() for _ in range(2)]

    def run(self, Qp, Kp, Vp, out_host):
        w, g = self.w, self.g
        cur = torch.cuda.current_stream()
        for s_ in (self.s_in, self.s_cmp, self.s_out):
            s_.wait_stream(cur)
        u = 0
        for b in range(w.B):
            for hk in range(w.Hkv):
                sl, path = u & 1, self.slots[u & 1]
                with torch.cuda.stream(self.s_in):
                    if u >= 2:
                        self.s_in.wait_event(self.cmp_done[sl])       # the slot's inputs were read by unit u-2
                    path.Q.copy_(Qp[b:b + 1, hk * g:(hk + 1) * g], non_blocking=True)
                    path.K.copy_(Kp[b:b + 1, hk:hk + 1], non_blocking=True)
                    path.V.copy_(Vp[b:b + 1, hk:hk + 1], non_blocking=True)
                    self.in_done[sl].record(self.s_in)
                with torch.cuda.stream(self.s_cmp):
                    self.s_cmp.wait_event(self.in_done[sl])
                    if u >= 2:
                        self.s_cmp.wait_event(self.out_done[sl])     # the slot's output was copied out (unit u-2)
                    path.step()
                    self.cmp_done[sl].record(self.s_cmp)
                with torch.cuda.stream(self.s_out):
                    self.s_out.wait_event(self.cmp_done[sl])
                    out_host[b:b + 1, hk * g:(hk + 1) * g].copy_(path.out, non_blocking=True)
                    self.out_done[sl].record(self.s_out)
                u += 1
        for s_ in (self.s_in, self.s_cmp, self.s_out):
            cur.wait_stream(s_)

    def status(self) -> int:
        return max(int(p_.status.item()) for p_ in self.slots)


def run_query_block(args, w: wl.Workload):
    """`--lq N`: the same path for a query block of the last N rows against the full K, V (Algorithm 2's query
    block; chunked prefill): select on the block's tail queries, quantize the block and K, V, fused attention with
    Lq = N.  One JSON line with the metric on the block's causal pairs; device-resident inputs; one GPU."""
    import ctypes
    from paper_2608_27875_b200 import api, build
    build.build()
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    L, Lq, D, W = w.L, args.lq, w.D, w.window
    assert 0 < Lq <= L
    Q, K, V = (t.to(dev) for t in wl.make_inputs(w))
    Qb = Q[:, :, L - Lq:].contiguous()
    mode = api.WINDOW_FIXED_TAIL if args.fixed_tail else api.WINDOW_SLIDING
    nbq, nb = -(-Lq // 64), -(-L // 64)
    e = lambda *sh, dt=torch.uint8: torch.empty(*sh, dtype=dt, device=dev)   # noqa: E731
    idx = e(w.B, w.Hq, w.k, dt=torch.int32)
    sel_ws = e(max(16, api.hyq_select_vertical_workspace(w.B, w.Hq, w.Hkv, Lq, L, D, W, w.k)))
    qc, kc, vc = (e(w.B, h, n, api.code_row_bytes(f, D)) for h, n, f in zip((w.Hq, w.Hkv, w.Hkv), (Lq, L, L), w.fmts))
    qs, ks, vs = e(w.B, w.Hq, nbq, dt=torch.float32), e(w.B, w.Hkv, nb, dt=torch.float32), e(w.B, w.Hkv, nb, dt=torch.float32)
    out = e(w.B, w.Hq, Lq, D, dt=torch.float32)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    a = api.make_attn_args(Qb, K, V, qc, kc, vc, qs, ks, vs, w.fmts, idx, W, out, status_word=status, window_mode=mode)
    ws = e(max(16, api.hyq_hybrid_attention_prefill_workspace(a)))
    a.workspace, a.workspace_bytes = ws.data_ptr(), ws.numel()
    kev = [torch.cuda.Event(enable_timing=True) for _ in range(2)]
    for ev in kev:
        ev.record()
    a.ev_kernel_start, a.ev_kernel_stop = (ev.cuda_event for ev in kev)

    def step():
        api.hyq_select_vertical(Qb, K, W, w.k, workspace=sel_ws, out=idx)
        api.hyq_quantize_blocks(Qb, w.q_fmt, codes=qc, scales=qs)
        api.hyq_quantize_blocks(K, w.k_fmt, codes=kc, scales=ks)
        api.hyq_quantize_blocks(V, w.v_fmt, codes=vc, scales=vs)
        rc = api.lib().hyq_hybrid_attention_prefill(ctypes.byref(a), torch.cuda.current_stream().cuda_stream)
        assert rc == 0, rc

    for _ in range(max(3, args.warmup)):
        step()
    torch.cuda.synchronize()
    sampler = ClockSampler(0)
    sampler.start()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ev0.record()
    for _ in range(args.steps):
        step()
    ev1.record()
    torch.cuda.synchronize()
    clocks = sampler.stop()
    assert int(status.item()) == 0, "attention kernel reported a device-side error"
    ms = ev0.elapsed_time(ev1) / args.steps
    k_ms = kev[0].elapsed_time(kev[1])
    off = L - Lq
    pairs = w.B * w.Hq * (L * (L + 1) - off * (off + 1)) // 2
    pos = torch.arange(off, L, device=dev)
    if args.fixed_tail:
        n_win = int(torch.clamp(pos - (L - W) + 1, min=0).sum()) * w.B * w.Hq
        lim = torch.clamp(pos, max=L - W - 1)
    else:
        n_win = int(torch.clamp(pos + 1, max=W).sum()) * w.B * w.Hq
        lim = pos - W
    n_vl = int((idx.long().unsqueeze(-1) <= lim.view(1, 1, 1, -1)).sum()) if w.k else 0
    n_fp = n_win + n_vl
    peaks = measured_peaks()
    flops = 4 * D * pairs
    t_meas = 4 * D * (n_fp / (peaks["bf16_tflops"] * 1e12) + (pairs - n_fp) / (2 * peaks["bf16_tflops"] * 1e12))
    t_nom = 4 * D * (n_fp / (NOMINAL["bf16_tflops"] * 1e12) + (pairs - n_fp) / (NOMINAL["lowbit_tflops"] * 1e12))
    print(json.dumps({
        "metric": METRIC, "value": flops / (ms * 1e-3) / 1e12, "unit": "TFLOPS", "n_gpus": 1, "steps": args.steps,
        "warmup": max(3, args.warmup), "ms_per_step": ms, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": DTYPE_NOTE.get(w.q_fmt, "mixed"), "data": "synthetic",
        "config": {"workload": f"{w.name}, query block of the last {Lq} rows of {L}", "B": w.B, "Hq": w.Hq, "Hkv": w.Hkv,
                   "L": L, "Lq": Lq, "D": D, "window": W, "window_form": "fixed tail" if args.fixed_tail else "sliding",
                   "k": w.k, "formats": list(w.fmts), "step": "select + quantize Q block, K, V + fused attention",
                   "l2": "K, V and their codes exceed L2" if 4 * w.B * w.Hkv * L * D > 126e6 else "inputs fit L2"},
        "roofline": {"bound": "tensor", "kernel": "attn_tc_kernel", "achieved": flops / (k_ms * 1e-3) / 1e12,
                     "peak": flops / t_meas / 1e12, "unit": "TFLOP/s", "frac": t_meas * 1e3 / k_ms, "traffic": None,
                     "kernel_ms": k_ms, "frac_nominal": t_nom * 1e3 / k_ms, "fp_pair_share": n_fp / pairs,
                     "peak_source": peaks["source"]},
        "gpu_launches": launches_per_step(w) * args.steps,
        "clocks": clocks}))


def run_decode(args, w: wl.Workload):
    """`--decode`: the decode side on the same cache shape.  Freeze (Algorithm 4) builds the hybrid K4V4 cache
    of `--batch` sequences from a synthetic prefill cache (vertical sets from Algorithm 1 on the first query head
    of every KV group), the staging buffer is filled, and the timed step is one hyq_hybrid_attention_decode call
    (Algorithm 3: slice kernel + merge kernel) for one new token per sequence, over cache replicas used
    round-robin so that no call finds its cache in L2.  One JSON line; one GPU."""
    from paper_2608_27875_b200 import api, build, decode_api as dapi
    build.build()
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    w = w.scaled(B=args.batch)
    g = w.Hq // w.Hkv
    kv_fmt = {"int4": wl.FMT_INT4, "int8": wl.FMT_INT8, "fp8": wl.FMT_FP8_E4M3}[args.kv_format]
    Q, K, V = wl.make_inputs(w)
    K, V = K.to(dev), V.to(dev)
    q_tail = Q[:, ::g].contiguous().to(dev)                 # Algorithm 1 with H = H_KV heads
    idx = api.hyq_select_vertical(q_tail, K, w.window, w.k)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    cache = dapi.hyq_freeze(K, V, idx, w.window, w.Hq, staging_capacity=args.staging, fmt=kv_fmt)
    torch.cuda.synchronize()
    e0.record()
    dapi.hyq_freeze(K, V, idx, w.window, w.Hq, staging_capacity=args.staging, cache=cache)
    e1.record()
    torch.cuda.synchronize()
    freeze_ms = e0.elapsed_time(e1)
    gen = torch.Generator(device=dev).manual_seed(w.seed + 5)
    new_rows = [(torch.randn(w.B, w.Hkv, w.D, device=dev, generator=gen).to(torch.bfloat16),
                 torch.randn(w.B, w.Hkv, w.D, device=dev, generator=gen).to(torch.bfloat16)) for _ in range(args.staging)]
    # Replicas of the cache at different addresses, used round-robin: a call never finds its cache in L2
    # (more than three L2 sizes of other replicas are read in between) and no flush kernel dirties L2
    # right before a timed call.
    by = cache.bytes_read_per_token()
    n_rep = 1 + int(np.ceil(3 * 126e6 / by))
    caches = [cache] + [dapi.hyq_freeze(K, V, idx, w.window, w.Hq, staging_capacity=args.staging, fmt=kv_fmt)
                        for _ in range(n_rep - 1)]
    for c in caches:
        for kn, vn in new_rows:
            c.append(kn, vn)
    q = Q[:, :, -1].contiguous().to(dev)
    out = torch.empty(w.B, w.Hq, w.D, dtype=torch.bfloat16, device=dev)
    ws = torch.empty(max(16, dapi.hyq_hybrid_attention_decode_workspace(cache, args.splits)), dtype=torch.uint8, device=dev)
    call = lambda i: dapi.hyq_hybrid_attention_decode(q, caches[i % n_rep], splits=args.splits, out=out, workspace=ws)   # noqa: E731
    for i in range(max(3, args.warmup)):
        call(i)
    torch.cuda.synchronize()
    sampler = ClockSampler(0)
    sampler.start()
    e0.record()
    for i in range(args.steps):
        call(i)
    e1.record()
    torch.cuda.synchronize()
    clocks = sampler.stop()
    ms = e0.elapsed_time(e1) / args.steps
    # end to end: the token's query from pinned host memory, the output back to the host, every step
    q_host, out_host = q.cpu().pin_memory(), torch.empty(out.shape, dtype=out.dtype).pin_memory()
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    for i in range(args.steps):
        q.copy_(q_host, non_blocking=True)
        call(i)
        out_host.copy_(out, non_blocking=True)
        torch.cuda.synchronize()
    e2e_ms = (time.perf_counter() - t0) / args.steps * 1e3
    cache = caches[(args.steps - 1) % n_rep]
    by = cache.bytes_read_per_token()
    peaks = measured_peaks()
    rows = w.L + args.staging
    # CPU baseline: the oracle on one sequence's cache (Freeze + one token), all heads
    import oracle
    from oracle import decode as od
    kb, vb = wl.bits(K[:1].cpu()), wl.bits(V[:1].cpu())
    ref = od.freeze(kb, vb, idx[:1].cpu().numpy(), w.window, fmts=(kv_fmt, kv_fmt), staging_capacity=args.staging)
    for kn, vn in new_rows:
        od.append_staging(ref, wl.bits(kn[:1].cpu()), wl.bits(vn[:1].cpu()))
    t0 = time.perf_counter()
    want, _ = od.decode_attention(wl.bits(q[:1].cpu()), ref)
    cpu_s = time.perf_counter() - t0
    err = np.abs(out[:1].float().cpu().numpy() - want)
    print(json.dumps({
        "metric": "hybrid decode attention latency per token step", "value": ms * 1e3, "unit": "us", "n_gpus": 1,
        "steps": args.steps, "warmup": max(3, args.warmup), "ms_per_step": ms, "higher_is_better": False,
        "scaling": "weak", "vs_baseline": None,
        "dtype": f"{args.kv_format} codes -> fp16 in registers, fp16 / bf16 mma.sync with f32 accumulation", "data": "synthetic",
        "config": {"workload": f"{w.name} cache shape, decode of one token per sequence", "B": w.B, "Hq": w.Hq,
                   "Hkv": w.Hkv, "N": w.L, "D": w.D, "window": w.window, "k": w.k, "staging_rows": args.staging,
                   "format": {"int4": "K4V4", "int8": "K8V8 (INT8)", "fp8": "K8V8 (FP8 e4m3)"}[args.kv_format] + ", group 64", "splits": args.splits, "cached_rows_per_head": rows,
                   "l2": f"{n_rep} cache replicas used round-robin ({by * (n_rep - 1) / 1e6:.0f} MB read between reuses)",
                   "freeze_ms": freeze_ms},
        "roofline": {"bound": "hbm", "kernel": "decode_kernel + decode_merge_kernel (one call)",
                     "achieved": by / (ms * 1e-3) / 1e9, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                     "frac": by / (ms * 1e-3) / 1e9 / peaks["hbm_gbs"], "traffic": (NCU_DECODE_TRAFFIC_BYTES_B4 * w.B // 4 if (w.name, w.L, args.staging, args.kv_format) == ("c2", 32768, 128, "int4") else None),
                     "bytes_per_call": by, "peak_source": peaks["source"]},
        "cpu_baseline": {"value": cpu_s * 1e6 * w.B, "unit": "us", "cores": oracle.num_threads(), "kind": "oracle",
                         "sample": "oracle attention of one sequence (all heads) timed, scaled by the batch size"},
        "e2e": {"value": e2e_ms * 1e3, "unit": "us", "h2d_bytes_per_step": q_host.numel() * 2,
                "d2h_bytes_per_step": out_host.numel() * 2},
        "check": {"max_abs_err_vs_oracle_seq0": float(err.max())},
        "gpu_launches": 2 * args.steps, "clocks": clocks}))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--config", default="c2", choices=sorted(wl.CONFIGS))
    ap.add_argument("--impl", default="hyq", choices=["hyq", "reference"])
    ap.add_argument("--seq", type=int, default=0, help="override the sequence length (profiling on a smaller case)")
    ap.add_argument("--cpu-budget", type=float, default=15.0, help="seconds of oracle time for cpu_baseline")
    ap.add_argument("--lq", type=int, default=0, help="measure a query block of the last LQ rows against the full K, V")
    ap.add_argument("--fixed-tail", action="store_true", help="with --lq: Algorithm 2's fixed tail window")
    ap.add_argument("--decode", action="store_true", help="measure the decode side (Freeze + one-token attention)")
    ap.add_argument("--batch", type=int, default=8, help="with --decode: sequences in the batch")
    ap.add_argument("--staging", type=int, default=128, help="with --decode: staged rows (W_s, all filled)")
    ap.add_argument("--splits", type=int, default=0, help="with --decode: slices per KV head (0 = library's choice)")
    ap.add_argument("--kv-format", default="int4", choices=["int4", "int8", "fp8"], help="with --decode: cache code format (K4V4 / K8V8 / FP8 e4m3)")
    ap.add_argument("--strong", action="store_true",
                    help="strong scaling: ONE batch of the workload, its (batch, KV head) units sharded over the ranks "
                         "(default: every rank runs its own full batch)")
    ap.add_argument("--method-error", action="store_true",
                    help="also report the method's error against exact attention (always on for c4)")
    ap.add_argument("--formats", default="", choices=["", *sorted(FORMAT_SETS)],
                    help="override the workload's (Q, K, V) low-bit formats (default: as the workload defines them)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "hyq" else args.warmup
    w = wl.CONFIGS[args.config]
    if args.seq:
        w = w.scaled(L=args.seq, k=max(1, w.k * args.seq // w.L), n_plant=max(1, w.n_plant * args.seq // w.L))
    if args.formats:
        fq, fk, fv = FORMAT_SETS[args.formats]
        w = w.scaled(q_fmt=fq, k_fmt=fk, v_fmt=fv)
    if args.impl == "reference":
        run_reference(args, w)
        return
    if args.lq:
        run_query_block(args, w)
        return
    if args.decode:
        run_decode(args, w)
        return

    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        # launched plainly: start the N ranks here (one process per GPU; NCCL only for the barrier and the max-reduction)
        import socket
        import torch.multiprocessing as mp
        with socket.socket() as s_:
            s_.bind(("127.0.0.1", 0))
            port = s_.getsockname()[1]
        mp.spawn(_spawned_rank, args=(args.gpus, port, sys.argv[1:]), nprocs=args.gpus, join=True)
        return
    run_hyq(args, w)


def _spawned_rank(rank: int, world: int, port: int, argv):
    os.environ.update(RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world), MASTER_ADDR="127.0.0.1",
                      MASTER_PORT=str(port))
    sys.argv = [sys.argv[0]] + list(argv)
    main()


def run_hyq(args, w):
    import ctypes
    from paper_2608_27875_b200 import api, build, sharding
    rank, world = int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1"))
    if world != args.gpus:
        raise SystemExit(f"bench.py: --gpus {args.gpus} but the launcher started {world} rank(s)")
    if torch.cuda.device_count() < (world if "LOCAL_RANK" in os.environ else 1):
        raise SystemExit(f"bench.py: {world} ranks on one node need {world} GPUs, found {torch.cuda.device_count()}")
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if rank == 0 or world == 1:
        build.build()
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)
        dist.barrier()
    api.lib()

    if args.strong:
        run_strong(args, w, api, sharding, rank, world, dev)
        return
    # every rank runs its own full batch of the workload (units = (batch, kv head) groups; no collective)
    wr = w.scaled(seed=w.seed + 17 * rank)
    Q, K, V = wl.make_inputs(wr)
    Qp, Kp, Vp = (t.pin_memory() for t in (Q, K, V))
    path = DevicePath(wr, dev)
    path.load(Qp, Kp, Vp)
    torch.cuda.synchronize()

    def barrier():
        if world > 1:
            torch.distributed.barrier()
        torch.cuda.synchronize()

    for _ in range(args.warmup):
        path.step()
    barrier()
    assert int(path.status.item()) == 0, "attention kernel reported a device-side error"

    sampler = ClockSampler(local)
    sampler.start()
    parts = np.zeros(3)
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    # one pair of events per timed step for the library to record around the attention kernel proper
    kevs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
    for a_, b_ in kevs:                 # (torch creates the CUDA event at the first record)
        a_.record()
        b_.record()
    barrier()
    ev0.record()
    for n in range(args.steps):
        path.step(timed=True, kernel_events=kevs[n])
    ev1.record()
    barrier()
    total_ms = ev0.elapsed_time(ev1)
    kern_in_loop = [a_.elapsed_time(b_) for a_, b_ in kevs]
    # per-part times of the last step (events are re-recorded every step)
    parts = np.array([path.ev[n].elapsed_time(path.ev[n + 1]) for n in range(3)])
    clocks = sampler.stop()
    assert int(path.status.item()) == 0, "attention kernel reported a device-side error"

    # the dominant kernel alone: attention call (pre-pass + kernel) re-timed over the same inputs
    attn_ms, kern_ms_l = [], []
    for _ in range(max(3, min(args.steps, 10))):
        path.ev[0].record()
        path.args.ev_kernel_start, path.args.ev_kernel_stop = (e_.cuda_event for e_ in path.kev)
        rc = api.lib().hyq_hybrid_attention_prefill(ctypes.byref(path.args), torch.cuda.current_stream().cuda_stream)
        path.ev[1].record()
        torch.cuda.synchronize()
        assert rc == 0
        attn_ms.append(path.ev[0].elapsed_time(path.ev[1]))
        kern_ms_l.append(path.kev[0].elapsed_time(path.kev[1]))
    attn_call_ms = float(np.mean(attn_ms))
    kern_ms_isolated = float(np.mean(kern_ms_l))
    kern_ms = float(np.median(kern_in_loop))                 # the figure of record: inside the timed steps

    total_ms = sharding.max_over_ranks(total_ms, dev)
    ms_per_step = total_ms / args.steps
    flops = wr.flops
    value = world * flops / (ms_per_step * 1e-3) / 1e12

    # end to end through host buffers: H2D of Q, K, V, the path, D2H of the output; the (batch, KV head) units
    # are pipelined so that the copies of neighbouring units overlap the kernels of the current one
    out_host = torch.empty(path.out.shape, dtype=path.out.dtype).pin_memory()
    pipe = PipelinedHostPath(wr, dev)
    e2e_steps = max(2, min(args.steps, 5))
    e2e_ms = []
    for n in range(e2e_steps + 1):
        barrier()
        t0 = time.perf_counter()
        pipe.run(Qp, Kp, Vp, out_host)
        torch.cuda.synchronize()
        if n > 0:
            e2e_ms.append((time.perf_counter() - t0) * 1e3)
    assert pipe.status() == 0, "attention kernel reported a device-side error"
    # the pipelined units must reproduce the whole-batch result bit for bit (checked on the last unit)
    g_ = wr.Hq // wr.Hkv
    assert torch.equal(out_host[wr.B - 1:, wr.Hq - g_:].to(dev), path.out[wr.B - 1:, wr.Hq - g_:]), "pipelined e2e differs"
    e2e_ms_max = sharding.max_over_ranks(float(np.mean(e2e_ms)), dev)
    e2e_val = world * flops / (e2e_ms_max * 1e-3) / 1e12
    # the same with the output stored as bf16 (RNE of the fp32 result, the dtype of Q, K, V): half the D2H bytes
    out_host16 = torch.empty(path.out.shape, dtype=torch.bfloat16).pin_memory()
    pipe16 = PipelinedHostPath(wr, dev, torch.bfloat16)
    e2e16_ms = []
    for n in range(e2e_steps + 1):
        barrier()
        t0 = time.perf_counter()
        pipe16.run(Qp, Kp, Vp, out_host16)
        torch.cuda.synchronize()
        if n > 0:
            e2e16_ms.append((time.perf_counter() - t0) * 1e3)
    assert pipe16.status() == 0, "attention kernel reported a device-side error"
    assert torch.equal(out_host16[wr.B - 1:, wr.Hq - g_:].to(dev), path.out[wr.B - 1:, wr.Hq - g_:].to(torch.bfloat16)), "bf16 e2e differs"
    e2e16_ms_max = sharding.max_over_ranks(float(np.mean(e2e16_ms)), dev)
    h2d = sum(t.numel() * t.element_size() for t in (Q, K, V))
    d2h = out_host.numel() * out_host.element_size()

    if rank != 0:
        if world > 1:
            torch.distributed.destroy_process_group()
        return

    # roofline of the attention kernel (tensor-bound): mixed-precision time at measured peaks
    peaks = measured_peaks()
    idx = path.idx.cpu().numpy()
    n_fp = fp_pairs(wr, idx)
    t_roof_meas, _, bytes_min = roofline_seconds(wr, n_fp, peaks["bf16_tflops"], 2 * peaks["bf16_tflops"], peaks["hbm_gbs"])
    t_roof_nom, _, _ = roofline_seconds(wr, n_fp, NOMINAL["bf16_tflops"], NOMINAL["lowbit_tflops"], NOMINAL["hbm_gbs"])
    k_ms = kern_ms if kern_ms else attn_call_ms
    achieved = flops / (k_ms * 1e-3) / 1e12
    peak_eff = flops / t_roof_meas / 1e12
    sus = peaks.get("bf16_tflops_sustained")
    t_roof_sus = roofline_seconds(wr, n_fp, sus, 2 * sus, peaks["hbm_gbs"])[0] if sus else None
    roofline = {
        "bound": "tensor", "kernel": "attn_tc_kernel", "achieved": achieved, "peak": peak_eff, "unit": "TFLOP/s",
        "frac": achieved / peak_eff, "traffic": NCU_TRAFFIC_BYTES.get(w.name),
        "peak_source": f"{peaks['source']}: bf16 {peaks['bf16_tflops']} TFLOP/s for the full-precision pairs, 2x that "
                       f"(nominal 8-bit:16-bit ratio) for the low-bit pairs; peak = flops / mixed roofline time",
        "kernel_ms": k_ms, "kernel_ms_isolated": kern_ms_isolated,
        "timed": "median over the timed steps of the library's own events around the attention kernel (kernel_ms_isolated: "
                 "the same events in a separate loop with a synchronize between launches)",
        "fp_pair_share": n_fp / wr.causal_pairs, "roofline_ms_measured": t_roof_meas * 1e3,
        "roofline_ms_nominal": t_roof_nom * 1e3, "frac_nominal": (t_roof_nom * 1e3) / k_ms,
        "frac_whole_step": (t_roof_meas * 1e3) / ms_per_step,
        "frac_isolated": (t_roof_meas * 1e3) / kern_ms_isolated if kern_ms_isolated else None,
        "frac_nominal_whole_step": (t_roof_nom * 1e3) / ms_per_step, "min_bytes": bytes_min,
        "frac_at_sustained_peak": (t_roof_sus * 1e3) / k_ms if t_roof_sus else None,
        "sustained_note": "context only: the same fraction against the sustained bf16 figure of MEASURED_PEAKS.json (a matmul "
                          "looped for seconds, at the clocks it falls to); `frac` keeps the burst figure, the larger denominator, "
                          "because the timed region here is a fraction of a second",
        "nominal_definition": "the workload definition's roofline: full-precision pairs at 2250 TFLOP/s dense bf16, low-bit "
                              "pairs at 4500 TFLOP/s dense INT8/FP8, or the minimum bytes at 8 TB/s if larger (frac_nominal); "
                              "`frac` and `peak` use this pool's measured bf16 matmul rate instead, as the measurement "
                              "contract asks",
    }

    t_cpu, pairs_cpu, desc, cores = oracle_sample(w, args.cpu_budget)
    cpu = {"value": 4 * w.D * pairs_cpu / t_cpu / 1e12, "unit": "TFLOPS", "cores": cores, "kind": "oracle", "sample": desc}

    method_error = method_error_report(wr, path, Q, K, V) if (args.method_error or w.name == "c4") else None

    line = {
        "metric": METRIC, "value": value, "unit": "TFLOPS", "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": DTYPE_NOTE[w.q_fmt],
        "data": "synthetic",
        "config": workload_config(w, world, args.strong),
        "config_notes": {"l2": "inputs larger than L2 (Q+K+V bf16 = %.0f MB per step)" % (h2d / 1e6),
                         "step": "select + quantize Q,K,V + fused attention (pre-pass included)", "out_dtype": "fp32"},
        "step_parts_ms": {"select": float(parts[0]), "quantize": float(parts[1]), "attention_call": float(parts[2])},
        "attention_only_tflops": flops / (attn_call_ms * 1e-3) / 1e12,
        "roofline": roofline, "cpu_baseline": cpu,
        "e2e_bf16_out": {"value": world * flops / (e2e16_ms_max * 1e-3) / 1e12, "unit": "TFLOPS", "h2d_bytes_per_step": h2d,
                         "d2h_bytes_per_step": d2h // 2, "ms_per_step": e2e16_ms_max,
                         "how": "as e2e, with the output stored as bf16 (round-to-nearest of the fp32 result)"},
        "e2e": {"value": e2e_val, "unit": "TFLOPS", "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "ms_per_step": e2e_ms_max, "steps": e2e_steps,
                "how": "pinned host Q,K,V -> H2D -> select, quantize, attention -> D2H of the fp32 output, pipelined over the "
                       f"{wr.B * wr.Hkv} (batch, KV head) units on three streams"},
        "gpu_launches": path.launches_per_step * args.steps,
        "clocks": clocks,
    }
    if method_error is not None:
        line["method_error"] = method_error
    print(json.dumps(line))
    if world > 1:
        torch.distributed.destroy_process_group()


def run_strong(args, w, api, sharding, rank, world, dev):
    """`--strong`: ONE batch of the workload; its (batch, KV head) units are sharded over the ranks by
    sharding.shard_units and every rank runs the whole path on its own units (device-resident inputs, no collective on
    the data path).  value = the batch's FLOPs / the slowest rank's time.  The end-to-end leg goes through
    sharding.run_sharded from pinned host tensors, every rank writing its slices of the output."""
    import torch.distributed as dist
    g = w.Hq // w.Hkv
    wu = w.scaled(B=1, Hq=g, Hkv=1)
    Q, K, V = wl.make_inputs(w)
    mine = sharding.shard_units(w.B, w.Hkv, world, rank)
    paths = []
    for b, hk in mine:
        p_ = DevicePath(wu, dev)
        p_.load(Q[b:b + 1, hk * g:(hk + 1) * g].contiguous(), K[b:b + 1, hk:hk + 1].contiguous(), V[b:b + 1, hk:hk + 1].contiguous())
        paths.append(p_)
    torch.cuda.synchronize()

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(args.warmup):
        for p_ in paths:
            p_.step()
    barrier()
    sampler = ClockSampler(dev.index)
    sampler.start()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    ev0.record()
    for _ in range(args.steps):
        for p_ in paths:
            p_.step()
    ev1.record()
    barrier()
    ms = sharding.max_over_ranks(ev0.elapsed_time(ev1), dev) / args.steps
    clocks = sampler.stop()
    assert all(int(p_.status.item()) == 0 for p_ in paths), "attention kernel reported a device-side error"
    # end to end: pinned host batch -> each rank's units through the public wrapper -> the rank's slices of the output
    Qp, Kp, Vp = (t.pin_memory() for t in (Q, K, V))
    out_host = torch.zeros(w.B, w.Hq, w.L, w.D, dtype=torch.float32).pin_memory()
    slot = DevicePath(wu, dev)

    def unit_prefill(q, k_, v, window, k_sel, fmts):
        slot.load(q, k_, v)
        slot.step()
        return slot.out

    e2e = []
    for n in range(3):
        barrier()
        t0 = time.perf_counter()
        sharding.run_sharded(Qp, Kp, Vp, w.window, w.k, w.fmts, prefill_fn=unit_prefill, out=out_host, world=world, rank=rank)
        torch.cuda.synchronize()
        if n > 0:
            e2e.append((time.perf_counter() - t0) * 1e3)
    e2e_ms = sharding.max_over_ranks(float(np.mean(e2e)), dev)
    if mine:
        b, hk = mine[-1]
        assert torch.equal(out_host[b:b + 1, hk * g:(hk + 1) * g].to(dev), paths[-1].out), "sharded e2e differs from the device-resident run"
    if rank == 0:
        h2d = sum(t.numel() * t.element_size() for t in (Q, K, V))
        print(json.dumps({
            "metric": METRIC, "value": w.flops / (ms * 1e-3) / 1e12, "unit": "TFLOPS", "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "strong", "vs_baseline": None,
            "dtype": DTYPE_NOTE[w.q_fmt], "data": "synthetic", "config": workload_config(w, world, True),
            "config_notes": {"sharding": f"{w.B * w.Hkv} (batch, KV head) units over {world} rank(s), contiguous balanced ranges, "
                                         f"one launch sequence per unit, no collective on the data path",
                             "l2": "inputs larger than L2" if h2d > 126e6 else "inputs fit L2"},
            "e2e": {"value": w.flops / (e2e_ms * 1e-3) / 1e12, "unit": "TFLOPS", "h2d_bytes_per_step": h2d,
                    "d2h_bytes_per_step": out_host.numel() * 4, "ms_per_step": e2e_ms,
                    "how": "sharding.run_sharded: pinned host batch -> each rank's units H2D -> path -> D2H into the rank's output slices"},
            "gpu_launches": sum(p_.launches_per_step for p_ in paths) * args.steps, "clocks": clocks}))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
