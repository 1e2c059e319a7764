#!/usr/bin/env python
"""Benchmark of the halted-prefill block step on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--seq T]

One *step* = one pass of the whole hot path (dash_layer_step: RMSNorm, QKV
projection, rotary embedding, causal GQA attention over the packed active set,
output projection, delta score + residual + halting rule, scatter, compaction)
over one batch of synthetic tokens.  The workload at every N is the
Qwen2.5-7B-shaped single layer at 8192 tokens, bf16, with the threshold at the
40th percentile of the relative delta (60 % of the tokens stay active).  With
N > 1 every rank runs its own batch (weak scaling, no data-path collective).

Prints one JSON line (rank 0).  `--impl reference` times the CPU oracle, as it
stands, on the host cores on a bounded sample of the same workload.
"""
from __future__ import annotations

import argparse
import json
import math
import os
import statistics
import subprocess
import sys
import threading
import time

import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2604_18103_b200 import workloads as wl  # noqa: E402

METRIC = "active_token_prefill_tokens_per_s_per_layer"
UNIT = "tokens/s"
L2_FLUSH_BYTES = 256 << 20


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            d = json.load(f)
        return {"hbm_gbs": d["hbm_gbs"], "bf16_tflops": d["bf16_tflops"], "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "source": "fallback"}


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.rows, self.proc = index, [], None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits", "-lms", "100",
                                          "-i", str(self.index)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.t = threading.Thread(target=self._read, daemon=True)
            self.t.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([x.strip() for x in line.split(",")])

    def stop(self, first: int = 0):
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        for r in self.rows[max(0, first - 1):]:
            try:
                sm.append(float(r[1])); mx.append(float(r[2]))
            except Exception:
                continue
            for name, col in (("hw_slowdown", 5), ("hw_thermal_slowdown", 6), ("sw_thermal_slowdown", 7), ("sw_power_cap", 8)):
                if len(r) > col and r[col].lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


def attention_flops(cu, Hq, D):
    """Algorithmic FLOPs of the causal attention: 4 Hq D per (query, key <= query) pair."""
    tot = 0
    for s in range(len(cu) - 1):
        n = int(cu[s + 1]) - int(cu[s])
        tot += n * (n + 1) // 2
    return 4.0 * Hq * D * tot


# --------------------------------------------------------------------------- ours
def run_ours(args):
    from paper_2604_18103_b200 import build as dash_build
    from paper_2604_18103_b200 import dash

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py: no CUDA device (the product path has no CPU fallback)")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)
    if rank == 0:
        dash_build.build()
    if world > 1:
        dist.barrier()
    dash.lib()

    T = args.seq
    w = wl.config2(T=T, seed=1 + rank)
    sh = w.shape
    S = w.S
    H_host = w.tensors["H"].pin_memory()
    pos_host = wl.positions(w.cu).pin_memory()
    tok_host = torch.arange(T, dtype=torch.int32).pin_memory()
    cu_host = w.cu.pin_memory()
    layer = dash.Layer(sh, w.weights[0], dev, tau=0.0)
    lay = dash.dash_layer_workspace(layer, T, S)
    ws = dash.workspace(lay.total, dev)
    H = torch.empty(T, sh.d, dtype=sh.dtype, device=dev)
    pos = torch.empty(T, dtype=torch.int32, device=dev)
    tok = torch.empty(T, dtype=torch.int32, device=dev)
    cu = torch.empty(S + 1, dtype=torch.int32, device=dev)
    x_full = torch.zeros(T, sh.d, dtype=sh.dtype, device=dev)
    H_next = torch.zeros(T, sh.d, dtype=sh.dtype, device=dev)
    tok_next = torch.zeros(T, dtype=torch.int32, device=dev)
    pos_next = torch.zeros(T, dtype=torch.int32, device=dev)
    cu_next = torch.zeros(S + 1, dtype=torch.int32, device=dev)
    n_next = torch.zeros(1, dtype=torch.int32, device=dev)
    r = torch.zeros(T, dtype=torch.float32, device=dev)
    mask = torch.zeros(T, dtype=torch.uint8, device=dev)
    flush = torch.empty(L2_FLUSH_BYTES, dtype=torch.uint8, device=dev)
    flush_src = torch.zeros(L2_FLUSH_BYTES // 4, dtype=torch.int32, device=dev)
    # host-side result buffers of the end-to-end arm
    x_full_h = torch.empty(T, sh.d, dtype=sh.dtype).pin_memory()
    H_next_h = torch.empty(T, sh.d, dtype=sh.dtype).pin_memory()
    r_h = torch.empty(T, dtype=torch.float32).pin_memory()
    mask_h = torch.empty(T, dtype=torch.uint8).pin_memory()
    tok_next_h = torch.empty(T, dtype=torch.int32).pin_memory()
    cu_next_h = torch.empty(S + 1, dtype=torch.int32).pin_memory()

    def h2d():
        H.copy_(H_host, non_blocking=True); pos.copy_(pos_host, non_blocking=True)
        tok.copy_(tok_host, non_blocking=True); cu.copy_(cu_host, non_blocking=True)

    def d2h():
        x_full_h.copy_(x_full, non_blocking=True); H_next_h.copy_(H_next, non_blocking=True)
        r_h.copy_(r, non_blocking=True); mask_h.copy_(mask, non_blocking=True)
        tok_next_h.copy_(tok_next, non_blocking=True); cu_next_h.copy_(cu_next, non_blocking=True)

    def step():
        dash.dash_layer_step(layer, H, tok, pos, cu, T, x_full, H_next, tok_next, pos_next, cu_next, n_next, r, mask, ws)

    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    h2d()
    # threshold at the 40th percentile of the measured relative delta (harness work, untimed)
    step()
    torch.cuda.synchronize()
    K = dash.dash_keep_count(T, w.rho)
    tau = float(torch.topk(r, K).values[-1].item())
    layer.set_tau(tau)
    for _ in range(max(args.warmup, 3)):
        step()
    torch.cuda.synchronize()
    n_active = int(n_next.item())

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def timed(fn, steps, pre=None, post=None):
        """Per-step CUDA-event timing on the current stream; L2 flushed between steps outside the events."""
        evs = []
        barrier()
        for _ in range(steps):
            flush.zero_()          # write a buffer larger than L2 ...
            flush_src.sum()        # ... then read another one, so the timed kernels do not inherit dirty-line write-backs
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            if pre:
                pre()
            fn()
            if post:
                post()
            b.record()
            evs.append((a, b))
        barrier()
        return [a.elapsed_time(b) for a, b in evs]

    if rank == 0:                                   # the sampler needs a moment before its first line
        t_s = time.time()
        while not sampler.rows and time.time() - t_s < 5.0:
            step()
            torch.cuda.synchronize()
    n_before = len(sampler.rows)
    t_wall0 = time.time()
    ms = timed(step, args.steps)
    wall = time.time() - t_wall0
    ms_e2e = timed(step, max(3, min(args.steps, 10)), pre=h2d, post=d2h)

    # the dominant kernel alone (same launch configuration as inside the step)
    nq = (sh.Hq + 2 * sh.Hkv) * sh.D
    es = 2
    QKV = ws[lay.QKV:lay.QKV + T * nq * es].view(sh.dtype).view(T, nq)
    Q = QKV[:, :sh.Hq * sh.D].view(T, sh.Hq, sh.D)
    Kt = QKV[:, sh.Hq * sh.D:(sh.Hq + sh.Hkv) * sh.D].view(T, sh.Hkv, sh.D)
    V = QKV[:, (sh.Hq + sh.Hkv) * sh.D:].view(T, sh.Hkv, sh.D)
    Obuf = ws[lay.O:lay.O + T * sh.Hq * sh.D * es].view(sh.dtype).view(T, sh.Hq, sh.D)
    attn_ws = dash.workspace(256, dev)
    ms_attn = timed(lambda: dash.dash_varlen_attention(Q, Kt, V, cu, T, O=Obuf, ws=attn_ws), max(5, min(args.steps, 20)))
    # the two HBM-bound kernels alone, for the record
    U = ws[lay.U:lay.U + T * sh.d * es].view(sh.dtype).view(T, sh.d)
    Ht = ws[lay.Ht:lay.Ht + T * sh.d * es].view(sh.dtype).view(T, sh.d)
    ms_norm = timed(lambda: dash.dash_delta_norm(U, H, r_out=r, Hres_out=Ht, tau=tau, cu_seqlens=cu, mask_out=mask), 10)
    cws = dash.workspace(dash.dash_workspace_bytes(dash.WS_COMPACT, T, S), dev)
    ms_comp = timed(lambda: dash.dash_compact(mask, cu, rows=[Ht], rows_out=[H_next], pos_in=pos, tok_in=tok, want_idx=False, ws=cws), 10)
    status = dash.dash_check_status()
    clocks = sampler.stop(n_before) if rank == 0 else None

    def reduce_max(x):
        if world == 1:
            return x
        t = torch.tensor([x], dtype=torch.float64, device=dev)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        return float(t.item())

    t_step = reduce_max(sum(ms) / len(ms))
    t_e2e = reduce_max(sum(ms_e2e) / len(ms_e2e))
    t_attn = statistics.mean(ms_attn)
    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    peaks = measured_peaks()
    fl = attention_flops(w.cu.tolist(), sh.Hq, sh.D)
    ach = fl / (t_attn * 1e-3) / 1e12
    norm_bytes = T * (3 * sh.d * es + 5)
    comp_bytes = n_active * (2 * sh.d * es + 16) + T * 9
    h2d_bytes = H_host.numel() * es + (2 * T + S + 1) * 4
    d2h_bytes = 2 * T * sh.d * es + T * 4 + T + T * 4 + (S + 1) * 4
    out = {
        "metric": METRIC, "value": world * T / (t_step * 1e-3), "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": t_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16", "data": "synthetic",
        "config": {"workload": f"configs[1]: Qwen2.5-7B-shaped single layer, bf16, batch 1, seq {T}, threshold at 40th percentile "
                               f"({n_active} of {T} tokens stay active)", "tokens_per_step_per_gpu": T, "n_active_after": n_active,
                   "tau": tau, "l2": f"flushed between timed steps ({L2_FLUSH_BYTES >> 20} MiB write, then {L2_FLUSH_BYTES >> 20} MiB read)",
                   "status_word": status},
        "e2e": {"value": world * T / (t_e2e * 1e-3), "unit": UNIT, "ms_per_step": t_e2e, "h2d_bytes_per_step": h2d_bytes,
                "d2h_bytes_per_step": d2h_bytes},
        "gpu_launches": 6 * args.steps,
        "gpu_launches_note": "per step: rmsnorm, rope, attention, delta_norm(+residual+threshold), scatter, compact "
                             "(+2 cuBLASLt GEMMs and 1 memset that are not this library's kernels)",
        "clocks": clocks,
        "roofline": {"kernel": "attention_kernel<128> (dash_varlen_attention)", "bound": "tensor", "achieved": ach,
                     "peak": peaks["bf16_tflops"], "unit": "TFLOP/s", "frac": ach / peaks["bf16_tflops"], "peak_source": peaks["source"],
                     "frac_of_nominal_2250": ach / 2250.0, "ms_per_launch": t_attn, "flops_per_launch": fl, "traffic": None},
        "hbm_kernels": {
            "delta_norm_fused": {"ms": statistics.mean(ms_norm), "GBps": norm_bytes / (statistics.mean(ms_norm) * 1e-3) / 1e9,
                                 "frac": norm_bytes / (statistics.mean(ms_norm) * 1e-3) / 1e9 / peaks["hbm_gbs"], "bytes": norm_bytes},
            "compact": {"ms": statistics.mean(ms_comp), "GBps": comp_bytes / (statistics.mean(ms_comp) * 1e-3) / 1e9,
                        "frac": comp_bytes / (statistics.mean(ms_comp) * 1e-3) / 1e9 / peaks["hbm_gbs"], "bytes": comp_bytes},
            "peak_GBps": peaks["hbm_gbs"], "l2": "flushed"},
        "wall_s_timed_region": wall,
    }
    if world == 1 and not args.no_cpu_baseline:
        out["cpu_baseline"] = cpu_baseline(T, budget_s=args.cpu_budget)
    print(json.dumps(out))
    if world > 1:
        dist.destroy_process_group()


# ------------------------------------------------------------------- CPU oracle arm
def cpu_baseline(T: int, budget_s: float = 20.0, seed: int = 1):
    """Times the CPU oracle, as it stands, on a bounded sample of the same workload and scales to tokens/s.

    Sample: the O(n d^2) steps (RMSNorm, projections, rotary embedding, output projection, score, halting rule,
    scatter, compaction) on the first m tokens, scaled by n/m; the brute-force attention on q seeded query rows
    (all heads), scaled by the exact (query, key) pair count."""
    import numpy as np
    from oracle import dash_oracle as oc
    w = wl.config2(T=T, seed=seed)
    sh, W = w.shape, w.weights[0]
    m = min(T, 1024)
    Hm = w.tensors["H"][:m]
    cu_m = np.array([0, m], dtype=np.int32)
    pos_m = np.arange(m)
    t0 = time.perf_counter()
    Hn = oc.rmsnorm(Hm, W["rms_w"], sh.rms_eps)
    Q = oc.rope((Hn @ oc.f64(W["Wq"])).reshape(m, sh.Hq, sh.D), pos_m, sh.rope_base)
    Kk = oc.rope((Hn @ oc.f64(W["Wk"])).reshape(m, sh.Hkv, sh.D), pos_m, sh.rope_base)
    V = (Hn @ oc.f64(W["Wv"])).reshape(m, sh.Hkv, sh.D)
    U = np.zeros((m, sh.Hq * sh.D)) @ oc.f64(W["Wo"])
    r = oc.delta_norm(U + 1.0, Hm)
    mask = oc.select(r, cu_m, oc.THRESHOLD, tau=float(np.median(r)))
    Ht = oc.residual(Hm, U)
    oc.scatter(Ht, np.arange(m), None, 2, np.zeros_like(Ht))
    oc.compact(mask, cu_m, rows=[Ht], pos_in=pos_m)
    t_lin = (time.perf_counter() - t0) * (T / m)
    # attention: seeded rows of the full-length problem
    g = torch.Generator().manual_seed(seed)
    Qf = torch.randn(T, sh.Hq, sh.D, generator=g).to(torch.bfloat16)
    Kf = torch.randn(T, sh.Hkv, sh.D, generator=g).to(torch.bfloat16)
    Vf = torch.randn(T, sh.Hkv, sh.D, generator=g).to(torch.bfloat16)
    Qd, Kd, Vd = oc.f64(Qf), oc.f64(Kf), oc.f64(Vf)
    cu = np.array([0, T], dtype=np.int32)
    q, rows_done, pairs_done, t_attn = 8, 0, 0, 0.0
    while t_attn < 0.6 * budget_s and rows_done < T:
        rows = np.sort(torch.randint(0, T, (q,), generator=g).numpy())
        t1 = time.perf_counter()
        oc.attention(Qd, Kd, Vd, cu, rows=rows)
        t_attn += time.perf_counter() - t1
        rows_done += q
        pairs_done += int(np.sum(rows + 1))
        q = min(q * 2, 256)
    total_pairs = T * (T + 1) // 2
    t_attn_full = t_attn * total_pairs / max(pairs_done, 1)
    t_total = t_lin + t_attn_full
    return {"value": T / t_total, "unit": UNIT, "cores": oc.num_threads(), "kind": "oracle",
            "sample": f"O(n d^2) steps timed on the first {m} of {T} tokens and scaled by n/m ({t_lin:.1f} s scaled); brute-force "
                      f"attention timed on {rows_done} seeded query rows x {sh.Hq} heads ({t_attn:.1f} s) and scaled by the exact "
                      f"pair count ({t_attn_full:.0f} s extrapolated)",
            "est_seconds_per_step": t_total}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    vals = []
    per_step_budget = max(5.0, min(30.0, 120.0 / max(1, args.steps + args.warmup)))
    for i in range(args.warmup + args.steps):
        b = cpu_baseline(args.seq, budget_s=per_step_budget)
        if i >= args.warmup:
            vals.append(b)
    v = statistics.mean(x["value"] for x in vals)
    last = vals[-1]
    out = {"impl": "reference", "metric": METRIC, "value": v, "unit": UNIT, "n_gpus": int(os.environ.get("WORLD_SIZE", "1")),
           "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * args.seq / v, "higher_is_better": True,
           "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
           "config": {"workload": f"configs[1]: Qwen2.5-7B-shaped single layer, seq {args.seq} (CPU oracle, bounded sample per step)"},
           "cpu_baseline": {"value": v, "unit": UNIT, "cores": last["cores"], "kind": "oracle", "sample": last["sample"]},
           "e2e": {"value": v, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(out))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--seq", type=int, default=8192)
    ap.add_argument("--cpu-budget", type=float, default=20.0)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
