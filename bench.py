#!/usr/bin/env python
"""Benchmark of the selective-KV attention hot path.

A "step" is one planning step of the workload: one group store (the K/V of one group rewritten in
place in every layer, Sec. 3.2), the gather plan (built at the first layer, reused by the
others), and one `enl_attend` per layer (attention + fused per-group mass, plus the split merge
when KV splits are used).  Layers run sequentially on one stream, as in the planner.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload planner|long|long_scoring|concurrent|decode|tiny]
    python bench.py --impl reference      # the float64 CPU oracle, timed on the host cores

Prints ONE JSON line.  `value` is algorithmic TFLOP/s for prefill workloads (QK^T and PV, causal half
counted once, padding and masked work not credited) and algorithmic GB/s for the decode workload.
The default run (planner) also times a short leg of the decode workload and reports it under the key
`decode` (its own value in GB/s, roofline, e2e and clocks): the metric has a tensor half and an HBM half.
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
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np
import torch

FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}

# dram__bytes_read.sum + dram__bytes_write.sum per attention launch from the ncu capture summarised in
# profiles/ (same kernel, same workload shape); None until a capture exists for the workload.
NCU_TRAFFIC_BYTES = {
    "planner": 15.43e6 + 0.0,         # attn_kernel<128> incl. the in-kernel split merge, profiles/attn_kernel_planner.md
    "long": 45.18e6 + 1.80e6,         # attn_kernel<128>, one launch, profiles/attn_kernel_planner.md
    "decode": 140.67e6 + 4.71e6,      # decode_kernel<128>, profiles/decode_kernel_decode.md
}


def load_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            d = json.load(f)
        d["_source"] = "measured"
        return d
    d = dict(FALLBACK_PEAKS)
    d["_source"] = "fallback"
    return d


# ---- algorithmic work ---------------------------------------------------------------------------
def prefill_flops_per_layer(wl) -> float:
    f = 0.0
    for b in range(wl.batch):
        S, tn, nn = wl.selected_tokens(b), wl.n_q[b], wl.n_new[b]
        vis_new = tn * (nn - tn) + tn * (tn + 1) / 2.0
        f += 4.0 * wl.n_q_heads * wl.head_dim * (tn * S + vis_new)
    return f


def kv_bytes_per_token(wl) -> int:
    return 2 * wl.n_kv_heads * wl.head_dim * 2


def prefill_bytes_per_layer(wl) -> float:
    by = 0.0
    for b in range(wl.batch):
        S, tn, nn, G = wl.selected_tokens(b), wl.n_q[b], wl.n_new[b], len(wl.sel_local[b])
        by += (S + nn) * kv_bytes_per_token(wl) + 2 * tn * wl.n_q_heads * wl.head_dim * 2 + 4 * tn * wl.n_q_heads * (G + 1)
    return by


def decode_bytes_per_layer(wl, t: int) -> float:
    return (wl.selected_tokens(0) + t + 1) * kv_bytes_per_token(wl)


class ClockSampler:
    """nvidia-smi clocks and throttle reasons while the timed region runs."""

    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.rows, self._stop, self._t = index, [], threading.Event(), None

    def _run(self):
        while not self._stop.is_set():
            try:
                o = subprocess.run(["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                                    "-i", str(self.index)], capture_output=True, text=True, timeout=5).stdout.strip()
                if o:
                    self.rows.append([x.strip() for x in o.splitlines()[0].split(",")])
            except Exception:
                pass
            self._stop.wait(0.1)

    def __enter__(self):
        self._t = threading.Thread(target=self._run, daemon=True)
        self._t.start()
        return self

    def __exit__(self, *a):
        self._stop.set()
        self._t.join(timeout=10)

    def summary(self):
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            try:
                sm.append(float(r[0])); mx.append(float(r[1]))
            except Exception:
                continue
            for n, v in zip(names, r[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


# ---- the oracle arm (also the cpu_baseline leg) -------------------------------------------------
def oracle_sample(wl, seconds_target: float = 15.0):
    """Times the float64 oracle, as it stands, on a bounded sample of the workload: episode 0, all q heads,
    layer after layer (for a decode workload: step after step of layer 0) until about `seconds_target`
    seconds of CPU work have been done; a layer too long for that contributes evenly spaced query rows.
    Returns (value in the metric's unit, unit, seconds, dict)."""
    from oracle import enl_oracle as orc
    b = 0
    S = wl.selected_tokens(b)
    offs = wl.pool_offsets(b)
    work, dt, n_calls, n_rows = 0.0, 0.0, 0, 0
    layer, t_dec = 0, wl.decode_steps - 1 if wl.decode_steps else 0
    row_budget = None
    dec_layers = min(4, wl.n_layers)            # decode: a few layers' pools are drawn once, then step after step
    drawn = {}

    def draw(layer):
        if layer not in drawn:
            k, v = wl.pool_kv(layer, b, "cpu")
            drawn[layer] = ([k[offs[g]:offs[g + 1]] for g in wl.sel_local[b]],
                            [v[offs[g]:offs[g + 1]] for g in wl.sel_local[b]], wl.new_qkv(layer, "cpu"))
        return drawn[layer]

    while dt < seconds_target:
        if wl.decode_steps:
            if layer >= dec_layers:
                layer, t_dec = 0, t_dec - 1
            if t_dec < 0:
                break
        elif layer >= wl.n_layers:
            break
        ks, vs, (q, kn, vn) = draw(layer)
        if not wl.decode_steps:
            drawn.pop(layer)                     # prefill: one pass per layer, do not keep the pool
        if wl.decode_steps:
            q, kn, vn = q[t_dec:t_dec + 1], kn[:t_dec + 1], vn[:t_dec + 1]
            rows = [0]
        else:
            q, kn, vn = q[:wl.n_q[b]], kn[:wl.n_new[b]], vn[:wl.n_new[b]]
            n_q = q.shape[0]
            if row_budget is None:
                # calibrate on the most expensive row, then size one layer's share of the sample
                t0 = time.perf_counter()
                orc.attend_slots(wl.n_q_heads, wl.n_kv_heads, wl.head_dim, ks, vs, q, kn, vn, rows=[n_q - 1])
                row_budget = int(max(1, min(n_q, seconds_target / max(time.perf_counter() - t0, 1e-5))))
            rows = sorted(set(np.linspace(0, n_q - 1, row_budget).astype(int).tolist()))
        n_q, n_new = q.shape[0], kn.shape[0]
        t0 = time.perf_counter()
        orc.attend_slots(wl.n_q_heads, wl.n_kv_heads, wl.head_dim, ks, vs, q, kn, vn, rows=rows)
        dt += time.perf_counter() - t0
        n_calls += 1
        n_rows += len(rows)
        if wl.decode_steps:
            work += decode_bytes_per_layer(wl, t_dec)
        else:
            work += sum(4.0 * wl.n_q_heads * wl.head_dim * (S + (n_new - n_q) + r + 1) for r in rows)
        layer += 1
    if wl.decode_steps:
        value, unit = work / dt / 1e9, "GB/s"
        what = f"{n_calls} (layer, step) pairs: layers 0..{dec_layers - 1} of steps {max(t_dec, 0)}..{wl.decode_steps - 1}"
    else:
        value, unit = work / dt / 1e12, "TFLOP/s"
        what = f"layers 0..{n_calls - 1}, {n_rows} query rows in all"
    info = {"value": value, "unit": unit, "cores": orc.threads(), "kind": "oracle",
            "sample": f"episode 0, {what} x {wl.n_q_heads} heads, {S} cached keys, {dt:.1f} s of oracle time"}
    return value, unit, dt, info


def run_reference(args, wl, rank):
    if rank != 0:
        return
    times = []
    info = None
    for i in range(args.warmup + args.steps):
        value, unit, dt, info = oracle_sample(wl, seconds_target=max(1.0, min(15.0, 90.0 / (args.warmup + args.steps))))
        if i >= args.warmup:
            times.append((value, dt))
    value = float(np.mean([t[0] for t in times]))
    line = {"impl": "reference", "metric": metric_name(wl), "value": value, "unit": unit, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": float(np.mean([t[1] for t in times]) * 1e3),
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": wl.name, "note": "each step is a bounded sample of the workload (see cpu_baseline.sample)"},
            "cpu_baseline": dict(info, value=value),
            "e2e": {"value": value, "unit": unit, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


def metric_name(wl):
    if wl.decode_steps:
        return "selective-KV decode attention HBM GB/s (one decode step, all layers)"
    return "selective-KV attention TFLOP/s (one planning step, all layers)"


# ---- the CUDA arm --------------------------------------------------------------------------------
def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--layers", type=int, default=0, help="override the workload's layer count (profiling)")
    ap.add_argument("--impl", default="enl", choices=["enl", "reference"])
    ap.add_argument("--workload", default="planner")
    ap.add_argument("--split", type=int, default=0, help="KV splits (0 = library chooses)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-decode-leg", action="store_true", help="planner run without the decode leg")
    args = ap.parse_args()
    if args.warmup < 3 and args.impl == "enl":
        args.warmup = 3
    return args


MIN_TIMED_MS = 300.0        # the K timed steps are repeated until the timed region is at least this long (clock samples)


def run_cuda(args, workload, steps, warmup, want_e2e, want_cpu, rank, world, local):
    """One workload through the C ABI: returns the fields of its JSON line."""
    from paper_2510_18546_b200 import enl, synth
    from paper_2510_18546_b200.dist import max_over_ranks, barrier
    dev = torch.device(f"cuda:{local}")
    wl = synth.make(workload)
    if args.layers > 0:
        wl.n_layers = args.layers
    # weak scaling: every rank runs its own replica of the workload (episodes are independent; no
    # data-path collective).  Rank r draws its values from seed + r.
    wl.seed += rank

    L = wl.n_layers
    tq = wl.decode_steps if wl.decode_steps else int(sum(wl.n_q))
    cache = enl.enl_cache_create(L, wl.n_q_heads, wl.n_kv_heads, wl.head_dim, wl.n_groups, wl.pool_tokens,
                                 device=local, max_batch=wl.batch, max_q_tokens=max(tq, 1))
    stream = torch.cuda.current_stream(dev).cuda_stream
    store_src = []                       # per layer: (group id, K, V) rewritten every step
    for layer in range(L):
        for b in range(wl.batch):
            k, v = wl.pool_kv(layer, b, dev)
            offs = wl.pool_offsets(b)
            for g in range(len(wl.pool_lens[b])):
                enl.enl_group_store(cache, wl.group_base[b] + g, layer, k[offs[g]:offs[g + 1]], v[offs[g]:offs[g + 1]])
            if b == 0:
                g = int(wl.sel_local[0][0]) if len(wl.sel_local[0]) else 0
                store_src.append((wl.group_base[0] + g, k[offs[g]:offs[g + 1]].clone(), v[offs[g]:offs[g + 1]].clone()))
        torch.cuda.synchronize(dev)
    qs, kns, vns = [], [], []
    for layer in range(L):
        q, kn, vn = wl.new_qkv(layer, dev)
        qs.append(q); kns.append(kn); vns.append(vn)
    sel = wl.sel_ids()
    cs, cq, cn = wl.cu()
    multi = wl.batch > 1
    G = int(np.max(np.diff(cs))) if len(sel) else 0
    outs = [torch.empty(tq if not wl.decode_steps else 1, wl.n_q_heads, wl.head_dim, dtype=torch.bfloat16, device=dev)
            for _ in range(L)]
    masses = [torch.empty(outs[0].shape[0], wl.n_q_heads, G + 1, dtype=torch.float32, device=dev) for _ in range(L)]

    def attend(layer, q, kn, vn, out, mass, t=None):
        if wl.decode_steps:
            enl.enl_attend(cache, layer, sel, q[t:t + 1], kn, vn, out, mass, n_q=1, n_new=t + 1,
                           split_hint=args.split, stream=stream)
        else:
            enl.enl_attend(cache, layer, sel, q, kn, vn, out, mass, cu_sel=cs if multi else None,
                           cu_q=cq if multi else None, cu_new=cn if multi else None, split_hint=args.split,
                           stream=stream)

    store_ks, store_vs = [x[1] for x in store_src], [x[2] for x in store_src]
    store_pages = (int(store_ks[0].shape[0]) + 15) // 16
    store_launches = ((L + 63) // 64) * max(1, (store_pages + 63) // 64)

    def store_step():
        # the group's K/V of every layer rewritten in place by one launch (Sec. 3.2: a group's rows of all layers
        # come out of one prefill)
        enl.enl_group_store_all_layers(cache, store_src[0][0], store_ks, store_vs, stream=stream)

    def step(i, timed_events=None):
        t = (i % wl.decode_steps) if wl.decode_steps else None
        store_step()
        # the attention launches of a step run back to back (chained by programmatic dependent launch, as in
        # use); one pair of events around the L of them gives the kernel's average duration in that context
        if timed_events is not None:
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
        for layer in range(L):
            attend(layer, qs[layer], kns[layer], vns[layer], outs[layer], masses[layer], t)
        if timed_events is not None:
            e1.record()
            timed_events.append((e0, e1))
        return t

    for i in range(warmup):
        step(i)
    torch.cuda.synchronize(dev)
    plan = enl.enl_plan_inspect(cache)
    n_splits = plan["n_splits"]
    barrier()
    torch.cuda.synchronize(dev)
    # EXACTLY `steps` steps per timed region; a region shorter than MIN_TIMED_MS is repeated (same steps again) so
    # that the clock sampler sees the GPU under this load for long enough, and the regions are averaged
    evs, regions = [], []
    with ClockSampler(local) as clk:
        while True:
            e_beg, e_end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e_beg.record()
            for i in range(steps):
                step(warmup + i, evs)
            e_end.record()
            torch.cuda.synchronize(dev)
            regions.append(max_over_ranks(e_beg.elapsed_time(e_end)))      # every rank takes the same decision
            if sum(regions) >= MIN_TIMED_MS or len(regions) >= 50:
                break
    barrier()
    ms_step = float(np.mean(regions)) / steps
    status = enl.enl_cache_status(cache)

    # the dominant kernel's own duration, from the events inside the timed region: the attention launches of a step / L
    attend_ms = float(np.mean([a.elapsed_time(b) for a, b in evs])) / L

    if wl.decode_steps:
        ts = [(warmup + i) % wl.decode_steps for i in range(steps)]
        work_step = float(np.mean([decode_bytes_per_layer(wl, t) for t in ts])) * L
        value, unit, bound = work_step * world / (ms_step * 1e-3) / 1e9, "GB/s", "hbm"
        per_launch = work_step / L
        achieved = per_launch / (attend_ms * 1e-3) / 1e9
    else:
        work_step = prefill_flops_per_layer(wl) * L
        value, unit, bound = work_step * world / (ms_step * 1e-3) / 1e12, "TFLOP/s", "tensor"
        per_launch = work_step / L
        achieved = per_launch / (attend_ms * 1e-3) / 1e12
    peaks = load_peaks()
    clocks = clk.summary()
    if bound == "hbm":
        peak, which = peaks["hbm_gbs"], "copy bandwidth"
        fracs = {}
    else:
        # two measured denominators: the GEMM burst figure suits a short timed region at full clocks, the sustained
        # figure a region long enough to reach the power cap; `frac` takes the one that matches this run
        burst = sum(regions) < 1000.0 and "sw_power_cap" not in clocks["reasons"]
        peak = peaks["bf16_tflops"] if burst else peaks["bf16_tflops_sustained"]
        which = "burst bf16 GEMM" if burst else "sustained bf16 GEMM"
        fracs = {"frac_burst": achieved / peaks["bf16_tflops"], "frac_sustained": achieved / peaks["bf16_tflops_sustained"],
                 "peak_burst": peaks["bf16_tflops"], "peak_sustained": peaks["bf16_tflops_sustained"]}
    roofline = {"bound": bound, "achieved": achieved, "peak": peak, "unit": unit, "frac": achieved / peak, **fracs,
                "traffic": NCU_TRAFFIC_BYTES.get(wl.name),
                "peak_source": f"{peaks['_source']} ({which})",
                "kernel": (f"decode_kernel<{wl.head_dim}> (split merge fused)" if wl.decode_steps else
                           f"attn_kernel<{wl.head_dim}>" + (" + combine_kernel" if plan["merge_kind"] == 1 else
                                                            " (split merge by CTA pairs)" if plan["merge_kind"] == 2 else "")),
                "launch_ms": attend_ms,
                "algorithmic_per_launch": per_launch}

    # ---- end to end through the C ABI with host buffers ----
    e2e = None
    if want_e2e:
        hq = [x.cpu().pin_memory() for x in qs]
        hk = [x.cpu().pin_memory() for x in kns]
        hv = [x.cpu().pin_memory() for x in vns]
        ho = [torch.empty_like(o, device="cpu").pin_memory() for o in outs]
        hm = [torch.empty_like(m, device="cpu").pin_memory() for m in masses]
        # Two sets of device input buffers and two copy streams: the upload of layer l + 1 and the download of
        # layer l - 1 run while layer l computes (PCIe is full duplex); events order them against the stream the
        # library launches on.
        # A layer's q | k_new | v_new travel as one copy, and so do its out | mass: fewer, larger transfers and half
        # the host calls per layer (the C ABI takes plain pointers, so the tensors are views into the packed buffers).
        # Queuing a whole step's uploads, attends and downloads at once was slower: the link carries about 65 GB/s
        # in both directions together, and the per-layer interleaving keeps both directions busy all the time.
        def packed(parts, device, pin=False):
            sizes = [(x.nbytes + 255) // 256 * 256 for x in parts]
            buf = torch.empty(sum(sizes), dtype=torch.uint8, device=device)
            if pin:
                buf = buf.pin_memory()
            views, off = [], 0
            for x, n in zip(parts, sizes):
                views.append(buf[off:off + x.nbytes].view(x.dtype).view(x.shape))
                off += n
            return buf, views
        dbuf, hin, dout, hout = [], [], [], []
        if not wl.decode_steps:
            dbuf = [packed((qs[0], kns[0], vns[0]), dev) for _ in range(2)]
        for layer in range(L):
            if not wl.decode_steps:
                hb, hv3 = packed((qs[layer], kns[layer], vns[layer]), "cpu", pin=True)
                for dst, src in zip(hv3, (hq[layer], hk[layer], hv[layer])):
                    dst.copy_(src)
                hin.append(hb)
            dout.append(packed((outs[layer], masses[layer]), dev))
            hout.append(torch.empty(dout[-1][0].numel(), dtype=torch.uint8).pin_memory())
        main = torch.cuda.current_stream(dev)
        s_up, s_dn = torch.cuda.Stream(dev), torch.cuda.Stream(dev)
        ev_free = [None, None]

        def e2e_step(i):
            t = (i % wl.decode_steps) if wl.decode_steps else None
            bi = bo = 0
            store_step()
            for layer in range(L):
                if wl.decode_steps:
                    # the step's inputs: one query row and the new token's K/V row, appended to the
                    # caller-owned device buffer that already holds the rows of earlier steps
                    qs[layer][t:t + 1].copy_(hq[layer][t:t + 1], non_blocking=True)
                    kns[layer][t:t + 1].copy_(hk[layer][t:t + 1], non_blocking=True)
                    vns[layer][t:t + 1].copy_(hv[layer][t:t + 1], non_blocking=True)
                    bi += hq[layer][t:t + 1].nbytes + 2 * hk[layer][t:t + 1].nbytes
                    attend(layer, qs[layer], kns[layer], vns[layer], dout[layer][1][0], dout[layer][1][1], t)
                else:
                    din, (dq, dk, dv) = dbuf[layer & 1]
                    with torch.cuda.stream(s_up):
                        if ev_free[layer & 1] is not None:
                            s_up.wait_event(ev_free[layer & 1])      # the attend that last read this buffer set
                        din.copy_(hin[layer], non_blocking=True)
                        ev_up = torch.cuda.Event()
                        ev_up.record(s_up)
                    main.wait_event(ev_up)
                    bi += hq[layer].nbytes + hk[layer].nbytes + hv[layer].nbytes
                    attend(layer, dq, dk, dv, dout[layer][1][0], dout[layer][1][1], t)
                ev_done = torch.cuda.Event()
                ev_done.record(main)
                ev_free[layer & 1] = ev_done
                with torch.cuda.stream(s_dn):
                    s_dn.wait_event(ev_done)
                    hout[layer].copy_(dout[layer][0], non_blocking=True)
                bo += ho[layer].nbytes + hm[layer].nbytes
            ev_last = torch.cuda.Event()
            ev_last.record(s_dn)
            main.wait_event(ev_last)                                 # the step ends when its results are on the host
            return bi, bo

        for i in range(3):
            e2e_step(i)
        torch.cuda.synchronize(dev)
        barrier()
        n_e2e = max(3, min(steps, 10))
        a, b_ = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for i in range(n_e2e):
            bi, bo = e2e_step(warmup + i)
        b_.record()
        torch.cuda.synchronize(dev)
        barrier()
        e2e_ms = max_over_ranks(a.elapsed_time(b_)) / n_e2e
        scale = 1e9 if wl.decode_steps else 1e12
        e2e = {"value": work_step * world / (e2e_ms * 1e-3) / scale, "unit": unit, "ms_per_step": e2e_ms,
               "h2d_bytes_per_step": int(bi), "d2h_bytes_per_step": int(bo), "steps": n_e2e}

    # the clustering reduce over the scoring pass's masses (Sec. 3.3): objects = spans of 32 new tokens
    cluster = None
    if wl.name == "long_scoring":
        n_groups = G
        obj_off = list(range(0, tq + 1, 32))
        avg = torch.empty(len(obj_off) - 1, n_groups, dtype=torch.float32, device=dev)
        asg = torch.empty(len(obj_off) - 1, dtype=torch.int32, device=dev)
        for _ in range(3):
            enl.enl_cluster_assign(masses, obj_off, n_groups, 1.0 / n_groups, avg, asg, stream=stream)
        ca, cb = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        ca.record()
        for _ in range(20):
            enl.enl_cluster_assign(masses, obj_off, n_groups, 1.0 / n_groups, avg, asg, stream=stream)
        cb.record()
        torch.cuda.synchronize(dev)
        c_ms = ca.elapsed_time(cb) / 20
        c_bytes = float(L) * tq * wl.n_q_heads * n_groups * 4
        cluster = {"ms": c_ms, "algorithmic_bytes": c_bytes, "achieved_gbs": c_bytes / (c_ms * 1e-3) / 1e9,
                   "frac_of_hbm_peak": c_bytes / (c_ms * 1e-3) / 1e9 / load_peaks()["hbm_gbs"],
                   "objects": len(obj_off) - 1, "groups": n_groups, "layers": L,
                   "note": "enl_cluster_assign over the masses of the scoring layers; masses (%.0f MB) exceed L2" % (c_bytes / 1e6)}
        # the same decision with the sums taken inside the attention kernel (group_mass_sum): the per-row masses of
        # all layers go through ONE reused buffer and are never read back
        sums = torch.zeros(len(obj_off) - 1, G + 1, dtype=torch.float32, device=dev)

        def fused_pass():
            sums.zero_()
            for layer in range(L):
                enl.enl_attend(cache, layer, sel, qs[layer], kns[layer], vns[layer], outs[layer], masses[0],
                               group_mass_sum=sums, obj_off=obj_off, stream=stream)
            enl.enl_cluster_assign_sums(sums, obj_off, n_groups, wl.n_q_heads, L, 1.0 / n_groups, avg, asg, stream=stream)

        def plain_pass():
            for layer in range(L):
                attend(layer, qs[layer], kns[layer], vns[layer], outs[layer], masses[layer])
            enl.enl_cluster_assign(masses, obj_off, n_groups, 1.0 / n_groups, avg, asg, stream=stream)

        times = {}
        for name_, fn in (("plain", plain_pass), ("fused", fused_pass)):
            for _ in range(2):
                fn()
            fa, fb = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            fa.record()
            for _ in range(5):
                fn()
            fb.record()
            torch.cuda.synchronize(dev)
            times[name_] = fa.elapsed_time(fb) / 5
        cluster["scoring_pass_ms"] = {"attends_then_cluster_assign": times["plain"], "attends_with_mass_sums": times["fused"]}
        cluster["mass_bytes_kept_per_layer"] = {"plain": float(tq) * wl.n_q_heads * (G + 1) * 4, "fused": 0.0,
                                                "fused_note": "one reused buffer of that size + %.1f MB of sums" % (sums.nbytes / 1e6)}

    # the slow tier (Sec. 3.2): push the step's selected groups out to pinned host memory, time loading them back
    tier = None
    if wl.name == "planner" and want_e2e:
        enl.enl_tier_enable(cache, wl.pool_tokens)
        ids = [int(x) for x in sel]
        t_ms, moved = [], 0
        for _ in range(3):
            for gid in ids:
                enl.enl_group_evict(cache, gid, stream=stream)
            torch.cuda.synchronize(dev)
            ta, tb = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            ta.record()
            st_ = enl.enl_step_prepare(cache, ids, stream=stream)
            tb.record()
            torch.cuda.synchronize(dev)
            t_ms.append(ta.elapsed_time(tb))
            moved = st_["bytes_h2d"]
        again = enl.enl_step_prepare(cache, ids, stream=stream)
        tier = {"load_ms": float(np.median(t_ms)), "bytes_h2d": int(moved), "gbs": moved / (np.median(t_ms) * 1e-3) / 1e9,
                "groups": len(ids), "layers": L, "hit_rate_when_repeated": again["n_hit"] / max(len(ids), 1),
                "note": "enl_step_prepare after evicting the step's selected groups: one kernel copies their pages "
                        "of all layers from the pinned host pool"}

    cpu = None
    if rank == 0 and world == 1 and want_cpu:
        wl0 = synth.make(workload)
        _, _, _, cpu = oracle_sample(wl0)

    # attention (+ merge kernel when the splits go through the scratch buffer) + page scatter
    launches_per_step = L * (1 + (1 if plan["merge_kind"] == 1 else 0)) + store_launches
    enl.enl_cache_free(cache)
    del qs, kns, vns, outs, masses, store_src
    torch.cuda.empty_cache()
    if True:
        line = {"metric": metric_name(wl), "value": value, "unit": unit, "n_gpus": world, "steps": steps,
                "warmup": warmup, "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
                "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
                "config": {"workload": wl.name, "layers": L, "q_heads": wl.n_q_heads, "kv_heads": wl.n_kv_heads,
                           "head_dim": wl.head_dim, "batch": wl.batch, "pool_groups": wl.n_groups,
                           "selected_groups": int(len(sel)), "selected_tokens": int(sum(wl.selected_tokens(b) for b in range(wl.batch))),
                           "new_tokens": int(sum(wl.n_new)) if not wl.decode_steps else 1,
                           "kv_splits": n_splits, "parallelism": f"replicas x{world}", "timed_regions": len(regions),
                           "l2": "inputs larger than L2: every layer of a step reads its own pages and tensors"},
                "roofline": roofline, "cpu_baseline": cpu, "e2e": e2e,
                "gpu_launches": launches_per_step * steps * len(regions),
                "clocks": dict(clocks, sm_cycles_per_step=(ms_step * 1e3 * clocks["sm_mhz"]) if clocks["sm_mhz"] else None),
                "status": "ok" if status == 0 else enl.strerror(status), "cluster_reduce": cluster, "slow_tier": tier,
                "fraction_of_nominal": achieved / (8000.0 if bound == "hbm" else 2250.0)}
        return line


def main():
    args = parse_args()
    from paper_2510_18546_b200 import synth
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if args.impl == "reference":
        wl = synth.make(args.workload)
        if args.layers > 0:
            wl.n_layers = args.layers
        run_reference(args, wl, rank)
        return
    from paper_2510_18546_b200.dist import init_process_group
    torch.cuda.set_device(torch.device(f"cuda:{local}"))
    init_process_group(world, rank, backend="nccl")
    line = run_cuda(args, args.workload, args.steps, args.warmup, not args.no_e2e, not args.no_cpu_baseline, rank, world, local)
    if args.workload == "planner" and not args.no_decode_leg:
        # the HBM half of the metric: a short leg of the decode workload (one query token per step over ~33k cached keys)
        dec = run_cuda(args, "decode", max(3, min(args.steps, 40)), 3, not args.no_e2e, False, rank, world, local)
        line["decode"] = {k: dec[k] for k in ("metric", "value", "unit", "steps", "warmup", "ms_per_step", "config", "roofline",
                                              "e2e", "gpu_launches", "clocks", "status", "fraction_of_nominal")}
        line["gpu_launches"] += dec["gpu_launches"]
    if rank == 0:
        print(json.dumps(line), flush=True)


if __name__ == "__main__":
    main()
