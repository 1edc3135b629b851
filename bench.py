#!/usr/bin/env python
"""Benchmark of the D2O hot path on B200.

One bench *step* is one pass of the whole path over one synthetic batch:
  per layer: column sums + density (d2o_layer_stats) -> budgets (d2o_layer_budgets)
  -> all layers: eviction + similarity + merge (d2o_prefill_compress_layers)
  -> the decode loop (`decode_steps` tokens, all layers per step, through d2o_decode_steps: the inputs
     of every step are resident, which is what that entry point asks for).
The headline value is compressed decode steps/s (tokens/s = steps/s x sequences); the
prompt-stage times are reported beside it, and so is the decode loop with one d2o_decode_step call
per token.  Inputs are generated once, seeded, and are resident in HBM before the timed region; the
`e2e` leg repeats the decode loop through the host-buffer entry points with pinned host q/k/v/out,
every step's bytes crossing inside the timed region.  `--single-step-calls` runs every leg through the
one-call-per-layer / one-call-per-token entry points instead.

The default workload is the Llama-3-8B-shaped config (16 sequences, prompt 8192, 1.7 GB of cache
streamed per decode step).  `per_config` holds a shorter measurement of the other configs (fewer
passes and decode steps, prompts generated layer by layer so that the largest batch fits), each
also with the upper clamp of the layer budgets removed.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config cfg2] [--impl reference]
"""
from __future__ import annotations

import argparse
import dataclasses
import json
import os
import socket
import statistics
import subprocess
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import torch  # noqa: E402

from paper_2406_13035_b200 import workloads as W  # noqa: E402

METRIC = "compressed decode steps/s (x sequences = tokens/s); prefill-compress ms; fraction of HBM roofline"
NOMINAL_HBM_GBS = 8000.0          # the figure the metric quotes; the measured copy bandwidth is the other denominator
# dram__bytes_read.sum + dram__bytes_write.sum of the decode_kernel launches of one step under ncu (the full-size
# workload, counters that take one pass), divided by the algorithmic bytes of that step, per workload the counters were
# taken on (None: not captured for this kernel build)
DECODE_TRAFFIC_RATIO = {"cfg1": 1.005, "cfg2": 1.040}
NO_CHAIN = False                  # --single-step-calls: one d2o_decode_step call per token in the timed passes too


def parse():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--config", default="cfg2")
    ap.add_argument("--decode-steps", type=int, default=0, help="override the config's decode steps")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--stages", type=int, default=0, help="stages of the decode kernel's ring (0 = auto)")
    ap.add_argument("--decode-warps", type=int, default=0, help="consumer warps per decode CTA (0 = auto)")
    ap.add_argument("--smem-rows", type=int, default=0,
                    help="decode kernel: rows of a slice with their logits in shared memory (0 = auto)")
    ap.add_argument("--long-pairs", type=int, default=0,
                    help="decode: (layer, sequence) pairs in the long-slice launch (0 = auto, -1 = never)")
    ap.add_argument("--no-l2-hints", action="store_true", help="decode kernel: copies without L2 eviction hints")
    ap.add_argument("--ffma-similarity", action="store_true", help="prompt-stage similarity on the FFMA kernel")
    ap.add_argument("--ffma-stats", action="store_true", help="column sums of the prompt attention on the FFMA kernels")
    ap.add_argument("--full-cache", action="store_true", help="also time the uncompressed decode-attention kernel")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-per-config", action="store_true", help="skip the shorter measurements of the other configs")
    ap.add_argument("--unclamped", action="store_true", help="run the main config without the upper budget clamp")
    ap.add_argument("--layers-per-call", type=int, default=0)
    ap.add_argument("--single-step-calls", action="store_true",
                    help="decode with one d2o_decode_step call per token instead of d2o_decode_steps")
    ap.add_argument("--layers", type=int, default=0, help="override the number of layers (profiling captures)")
    ap.add_argument("--batch", type=int, default=0, help="override the number of sequences (the serving sweep of config 4)")
    return ap.parse_args()


# --------------------------------------------------------------------------------------- clocks
class ClockSampler:
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.proc = index, None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                          "-lms", "200", "-i", str(self.index)], stdout=subprocess.PIPE,
                                         stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None

    def stop(self):
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
            out, _ = self.proc.communicate()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in out.strip().splitlines():
            f = [x.strip() for x in line.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1])); mx.append(float(f[2]))
            except ValueError:
                continue
            for n, v in zip(names, f[5:9]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


# --------------------------------------------------------------------------------------- helpers
def max_over_ranks(values, world: int, device):
    """Element-wise maximum of a list of per-rank timings over all ranks (the replicas share no data path: this is
    the only exchange).  Returns the list unchanged for a single rank."""
    if world <= 1:
        return [float(v) for v in values]
    t = torch.tensor([float(v) for v in values], device=device, dtype=torch.float64)
    torch.distributed.all_reduce(t, op=torch.distributed.ReduceOp.MAX)
    return t.tolist()


def whole_job_rate(per_gpu_units: float, world: int, ms: float) -> float:
    """Units all ranks processed per second, given the slowest rank's time."""
    return world * per_gpu_units / (ms * 1e-3)


def workload_string(wl: W.Workload, nd: int) -> str:
    return (f"{wl.name}: L={wl.n_layers} Hq={wl.n_q_heads} Hkv={wl.n_kv_heads} d={wl.d_head} {wl.dtype} "
            f"B={wl.batch} P={wl.prompt_len} rho={wl.rho} max_budget={wl.max_budget or wl.prompt_len} decode_steps={nd}")


def algorithmic_decode_bytes(wl: W.Workload, rows_held: float) -> float:
    """Bytes one decode step over all layers must move: K_c and V_c rows once, per-row score/pos/norm read (12 B)
    and score write (4 B), q/k/v in and out once.  `rows_held` = cache rows summed over (sequence, layer, KV
    head)."""
    e = 4 if wl.dtype == "f32" else 2
    rows = float(rows_held)
    per_row = 2 * wl.d_head * e + 16
    io = wl.n_layers * wl.batch * (2 * wl.n_q_heads + 2 * wl.n_kv_heads) * wl.d_head * e
    return rows * per_row + io


def load_peaks():
    pk_path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    return json.load(open(pk_path)) if os.path.exists(pk_path) else {}


def make_context(B, wl: W.Workload, nd: int, device, args):
    cfg = B.make_config(n_layers=wl.n_layers, batch=wl.batch, n_q_heads=wl.n_q_heads, n_kv_heads=wl.n_kv_heads,
                        d_head=wl.d_head, dtype=wl.dtype, prompt_len=wl.prompt_len, max_new_tokens=nd, rho=wl.rho,
                        n_sink=wl.n_sink, window=wl.window, nm_ratio=wl.nm_ratio, beta=wl.beta,
                        density_temp=wl.density_temp, min_budget=wl.min_budget, max_budget=wl.max_budget)
    ctx = B.D2OContext(cfg, device)
    if (args.stages or args.no_l2_hints or args.ffma_similarity or args.ffma_stats or args.decode_warps
            or args.smem_rows or args.long_pairs):
        ctx.d2o_set_tuning(args.stages, 0 if args.no_l2_hints else 1, 1 if args.ffma_similarity else 0,
                           1 if args.ffma_stats else 0, args.decode_warps, args.smem_rows, args.long_pairs)
    return ctx


def decode_inputs(streams, nd: int):
    dq, dk, dv = [], [], []
    for _ in range(nd):
        qs, ks, vs = zip(*[s.decode() for s in streams])
        dq.append(torch.stack(qs)); dk.append(torch.stack(ks)); dv.append(torch.stack(vs))
    return torch.stack(dq), torch.stack(dk), torch.stack(dv)


def ev():
    return torch.cuda.Event(enable_timing=True)


def kernels_per_pass(wl: W.Workload) -> int:
    """Launches of the library's kernels in the prompt stage of one pass: 2 attention sweeps + density per layer,
    budgets once, and select, gather, similarity, neighbour reduce (16-bit only), segments, merge per layer."""
    L = wl.n_layers
    return L * 3 + 1 + L * (5 if wl.dtype == "f32" else 6)


def roofline_of_decode(wl, budgets, nd, decode_ms, launches_per_step, peaks):
    """`budgets`: host int tensor [B, L, Hkv]."""
    P = wl.prompt_len
    rows = 0.0
    for s in range(nd):
        rows += float(torch.clamp(budgets.double(), max=P + s).sum())          # cache rows held before step s
    bytes_per_step = algorithmic_decode_bytes(wl, rows / nd)
    step_ms = decode_ms / nd
    peak = float(peaks.get("hbm_gbs", 6650.0))
    achieved = bytes_per_step / (step_ms * 1e-3) / 1e9
    return bytes_per_step, achieved, peak


# --------------------------------------------------------------------------------------- the measured path
def measure_resident(ctx, wl, prompts, dq, dk, dv, nd, lpc, warmup, steps, world, device, want_steps=True):
    """`steps` timed passes of the whole path with every input resident; returns per-phase milliseconds (mean over
    the passes), the budgets, the launch count, and the decode-step percentiles of one extra pass."""
    L = wl.n_layers
    # all layers per call: the decode steps of a pass go through the multi-step entry point (their inputs are all
    # resident, which is what it asks for); the extra pass below steps call by call
    chain = (lpc == L) and not NO_CHAIN
    dout = torch.empty_like(dq) if chain else torch.empty_like(dq[0])
    launches = {"n": 0, "decode_seen": ctx.d2o_get_stats().decode_launches}

    def one_pass(timed: bool, step_events=None):
        e = [ev() for _ in range(5)]
        e[0].record()
        if NO_CHAIN:
            for l in range(L):
                ctx.d2o_layer_stats(l, prompts[l][0], prompts[l][1])
        else:
            ctx.d2o_layer_stats_layers(0, L, [p[0] for p in prompts], [p[1] for p in prompts])
        e[1].record()
        budgets = ctx.d2o_layer_budgets()
        e[2].record()
        if NO_CHAIN:
            for l in range(L):
                ctx.d2o_prefill_compress(l, prompts[l][1], prompts[l][2])
        else:                                             # every layer's K and V are resident: one call
            ctx.d2o_prefill_compress_layers(0, L, [p[1] for p in prompts], [p[2] for p in prompts])
        e[3].record()
        if chain and step_events is None:
            ctx.d2o_decode_steps(0, L, nd, dq, dk, dv, dout)
        else:
            o = dout[0] if chain else dout
            for s in range(nd):
                for l0 in range(0, L, lpc):
                    l1 = min(L, l0 + lpc)
                    ctx.d2o_decode_step(l0, l1, dq[s, l0:l1], dk[s, l0:l1], dv[s, l0:l1], o[l0:l1])
                if step_events is not None:
                    step_events[s + 1].record()
        e[4].record()
        dl = ctx.d2o_get_stats().decode_launches      # the library counts its decode launches (a step may take two)
        if timed:
            launches["n"] += kernels_per_pass(wl) + (dl - launches["decode_seen"])
        launches["decode_seen"] = dl
        return e, budgets

    def sync_all():
        torch.cuda.synchronize()
        if world > 1:
            torch.distributed.barrier()

    for _ in range(warmup):
        one_pass(False)
    sync_all()
    sampler = ClockSampler(torch.cuda.current_device())
    sampler.start()
    t_wall = time.perf_counter()
    passes = []
    sync_all()
    for _ in range(steps):
        passes.append(one_pass(True))
    sync_all()
    t_wall = time.perf_counter() - t_wall
    clocks = sampler.stop()
    step_pct = None
    if want_steps:
        # one more pass, outside the timed ones, with an event after every decode step: the spread of the step times
        step_ev = [ev() for _ in range(nd + 1)]
        extra = one_pass(False, step_ev)
        step_ev[0] = extra[0][3]
        torch.cuda.synchronize()
        step_us = sorted(step_ev[i].elapsed_time(step_ev[i + 1]) * 1e3 for i in range(nd))
        step_pct = {"p50": round(step_us[nd // 2], 2), "p99": round(step_us[min(nd - 1, (nd * 99) // 100)], 2),
                    "max": round(step_us[-1], 2), "mean": round(step_ev[0].elapsed_time(step_ev[nd]) * 1e3 / nd, 2),
                    "entry_point": "d2o_decode_step, one call per token (an event after every call)"}
    seg = [[p[0][i].elapsed_time(p[0][i + 1]) for i in range(4)] for p in passes]          # ms
    means = [statistics.mean(s[i] for s in seg) for i in range(4)]
    means.append(sum(means))
    stats_ms, budget_ms, compress_ms, decode_ms, pass_ms = max_over_ranks(means, world, device)
    return dict(stats_ms=stats_ms, budget_ms=budget_ms, compress_ms=compress_ms, decode_ms=decode_ms, pass_ms=pass_ms,
                budgets=passes[-1][1], launches=launches["n"], clocks=clocks, wall_s=t_wall, step_pct=step_pct,
                chained=chain)


def measure_streamed(B, wl, nd, warmup, steps, device, args, with_lse=False):
    """The same path with the prompt tensors of one layer at a time on the device (regenerated from their seeds for
    the compression stage), so that batches whose prompts do not fit all at once can be measured.  Only the library
    calls are inside the event pairs.  Returns the same per-phase means as measure_resident."""
    L = wl.n_layers
    chain = not NO_CHAIN
    ctx = make_context(B, wl, 2 * nd if chain else nd, device, args)
    acc = []
    single_ms = []
    lse_ms = None
    for it in range(warmup + steps):
        t_stats = t_comp = 0.0
        pend = []
        sgroup = 1 if NO_CHAIN else 2                     # layers whose Q and K are on the device together
        for l0 in range(0, L, sgroup):
            l1 = min(L, l0 + sgroup)
            Qs, Ks = [], []
            for l in range(l0, l1):
                Q, K, _ = W.LayerStream(wl, l, device).prompt()
                Qs.append(Q); Ks.append(K)
            a, b = ev(), ev()
            a.record()
            if sgroup == 1:
                ctx.d2o_layer_stats(l0, Qs[0], Ks[0])
            else:
                ctx.d2o_layer_stats_layers(l0, l1, Qs, Ks)
            b.record()
            pend.append((0, a, b))
            del Qs, Ks, Q, K
        a, b = ev(), ev()
        a.record(); budgets = ctx.d2o_layer_budgets(); b.record()
        pend.append((1, a, b))
        streams = []
        group = 1 if NO_CHAIN else 4                      # layers whose K and V are on the device together
        for l0 in range(0, L, group):
            l1 = min(L, l0 + group)
            Ks, Vs = [], []
            for l in range(l0, l1):
                s = W.LayerStream(wl, l, device)
                _, K, V = s.prompt()
                Ks.append(K); Vs.append(V)
                streams.append(s)
            a, b = ev(), ev()
            a.record()
            if group == 1:
                ctx.d2o_prefill_compress(l0, Ks[0], Vs[0])
            else:
                ctx.d2o_prefill_compress_layers(l0, l1, Ks, Vs)
            b.record()
            pend.append((2, a, b))
            del Ks, Vs, K, V
        dq, dk, dv = decode_inputs(streams, nd)
        dout = torch.empty_like(dq) if chain else torch.empty_like(dq[0])
        a, b = ev(), ev()
        a.record()
        if chain:
            ctx.d2o_decode_steps(0, L, nd, dq, dk, dv, dout)
        else:
            for s in range(nd):
                ctx.d2o_decode_step(0, L, dq[s], dk[s], dv[s], dout)
        b.record()
        pend.append((3, a, b))
        if chain:
            # the same number of further tokens, one call per token (same inputs again: the sizes are what matters)
            a2, b2 = ev(), ev()
            a2.record()
            for s in range(nd):
                ctx.d2o_decode_step(0, L, dq[s], dk[s], dv[s], dout[0])
            b2.record()
        torch.cuda.synchronize()
        if chain and it >= warmup:
            single_ms.append(a2.elapsed_time(b2))
        tot = [0.0, 0.0, 0.0, 0.0]
        for k, a, b in pend:
            tot[k] += a.elapsed_time(b)
        if it >= warmup:
            acc.append(tot)
        del dq, dk, dv, dout, streams
    st = ctx.d2o_get_stats()
    if st.error_word != 0:
        raise RuntimeError(f"device error word {st.error_word} ({st.error_detail:#x})")
    if with_lse:
        # column sums with the row normalisers supplied by the caller (what a fused prefill attention kernel hands
        # over): one sweep instead of two.  Timed on layer 0 and scaled to all layers.
        Q, K, _ = W.LayerStream(wl, 0, device).prompt()
        lse = torch.zeros(wl.batch, wl.n_q_heads, wl.prompt_len, dtype=torch.float32, device=device)
        ctx.d2o_layer_stats(0, Q, K, lse)
        a, b = ev(), ev()
        a.record()
        for _ in range(3):
            ctx.d2o_layer_stats(0, Q, K, lse)
        b.record()
        torch.cuda.synchronize()
        lse_ms = a.elapsed_time(b) / 3 * L
        del Q, K, lse
    ctx.close()
    del ctx
    torch.cuda.empty_cache()
    m = [statistics.mean(x[i] for x in acc) for i in range(4)]
    return dict(stats_ms=m[0], budget_ms=m[1], compress_ms=m[2], decode_ms=m[3], pass_ms=sum(m), budgets=budgets,
                stats_with_lse_ms=lse_ms, merges_discards=[int(st.merges), int(st.discards)],
                decode_single_calls_ms=statistics.mean(single_ms) if single_ms else None)


def full_cache_decode(B, wl, nd, device, peak, world=1):
    """Decode attention over the uncompressed cache of prompt + generated tokens (all layers per call)."""
    L, P = wl.n_layers, wl.prompt_len
    n_sl = L * wl.batch * wl.n_kv_heads
    nf = min(nd, 32)
    cap = P + nf
    td = W.TORCH_DTYPES[wl.dtype]
    g = torch.Generator(device=device).manual_seed(wl.seed + 99)
    kc = torch.empty(n_sl, cap, wl.d_head, device=device, dtype=td)
    vc = torch.empty(n_sl, cap, wl.d_head, device=device, dtype=td)
    step = max(1, n_sl // 64)
    for i in range(0, n_sl, step):                       # filled piecewise: no fp32 copy of the whole cache
        kc[i:i + step] = torch.randn(min(step, n_sl - i), cap, wl.d_head, generator=g, device=device).to(td)
        vc[i:i + step] = torch.randn(min(step, n_sl - i), cap, wl.d_head, generator=g, device=device).to(td)
    fq = (2 * torch.randn(nf, n_sl, wl.group, wl.d_head, generator=g, device=device)).to(td)
    fk = torch.randn(nf, n_sl, wl.d_head, generator=g, device=device).to(td)
    fv = torch.randn(nf, n_sl, wl.d_head, generator=g, device=device).to(td)
    fo = torch.empty_like(fq[0])
    for s in range(min(3, nf)):
        B.d2o_full_decode_step(kc, vc, P + s, fq[s], fk[s], fv[s], fo)
    torch.cuda.synchronize()
    e0, e1 = ev(), ev()
    e0.record()
    for s in range(nf):
        B.d2o_full_decode_step(kc, vc, P + s, fq[s], fk[s], fv[s], fo)
    e1.record()
    torch.cuda.synchronize()
    fms = max_over_ranks([e0.elapsed_time(e1)], world, device)[0]
    esz = 4 if wl.dtype == "f32" else 2
    fbytes = n_sl * (P + (nf - 1) / 2.0 + 1) * 2 * wl.d_head * esz
    del kc, vc
    torch.cuda.empty_cache()
    return {"kernel": "full_decode_kernel", "us_per_step": round(fms * 1e3 / nf, 2), "steps": nf,
            "cache_rows": [P, P + nf], "achieved_GBps": round(fbytes / (fms * 1e-3 / nf) / 1e9, 1),
            "frac_of_hbm_peak": round(fbytes / (fms * 1e-3 / nf) / 1e9 / peak, 4)}


def tensor_phase_rates(wl, budgets, stats_ms, compress_ms, peaks):
    """Algorithmic flops of the two tensor-core phases over their durations (each phase also holds the small kernels
    around its contraction, so these are lower bounds for the contraction kernels themselves)."""
    if wl.dtype == "f32":
        return None
    P, L = wl.prompt_len, wl.n_layers
    tpeak = float(peaks.get("bf16_tflops_sustained", 1400.0))
    Le = P - budgets.double()                                     # evicted rows per (sequence, layer, KV head)
    sim_flops = float((2.0 * Le * budgets.double() * wl.d_head).sum())
    attn_flops = 2.0 * wl.batch * wl.n_q_heads * L * float(P) * P * wl.d_head      # two causal sweeps of P^2 d
    return [
        {"phase": "d2o_layer_stats (attn_tc_kernel x 2 sweeps + density)", "bound": "tensor",
         "achieved": round(attn_flops / (stats_ms * 1e-3) / 1e12, 1), "peak": tpeak, "unit": "TFLOP/s",
         "frac": round(attn_flops / (stats_ms * 1e-3) / 1e12 / tpeak, 4)},
        {"phase": "d2o_prefill_compress (select, sim_tc_kernel, reduce, segments, merge)", "bound": "tensor",
         "achieved": round(sim_flops / (compress_ms * 1e-3) / 1e12, 1), "peak": tpeak, "unit": "TFLOP/s",
         "frac": round(sim_flops / (compress_ms * 1e-3) / 1e12 / tpeak, 4)}]


def per_config_entry(B, wl, device, args, peaks, full_cache=False):
    """A shorter measurement of one config: 1 warm-up + 2 timed passes, at most 64 decode steps."""
    nd = min(wl.decode_steps, 64)
    m = measure_streamed(B, wl, nd, 1, 2, device, args, with_lse=(wl.dtype != "f32"))
    bytes_per_step, achieved, peak = roofline_of_decode(wl, m["budgets"], nd, m["decode_ms"], 1, peaks)
    out = {"workload": workload_string(wl, nd), "decode_us_per_step": round(m["decode_ms"] * 1e3 / nd, 2),
           "decode_entry_point": "d2o_decode_step" if NO_CHAIN else "d2o_decode_steps",
           "decode_us_per_step_single_calls": (None if m["decode_single_calls_ms"] is None
                                               else round(m["decode_single_calls_ms"] * 1e3 / nd, 2)),
           "tokens_per_s": round(wl.batch * nd / (m["decode_ms"] * 1e-3), 1),
           "frac_of_measured_hbm": round(achieved / peak, 4), "frac_of_nominal_hbm": round(achieved / NOMINAL_HBM_GBS, 4),
           "achieved_GBps": round(achieved, 1), "stats_ms": round(m["stats_ms"], 3),
           "stats_with_lse_ms": None if m["stats_with_lse_ms"] is None else round(m["stats_with_lse_ms"], 3),
           "budgets_ms": round(m["budget_ms"], 3), "prefill_compress_ms": round(m["compress_ms"], 3),
           "budgets_min_max": [int(m["budgets"].min()), int(m["budgets"].max())],
           "merges_discards": m["merges_discards"],
           "tensor_phases": tensor_phase_rates(wl, m["budgets"], m["stats_ms"], m["compress_ms"], peaks)}
    if full_cache:
        f = full_cache_decode(B, wl, nd, device, peak)
        f["compressed_over_full_speedup"] = round(f["us_per_step"] / out["decode_us_per_step"], 2)
        out["full_cache_decode"] = f
    return out


def run_ours(args, wl, rank, world, device):
    from paper_2406_13035_b200 import binding as B
    from paper_2406_13035_b200 import build
    if rank == 0:
        build.build_library()
    if world > 1:
        torch.distributed.barrier()
    B.load_library()
    peaks = load_peaks()
    nd = args.decode_steps or wl.decode_steps
    ctx = make_context(B, wl, nd, device, args)
    # every rank works on its own sequences: same shapes, rank-dependent seed (weak scaling, no exchange)
    wl_r = dataclasses.replace(wl, seed=wl.seed + 7919 * rank)
    streams = [W.LayerStream(wl_r, l, device) for l in range(wl.n_layers)]
    prompts = [s.prompt() for s in streams]
    dq, dk, dv = decode_inputs(streams, nd)
    L = wl.n_layers
    lpc = args.layers_per_call or L
    m = measure_resident(ctx, wl, prompts, dq, dk, dv, nd, lpc, args.warmup, args.steps, world, device)
    budgets, decode_ms = m["budgets"], m["decode_ms"]
    steps_per_s = nd / (decode_ms * 1e-3)
    calls_per_step = (L + lpc - 1) // lpc
    bytes_per_step, achieved, peak = roofline_of_decode(wl, budgets, nd, decode_ms, calls_per_step, peaks)
    bytes_per_launch = bytes_per_step / calls_per_step
    launch_us = decode_ms * 1e3 / (nd * calls_per_step)
    ratio = DECODE_TRAFFIC_RATIO.get(wl.name) if lpc == L else None
    roofline = {"bound": "hbm", "kernel": "decode_kernel", "achieved": round(achieved, 1), "peak": peak,
                "unit": "GB/s", "frac": round(achieved / peak, 4),
                "peak_source": "measured" if "hbm_gbs" in peaks else "fallback",
                "frac_of_nominal_8TBps": round(achieved / NOMINAL_HBM_GBS, 4),
                "algorithmic_bytes_per_launch": int(bytes_per_launch), "avg_launch_us": round(launch_us, 2),
                "traffic": int(ratio * bytes_per_launch) if ratio else None,
                "traffic_source": ("ncu dram__bytes_read.sum + dram__bytes_write.sum of four decode_kernel launches of "
                                   "this workload at full size (a one-pass capture), as a ratio to the algorithmic "
                                   "bytes of the captured run, times the algorithmic bytes of this run") if ratio else None}

    def sync_all():
        torch.cuda.synchronize()
        if world > 1:
            torch.distributed.barrier()

    # end to end: the decode loop through the host-buffer entry point
    e2e = None
    if not args.no_e2e:
        for l in range(L):
            ctx.d2o_prefill_compress(l, prompts[l][1], prompts[l][2])
        n_e2e = min(nd, 64)
        # one pinned block per step holding q | k | v back to back: the library then moves them in one transfer
        nq, nk = dq[0].numel(), dk[0].numel()
        hall = torch.empty((n_e2e, nq + 2 * nk), dtype=dq.dtype).pin_memory()
        hall[:, :nq] = dq[:n_e2e].reshape(n_e2e, nq).cpu()
        hall[:, nq:nq + nk] = dk[:n_e2e].reshape(n_e2e, nk).cpu()
        hall[:, nq + nk:] = dv[:n_e2e].reshape(n_e2e, nk).cpu()
        hq = [hall[s, :nq].view(dq[0].shape) for s in range(n_e2e)]
        hk = [hall[s, nq:nq + nk].view(dk[0].shape) for s in range(n_e2e)]
        hv = [hall[s, nq + nk:].view(dv[0].shape) for s in range(n_e2e)]
        ho = torch.empty(dq[0].shape, dtype=dq.dtype).pin_memory()
        n_warm = min(3, n_e2e)

        def recompress():
            ctx.d2o_prefill_compress_layers(0, L, [p[1] for p in prompts], [p[2] for p in prompts])

        for s in range(n_warm):                           # untimed: the entry point's first calls
            ctx.d2o_decode_step_host(0, L, hq[s], hk[s], hv[s], ho)
        n_rep = 3                                         # timed runs of n_e2e steps each; the median is reported

        def timed(run):
            times = []
            for _ in range(n_rep):
                recompress()
                sync_all()
                e0, e1 = ev(), ev()
                e0.record()
                run()
                e1.record()
                sync_all()
                times.append(max_over_ranks([e0.elapsed_time(e1)], world, device)[0])
            return statistics.median(times), times

        def run_single():
            for s in range(n_e2e):
                ctx.d2o_decode_step_host(0, L, hq[s], hk[s], hv[s], ho)

        ms_single, all_single = timed(run_single)
        ms, all_ms = ms_single, all_single
        if not NO_CHAIN:
            # the same steps through the multi-step host entry point: every step's inputs still cross from pinned
            # host memory and its output crosses back inside the timed region, but beside the neighbouring steps' kernels
            recompress()
            hq2 = dq[:n_e2e].cpu().pin_memory(); hk2 = dk[:n_e2e].cpu().pin_memory(); hv2 = dv[:n_e2e].cpu().pin_memory()
            ho2 = torch.empty_like(hq2).pin_memory()
            # untimed: the first call creates the library's two copy streams
            ctx.d2o_decode_steps_host(0, L, n_warm, hq2[:n_warm], hk2[:n_warm], hv2[:n_warm], ho2[:n_warm])
            ms, all_ms = timed(lambda: ctx.d2o_decode_steps_host(0, L, n_e2e, hq2, hk2, hv2, ho2))
            del hq2, hk2, hv2, ho2
        e2e = {"value": round(whole_job_rate(wl.batch * n_e2e, world, ms), 2), "unit": "token-steps/s",
               "h2d_bytes_per_step": int((nq + 2 * nk) * hall.element_size()),
               "d2h_bytes_per_step": int(ho.numel() * ho.element_size()), "steps": n_e2e,
               "runs": f"median of {n_rep} timed runs of {n_e2e} steps after {n_warm} untimed steps",
               "us_per_step_runs": [round(x * 1e3 / n_e2e, 2) for x in all_ms],
               "us_per_step": round(ms * 1e3 / n_e2e, 2),
               "entry_point": "d2o_decode_step_host" if NO_CHAIN else "d2o_decode_steps_host",
               "us_per_step_single_calls": round(ms_single * 1e3 / n_e2e, 2)}
    st = ctx.d2o_get_stats()
    if st.error_word != 0:
        raise RuntimeError(f"device error word {st.error_word} ({st.error_detail:#x})")
    ctx.close()
    del ctx, prompts, dq, dk, dv, streams
    torch.cuda.empty_cache()
    full = None
    if args.full_cache or wl.name.startswith("cfg4"):
        full = full_cache_decode(B, wl, nd, device, peak, world)
        full["compressed_over_full_speedup"] = round(full["us_per_step"] / (decode_ms * 1e3 / nd), 2)
    res = {
        "metric": METRIC, "value": round(whole_job_rate(wl.batch * nd, world, decode_ms), 2), "unit": "token-steps/s",
        "n_gpus": world, "steps": args.steps, "warmup": args.warmup, "ms_per_step": round(m["pass_ms"], 3),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": wl.dtype, "data": "synthetic",
        "config": {"workload": workload_string(wl, nd),
                   "l2": "decode working set (K_c+V_c of all layers) exceeds the 126 MB L2; prompt tensors exceed it too",
                   "layers_per_decode_call": lpc, "decode_ring_stages": args.stages or "auto",
                   "sequences_per_gpu": wl.batch, "parallelism": "replicas (independent sequences per GPU)"},
        "decode_steps_per_s_per_gpu": round(steps_per_s, 2), "decode_us_per_step": round(decode_ms * 1e3 / nd, 2),
        "decode_entry_point": ("d2o_decode_steps (all decode steps of a pass in one call, inputs resident)"
                               if m["chained"] else "d2o_decode_step (one call per token)"),
        "decode_step_us_single_calls": m["step_pct"],
        "stats_ms": round(m["stats_ms"], 3), "budgets_ms": round(m["budget_ms"], 3),
        "prefill_compress_ms": round(m["compress_ms"], 3), "decode_ms": round(decode_ms, 3),
        "wall_s": round(m["wall_s"], 3), "budgets_min_max": [int(budgets.min()), int(budgets.max())],
        "merges_discards": [int(st.merges), int(st.discards)],
        "roofline": roofline, "tensor_phases": tensor_phase_rates(wl, budgets, m["stats_ms"], m["compress_ms"], peaks),
        "full_cache_decode": full, "e2e": e2e, "gpu_launches": m["launches"], "clocks": m["clocks"],
    }
    # the other configs, shorter (rank 0 of a single-GPU run only: they are context for the headline, not part of it)
    if not args.no_per_config and world == 1 and args.config == "cfg2" and not (args.layers or args.batch):
        per = {}
        todo = [("cfg2_unclamped", dataclasses.replace(wl, max_budget=0, name="cfg2[unclamped]"), False)]
        for name in ("cfg1", "cfg3"):
            c = W.CONFIGS[name]
            todo.append((name, c, False))
            todo.append((name + "_unclamped", dataclasses.replace(c, max_budget=0, name=f"{name}[unclamped]"), False))
        for bsz in (1, 8, 32, 64):
            c = dataclasses.replace(W.CONFIGS["cfg4"], batch=bsz, name=f"cfg4[B={bsz}]")
            todo.append((f"cfg4_B{bsz}", c, True))
        todo.append(("cfg4_B8_unclamped", dataclasses.replace(W.CONFIGS["cfg4"], max_budget=0, name="cfg4[B=8,unclamped]"),
                     False))
        # the multi-turn (streaming) shape of the paper's appendix: fixed budget 2048 = 48 important + 2000 recent tokens
        todo.append(("streaming_session", W.CONFIGS["session"], False))
        for key, c, fc in todo:
            try:
                per[key] = per_config_entry(B, c, device, args, peaks, full_cache=fc)
            except Exception as exc:                      # keep the headline line even if a side measurement fails
                per[key] = {"workload": workload_string(c, min(c.decode_steps, 64)), "error": repr(exc)[:300]}
                torch.cuda.empty_cache()
        res["per_config"] = per
    return res


# --------------------------------------------------------------------------------------- CPU oracle leg
def oracle_sample(wl: W.Workload, n_slices: int, n_steps: int, threads: int = 1):
    """Times the oracle on `n_slices` slices of layer 0 of the workload: column sums of their query heads,
    compression at the uniform budget rho * P, `n_steps` decode steps.  Returns (seconds for the prompt stage per
    slice, seconds per decode step of one slice, slices)."""
    import numpy as np
    from oracle import d2o_oracle as O
    from threadpoolctl import threadpool_limits
    s = W.LayerStream(dataclasses.replace(wl, batch=1), 0, "cpu")
    Q, K, V = s.prompt()
    G = wl.group
    picks = [(0, h) for h in range(min(n_slices, wl.n_kv_heads))]
    dec = [s.decode() for _ in range(n_steps)]

    class PerHead:
        """[b, h] -> float64 [P, d] of one head, converted on demand."""

        def __init__(self, t):
            self.t = t

        def __getitem__(self, i):
            return self.t[i].double().numpy()

    with threadpool_limits(limits=threads):
        orc = O.OracleStack(n_layers=1, batch=1, n_q_heads=wl.n_q_heads, n_kv_heads=wl.n_kv_heads,
                            d_head=wl.d_head, dtype=wl.dtype, prompt_len=wl.prompt_len, rho=wl.rho, n_sink=wl.n_sink,
                            window=wl.window, nm_ratio=wl.nm_ratio, beta=wl.beta, min_budget=wl.min_budget)
        t0 = time.perf_counter()
        heads = [(b, h * G + g) for b, h in picks for g in range(G)]
        orc.layer_stats(0, PerHead(Q), PerHead(K), heads)
        orc.budgets = np.full((1, 1, wl.n_kv_heads), int(round(wl.rho * wl.prompt_len)), dtype=np.int64)
        orc.prefill_compress(0, PerHead(K), PerHead(V), picks)
        t1 = time.perf_counter()
        for i, (q, k, v) in enumerate(dec):
            orc.decode_step(0, q.double().numpy(), k.double().numpy(), v.double().numpy(), i, picks)
        t2 = time.perf_counter()
    return (t1 - t0) / len(picks), (t2 - t1) / (len(picks) * max(1, n_steps)), len(picks)


def cpu_baseline(wl: W.Workload, n_slices=0, n_steps=64):
    if n_slices <= 0:
        # about 10 s of prompt-stage oracle work: one query head of 4096 positions costs about a quarter second
        per_slice = 0.25 * wl.group * (wl.prompt_len / 4096.0) ** 2
        n_slices = max(1, min(16, int(10.0 / per_slice)))
    prompt_s, step_s, n = oracle_sample(wl, n_slices, n_steps)
    total_slices = wl.n_layers * wl.batch * wl.n_kv_heads
    return {"value": round(wl.batch / (step_s * total_slices), 4), "unit": "token-steps/s", "cores": 1,
            "host_cores": os.cpu_count(), "kind": "oracle",
            "sample": f"{n} slices of layer 0 of one sequence (column sums, compression, {n_steps} decode steps), one "
                      f"NumPy thread of the host's {os.cpu_count()} cores; {step_s * 1e3:.3f} ms per slice-step and "
                      f"{prompt_s:.2f} s prompt stage per slice, extrapolated linearly to all {total_slices} slices"}


def run_reference(args, wl):
    vals = []
    nd = 16
    for _ in range(min(args.warmup, 1)):
        oracle_sample(wl, 1, 2)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        vals.append(oracle_sample(wl, 1, nd))
    wall = time.perf_counter() - t0
    step_s = statistics.mean(v[1] for v in vals)
    prompt_s = statistics.mean(v[0] for v in vals)
    total_slices = wl.n_layers * wl.batch * wl.n_kv_heads
    value = round(wl.batch / (step_s * total_slices), 4)
    sample = (f"per bench step: 1 slice of layer 0 of one sequence (column sums, compression, {nd} decode steps), one "
              f"NumPy thread of the host's {os.cpu_count()} cores; extrapolated linearly to all {total_slices} slices")
    return {"impl": "reference", "metric": METRIC, "value": value, "unit": "token-steps/s", "n_gpus": 1,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": round(wall / max(1, args.steps) * 1e3, 2),
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": workload_string(wl, args.decode_steps or wl.decode_steps)},
            "prompt_stage_s_per_slice": round(prompt_s, 3),
            "cpu_baseline": {"value": value, "unit": "token-steps/s", "cores": 1, "host_cores": os.cpu_count(),
                             "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": "token-steps/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}


def spawn_ranks(n: int) -> int:
    """`--gpus N` without a launcher: start N ranks of this script on this node, one per GPU."""
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    return subprocess.call(cmd)


def main():
    global NO_CHAIN
    args = parse()
    NO_CHAIN = args.single_step_calls
    wl = W.CONFIGS[args.config] if args.config in W.CONFIGS else W.twin(args.config.replace("_twin", ""))
    if args.batch:
        wl = dataclasses.replace(wl, batch=args.batch, name=f"{wl.name}[B={args.batch}]")
    if args.layers:
        wl = dataclasses.replace(wl, n_layers=args.layers, name=f"{wl.name}[{args.layers} layers]")
    if args.unclamped:
        wl = dataclasses.replace(wl, max_budget=0, name=f"{wl.name}[unclamped]")
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if args.impl == "reference":
        if rank == 0:
            print(json.dumps(run_reference(args, wl)), flush=True)
        return
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        sys.exit(spawn_ranks(args.gpus))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    device = f"cuda:{local}"
    if world > 1:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        torch.distributed.init_process_group("nccl", device_id=torch.device(device))
    res = run_ours(args, wl, rank, world, device)
    if rank == 0:
        if not args.no_cpu_baseline and world == 1:
            res["cpu_baseline"] = cpu_baseline(wl)
        print(json.dumps(res), flush=True)
    if world > 1:
        torch.distributed.barrier()
        torch.distributed.destroy_process_group()


if __name__ == "__main__":
    main()
