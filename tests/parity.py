"""GPU-vs-oracle parity harness (test infrastructure).

Runs one workload through the C-ABI library on the GPU and through the float64 oracle on the
CPU, on the same seeded tensors, and compares stage by stage:
  column sums and densities, budgets, retained sets, nearest neighbours, tau_0, merged caches,
  then every decode step (outputs, victim, cache content, scores, tau).

Where floating point decides an index (Top-N boundary, arg-min victim, arg-max neighbour,
threshold test) the GPU decides in float32 and the oracle in float64.  A disagreement is a
*tolerated tie* only if the oracle's own gap between the two candidates is below `tie_rtol`
(1e-6 relative); the oracle then replays the GPU's choice ("tie-follow") so that later stages
stay comparable, and the event is counted in the report.
"""
from __future__ import annotations

import copy
import math
from dataclasses import dataclass, field
from typing import Dict, List, Optional, Tuple

import numpy as np
import torch

from oracle import d2o_oracle as O
from paper_2406_13035_b200 import binding as B
from paper_2406_13035_b200 import workloads as W

TIE_RTOL = 1e-6


@dataclass
class Report:
    ties: Dict[str, int] = field(default_factory=lambda: dict(budget=0, topn=0, nn=0, mask=0, victim=0,
                                                               dec_nn=0, dec_merge=0))
    max_err: Dict[str, float] = field(default_factory=dict)
    checked_slices: int = 0
    steps: int = 0
    merges: int = 0
    discards: int = 0

    def err(self, key: str, v: float):
        self.max_err[key] = max(self.max_err.get(key, 0.0), float(v))


def tolerances(dtype: str):
    """(relative-to-scale tolerance for fp32, absolute tolerance for 16-bit) of outputs and merged K/V."""
    return (1e-5, 0.0) if dtype == "f32" else (0.0, 2e-2)


def close(got: np.ndarray, ref: np.ndarray, dtype: str) -> float:
    """Error measure normalised so that <= 1 passes: fp32 -> |diff| / (1e-5 * max(|ref|, rms));
    fp16/bf16 -> |diff| / 2e-2."""
    got = np.asarray(got, np.float64)
    ref = np.asarray(ref, np.float64)
    rel, ab = tolerances(dtype)
    if ab > 0:
        return float(np.max(np.abs(got - ref)) / ab) if got.size else 0.0
    scale = np.maximum(np.abs(ref), math.sqrt(float(np.mean(ref * ref))) if ref.size else 1.0)
    return float(np.max(np.abs(got - ref) / (rel * np.maximum(scale, 1e-30)))) if got.size else 0.0


def np64(t: torch.Tensor) -> np.ndarray:
    return t.detach().to("cpu", torch.float64).numpy()


def make_ctx(wl: W.Workload, device="cuda:0", **over) -> B.D2OContext:
    kw = dict(n_layers=wl.n_layers, batch=wl.batch, n_q_heads=wl.n_q_heads, n_kv_heads=wl.n_kv_heads,
              d_head=wl.d_head, dtype=wl.dtype, prompt_len=wl.prompt_len, max_new_tokens=wl.decode_steps,
              rho=wl.rho, n_sink=wl.n_sink, window=wl.window, nm_ratio=wl.nm_ratio, beta=wl.beta,
              density_temp=wl.density_temp, min_budget=wl.min_budget, max_budget=wl.max_budget)
    kw.update(over)
    return B.D2OContext(B.make_config(**kw), device)


def make_oracle(wl: W.Workload, cfg: B.D2OConfig) -> O.OracleStack:
    # float parameters take the values the C floats hold
    return O.OracleStack(n_layers=cfg.n_layers, batch=cfg.batch, n_q_heads=cfg.n_q_heads,
                         n_kv_heads=cfg.n_kv_heads, d_head=cfg.d_head, dtype=wl.dtype, prompt_len=cfg.prompt_len,
                         rho=float(cfg.rho), n_sink=cfg.n_sink, window=cfg.window, nm_ratio=float(cfg.nm_ratio),
                         beta=float(cfg.beta), density_temp=float(cfg.density_temp), min_budget=cfg.min_budget,
                         head_reduce=cfg.head_reduce, tau_override=float(cfg.tau_override),
                         max_budget=cfg.max_budget)


def run_parity(wl: W.Workload, device="cuda:0", slices: Optional[List[Tuple[int, int, int]]] = None,
               steps: Optional[int] = None, tie_rtol: float = TIE_RTOL, ctx_over: Optional[dict] = None,
               layers_per_call: Optional[int] = None, decode_stages: int = 0, decode_l2_hints: int = 1,
               similarity_path: int = 0, stats_path: int = 0, decode_warps: int = 0,
               decode_smem_rows: int = 0, decode_long_pairs: int = 0,
               check_stats_all: Optional[bool] = None) -> Report:
    """`slices`: (layer, b, kv_head) triples checked against the oracle (None = all).
    The GPU always runs the whole workload."""
    rep = Report()
    ctx = make_ctx(wl, device, **(ctx_over or {}))
    cfg = ctx.cfg
    if (decode_stages or not decode_l2_hints or similarity_path or stats_path or decode_warps or decode_smem_rows
            or decode_long_pairs):
        ctx.d2o_set_tuning(decode_stages, decode_l2_hints, similarity_path, stats_path, decode_warps,
                           decode_smem_rows, decode_long_pairs)
    orc = make_oracle(wl, cfg)
    L, Bn, Hq, Hkv, G, P = wl.n_layers, wl.batch, wl.n_q_heads, wl.n_kv_heads, wl.group, wl.prompt_len
    all_slices = [(l, b, h) for l in range(L) for b in range(Bn) for h in range(Hkv)]
    chk = all_slices if slices is None else slices
    rep.checked_slices = len(chk)
    chk_by_layer: Dict[int, List[Tuple[int, int]]] = {}
    for l, b, h in chk:
        chk_by_layer.setdefault(l, []).append((b, h))
    streams = [W.LayerStream(wl, l, device) for l in range(L)]
    # ---------------- (1) statistics
    KV = []
    for l in range(L):
        Q, K, V = streams[l].prompt()
        ctx.d2o_layer_stats(l, Q, K)
        KV.append((K, V))
        if l in chk_by_layer:
            heads = sorted({(b, h * G + g) for b, h in chk_by_layer[l] for g in range(G)})
            Qc, Kc = Q.cpu(), K.cpu()
            orc.layer_stats(l, _lazy64(Qc), _lazy64(Kc), heads)
            cs = ctx.colsum(l).cpu().double().numpy()
            for b, hq in heads:
                ref = orc.colsum[l, b, hq]
                rep.err("colsum_rel", np.max(np.abs(cs[b, hq] - ref) / np.maximum(np.abs(ref), 1e-6)))
        del Q
    budgets = ctx.d2o_layer_budgets().numpy().astype(np.int64)
    F_gpu = ctx.density().cpu().numpy()
    for l, b, h in chk:
        for g in range(G):
            ref = orc.F[b, l, h * G + g]
            rep.err("density_rel", abs(F_gpu[b, l, h * G + g] - ref) / max(abs(ref), 1e-12))
    # budgets: the oracle's pure function on the GPU's densities must give the GPU's integers
    orc_b = orc.layer_budgets(F_gpu)
    rep.ties["budget"] = int((orc_b != budgets).sum())
    orc.budgets = budgets.copy()                       # budget-follow
    tabs = ctx.tables()
    for b in range(Bn):
        for l in range(L):
            S, T, M = orc.slice_params(b, l)
            assert int(tabs[1][b, l]) == M, f"window mismatch at b={b} l={l}: {int(tabs[1][b, l])} vs {M}"
    # ---------------- (2) prompt-stage compression
    for l in range(L):
        K, V = KV[l]
        ctx.d2o_prefill_compress(l, K, V)
        if l not in chk_by_layer:
            continue
        K64, V64 = _lazy64(K.cpu()), _lazy64(V.cpu())
        for b, h in chk_by_layer[l]:
            _check_prefill_slice(rep, ctx, orc, wl, l, b, h, K64, V64, tabs, tie_rtol)
    KV.clear()
    # ---------------- (3) decode steps
    n_steps = wl.decode_steps if steps is None else steps
    lpc = L if layers_per_call is None else layers_per_call
    for step in range(n_steps):
        t = P + step
        qs, ks, vs = zip(*[streams[l].decode() for l in range(L)])
        q, k, v = torch.stack(qs), torch.stack(ks), torch.stack(vs)
        out = torch.empty_like(q)
        for l0 in range(0, L, lpc):
            l1 = min(L, l0 + lpc)
            ctx.d2o_decode_step(l0, l1, q[l0:l1].contiguous(), k[l0:l1].contiguous(), v[l0:l1].contiguous(),
                                out[l0:l1])
        qc, kc, vc, oc = np64(q), np64(k), np64(v), np64(out)
        for l, b, h in chk:
            _check_decode_slice(rep, ctx, orc, wl, l, b, h, qc[l], kc[l], vc[l], oc[l], t, tabs, tie_rtol)
        rep.steps += 1
    st = ctx.d2o_get_stats()
    assert st.error_word == 0, f"device error word {st.error_word} detail {st.error_detail:#x}"
    rep.gpu_stats = st
    ctx.close()
    return rep


class _lazy64:
    """Indexable view that converts one [P, d] head at a time to float64 (saves memory at full size)."""

    def __init__(self, t: torch.Tensor):
        self.t = t

    def __getitem__(self, idx):
        return self.t[idx].to(torch.float64).numpy()


def _gap_rel(a: float, b: float) -> float:
    return abs(a - b) / max(abs(a), abs(b), 1e-300)


def _check_prefill_slice(rep, ctx, orc, wl, l, b, h, K64, V64, tabs, tie_rtol):
    G, P = wl.group, wl.prompt_len
    got = ctx.slice_state(l, b, h, tabs)
    S, T, M = orc.slice_params(b, l)
    score = orc.group_score(l, b, h)
    force = {}
    orc.prefill_compress(l, K64, V64, [(b, h)])
    st = orc.slices[(l, b, h)]
    gpos = got["pos"].numpy().astype(np.int64)
    assert got["len"] == min(S, P)
    assert np.all(np.diff(gpos) > 0), "GPU retained positions must be ascending"
    if not np.array_equal(gpos, st.pos):
        # tolerated only if every swapped pair is a near-tie at the Top-N boundary
        only_gpu = sorted(set(gpos.tolist()) - set(st.pos.tolist()))
        only_orc = sorted(set(st.pos.tolist()) - set(gpos.tolist()))
        assert len(only_gpu) == len(only_orc)
        lo = min(score[only_orc].min(), score[only_gpu].min())
        hi = max(score[only_orc].max(), score[only_gpu].max())
        assert _gap_rel(lo, hi) <= tie_rtol, \
            f"retained set differs beyond a tie: layer {l} b {b} h {h}: {only_gpu} vs {only_orc}, gap {_gap_rel(lo, hi):.3e}"
        assert all(T <= j < P - M for j in only_gpu)
        rep.ties["topn"] += len(only_gpu)
        force["force_retained"] = gpos
        orc.prefill_compress(l, K64, V64, [(b, h)], force={(l, b, h): force})
        st = orc.slices[(l, b, h)]
    Le = P - min(S, P)
    if Le > 0:
        eidx, emx, enn = ctx.evict_lists(b, h, Le)
        np.testing.assert_array_equal(eidx.numpy(), st.log["evicted"])
        U = st.log["U"]
        mx_o, nn_o = st.log["mx"], st.log["nn"]
        gnn = enn.numpy().astype(np.int64)
        bad = np.nonzero(gnn != nn_o)[0]
        if bad.size:
            for i in bad:
                assert U[i, nn_o[i]] - U[i, gnn[i]] <= tie_rtol, \
                    f"nearest neighbour differs beyond a tie: row {i}: {gnn[i]} vs {nn_o[i]} gap {U[i, nn_o[i]] - U[i, gnn[i]]:.3e}"
            rep.ties["nn"] += int(bad.size)
            fnn = np.full(Le, -1, np.int64)
            fnn[bad] = gnn[bad]
            force["force_nn"] = fnn
            orc.prefill_compress(l, K64, V64, [(b, h)], force={(l, b, h): force})
            st = orc.slices[(l, b, h)]
            mx_o = st.log["mx"]
        rep.err("sim_abs", np.max(np.abs(emx.numpy() - mx_o)))
        rep.err("tau0_abs", abs(got["tau"] - st.tau))
        # merge mask of the GPU: rows whose Max(U) >= tau_0 in float32
        thr_gpu = np.float32(got["tau"]) if math.isnan(float(ctx.cfg.tau_override)) else np.float32(ctx.cfg.tau_override)
        gmask = emx.numpy() >= thr_gpu
        omask = st.log["merged"]
        flip = np.nonzero(gmask != omask)[0]
        if flip.size:
            for i in flip:
                assert abs(mx_o[i] - st.log["thr"]) <= 4e-6, \
                    f"merge decision differs beyond a tie: row {i}: mx {mx_o[i]} thr {st.log['thr']}"
            rep.ties["mask"] += int(flip.size)
            force["force_merged"] = gmask
            orc.prefill_compress(l, K64, V64, [(b, h)], force={(l, b, h): force})
            st = orc.slices[(l, b, h)]
    _compare_state(rep, got, st, wl.dtype, "prefill")


def _compare_state(rep, got, st, dtype, tag):
    gpos = got["pos"].numpy().astype(np.int64)
    order = np.argsort(gpos, kind="stable")
    assert np.array_equal(gpos[order], st.pos), f"{tag}: cache positions differ"
    Kg, Vg = got["K"].double().numpy()[order], got["V"].double().numpy()[order]
    eK, eV = close(Kg, st.K, dtype), close(Vg, st.V, dtype)
    rep.err(f"{tag}_K", eK)
    rep.err(f"{tag}_V", eV)
    if eK <= 1.0 and eV <= 1.0:
        # storage-follow: a merged value that sits on a rounding boundary of the cache dtype may round
        # either way (float32 vs float64 arithmetic).  The flip is within tolerance, but one 16-bit ulp in a
        # key moves later logits by ~1e-3, so the oracle continues from the rows the GPU actually stored.
        rep.storage_flips = getattr(rep, "storage_flips", 0) + int((Kg != st.K).sum() + (Vg != st.V).sum())
        st.K, st.V = Kg.copy(), Vg.copy()
    sc = got["score"].double().numpy()[order]
    rep.err(f"{tag}_score_rel", np.max(np.abs(sc - st.score) / np.maximum(np.abs(st.score), 1e-6)))
    # the cached inverse norms belong to the stored keys
    Kg = got["K"].double().numpy()
    nrm = np.sqrt((Kg * Kg).sum(axis=1))
    rn = got["rnorm"].double().numpy()
    ok = nrm > 0
    rep.err(f"{tag}_rnorm_rel", np.max(np.abs(rn[ok] * nrm[ok] - 1.0)) if ok.any() else 0.0)


def _check_decode_slice(rep, ctx, orc, wl, l, b, h, q, k, v, out, t, tabs, tie_rtol):
    G = wl.group
    key = (l, b, h)
    before = copy.deepcopy(orc.slices[key])
    got = ctx.slice_state(l, b, h, tabs)
    gset = set(got["pos"].tolist())
    qs, ks, vs = q[b, h * G:(h + 1) * G], k[b, h], v[b, h]

    def attempt(force_victim=None, force_nn=None, tau_override=None):
        st = copy.deepcopy(before)
        o, log = O.decode_step_slice(st, qs, ks, vs, t, orc.beta,
                                     orc.tau_override if tau_override is None else tau_override,
                                     force_victim, force_nn)
        return st, o, log

    st, o, log = attempt()
    fv = fn = None
    if log.evicted and set(st.pos.tolist()) != gset:
        gone = sorted((set(before.pos.tolist()) | {t}) - gset)
        assert len(gone) == 1, f"GPU cache lost {gone} at t={t}"
        assert log.victim_gap <= tie_rtol and gone[0] == log.runner_up_pos, \
            f"victim differs beyond a tie at t={t} slice {key}: GPU {gone[0]} oracle {log.victim_pos} gap {log.victim_gap:.3e}"
        rep.ties["victim"] += 1
        fv = gone[0]
        st, o, log = attempt(force_victim=fv)
    # merged / discarded and neighbour choice show in the cache content
    e = _state_err(got, st, wl.dtype)
    if log.evicted and e > 1.0:
        tried = False
        if abs(log.mx - log.tau) <= 4e-6:                     # threshold tie: replay the other decision
            alt = float("inf") if log.merged else float("-inf")
            st2, o2, log2 = attempt(force_victim=fv, tau_override=alt)
            st2.tau = st.tau
            if _state_err(got, st2, wl.dtype) <= 1.0:
                st, o, log, tried = st2, o2, log2, True
                rep.ties["dec_merge"] += 1
        if not tried and log.nn_gap <= tie_rtol:              # neighbour tie
            st2, o2, log2 = attempt(force_victim=fv, force_nn=log.nn_runner_pos)
            if _state_err(got, st2, wl.dtype) <= 1.0:
                st, o, log, tried = st2, o2, log2, True
                rep.ties["dec_nn"] += 1
        assert tried, f"cache content differs at t={t} slice {key}: err {e:.3f} (mx {log.mx}, tau {log.tau}, nn_gap {log.nn_gap})"
    orc.slices[key] = st
    rep.err("out", close(out[b, h * G:(h + 1) * G], o, wl.dtype))
    _compare_state(rep, got, st, wl.dtype, "decode")
    orc.slices[key] = st
    rep.err("tau_abs", abs(got["tau"] - st.tau))
    if log.evicted:
        rep.merges += int(log.merged)
        rep.discards += int(not log.merged)


def _state_err(got, st, dtype) -> float:
    gpos = got["pos"].numpy().astype(np.int64)
    order = np.argsort(gpos, kind="stable")
    if not np.array_equal(gpos[order], st.pos):
        return float("inf")
    return max(close(got["K"].double().numpy()[order], st.K, dtype),
               close(got["V"].double().numpy()[order], st.V, dtype))


def assert_report(rep: Report, dtype: str, max_tie_frac: float = 0.01):
    e = rep.max_err
    assert e.get("colsum_rel", 0) < 2e-4, e
    assert e.get("density_rel", 0) < 2e-4, e
    assert e.get("sim_abs", 0) < 5e-6, e
    assert e.get("tau0_abs", 0) < 5e-6, e
    for k in ("prefill_K", "prefill_V", "decode_K", "decode_V", "out"):
        assert e.get(k, 0) <= 1.0, (k, e)
    for k in ("prefill_score_rel", "decode_score_rel"):
        assert e.get(k, 0) < 2e-4, (k, e)
    assert e.get("tau_abs", 0) < 1e-5, e
    assert e.get("prefill_rnorm_rel", 0) < 1e-5 and e.get("decode_rnorm_rel", 0) < 1e-5, e
    assert rep.ties["budget"] == 0, rep.ties
    decisions = max(1, rep.checked_slices * max(1, rep.steps))
    assert sum(rep.ties.values()) <= max(2, max_tie_frac * decisions), rep.ties
