"""GPU-vs-oracle parity harness (test infrastructure).

Runs one workload through the C-ABI library on the GPU and through the float64 oracle on the
CPU, on the same seeded tensors, and compares stage by stage:
  column sums and densities, budgets, retained sets, nearest neighbours, tau_0, merged caches,
  then every decode step (outputs, victim, cache content, scores, tau).

Where floating point decides an index (Top-N boundary, arg-min victim, arg-max neighbour,
threshold test) the GPU decides in float32 and the oracle in float64.  A disagreement is a
*tolerated tie* only if the oracle's own gap between the two candidates is below `tie_rtol`
(1e-6 relative); the harness then replays the GPU's choice ("tie-follow") by composing the oracle's
step functions itself, so that later stages stay comparable, and the event is counted in the report.

Cache content: for float32 caches the oracle keeps its own trajectory over all steps and the merged
rows are compared at the 1e-5 tolerance.  For 16-bit caches a merged value that sits on a rounding
boundary of the cache dtype may round either way in float32 (GPU) and float64 (oracle) arithmetic; one
16-bit ulp in a key moves later logits by ~1e-3, so after a comparison that passed the oracle continues
from the rows the GPU stored ("storage-follow").  Every adopted element is checked: it must lie in a
row that was merged in this very step, and it must be the rounding of some value within a few float32 ulps
(relative to the row's scale) of the oracle's unrounded value.
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
# |exact - rounding boundary| of an adopted 16-bit element, relative to the row's scale: a few float32 ulps for the
# two-term merge of a decode step, more for a prompt-stage row that sums up to hundreds of float32 terms
BOUNDARY_RTOL = {"decode": 4e-6, "prefill": 2e-5}


@dataclass
class Report:
    ties: Dict[str, int] = field(default_factory=lambda: dict(budget=0, topn=0, nn=0, mask=0, victim=0,
                                                               dec_nn=0, dec_merge=0))
    max_err: Dict[str, float] = field(default_factory=dict)
    checked_slices: int = 0
    steps: int = 0
    merges: int = 0
    discards: int = 0
    storage_flips: int = 0

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


def make_oracle(wl: W.Workload, cfg: B.D2OConfig, prompt_lens=None) -> O.OracleStack:
    # float parameters take the values the C floats hold
    return O.OracleStack(n_layers=cfg.n_layers, batch=cfg.batch, n_q_heads=cfg.n_q_heads,
                         n_kv_heads=cfg.n_kv_heads, d_head=cfg.d_head, dtype=wl.dtype, prompt_len=cfg.prompt_len,
                         rho=float(cfg.rho), n_sink=cfg.n_sink, window=cfg.window, nm_ratio=float(cfg.nm_ratio),
                         beta=float(cfg.beta), density_temp=float(cfg.density_temp), min_budget=cfg.min_budget,
                         head_reduce=cfg.head_reduce, tau_override=float(cfg.tau_override),
                         max_budget=cfg.max_budget, feature=("k", "v")[cfg.sim_feature],
                         policy=("weighted", "average")[cfg.merge_policy],
                         budget_rule=("layer", "head", "exp_decay")[cfg.budget_rule], prompt_lens=prompt_lens)


def run_parity(wl: W.Workload, device="cuda:0", slices: Optional[List[Tuple[int, int, int]]] = None,
               steps: Optional[int] = None, tie_rtol: float = TIE_RTOL, ctx_over: Optional[dict] = None,
               layers_per_call: Optional[int] = None, decode_stages: int = 0, decode_l2_hints: int = 1,
               similarity_path: int = 0, stats_path: int = 0, decode_warps: int = 0,
               decode_smem_rows: int = 0, decode_long_pairs: int = 0,
               check_stats_all: Optional[bool] = None, prompt_hook=None, decode_hook=None,
               max_ties: Optional[int] = None, prompt_lens=None) -> Report:
    """`slices`: (layer, b, kv_head) triples checked against the oracle (None = all).
    The GPU always runs the whole workload.  `prompt_hook(layer, Q, K, V)` and `decode_hook(step, q, k, v)` may
    return edited input tensors (both sides then see the edited ones)."""
    rep = Report()
    ctx = make_ctx(wl, device, **(ctx_over or {}))
    cfg = ctx.cfg
    if (decode_stages or not decode_l2_hints or similarity_path or stats_path or decode_warps or decode_smem_rows
            or decode_long_pairs):
        ctx.d2o_set_tuning(decode_stages, decode_l2_hints, similarity_path, stats_path, decode_warps,
                           decode_smem_rows, decode_long_pairs)
    orc = make_oracle(wl, cfg, prompt_lens)
    if prompt_lens is not None:                        # ragged batch: the tensors stay padded to wl.prompt_len
        ctx.d2o_set_prompt_lens(prompt_lens)
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
        if prompt_hook is not None:
            Q, K, V = prompt_hook(l, Q, K, V)
        ctx.d2o_layer_stats(l, Q, K)
        KV.append((K, V))
        if l in chk_by_layer:
            heads = sorted({(b, h * G + g) for b, h in chk_by_layer[l] for g in range(G)})
            Qc, Kc = Q.cpu(), K.cpu()
            orc.layer_stats(l, _lazy64(Qc), _lazy64(Kc), heads)
            cs = ctx.colsum(l).cpu().double().numpy()
            for b, hq in heads:
                ref = orc.colsum[l, b, hq, :orc.Pb[b]]
                rep.err("colsum_rel", np.max(np.abs(cs[b, hq, :orc.Pb[b]] - ref) / np.maximum(np.abs(ref), 1e-6)))
        del Q
    budgets = ctx.d2o_layer_budgets().numpy().astype(np.int64)
    F_gpu = ctx.density().cpu().numpy()
    for l, b, h in chk:
        for g in range(G):
            ref = orc.F[b, l, h * G + g]
            rep.err("density_rel", abs(F_gpu[b, l, h * G + g] - ref) / max(abs(ref), 1e-12))
    # budgets: the oracle's pure function on the GPU's densities must give the GPU's integers
    orc_b = orc.layer_budgets(F_gpu)                   # [B, L, Hkv]
    gpu_b = budgets[:, :, None] if budgets.ndim == 2 else budgets
    rep.ties["budget"] = int((orc_b != gpu_b).sum())
    orc.budgets = np.broadcast_to(gpu_b, orc_b.shape).copy()     # budget-follow
    tabs = ctx.tables()
    for b in range(Bn):
        for l in range(L):
            for h in range(Hkv):
                S, T, M = orc.slice_params(b, l, h)
                assert int(tabs[1][b, l, h]) == M, f"window mismatch at b={b} l={l} h={h}: {int(tabs[1][b, l, h])} vs {M}"
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
        qs, ks, vs = zip(*[streams[l].decode() for l in range(L)])
        q, k, v = torch.stack(qs), torch.stack(ks), torch.stack(vs)
        if decode_hook is not None:
            q, k, v = decode_hook(step, q, k, v)
        out = torch.empty_like(q)
        for l0 in range(0, L, lpc):
            l1 = min(L, l0 + lpc)
            ctx.d2o_decode_step(l0, l1, q[l0:l1].contiguous(), k[l0:l1].contiguous(), v[l0:l1].contiguous(),
                                out[l0:l1])
        qc, kc, vc, oc = np64(q), np64(k), np64(v), np64(out)
        for l, b, h in chk:
            _check_decode_slice(rep, ctx, orc, wl, l, b, h, qc[l], kc[l], vc[l], oc[l], step, tabs, tie_rtol)
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


def replay_prefill(orc, l, b, h, K64, V64, retained=None, nn_override=None, mask_override=None):
    """The steps of O.prefill_compress_slice, composed here so that the GPU's choice at a near-tie (kept set,
    neighbour of some evicted rows, merge mask) can take the place of the oracle's own.  Used only after a
    disagreement has been shown to be a tie."""
    S, T, M = orc.slice_params(b, l, h)
    Pb = orc.Pb[b]
    K, V = K64[b, h][:Pb], V64[b, h][:Pb]
    score = orc.group_score(l, b, h)
    if retained is None:
        retained, evicted = O.select_retained(score, S, T, M)
    else:
        retained = np.array(sorted(int(j) for j in retained), dtype=np.int64)
        keep = set(retained.tolist())
        evicted = np.array([j for j in range(Pb) if j not in keep], dtype=np.int64)
    Kc, Vc, Ke, Ve = K[retained], V[retained], K[evicted], V[evicted]
    U = O.cosine_matrix(O.feature_rows(Ke, Ve, orc.feature), O.feature_rows(Kc, Vc, orc.feature))
    mx, nn = O.nearest_neighbour(U)
    if nn_override is not None:
        for i, j in enumerate(nn_override):
            if j >= 0:
                nn[i] = j
                mx[i] = U[i, j]
    tau0 = O.initial_threshold(mx)
    thr = tau0 if math.isnan(orc.tau_override) else orc.tau_override
    mask = O.merge_mask(mx, thr) if mask_override is None else np.asarray(mask_override, bool)
    Km, Vm, den = O.weighted_merge(Kc, Vc, Ke, Ve, mx, nn, mask, orc.policy)
    touched = den > (O.E if orc.policy == "weighted" else 1.0)
    Kn = np.where(touched[:, None], O.round_storage(Km, orc.dtype), Kc)
    Vn = np.where(touched[:, None], O.round_storage(Vm, orc.dtype), Vc)
    st = O.SliceState(pos=retained.copy(), K=Kn, V=Vn, score=score[retained].copy(), tau=tau0, S=S, T=T, M=M,
                      dtype=orc.dtype, feature=orc.feature, policy=orc.policy)
    st.log = dict(retained=retained, evicted=evicted, mx=mx, nn=nn, den=den, U=U, thr=thr, merged=mask,
                  K_exact=Km, V_exact=Vm, touched=touched)
    orc.slices[(l, b, h)] = st
    return st


def replay_decode(st, q, k, v, t, beta, tau_override, victim_pos=None, nn_pos=None):
    """The steps of O.decode_step_slice with the GPU's victim and / or neighbour in place of the oracle's own."""
    out = O.decode_attend(st, q, k, v, t)
    log = O.StepLog(tau=st.tau)
    if st.pos.size <= st.S:
        return out, log
    ranked = O.victim_order(st, t)
    assert ranked
    vi = ranked[0] if victim_pos is None else int(np.nonzero(st.pos == victim_pos)[0][0])
    if len(ranked) > 1:
        a, b_ = st.score[ranked[0]], st.score[ranked[1]]
        log.victim_gap = abs(b_ - a) / max(abs(a), abs(b_), 1e-300)
        log.runner_up_pos = int(st.pos[ranked[1]])
    log.victim_pos, log.evicted = int(st.pos[vi]), True
    k_e, v_e = O.evict_row(st, vi)
    U, order = O.neighbour_order(st, k_e, v_e)
    nj = order[0] if nn_pos is None else int(np.nonzero(st.pos == nn_pos)[0][0])
    if len(order) > 1:
        log.nn_gap = float(U[order[0]] - U[order[1]])
        log.nn_runner_pos = int(st.pos[order[1]])
    O.compensate(st, k_e, v_e, nj, float(U[nj]), beta, tau_override, log)
    return out, log


def _thr_tie(mx: float, thr: float, tie_rtol: float) -> bool:
    # cosines and thresholds live on a unit scale: relative to max(|mx|, |thr|, 1)
    return abs(mx - thr) <= tie_rtol * max(abs(mx), abs(thr), 1.0)


def _check_prefill_slice(rep, ctx, orc, wl, l, b, h, K64, V64, tabs, tie_rtol):
    P = orc.Pb[b]
    got = ctx.slice_state(l, b, h, tabs)
    S, T, M = orc.slice_params(b, l, h)
    score = orc.group_score(l, b, h)
    orc.prefill_compress(l, K64, V64, [(b, h)])
    st = orc.slices[(l, b, h)]
    gpos = got["pos"].numpy().astype(np.int64)
    assert got["len"] == min(S, P)
    assert np.all(np.diff(gpos) > 0), "GPU retained positions must be ascending"
    follow = {}
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
        follow["retained"] = gpos
        st = replay_prefill(orc, l, b, h, K64, V64, **follow)
    Le = P - min(S, P)
    if Le > 0:
        eidx, emx, enn = ctx.evict_lists(b, h, Le)
        np.testing.assert_array_equal(eidx.numpy(), st.log["evicted"])
        U = st.log["U"]
        mx_o, nn_o = st.log["mx"], st.log["nn"]
        gnn = enn.numpy().astype(np.int64)
        assert gnn.min() >= 0 and gnn.max() < min(S, P), "neighbour slot out of range"
        bad = np.nonzero(gnn != nn_o)[0]
        if bad.size:
            for i in bad:
                assert U[i, nn_o[i]] - U[i, gnn[i]] <= tie_rtol, \
                    f"nearest neighbour differs beyond a tie: row {i}: {gnn[i]} vs {nn_o[i]} gap {U[i, nn_o[i]] - U[i, gnn[i]]:.3e}"
            rep.ties["nn"] += int(bad.size)
            fnn = np.full(Le, -1, np.int64)
            fnn[bad] = gnn[bad]
            follow["nn_override"] = fnn
            st = replay_prefill(orc, l, b, h, K64, V64, **follow)
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
                assert _thr_tie(mx_o[i], st.log["thr"], tie_rtol), \
                    f"merge decision differs beyond a tie: row {i}: mx {mx_o[i]} thr {st.log['thr']}"
            rep.ties["mask"] += int(flip.size)
            follow["mask_override"] = gmask
            st = replay_prefill(orc, l, b, h, K64, V64, **follow)
    _compare_state(rep, got, st, wl.dtype, "prefill", st.log.get("K_exact"), st.log.get("V_exact"),
                   st.log.get("touched"))


def _compare_state(rep, got, st, dtype, tag, K_exact=None, V_exact=None, merged_rows=None):
    """`K_exact`/`V_exact`: the oracle's unrounded merged rows ([len, d], or None when nothing was merged);
    `merged_rows`: boolean [len], the rows written by a merge in the step just compared."""
    gpos = got["pos"].numpy().astype(np.int64)
    order = np.argsort(gpos, kind="stable")
    assert np.array_equal(gpos[order], st.pos), f"{tag}: cache positions differ"
    Kg, Vg = got["K"].double().numpy()[order], got["V"].double().numpy()[order]
    eK, eV = close(Kg, st.K, dtype), close(Vg, st.V, dtype)
    rep.err(f"{tag}_K", eK)
    rep.err(f"{tag}_V", eV)
    if dtype != "f32" and eK <= 1.0 and eV <= 1.0:
        # storage-follow, 16-bit caches only (see the module docstring); every adopted element is checked
        for name, G_, R_, X_ in (("K", Kg, st.K, K_exact), ("V", Vg, st.V, V_exact)):
            diff = G_ != R_
            if not diff.any():
                continue
            assert merged_rows is not None and X_ is not None, f"{tag}: {name} differs in a step without a merge"
            rows = np.nonzero(diff.any(axis=1))[0]
            assert np.all(np.asarray(merged_rows)[rows]), f"{tag}: {name} differs outside the merged rows {rows}"
            # The GPU forms the merged value in float32: its unrounded value lies within tol of the oracle's exact one,
            # so what it stores must be the rounding of something in [exact - tol, exact + tol] (rounding is monotone)
            X_ = np.asarray(X_)
            scale = np.maximum(np.abs(X_), np.sqrt(np.mean(X_[rows] ** 2)))
            tol = BOUNDARY_RTOL[tag] * scale
            lo, hi = O.round_storage(X_ - tol, dtype), O.round_storage(X_ + tol, dtype)
            need = (np.abs(G_ - X_) - np.abs(R_ - X_))[diff] / scale[diff]      # how far past its own rounding
            rep.err(f"{tag}_boundary_rel", float(need.max()))
            bad = diff & ((G_ < lo) | (G_ > hi))
            assert not bad.any(), \
                f"{tag}: {int(bad.sum())} adopted {name} elements are not roundings of a value within {BOUNDARY_RTOL[tag]:.0e} of the exact one"
            rep.storage_flips += int(diff.sum())
        st.K, st.V = Kg.copy(), Vg.copy()
    sc = got["score"].double().numpy()[order]
    rep.err(f"{tag}_score_rel", np.max(np.abs(sc - st.score) / np.maximum(np.abs(st.score), 1e-6)))
    # the cached inverse norms belong to the stored rows the similarity is computed on
    Fg = O.feature_rows(got["K"].double().numpy(), got["V"].double().numpy(), st.feature)
    nrm = np.sqrt((Fg * Fg).sum(axis=1))
    rn = got["rnorm"].double().numpy()
    ok = nrm > 0
    rep.err(f"{tag}_rnorm_rel", np.max(np.abs(rn[ok] * nrm[ok] - 1.0)) if ok.any() else 0.0)
    assert np.all(rn[~ok] == 0.0), f"{tag}: a zero row must have inverse norm 0"


def _check_decode_slice(rep, ctx, orc, wl, l, b, h, q, k, v, out, step, tabs, tie_rtol):
    G = wl.group
    key = (l, b, h)
    t = orc.Pb[b] + step
    before = copy.deepcopy(orc.slices[key])
    got = ctx.slice_state(l, b, h, tabs)
    gset = set(got["pos"].tolist())
    qs, ks, vs = q[b, h * G:(h + 1) * G], k[b, h], v[b, h]

    def attempt(victim=None, nn=None, tau_override=None):
        st = copy.deepcopy(before)
        tov = orc.tau_override if tau_override is None else tau_override
        if victim is None and nn is None:
            o, log = O.decode_step_slice(st, qs, ks, vs, t, orc.beta, tov)
        else:
            o, log = replay_decode(st, qs, ks, vs, t, orc.beta, tov, victim, nn)
        return st, o, log

    st, o, log = attempt()
    fv = None
    if log.evicted and set(st.pos.tolist()) != gset:
        gone = sorted((set(before.pos.tolist()) | {t}) - gset)
        assert len(gone) == 1, f"GPU cache lost {gone} at t={t}"
        assert log.victim_gap <= tie_rtol and gone[0] == log.runner_up_pos, \
            f"victim differs beyond a tie at t={t} slice {key}: GPU {gone[0]} oracle {log.victim_pos} gap {log.victim_gap:.3e}"
        rep.ties["victim"] += 1
        fv = gone[0]
        st, o, log = attempt(victim=fv)
    # merged / discarded and neighbour choice show in the cache content
    e = _state_err(got, st, wl.dtype)
    if log.evicted and e > 1.0:
        tried = False
        if _thr_tie(log.mx, log.tau, tie_rtol):               # threshold tie: replay the other decision
            alt = float("inf") if log.merged else float("-inf")
            st2, o2, log2 = attempt(victim=fv, tau_override=alt)
            st2.tau = st.tau
            if _state_err(got, st2, wl.dtype) <= 1.0:
                st, o, log, tried = st2, o2, log2, True
                rep.ties["dec_merge"] += 1
        if not tried and log.nn_gap <= tie_rtol:              # neighbour tie
            st2, o2, log2 = attempt(victim=fv, nn=log.nn_runner_pos)
            if _state_err(got, st2, wl.dtype) <= 1.0:
                st, o, log, tried = st2, o2, log2, True
                rep.ties["dec_nn"] += 1
        assert tried, f"cache content differs at t={t} slice {key}: err {e:.3f} (mx {log.mx}, tau {log.tau}, nn_gap {log.nn_gap})"
    orc.slices[key] = st
    rep.err("out", close(out[b, h * G:(h + 1) * G], o, wl.dtype))
    Kx = Vx = rows = None
    if log.merged:
        rows = st.pos == log.nn_pos
        Kx = np.where(rows[:, None], log.K_exact[None, :], st.K)
        Vx = np.where(rows[:, None], log.V_exact[None, :], st.V)
    _compare_state(rep, got, st, wl.dtype, "decode", Kx, Vx, rows)
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


def assert_report(rep: Report, dtype: str, max_ties: int = 0):
    """`max_ties`: tolerated near-ties (counted and reported).  The committed configurations produce none."""
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
    assert sum(rep.ties.values()) <= max_ties, rep.ties
