"""Plain CPU oracle for the D2O KV-cache compression hot path (arXiv 2406.13035).

TEST INFRASTRUCTURE ONLY.  This file is the slow, obviously-correct statement of
what the path computes, written from the paper's equations in float64 NumPy.
It shares no code with the CUDA library and must never be imported by the
product path; only the tests, the smoke check and the benchmark's CPU-baseline
leg call it.

Notation follows the paper: ``P`` = L_prompt, ``S`` = S_l (cache size of one
layer), ``T`` sink tokens, ``M`` recent window, ``N = S - T - M`` heavy hitters,
``K_c/V_c`` the conserved cache, ``K_e/V_e`` the evicted tokens, ``U`` the
cosine-similarity matrix, ``tau`` the EMA threshold, ``beta`` its smoothing
constant.  One *slice* is one (sequence, layer, KV head) with its ``G`` query
heads; slices are independent once the layer budgets are known.

Arithmetic is float64 on the (already storage-dtype-rounded) inputs.  The only
places where a storage dtype enters are the merged rows of ``K_c``/``V_c``,
which a real cache stores in the model dtype: they are rounded (nearest-even)
right after a merge, exactly where the cache is written.

Pins (tests/test_oracle_pins.py): closed forms, invariants, brute force and
library routines for every function below.  The end-to-end numeric values of a
compressed run have no published reference: *parity unpinned* beyond those
per-step pins.

The functions read top to bottom as the paper's steps.  Nothing in here replays
another implementation's choices: a harness that wants to follow a near-tie
composes the step functions itself.

Readings of points the paper leaves open are marked "Reading:" where they are
taken.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field
from typing import List, Optional, Tuple

import numpy as np

E = math.e  # weight of a conserved token in the merge: exp(self-similarity = 1)  (Eq. 12)


# --------------------------------------------------------------------------------------
# storage rounding
# --------------------------------------------------------------------------------------
def round_storage(x: np.ndarray, dtype: str) -> np.ndarray:
    """Round float64 values to the nearest value representable in the cache dtype
    ("f32", "f16", "bf16"; ties to even) and return them as float64."""
    x = np.asarray(x, dtype=np.float64)
    if dtype == "f32":
        return x.astype(np.float32).astype(np.float64)
    if dtype == "f16":
        return x.astype(np.float16).astype(np.float64)
    if dtype == "bf16":
        # bf16 = 8 significant bits (1 implicit + 7 stored) with the float32 exponent range.
        m, e = np.frexp(x)                       # x = m * 2**e, 0.5 <= |m| < 1
        r = np.rint(m * 256.0) / 256.0           # np.rint rounds half to even
        return np.ldexp(r, e)
    raise ValueError(f"unknown dtype {dtype!r}")


# --------------------------------------------------------------------------------------
# layer level: attention density and budgets (Section 4.1, Eq. 4, Eq. 5, Appendix A.2)
# --------------------------------------------------------------------------------------
def colsum_scores(Q: np.ndarray, K: np.ndarray, row_block: int = 512) -> np.ndarray:
    """Column sums of the prompt attention matrix of one query head (Eq. 4, Eq. 6 case 1).

    ``A_p = Softmax(Q K^T / sqrt(d))`` row by row, ``s_j = sum_i A_p[i, j]``.
    Reading: the softmax scale is 1/sqrt(d_head) (the paper drops head indices) and the
    prompt attention is causal (decoder-only models), so row ``i`` covers columns
    ``j <= i``; the sum runs over all ``P`` rows.  ``row_block`` only bounds memory:
    rows are independent and are visited in order."""
    Q = np.asarray(Q, dtype=np.float64)
    K = np.asarray(K, dtype=np.float64)
    P, d = Q.shape
    s = np.zeros(P, dtype=np.float64)
    cols = np.arange(P)
    for r0 in range(0, P, row_block):
        r1 = min(r0 + row_block, P)
        logits = Q[r0:r1] @ K.T / math.sqrt(d)                     # [rows, P]
        rows = np.arange(r0, r1)
        logits = np.where(cols[None, :] <= rows[:, None], logits, -np.inf)
        logits = logits - logits.max(axis=1, keepdims=True)
        A = np.exp(logits)
        A = A / A.sum(axis=1, keepdims=True)
        s += A.sum(axis=0)
    return s


def attention_density(s: np.ndarray) -> float:
    """F_v = Var(s) (Eq. 4).  Reading: population variance (divide by P)."""
    s = np.asarray(s, dtype=np.float64)
    mean = s.sum() / s.size
    return float(((s - mean) ** 2).sum() / s.size)


def layer_weights(F: np.ndarray, gamma: float = 1.0, head_reduce: int = 0) -> np.ndarray:
    """Un-normalised allocation weight of each layer.

    ``F`` is [L, H] (one density per layer and query head).
    head_reduce 0 (default; appendix form, Eq. for alpha_l^h): w_l = sum_h exp(-F_lh/gamma)
    head_reduce 1: w_l = exp(-mean_h(F_lh)/gamma)   (main-text form with a per-layer mean)
    head_reduce 2, 3: w_l = sum_h 1/F_lh, 1/mean_h(F_lh)   (the ablation's reciprocal-of-variance allocation)
    ``gamma`` = 1 is the paper's formula.  The common factor exp(F_min/gamma) is taken out
    for numerical stability; it cancels in the normalisation."""
    F = np.asarray(F, dtype=np.float64)
    if F.ndim == 1:
        F = F[:, None]
    if head_reduce == 0:
        return np.exp(-(F - F.min()) / gamma).sum(axis=1)
    if head_reduce == 1:
        Fm = F.sum(axis=1) / F.shape[1]
        return np.exp(-(Fm - Fm.min()) / gamma)
    # reciprocal-of-variance allocation (Section 5.4, setting 2): alpha_l proportional to 1 / F; per head (2) or on
    # the mean over heads (3); a zero variance counts as the smallest positive one
    tiny = 1e-300
    if head_reduce == 2:
        return np.minimum((1.0 / np.maximum(F, tiny)).sum(axis=1), 1e300)
    if head_reduce == 3:
        Fm = F.sum(axis=1) / F.shape[1]
        return np.minimum(1.0 / np.maximum(Fm, tiny), 1e300)
    raise ValueError("head_reduce must be 0, 1, 2 or 3")


def allocate_budgets(w: np.ndarray, S_tot: int, lo: int, cap: int) -> np.ndarray:
    """Integer sizes x_u = clip(lam * w_u, lo, cap) of allocation units (layers, or (layer, head) pairs)
    with the single scale ``lam`` that makes them add up to ``S_tot``, then floor + largest remainder.

    Reading (the paper gives S_u = alpha_u * S with sum alpha_u fixed, and is silent on bounds and on
    integer sizes): a unit cannot hold fewer than ``lo`` or more than ``cap`` tokens; the proportional
    rule is kept for every unit that neither bound touches (equal to the unclamped formula when no
    clamp binds); remainders go to the largest fractional parts, ties to the lower unit index."""
    w = np.maximum(np.asarray(w, dtype=np.float64), 1e-300)        # exp underflow: keep ratios finite
    n = w.size
    lo_f, hi_f = float(lo), float(cap)
    if not (n * lo_f <= S_tot <= n * hi_f):
        raise ValueError("global budget outside [n*min_budget, n*max_budget]")

    def total(lam: float) -> float:
        return float(np.clip(lam * w, lo_f, hi_f).sum())

    # total(lam) is continuous, piecewise linear and non-decreasing; its kinks are where
    # a unit leaves the lower clamp (lo/w_u) or reaches the upper one (cap/w_u).
    kinks = np.sort(np.concatenate([lo_f / w, hi_f / w]))
    k = 0
    while k < kinks.size and total(kinks[k]) < S_tot:
        k += 1
    if k == 0:
        lam = kinks[0]
    elif k == kinks.size:
        lam = kinks[-1]
    else:
        a, b = kinks[k - 1], kinks[k]
        mid = 0.5 * (a + b)
        free = (mid * w > lo_f) & (mid * w < hi_f)     # units on the linear part of this segment
        fixed = float(np.clip(mid * w, lo_f, hi_f)[~free].sum())
        wf = float(w[free].sum())
        lam = (S_tot - fixed) / wf if wf > 0.0 else b
        lam = min(max(lam, a), b)
    x = np.clip(lam * w, lo_f, hi_f)
    base = np.floor(x)
    rem = x - base
    S = base.astype(np.int64)
    left = S_tot - int(S.sum())
    assert 0 <= left <= n, "largest-remainder step out of range"
    order = sorted(range(n), key=lambda u: (-rem[u], u))
    for u in order:
        if left == 0:
            break
        if S[u] < cap:
            S[u] += 1
            left -= 1
    assert left == 0
    return S


def layer_budgets(F: np.ndarray, P: int, rho: float, min_budget: int = 1,
                  gamma: float = 1.0, head_reduce: int = 0, max_budget: int = 0) -> np.ndarray:
    """Integer cache size S_l of every layer (Eq. 5; constraint sum_l S_l = S*L*rho).

    Unclamped, S_l = alpha_l * P with alpha_l = L*rho*w_l / sum_l w_l.
    Reading: S_tot = floor(rho*L*P + 1/2); bounds ``min_budget`` and ``max_budget`` (``P`` unless
    given: the prompt has no more) and integer sizes as in allocate_budgets."""
    w = layer_weights(F, gamma, head_reduce)
    L = w.size
    S_tot = int(math.floor(rho * L * P + 0.5))
    cap = max_budget if max_budget > 0 else P
    return allocate_budgets(w, S_tot, min_budget, cap)


def head_budgets(F: np.ndarray, P: int, rho: float, group: int = 1, min_budget: int = 1,
                 gamma: float = 1.0, max_budget: int = 0) -> np.ndarray:
    """Per-head cache sizes S_l^h = alpha_l^h * S_total of the appendix ("Cache Size Allocation Based
    on Attention Variance"): alpha_l^h = exp(-F_lh) / sum_{l,h} exp(-F_lh), so that
    S_l = sum_h S_l^h and alpha_l = sum_h alpha_l^h.  Returns int64 [L, Hkv].

    Reading: the unit that owns cache rows is a KV head; with grouped queries its weight is the sum
    of the weights of its ``group`` query heads (the same sum that forms its attention score), and
    S_total = floor(rho * L * Hkv * P + 1/2) head-tokens, i.e. the same number of cache rows as the
    per-layer rule.  Bounds and integer sizes as in allocate_budgets."""
    F = np.asarray(F, dtype=np.float64)
    L, H = F.shape
    assert H % group == 0
    Hkv = H // group
    wq = np.exp(-(F - F.min()) / gamma).reshape(L, Hkv, group)     # [L, Hkv, G]
    w = np.zeros((L, Hkv))
    for g in range(group):                                         # query heads of a KV head, in order
        w = w + wq[:, :, g]
    w = w.reshape(-1)                                              # [L * Hkv]
    S_tot = int(math.floor(rho * (L * Hkv) * P + 0.5))
    cap = max_budget if max_budget > 0 else P
    return allocate_budgets(w, S_tot, min_budget, cap).reshape(L, Hkv)


def exp_decay_budgets(F: np.ndarray, P: int, min_budget: int = 1, gamma: float = 1.0,
                      max_budget: int = 0) -> np.ndarray:
    """The ablation's "Exponential Decay Allocation" (Section 5.4, setting 3): alpha_l = exp(-F_l),
    S_l = alpha_l * P.  The factor is not normalised, so the total is whatever the densities give.

    Reading: with several heads alpha_l is the mean over the query heads of exp(-F_lh / gamma)
    (a fraction in (0, 1]; one head gives the printed formula); S_l = floor(alpha_l * P + 1/2)
    clamped to [min_budget, max_budget]."""
    F = np.asarray(F, dtype=np.float64)
    if F.ndim == 1:
        F = F[:, None]
    e = np.exp(-F / gamma)
    alpha = np.zeros(F.shape[0])
    for h in range(F.shape[1]):                                    # query heads in order
        alpha = alpha + e[:, h]
    alpha = alpha / F.shape[1]
    cap = max_budget if max_budget > 0 else P
    S = np.floor(alpha * P + 0.5).astype(np.int64)
    return np.clip(S, min_budget, cap)


def window_size(S: int, T: int, window: int, nm_ratio: float) -> int:
    """Recent-window size M of a layer with cache size S.

    ``window`` > 0 fixes M; otherwise N:M = nm_ratio (3:1 in the paper, Section 5.1) with
    N + M + T = S, i.e. M = round((S - T) / (1 + nm_ratio)).  M is limited to S - T."""
    if window > 0:
        M = window
    else:
        M = int(math.floor((S - T) / (1.0 + nm_ratio) + 0.5))
    return max(0, min(M, S - T))


# --------------------------------------------------------------------------------------
# token level, prompt stage (Section 4.2: Eq. 7-12)
# --------------------------------------------------------------------------------------
def select_retained(score: np.ndarray, S: int, T: int, M: int) -> Tuple[np.ndarray, np.ndarray]:
    """Positions kept / evicted by Eq. 7-8: the first T (sinks), the last M (recent window)
    and the Top-N of AttnScore[T:P-M], N = S - T - M.

    Reading: equal scores are ordered by position (earlier first).  Returns
    (retained positions ascending, evicted positions ascending)."""
    score = np.asarray(score, dtype=np.float64)
    P = score.size
    if S >= P:
        return np.arange(P, dtype=np.int64), np.zeros(0, dtype=np.int64)
    N = S - T - M
    assert N >= 0 and T >= 0 and M >= 0
    cand = list(range(T, P - M))
    cand.sort(key=lambda j: (-score[j], j))
    keep = set(range(T)) | set(cand[:N]) | set(range(P - M, P))
    retained = np.array(sorted(keep), dtype=np.int64)
    evicted = np.array([j for j in range(P) if j not in keep], dtype=np.int64)
    return retained, evicted


def cosine_matrix(Ke: np.ndarray, Kc: np.ndarray) -> np.ndarray:
    """U[i, j] = k_i . k_j / (|k_i| |k_j|) for evicted i, conserved j (Eq. 9).
    Reading: a zero-norm key has similarity 0 to everything."""
    Ke = np.asarray(Ke, dtype=np.float64)
    Kc = np.asarray(Kc, dtype=np.float64)
    dots = Ke @ Kc.T
    ne = np.sqrt((Ke * Ke).sum(axis=1))
    nc = np.sqrt((Kc * Kc).sum(axis=1))
    den = ne[:, None] * nc[None, :]
    return np.where(den > 0.0, dots / np.where(den > 0.0, den, 1.0), 0.0)


def nearest_neighbour(U: np.ndarray) -> Tuple[np.ndarray, np.ndarray]:
    """Row maximum and its column (Eq. 9's Argmax).  Ties: lowest column."""
    if U.shape[0] == 0:
        return np.zeros(0), np.zeros(0, dtype=np.int64)
    nn = np.argmax(U, axis=1)          # first maximum
    mx = U[np.arange(U.shape[0]), nn]
    return mx, nn.astype(np.int64)


def initial_threshold(mx: np.ndarray) -> float:
    """tau_0 = mean over evicted tokens of their best similarity (Eq. 10, t = 0)."""
    return float(mx.sum() / mx.size) if mx.size else 0.0


def merge_mask(mx: np.ndarray, tau: float) -> np.ndarray:
    """m_i of Eq. 12 for the nearest neighbour of evicted token i: it is merged iff its best
    similarity is not lower than the threshold ("lower than tau: permanently discarded")."""
    return np.asarray(mx, dtype=np.float64) >= tau


def weighted_merge(Kc: np.ndarray, Vc: np.ndarray, Ke: np.ndarray, Ve: np.ndarray,
                   mx: np.ndarray, nn: np.ndarray, mask: np.ndarray,
                   policy: str = "weighted") -> Tuple[np.ndarray, np.ndarray, np.ndarray]:
    """Eq. 11-12 for all conserved tokens at once.

    ``mask[i]`` says whether evicted token i is merged into conserved token ``nn[i]``
    (m_ij = 1 iff j is i's nearest neighbour and i passed the threshold, see merge_mask).
    Reading of Eq. 12: the weight of evicted token i is
    exp(u_ij) m_ij / (sum_i' exp(u_i'j) m_i'j + e), so the weights of a conserved token
    and of everything merged into it sum to one.
    ``policy`` "average" is the ablation's average merging ("Merge Policy"): the conserved token and
    every token merged into it weigh the same, 1 / (1 + number merged).
    Returns (K_c', V_c', denominators; a conserved token's own weight is e, or 1, over its denominator)."""
    if policy not in ("weighted", "average"):
        raise ValueError("policy must be 'weighted' or 'average'")
    Kc = np.array(Kc, dtype=np.float64)
    Vc = np.array(Vc, dtype=np.float64)
    Lc = Kc.shape[0]
    own = E if policy == "weighted" else 1.0
    den = np.full(Lc, own, dtype=np.float64)
    Kn = own * Kc
    Vn = own * Vc
    for i in range(len(mx)):
        if mask[i]:
            j = int(nn[i])
            w = math.exp(mx[i]) if policy == "weighted" else 1.0
            den[j] += w
            Kn[j] += w * Ke[i]
            Vn[j] += w * Ve[i]
    return Kn / den[:, None], Vn / den[:, None], den


@dataclass
class SliceState:
    """Compressed cache of one (sequence, layer, KV head), kept in ascending position."""
    pos: np.ndarray        # int64 [len]   original token positions
    K: np.ndarray          # float64 [len, d], values representable in the cache dtype
    V: np.ndarray
    score: np.ndarray      # float64 [len]  accumulated attention (summed over the G query heads)
    tau: float
    S: int                 # cache size S_l
    T: int
    M: int
    dtype: str
    feature: str = "k"     # rows the similarity is computed on: keys (the method) or values (ablation)
    policy: str = "weighted"
    log: dict = field(default_factory=dict)


def feature_rows(K: np.ndarray, V: np.ndarray, feature: str) -> np.ndarray:
    """Rows that enter the similarity of Eq. 9: the keys in the method ("we compute the similarity
    matrix only on the key tokens"); the values in the ablation's "Feature choice" row V."""
    if feature == "k":
        return K
    if feature == "v":
        return V
    raise ValueError("feature must be 'k' or 'v'")


def prefill_compress_slice(K: np.ndarray, V: np.ndarray, score: np.ndarray, S: int, T: int, M: int,
                           dtype: str, tau_override: float = float("nan"), feature: str = "k",
                           policy: str = "weighted") -> SliceState:
    """Prompt-stage compression of one slice: eviction (Eq. 7-8), nearest-neighbour
    matching (Eq. 9), tau_0 (Eq. 10) and weighted merging (Eq. 11-12).

    ``score`` is the accumulated attention of the prompt (Eq. 6 case 1), already summed
    over the query heads that share this KV head (reading for grouped-query attention).
    Reading: similarities use the un-merged keys and all merges happen at once;
    every conserved slot (sinks and window included) can receive merges;
    a conserved token keeps its own accumulated score."""
    K = np.asarray(K, dtype=np.float64)
    V = np.asarray(V, dtype=np.float64)
    retained, evicted = select_retained(score, S, T, M)                      # Eq. 7-8
    Kc, Vc = K[retained], V[retained]
    Ke, Ve = K[evicted], V[evicted]
    U = cosine_matrix(feature_rows(Ke, Ve, feature), feature_rows(Kc, Vc, feature))   # Eq. 9
    mx, nn = nearest_neighbour(U)
    tau0 = initial_threshold(mx)                                             # Eq. 10, t = 0
    thr = tau0 if math.isnan(tau_override) else tau_override
    mask = merge_mask(mx, thr)
    Km, Vm, den = weighted_merge(Kc, Vc, Ke, Ve, mx, nn, mask, policy)       # Eq. 11-12
    touched = den > (E if policy == "weighted" else 1.0)
    Kn = np.where(touched[:, None], round_storage(Km, dtype), Kc)
    Vn = np.where(touched[:, None], round_storage(Vm, dtype), Vc)
    st = SliceState(pos=retained.copy(), K=Kn, V=Vn, score=np.asarray(score, np.float64)[retained].copy(),
                    tau=tau0, S=S, T=T, M=M, dtype=dtype, feature=feature, policy=policy)
    st.log = dict(retained=retained, evicted=evicted, mx=mx, nn=nn, den=den, U=U, thr=thr, merged=mask,
                  K_exact=Km, V_exact=Vm, touched=touched)
    return st


# --------------------------------------------------------------------------------------
# token generation (Eq. 2-3, Eq. 6 case 2, Eq. 7-8, Eq. 9, Eq. 10 case 2, Eq. 11-12)
# --------------------------------------------------------------------------------------
def softmax_attention(q: np.ndarray, K: np.ndarray, V: np.ndarray) -> Tuple[np.ndarray, np.ndarray]:
    """Eq. 3 for one query: returns (Softmax(q K^T / sqrt(d)) V, the probabilities)."""
    d = q.size
    z = K @ q / math.sqrt(d)
    z = z - z.max()
    p = np.exp(z)
    p = p / p.sum()
    return p @ V, p


@dataclass
class StepLog:
    victim_pos: int = -1
    victim_gap: float = float("inf")      # relative score gap to the runner-up victim
    runner_up_pos: int = -1
    mx: float = float("nan")
    nn_pos: int = -1
    nn_gap: float = float("inf")          # absolute similarity gap to the second-best neighbour
    nn_runner_pos: int = -1
    tau: float = float("nan")
    merged: bool = False
    evicted: bool = False
    K_exact: Optional[np.ndarray] = None  # the merged rows before storage rounding
    V_exact: Optional[np.ndarray] = None


def decode_attend(st: SliceState, q: np.ndarray, k: np.ndarray, v: np.ndarray, t: int) -> np.ndarray:
    """Append the new token (Eq. 2), attend over the cache including it (Eq. 3), and add the
    probabilities of the G query heads to AttnScore (Eq. 6 case 2).  Returns the outputs [G, d]."""
    q = np.asarray(q, dtype=np.float64).reshape(-1, np.asarray(k).size)
    st.pos = np.append(st.pos, t)
    st.K = np.vstack([st.K, np.asarray(k, np.float64)[None, :]])
    st.V = np.vstack([st.V, np.asarray(v, np.float64)[None, :]])
    st.score = np.append(st.score, 0.0)
    out = np.zeros_like(q)
    for g in range(q.shape[0]):
        o, p = softmax_attention(q[g], st.K, st.V)
        out[g] = o
        st.score += p
    return out


def victim_order(st: SliceState, t: int) -> List[int]:
    """Rows that may be evicted at step ``t`` (outside the T sinks and the M most recent positions,
    Eq. 7-8), worst first.  Reading: lowest score first, equal scores -> the later position first."""
    elig = [i for i in range(st.pos.size) if st.T <= st.pos[i] <= t - st.M]
    return sorted(elig, key=lambda i: (st.score[i], -st.pos[i]))


def evict_row(st: SliceState, vi: int) -> Tuple[np.ndarray, np.ndarray]:
    """Remove row ``vi`` from the cache; returns its key and value."""
    k_e, v_e = st.K[vi].copy(), st.V[vi].copy()
    keep = np.arange(st.pos.size) != vi
    st.pos, st.K, st.V, st.score = st.pos[keep], st.K[keep], st.V[keep], st.score[keep]
    return k_e, v_e


def neighbour_order(st: SliceState, k_e: np.ndarray, v_e: np.ndarray) -> Tuple[np.ndarray, List[int]]:
    """U = cosine of the evicted token with every remaining row (Eq. 9, one evicted token) and the
    rows ordered best first.  Reading: equal similarity -> the earlier position first."""
    U = cosine_matrix(feature_rows(k_e, v_e, st.feature)[None, :], feature_rows(st.K, st.V, st.feature))[0]
    return U, sorted(range(U.size), key=lambda j: (-U[j], st.pos[j]))


def compensate(st: SliceState, k_e: np.ndarray, v_e: np.ndarray, nj: int, mx: float, beta: float,
               tau_override: float, log: StepLog) -> None:
    """tau_t = beta * Max(U_t) + (1 - beta) * tau_{t-1} (Eq. 10), then merge the evicted token into row
    ``nj`` if mx >= tau_t, with weights e^{u}/(e^{u}+e) and e/(e^{u}+e) (Eq. 11-12 with one evicted
    token), else discard it.  Reading: the threshold is updated first, then compared; the neighbour
    keeps its own score; the merged rows are rounded to the cache dtype where they are stored."""
    st.tau = beta * mx + (1.0 - beta) * st.tau
    thr = st.tau if math.isnan(tau_override) else tau_override
    log.mx, log.nn_pos, log.tau = mx, int(st.pos[nj]), st.tau
    if merge_mask(np.array([mx]), thr)[0]:
        Km, Vm, _ = weighted_merge(st.K[nj][None, :], st.V[nj][None, :], k_e[None, :], v_e[None, :],
                                   np.array([mx]), np.array([0]), np.array([True]), st.policy)
        log.K_exact, log.V_exact = Km[0], Vm[0]
        st.K[nj] = round_storage(Km[0], st.dtype)
        st.V[nj] = round_storage(Vm[0], st.dtype)
        log.merged = True


def decode_step_slice(st: SliceState, q: np.ndarray, k: np.ndarray, v: np.ndarray, t: int, beta: float,
                      tau_override: float = float("nan")) -> Tuple[np.ndarray, StepLog]:
    """One generated token for one slice.  ``q`` [G, d], ``k``/``v`` [d], ``t`` = position of
    the new token.  Returns the attention outputs [G, d] (float64) and a log.

    Steps: append, attend, accumulate (decode_attend); if the cache now exceeds S: evict the
    lowest-scoring token outside the T sinks and the M most recent positions (victim_order,
    evict_row); cosine of the evicted token to every remaining one (neighbour_order);
    threshold update and merge-or-discard (compensate)."""
    out = decode_attend(st, q, k, v, t)
    log = StepLog(tau=st.tau)
    if st.pos.size <= st.S:
        return out, log
    ranked = victim_order(st, t)
    assert ranked, "no evictable slot: S < T + M"
    if len(ranked) > 1:
        a, b = st.score[ranked[0]], st.score[ranked[1]]
        log.victim_gap = abs(b - a) / max(abs(a), abs(b), 1e-300)
        log.runner_up_pos = int(st.pos[ranked[1]])
    log.victim_pos = int(st.pos[ranked[0]])
    log.evicted = True
    k_e, v_e = evict_row(st, ranked[0])
    U, order = neighbour_order(st, k_e, v_e)
    if len(order) > 1:
        log.nn_gap = float(U[order[0]] - U[order[1]])
        log.nn_runner_pos = int(st.pos[order[1]])
    compensate(st, k_e, v_e, order[0], float(U[order[0]]), beta, tau_override, log)
    return out, log


def full_attention_step(q: np.ndarray, K: np.ndarray, V: np.ndarray) -> np.ndarray:
    """Uncompressed decode attention (Eq. 3) for the G query heads of one KV head."""
    q = np.asarray(q, dtype=np.float64).reshape(-1, K.shape[1])
    return np.stack([softmax_attention(q[g], np.asarray(K, np.float64), np.asarray(V, np.float64))[0]
                     for g in range(q.shape[0])])


def group_score(colsum: np.ndarray, h: int, G: int) -> np.ndarray:
    """AttnScore of KV head ``h`` at the prompt stage from the per-query-head column sums [Hq, P].
    Reading (grouped-query attention; the paper does not treat it): one retained set per KV head,
    whose score is the sum over its G query heads' attention, at the prompt stage as in decode_attend."""
    return np.asarray(colsum, dtype=np.float64)[h * G:(h + 1) * G].sum(axis=0)


# --------------------------------------------------------------------------------------
# whole path for a small stack (used by the parity tests, the smoke check and the timed
# CPU baseline).  Tensors: Q [B,Hq,P,d], K/V [B,Hkv,P,d] per layer.
# --------------------------------------------------------------------------------------
class OracleStack:
    """``prompt_lens`` (one length per sequence, each <= prompt_len) makes the batch ragged: sequence b
    uses the first prompt_lens[b] positions of its tensors, its own budgets, and its generated tokens
    continue at position prompt_lens[b].  ``budget_rule``: "layer" (Eq. 5), "head" (per-head sizes of
    the appendix) or "exp_decay" (Section 5.4, setting 3)."""

    def __init__(self, *, n_layers: int, batch: int, n_q_heads: int, n_kv_heads: int, d_head: int,
                 dtype: str, prompt_len: int, rho: float, n_sink: int, window: int, nm_ratio: float,
                 beta: float, density_temp: float = 1.0, min_budget: int = 1, head_reduce: int = 0,
                 tau_override: float = float("nan"), max_budget: int = 0, feature: str = "k",
                 policy: str = "weighted", budget_rule: str = "layer",
                 prompt_lens: Optional[List[int]] = None):
        self.L, self.B, self.Hq, self.Hkv, self.d = n_layers, batch, n_q_heads, n_kv_heads, d_head
        self.G = n_q_heads // n_kv_heads
        self.dtype, self.P, self.rho = dtype, prompt_len, rho
        self.T, self.window, self.nm_ratio, self.beta = n_sink, window, nm_ratio, beta
        self.gamma, self.min_budget, self.head_reduce = density_temp, min_budget, head_reduce
        self.tau_override = tau_override
        self.max_budget = max_budget
        self.feature, self.policy, self.budget_rule = feature, policy, budget_rule
        self.Pb = [prompt_len] * batch if prompt_lens is None else [int(p) for p in prompt_lens]
        assert len(self.Pb) == batch and all(1 <= p <= prompt_len for p in self.Pb)
        self.colsum = np.zeros((self.L, self.B, self.Hq, self.P))
        self.F = np.zeros((self.B, self.L, self.Hq))
        self.budgets: Optional[np.ndarray] = None          # [B, L, Hkv]
        self.slices: dict = {}

    def layer_stats(self, layer: int, Q: np.ndarray, K: np.ndarray, heads: Optional[List[Tuple[int, int]]] = None):
        """Column sums and densities of one layer; ``heads`` restricts to (b, hq) pairs."""
        todo = heads if heads is not None else [(b, h) for b in range(self.B) for h in range(self.Hq)]
        for b, h in todo:
            Pb = self.Pb[b]
            s = colsum_scores(Q[b, h][:Pb], K[b, h // self.G][:Pb])
            self.colsum[layer, b, h, :Pb] = s
            self.F[b, layer, h] = attention_density(s)

    def layer_budgets(self, F: Optional[np.ndarray] = None) -> np.ndarray:
        """Cache size of every (sequence, layer, KV head), int64 [B, L, Hkv]; the per-layer rules give
        all KV heads of a layer the same size."""
        F = self.F if F is None else np.asarray(F, np.float64)
        out = np.zeros((self.B, self.L, self.Hkv), dtype=np.int64)
        for b in range(self.B):
            Pb = self.Pb[b]
            cap = self.max_budget if self.max_budget > 0 else Pb
            if self.budget_rule == "layer":
                out[b] = layer_budgets(F[b], Pb, self.rho, self.min_budget, self.gamma, self.head_reduce,
                                       cap)[:, None]
            elif self.budget_rule == "head":
                out[b] = head_budgets(F[b], Pb, self.rho, self.G, self.min_budget, self.gamma, cap)
            elif self.budget_rule == "exp_decay":
                out[b] = exp_decay_budgets(F[b], Pb, self.min_budget, self.gamma, cap)[:, None]
            else:
                raise ValueError("budget_rule must be 'layer', 'head' or 'exp_decay'")
        self.budgets = out
        return out

    def slice_params(self, b: int, layer: int, h: int = 0) -> Tuple[int, int, int]:
        S = int(self.budgets[b, layer, h])
        T = min(self.T, S)
        M = window_size(S, T, self.window, self.nm_ratio)
        return S, T, M

    def group_score(self, layer: int, b: int, h: int) -> np.ndarray:
        return group_score(self.colsum[layer, b, :, :self.Pb[b]], h, self.G)

    def prefill_compress(self, layer: int, K: np.ndarray, V: np.ndarray,
                         slices: Optional[List[Tuple[int, int]]] = None):
        """``slices`` restricts to (b, kv head) pairs."""
        todo = slices if slices is not None else [(b, h) for b in range(self.B) for h in range(self.Hkv)]
        for b, h in todo:
            S, T, M = self.slice_params(b, layer, h)
            Pb = self.Pb[b]
            self.slices[(layer, b, h)] = prefill_compress_slice(K[b, h][:Pb], V[b, h][:Pb],
                                                                self.group_score(layer, b, h), S, T, M,
                                                                self.dtype, self.tau_override, self.feature,
                                                                self.policy)

    def decode_step(self, layer: int, q: np.ndarray, k: np.ndarray, v: np.ndarray, step: int,
                    slices: Optional[List[Tuple[int, int]]] = None):
        """Token number ``step`` (0-based) after the prompt: q [B,Hq,d], k/v [B,Hkv,d] ->
        {(b,kvh): (out [G,d], StepLog)}; the new token of sequence b has position prompt_lens[b] + step."""
        todo = slices if slices is not None else [(b, h) for b in range(self.B) for h in range(self.Hkv)]
        res = {}
        for b, h in todo:
            res[(b, h)] = decode_step_slice(self.slices[(layer, b, h)], q[b, h * self.G:(h + 1) * self.G],
                                            k[b, h], v[b, h], self.Pb[b] + step, self.beta, self.tau_override)
        return res
