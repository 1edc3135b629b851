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

Pins (tests/test_oracle_*.py): closed forms, invariants, brute force and
library routines for every function below.  The end-to-end numeric values of a
compressed run have no published reference: *parity unpinned* beyond those
per-step pins.

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
    """Un-normalised inverse-variance-softmax weight of each layer.

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


def layer_budgets(F: np.ndarray, P: int, rho: float, min_budget: int = 1,
                  gamma: float = 1.0, head_reduce: int = 0, max_budget: int = 0) -> np.ndarray:
    """Integer cache size S_l of every layer (Eq. 5; constraint sum_l S_l = S*L*rho).

    Unclamped, S_l = alpha_l * P with alpha_l = L*rho*w_l / sum_l w_l.
    Reading (the paper is silent on all three):
      * a layer cannot hold fewer than ``min_budget`` or more than ``max_budget`` tokens
        (``P`` unless given: the prompt has no more), so
        S_l = clip(lam * w_l, min_budget, max_budget) with the single scale ``lam`` chosen so
        that the total is still S_tot (equal to the unclamped formula when no clamp binds);
      * S_tot = floor(rho*L*P + 1/2);
      * integer sizes by floor + largest remainder (ties: lower layer first)."""
    w = layer_weights(F, gamma, head_reduce)
    L = w.size
    S_tot = int(math.floor(rho * L * P + 0.5))
    cap = max_budget if max_budget > 0 else P
    lo, hi = float(min_budget), float(cap)
    if not (L * lo <= S_tot <= L * hi):
        raise ValueError("global budget outside [L*min_budget, L*max_budget]")
    w = np.maximum(w, 1e-300)        # exp underflow: keep ratios finite

    def total(lam: float) -> float:
        return float(np.clip(lam * w, lo, hi).sum())

    # total(lam) is continuous, piecewise linear and non-decreasing; its kinks are where
    # a layer leaves the lower clamp (lo/w_l) or reaches the upper one (hi/w_l).
    kinks = np.sort(np.concatenate([lo / w, hi / w]))
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
        free = (mid * w > lo) & (mid * w < hi)         # layers on the linear part of this segment
        fixed = float(np.clip(mid * w, lo, hi)[~free].sum())
        wf = float(w[free].sum())
        lam = (S_tot - fixed) / wf if wf > 0.0 else b
        lam = min(max(lam, a), b)
    x = np.clip(lam * w, lo, hi)
    base = np.floor(x)
    rem = x - base
    S = base.astype(np.int64)
    left = S_tot - int(S.sum())
    assert 0 <= left <= L, "largest-remainder step out of range"
    order = sorted(range(L), key=lambda l: (-rem[l], l))
    for l in order:
        if left == 0:
            break
        if S[l] < cap:
            S[l] += 1
            left -= 1
    assert left == 0
    return S


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


def weighted_merge(Kc: np.ndarray, Vc: np.ndarray, Ke: np.ndarray, Ve: np.ndarray,
                   mx: np.ndarray, nn: np.ndarray, tau: float) -> Tuple[np.ndarray, np.ndarray, np.ndarray]:
    """Eq. 11-12 for all conserved tokens at once.

    m_ij = 1 iff j is i's nearest neighbour and i passed the threshold (mx_i >= tau;
    "lower than tau: discarded").  Reading of Eq. 12: the weight of evicted token i is
    exp(u_ij) m_ij / (sum_i' exp(u_i'j) m_i'j + e), so the weights of a conserved token
    and of everything merged into it sum to one.  Returns (K_c', V_c', denominators)."""
    Kc = np.array(Kc, dtype=np.float64)
    Vc = np.array(Vc, dtype=np.float64)
    Lc = Kc.shape[0]
    den = np.full(Lc, E, dtype=np.float64)
    Kn = E * Kc
    Vn = E * Vc
    for i in range(mx.size):
        if mx[i] >= tau:
            j = int(nn[i])
            w = math.exp(mx[i])
            den[j] += w
            Kn[j] += w * Ke[i]
            Vn[j] += w * Ve[i]
    return Kn / den[:, None], Vn / den[:, None], den


def _merge_with_mask(Kc, Vc, Ke, Ve, mx, nn, mask):
    """weighted_merge with an explicit mask m_i instead of the threshold test (harness replay)."""
    passing = np.where(mask, mx, -np.inf)
    return weighted_merge(Kc, Vc, Ke, Ve, passing, nn, -1e300)


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
    log: dict = field(default_factory=dict)


def prefill_compress_slice(K: np.ndarray, V: np.ndarray, score: np.ndarray, S: int, T: int, M: int,
                           dtype: str, tau_override: float = float("nan"),
                           force_retained: Optional[np.ndarray] = None,
                           force_nn: Optional[np.ndarray] = None,
                           force_merged: Optional[np.ndarray] = None) -> SliceState:
    """Prompt-stage compression of one slice: eviction (Eq. 7-8), nearest-neighbour
    matching (Eq. 9), tau_0 (Eq. 10) and weighted merging (Eq. 11-12).

    ``score`` is the accumulated attention of the prompt (Eq. 6 case 1), already summed
    over the query heads that share this KV head (reading for grouped-query attention).
    Reading: similarities use the un-merged keys and all merges happen at once;
    every conserved slot (sinks and window included) can receive merges;
    a conserved token keeps its own accumulated score.
    ``force_*`` let a harness replay another implementation's choice at a near-tie: the kept
    positions, the neighbour column of some evicted rows (-1 = keep own), the merge mask."""
    K = np.asarray(K, dtype=np.float64)
    V = np.asarray(V, dtype=np.float64)
    retained, evicted = select_retained(score, S, T, M)
    if force_retained is not None:
        retained = np.array(sorted(int(j) for j in force_retained), dtype=np.int64)
        keep = set(retained.tolist())
        evicted = np.array([j for j in range(K.shape[0]) if j not in keep], dtype=np.int64)
    Kc, Vc = K[retained], V[retained]
    Ke, Ve = K[evicted], V[evicted]
    U = cosine_matrix(Ke, Kc)
    mx, nn = nearest_neighbour(U)
    if force_nn is not None:
        for i, j in enumerate(force_nn):
            if j >= 0:
                nn[i] = j
                mx[i] = U[i, j]
    tau0 = initial_threshold(mx)
    thr = tau0 if math.isnan(tau_override) else tau_override
    if force_merged is not None:
        # a merge mask is replayed by moving the threshold out of the way row by row
        Km, Vm, den = _merge_with_mask(Kc, Vc, Ke, Ve, mx, nn, np.asarray(force_merged, bool))
    else:
        Km, Vm, den = weighted_merge(Kc, Vc, Ke, Ve, mx, nn, thr)
    touched = den > E
    Kn = np.where(touched[:, None], round_storage(Km, dtype), Kc)
    Vn = np.where(touched[:, None], round_storage(Vm, dtype), Vc)
    st = SliceState(pos=retained.copy(), K=Kn, V=Vn, score=np.asarray(score, np.float64)[retained].copy(),
                    tau=tau0, S=S, T=T, M=M, dtype=dtype)
    st.log = dict(retained=retained, evicted=evicted, mx=mx, nn=nn, den=den, U=U, thr=thr,
                  merged=(np.asarray(force_merged, bool) if force_merged is not None
                          else ((mx >= thr) if mx.size else np.zeros(0, bool))))
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


def decode_step_slice(st: SliceState, q: np.ndarray, k: np.ndarray, v: np.ndarray, t: int, beta: float,
                      tau_override: float = float("nan"),
                      force_victim_pos: Optional[int] = None,
                      force_nn_pos: Optional[int] = None) -> Tuple[np.ndarray, StepLog]:
    """One generated token for one slice.  ``q`` [G, d], ``k``/``v`` [d], ``t`` = position of
    the new token.  Returns the attention outputs [G, d] (float64) and a log.

    Steps: append (Eq. 2); attention over the cache incl. the new token (Eq. 3);
    AttnScore += probabilities summed over the G query heads (Eq. 6 case 2); if the cache
    now exceeds S: evict the lowest-scoring token outside the T sinks and the M most
    recent positions (Eq. 7-8 keep S = T + N + M); U = cosine of the evicted key to every
    remaining key (Eq. 9); tau_t = beta*max(U) + (1-beta)*tau_{t-1} (Eq. 10);
    max(U) >= tau_t -> merge into the nearest neighbour with weights
    e^{u}/(e^{u}+e), e/(e^{u}+e) (Eq. 11-12 with one evicted token), else discard.
    Reading: victim ties -> the later position; neighbour ties -> the earlier position;
    the threshold is updated first, then compared; the neighbour keeps its own score.
    ``force_*`` let a harness replay another implementation's choice at a near-tie."""
    q = np.asarray(q, dtype=np.float64).reshape(-1, k.size)
    st.pos = np.append(st.pos, t)
    st.K = np.vstack([st.K, np.asarray(k, np.float64)[None, :]])
    st.V = np.vstack([st.V, np.asarray(v, np.float64)[None, :]])
    st.score = np.append(st.score, 0.0)
    out = np.zeros_like(q)
    for g in range(q.shape[0]):
        o, p = softmax_attention(q[g], st.K, st.V)
        out[g] = o
        st.score += p
    log = StepLog(tau=st.tau)
    if st.pos.size <= st.S:
        return out, log
    # ---- eviction of one token
    elig = [i for i in range(st.pos.size) if st.T <= st.pos[i] <= t - st.M]
    assert elig, "no evictable slot: S < T + M"
    ranked = sorted(elig, key=lambda i: (st.score[i], -st.pos[i]))   # lowest score, then latest position
    vi = ranked[0]
    if len(ranked) > 1:
        a, b = st.score[ranked[0]], st.score[ranked[1]]
        log.victim_gap = abs(b - a) / max(abs(a), abs(b), 1e-300)
        log.runner_up_pos = int(st.pos[ranked[1]])
    if force_victim_pos is not None:
        vi = int(np.nonzero(st.pos == force_victim_pos)[0][0])
    log.victim_pos = int(st.pos[vi])
    log.evicted = True
    k_e, v_e = st.K[vi].copy(), st.V[vi].copy()
    keep = np.arange(st.pos.size) != vi
    st.pos, st.K, st.V, st.score = st.pos[keep], st.K[keep], st.V[keep], st.score[keep]
    # ---- compensation
    U = cosine_matrix(k_e[None, :], st.K)[0]
    order = sorted(range(U.size), key=lambda j: (-U[j], st.pos[j]))
    nj = order[0]
    if len(order) > 1:
        log.nn_gap = float(U[order[0]] - U[order[1]])
        log.nn_runner_pos = int(st.pos[order[1]])
    if force_nn_pos is not None:
        nj = int(np.nonzero(st.pos == force_nn_pos)[0][0])
    mx = float(U[nj])
    st.tau = beta * mx + (1.0 - beta) * st.tau
    thr = st.tau if math.isnan(tau_override) else tau_override
    log.mx, log.nn_pos, log.tau = mx, int(st.pos[nj]), st.tau
    if mx >= thr:
        w_e = math.exp(mx) / (math.exp(mx) + E)
        w_c = E / (math.exp(mx) + E)
        st.K[nj] = round_storage(w_c * st.K[nj] + w_e * k_e, st.dtype)
        st.V[nj] = round_storage(w_c * st.V[nj] + w_e * v_e, st.dtype)
        log.merged = True
    return out, log


def full_attention_step(q: np.ndarray, K: np.ndarray, V: np.ndarray) -> np.ndarray:
    """Uncompressed decode attention (Eq. 3) for the G query heads of one KV head."""
    q = np.asarray(q, dtype=np.float64).reshape(-1, K.shape[1])
    return np.stack([softmax_attention(q[g], np.asarray(K, np.float64), np.asarray(V, np.float64))[0]
                     for g in range(q.shape[0])])


# --------------------------------------------------------------------------------------
# whole path for a small stack (used by the parity tests, the smoke check and the timed
# CPU baseline).  Tensors: Q [B,Hq,P,d], K/V [B,Hkv,P,d] per layer.
# --------------------------------------------------------------------------------------
class OracleStack:
    def __init__(self, *, n_layers: int, batch: int, n_q_heads: int, n_kv_heads: int, d_head: int,
                 dtype: str, prompt_len: int, rho: float, n_sink: int, window: int, nm_ratio: float,
                 beta: float, density_temp: float = 1.0, min_budget: int = 1, head_reduce: int = 0,
                 tau_override: float = float("nan"), max_budget: int = 0):
        self.L, self.B, self.Hq, self.Hkv, self.d = n_layers, batch, n_q_heads, n_kv_heads, d_head
        self.G = n_q_heads // n_kv_heads
        self.dtype, self.P, self.rho = dtype, prompt_len, rho
        self.T, self.window, self.nm_ratio, self.beta = n_sink, window, nm_ratio, beta
        self.gamma, self.min_budget, self.head_reduce = density_temp, min_budget, head_reduce
        self.tau_override = tau_override
        self.max_budget = max_budget
        self.colsum = np.zeros((self.L, self.B, self.Hq, self.P))
        self.F = np.zeros((self.B, self.L, self.Hq))
        self.budgets: Optional[np.ndarray] = None          # [B, L]
        self.slices: dict = {}
        self.t = prompt_len

    def layer_stats(self, layer: int, Q: np.ndarray, K: np.ndarray, heads: Optional[List[Tuple[int, int]]] = None):
        """Column sums and densities of one layer; ``heads`` restricts to (b, hq) pairs."""
        todo = heads if heads is not None else [(b, h) for b in range(self.B) for h in range(self.Hq)]
        for b, h in todo:
            s = colsum_scores(Q[b, h], K[b, h // self.G])
            self.colsum[layer, b, h] = s
            self.F[b, layer, h] = attention_density(s)

    def layer_budgets(self, F: Optional[np.ndarray] = None) -> np.ndarray:
        F = self.F if F is None else np.asarray(F, np.float64)
        self.budgets = np.stack([layer_budgets(F[b], self.P, self.rho, self.min_budget, self.gamma,
                                               self.head_reduce, self.max_budget) for b in range(self.B)])
        return self.budgets

    def slice_params(self, b: int, layer: int) -> Tuple[int, int, int]:
        S = int(self.budgets[b, layer])
        T = min(self.T, S)
        M = window_size(S, T, self.window, self.nm_ratio)
        return S, T, M

    def group_score(self, layer: int, b: int, h: int) -> np.ndarray:
        """AttnScore of one KV head at the prompt stage: the sum over its G query heads."""
        return self.colsum[layer, b, h * self.G:(h + 1) * self.G].sum(axis=0)

    def prefill_compress(self, layer: int, K: np.ndarray, V: np.ndarray,
                         slices: Optional[List[Tuple[int, int]]] = None, force: Optional[dict] = None):
        """``slices`` restricts to (b, kv head) pairs; ``force[(layer,b,h)]`` may hold the
        keyword overrides of prefill_compress_slice."""
        todo = slices if slices is not None else [(b, h) for b in range(self.B) for h in range(self.Hkv)]
        for b, h in todo:
            S, T, M = self.slice_params(b, layer)
            kw = (force or {}).get((layer, b, h), {})
            self.slices[(layer, b, h)] = prefill_compress_slice(K[b, h], V[b, h], self.group_score(layer, b, h),
                                                                S, T, M, self.dtype, self.tau_override, **kw)

    def decode_step(self, layer: int, q: np.ndarray, k: np.ndarray, v: np.ndarray, t: int,
                    slices: Optional[List[Tuple[int, int]]] = None, force: Optional[dict] = None):
        """q [B,Hq,d], k/v [B,Hkv,d] -> {(b,kvh): (out [G,d], StepLog)}."""
        todo = slices if slices is not None else [(b, h) for b in range(self.B) for h in range(self.Hkv)]
        res = {}
        for b, h in todo:
            f = (force or {}).get((layer, b, h), {})
            res[(b, h)] = decode_step_slice(self.slices[(layer, b, h)], q[b, h * self.G:(h + 1) * self.G],
                                            k[b, h], v[b, h], t, self.beta, self.tau_override,
                                            f.get("victim"), f.get("nn"))
        return res
