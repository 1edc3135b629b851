"""Pins of the CPU oracle: closed forms, invariants, brute force and library routines.

Nothing here touches the CUDA library.  Every oracle function is checked against something
that is not the oracle itself: a closed form (harmonic numbers, geometric EMA), a library
routine (numpy.var, scipy softmax / cdist), pure-Python brute force on tiny inputs, or an
invariant the paper states (budgets sum to S*L*rho, merge weights are convex, pure eviction
when nothing passes the threshold, full-cache equivalence when the budget is never reached).
"""
import math

import numpy as np
import pytest
import scipy.spatial.distance
import scipy.special

from oracle import d2o_oracle as O


def rng(seed):
    return np.random.default_rng(seed)


# ---------------------------------------------------------------- storage rounding
def test_round_storage_matches_torch():
    import torch
    x = rng(0).standard_normal(4096) * np.exp(rng(1).uniform(-20, 20, 4096))
    x = np.concatenate([x, [0.0, 1.0, -1.0, 1.00390625, 1.01171875, 65504.0, 3.0e-5]])
    for name, td in (("f32", torch.float32), ("f16", torch.float16), ("bf16", torch.bfloat16)):
        xs = x if name != "f16" else np.clip(x, -6e4, 6e4)
        ref = torch.tensor(xs, dtype=torch.float64).to(td).to(torch.float64).numpy()
        got = O.round_storage(xs, name)
        if name == "bf16":   # torch rounds double->float->bf16; direct rounding may differ only at float ties
            assert np.max(np.abs(got - ref) / np.maximum(np.abs(ref), 1e-300)) < 2 ** -8
            assert (got == ref).mean() > 0.999
        else:
            np.testing.assert_array_equal(got, ref)


def test_round_storage_bf16_ties_to_even():
    # 1 + 2^-8 is halfway between 1 and 1 + 2^-7 -> even mantissa (1.0); 1 + 3*2^-8 -> 1 + 2^-6
    assert O.round_storage(np.array([1.0 + 2 ** -8]), "bf16")[0] == 1.0
    assert O.round_storage(np.array([1.0 + 3 * 2 ** -8]), "bf16")[0] == 1.0 + 2 ** -6


# ---------------------------------------------------------------- O-1 column sums (Eq. 4 / Eq. 6)
def brute_colsum(Q, K):
    P, d = Q.shape
    s = [0.0] * P
    for i in range(P):
        z = [sum(Q[i, c] * K[j, c] for c in range(d)) / math.sqrt(d) for j in range(i + 1)]
        zmax = max(z)
        ez = [math.exp(a - zmax) for a in z]
        tot = sum(ez)
        for j in range(i + 1):
            s[j] += ez[j] / tot
    return np.array(s)


@pytest.mark.parametrize("P,d", [(1, 4), (7, 8), (33, 16), (64, 8)])
def test_colsum_brute_force(P, d):
    r = rng(P)
    Q, K = r.standard_normal((P, d)) * 2, r.standard_normal((P, d))
    np.testing.assert_allclose(O.colsum_scores(Q, K, row_block=5), brute_colsum(Q, K), rtol=1e-12, atol=1e-14)


def test_colsum_zero_query_is_harmonic():
    P, d = 200, 8
    K = rng(3).standard_normal((P, d))
    H = np.concatenate([[0.0], np.cumsum(1.0 / np.arange(1, P + 1))])
    np.testing.assert_allclose(O.colsum_scores(np.zeros((P, d)), K), H[P] - H[:P], rtol=1e-12)


def test_colsum_rows_sum_to_one_and_blocks_agree():
    P, d = 300, 16
    r = rng(4)
    Q, K = r.standard_normal((P, d)), r.standard_normal((P, d))
    s = O.colsum_scores(Q, K)
    assert abs(s.sum() - P) < 1e-9
    np.testing.assert_allclose(s, O.colsum_scores(Q, K, row_block=7), rtol=1e-12)
    assert O.colsum_scores(Q[:1], K[:1])[0] == 1.0
    # the last column only receives the last row's self-attention
    zl = K @ Q[-1] / math.sqrt(d)
    assert abs(s[-1] - scipy.special.softmax(zl)[-1]) < 1e-12


# ---------------------------------------------------------------- O-2 density (Eq. 4)
def test_density_is_population_variance():
    s = rng(5).gamma(0.3, size=777)
    assert abs(O.attention_density(s) - np.var(s)) < 1e-12 * np.var(s)
    s = s * (s.size / s.sum())                       # mean exactly 1, as column sums have
    assert abs(O.attention_density(s) - ((s * s).mean() - 1.0)) < 1e-9
    assert O.attention_density(np.ones(10)) == 0.0


# ---------------------------------------------------------------- O-3 budgets (Eq. 5, Appendix A.2)
def test_budgets_sum_and_bounds():
    r = rng(6)
    for trial in range(200):
        L = int(r.integers(1, 40))
        H = int(r.integers(1, 5))
        P = int(r.integers(16, 5000))
        rho = float(r.uniform(0.05, 1.0))
        smin = int(r.integers(1, 8))
        F = r.gamma(1.0, size=(L, H)) * float(r.choice([0.01, 1.0, 50.0, 1e4]))
        if L * smin > math.floor(rho * L * P + 0.5):
            continue
        S = O.layer_budgets(F, P, rho, smin)
        assert S.sum() == math.floor(rho * L * P + 0.5)          # sum_l S_l = S * L * rho
        assert S.min() >= smin and S.max() <= P
        w = O.layer_weights(F)
        for a in range(L):                                         # higher density weight -> not smaller cache
            for b in range(L):
                if w[a] > w[b]:
                    assert S[a] >= S[b] - 1


def test_budgets_equal_density_is_uniform():
    S = O.layer_budgets(np.full((8, 4), 3.7), 1000, 0.25)
    assert (S == 250).all()                                        # alpha_l = rho
    assert O.layer_budgets(np.array([[2.0]]), 1000, 0.3)[0] == 300  # L = 1


def test_budgets_large_temperature_is_the_uniform_allocation():
    # the ablation's "uniform allocation" alpha_l = rho (Section 5.4, setting 4) is the limit gamma -> infinity of
    # exp(-F / gamma): every layer gets rho * P whatever the densities are
    F = rng(11).gamma(1.0, size=(16, 8)) * 500.0
    S = O.layer_budgets(F, 2000, 0.2, 1, 1e30)
    assert (S == 400).all()


def test_budgets_reciprocal_of_variance_allocation():
    # Section 5.4, setting 2: alpha_l = (1 / F_l) / sum_l (1 / F_l) * L * rho.  F = 1, 2, 4 -> shares 4/7, 2/7, 1/7
    # of S_tot = 0.25 * 3 * 7000 = 5250
    S = O.layer_budgets(np.array([[1.0], [2.0], [4.0]]), 7000, 0.25, 1, 1.0, 2)
    assert S.tolist() == [3000, 1500, 750]
    assert O.layer_budgets(np.array([[1.0], [2.0], [4.0]]), 7000, 0.25, 1, 1.0, 3).tolist() == [3000, 1500, 750]
    # per head: w_l = sum_h 1 / F_lh; on the mean: w_l = 1 / mean_h F_lh
    F = np.array([[1.0, 4.0], [2.0, 2.0]])                          # rule 2: w = 1.25, 1.0; rule 3: w = 0.4, 0.5
    assert O.layer_budgets(F, 9000, 0.5, 1, 1.0, 2).tolist() == [5000, 4000]
    assert O.layer_budgets(F, 9000, 0.5, 1, 1.0, 3).tolist() == [4000, 5000]
    # the rule does not depend on the unit of F, nor on gamma
    r = rng(21)
    Fr = r.gamma(2.0, size=(12, 4)) + 0.1
    a = O.layer_budgets(Fr, 4096, 0.3, 8, 1.0, 2)
    assert (O.layer_budgets(Fr * 1024.0, 4096, 0.3, 8, 77.0, 2) == a).all()
    assert a.sum() == round(0.3 * 12 * 4096)
    w = (1.0 / Fr).sum(axis=1)
    for i in range(12):
        for j in range(12):
            if w[i] > w[j]:
                assert a[i] >= a[j] - 1


def test_budgets_match_softmax_formula_when_unclamped():
    r = rng(7)
    L, P, rho = 12, 4096, 0.3
    F = r.uniform(0.0, 0.5, size=(L, 1))
    alpha = scipy.special.softmax(-F[:, 0]) * L * rho              # Eq. 5
    x = alpha * P
    assert x.max() < P and x.min() > 1
    S = O.layer_budgets(F, P, rho)
    assert np.all(np.abs(S - x) < 1.0)
    assert abs(alpha.sum() - L * rho) < 1e-12
    # per-head form: alpha_l = sum_h alpha_l^h
    Fh = r.uniform(0.0, 0.5, size=(L, 4))
    ah = scipy.special.softmax(-Fh.reshape(-1)).reshape(L, 4).sum(axis=1) * L * rho
    Sh = O.layer_budgets(Fh, P, rho)
    assert np.all(np.abs(Sh - ah * P) < 1.0)
    # temperature: gamma rescales F
    Sg = O.layer_budgets(F * 10.0, P, rho, gamma=10.0)
    np.testing.assert_array_equal(Sg, S)


def test_budgets_clamped_cases():
    # one layer dominates the softmax: it saturates at P, the remainder is shared by weight
    F = np.array([[0.0], [50.0], [50.0], [51.0]])
    S = O.layer_budgets(F, 100, 0.5, min_budget=4)
    assert S.sum() == 200 and S[0] == 100
    assert S[1] == S[2] and S[1] > S[3] >= 4
    # brute force over lambda on a grid for a random case
    r = rng(8)
    F = r.gamma(2.0, size=(6, 1)) * 3
    P, rho, smin = 500, 0.4, 10
    w = O.layer_weights(F)
    S = O.layer_budgets(F, P, rho, smin)
    tot = math.floor(rho * 6 * P + 0.5)
    lo_l, hi_l = 0.0, 1e12
    for _ in range(200):                                           # bisection on the monotone total
        mid = 0.5 * (lo_l + hi_l)
        if np.clip(mid * w, smin, P).sum() < tot:
            lo_l = mid
        else:
            hi_l = mid
    x = np.clip(hi_l * w, smin, P)
    assert np.all(np.abs(S - x) < 1.0 + 1e-6)


def test_window_size_rule():
    assert O.window_size(256, 1, 32, 3.0) == 32
    assert O.window_size(101, 1, 0, 3.0) == 25                     # N:M = 3:1 with N + M + T = S
    assert O.window_size(5, 4, 32, 3.0) == 1
    for S in range(2, 300):
        M = O.window_size(S, 1, 0, 3.0)
        N = S - 1 - M
        assert N >= 0 and abs(N - 3 * M) <= 3


# ---------------------------------------------------------------- O-4 selection (Eq. 7-8)
def test_select_brute_force():
    r = rng(9)
    for trial in range(300):
        P = int(r.integers(4, 40))
        T = int(r.integers(0, 3))
        M = int(r.integers(0, 4))
        S = int(r.integers(T + M, P + 3))
        score = r.choice([0.1, 0.5, 1.0, 2.0, 3.0], size=P) if trial % 2 else r.random(P)
        ret, ev = O.select_retained(score, S, T, M)
        if S >= P:
            assert ret.tolist() == list(range(P)) and ev.size == 0
            continue
        assert ret.size == S and ev.size == P - S
        assert sorted(ret.tolist() + ev.tolist()) == list(range(P))
        assert all(j in ret for j in range(T)) and all(j in ret for j in range(P - M, P))
        mid = [j for j in ret if T <= j < P - M]
        # brute force: every kept candidate beats every evicted one under (score desc, pos asc)
        for a in mid:
            for b in ev:
                assert (score[a], -a) > (score[b], -b)


# ---------------------------------------------------------------- O-5 similarity (Eq. 9)
def test_cosine_matches_scipy_and_properties():
    r = rng(10)
    Ke, Kc = r.standard_normal((37, 16)), r.standard_normal((11, 16)) * 5
    U = O.cosine_matrix(Ke, Kc)
    np.testing.assert_allclose(U, 1.0 - scipy.spatial.distance.cdist(Ke, Kc, "cosine"), atol=1e-12)
    assert U.max() <= 1 + 1e-12 and U.min() >= -1 - 1e-12
    Kc[4] = 3.0 * Ke[20]                                           # scaled duplicate
    mx, nn = O.nearest_neighbour(O.cosine_matrix(Ke, Kc))
    assert nn[20] == 4 and abs(mx[20] - 1.0) < 1e-12
    Kc[7] = 0.0
    assert np.all(O.cosine_matrix(Ke, Kc)[:, 7] == 0.0)
    U2 = np.array([[0.5, 0.9, 0.9], [0.1, 0.1, 0.0]])
    mx, nn = O.nearest_neighbour(U2)
    assert nn.tolist() == [1, 0] and mx.tolist() == [0.9, 0.1]     # ties -> lowest column


# ---------------------------------------------------------------- O-6 / O-7 threshold and merge (Eq. 10-12)
def test_tau0_and_merge_weights():
    r = rng(11)
    Lc, Le, d = 6, 40, 8
    Kc, Vc = r.standard_normal((Lc, d)), r.standard_normal((Lc, d))
    Ke, Ve = r.standard_normal((Le, d)), r.standard_normal((Le, d))
    mx, nn = O.nearest_neighbour(O.cosine_matrix(Ke, Kc))
    tau0 = O.initial_threshold(mx)
    assert mx.min() <= tau0 <= mx.max() and abs(tau0 - np.mean(mx)) < 1e-15
    # tau = +inf: pure eviction, conserved rows unchanged bit for bit
    Kp, Vp, den = O.weighted_merge(Kc, Vc, Ke, Ve, mx, nn, O.merge_mask(mx, float("inf")))
    np.testing.assert_array_equal(den, np.full(Lc, math.e))
    np.testing.assert_allclose(Kp, Kc, rtol=1e-15)
    # tau = -inf: every evicted token is counted exactly once
    Km, Vm, den = O.weighted_merge(Kc, Vc, Ke, Ve, mx, nn, O.merge_mask(mx, float("-inf")))
    assert abs((den - math.e).sum() - np.exp(mx).sum()) < 1e-10
    # convexity: explicit weights reproduce the merged rows and sum to one
    for j in range(Lc):
        idx = np.nonzero(nn == j)[0]
        w_c = math.e / den[j]
        w_e = np.exp(mx[idx]) / den[j]
        assert abs(w_c + w_e.sum() - 1.0) < 1e-12 and 0 < w_c <= 1 and np.all((w_e > 0) & (w_e < 1))
        assert np.all(w_c >= w_e)                                   # the conserved token keeps the largest weight
        np.testing.assert_allclose(Km[j], w_c * Kc[j] + (w_e[:, None] * Ke[idx]).sum(0), atol=1e-12)
        np.testing.assert_allclose(Vm[j], w_c * Vc[j] + (w_e[:, None] * Ve[idx]).sum(0), atol=1e-12)
        lo = np.minimum(Kc[j], Ke[idx].min(0)) if idx.size else Kc[j]
        hi = np.maximum(Kc[j], Ke[idx].max(0)) if idx.size else Kc[j]
        assert np.all(Km[j] >= lo - 1e-12) and np.all(Km[j] <= hi + 1e-12)
    # threshold at tau0 merges exactly the rows with mx >= tau0
    K0, V0, den0 = O.weighted_merge(Kc, Vc, Ke, Ve, mx, nn, O.merge_mask(mx, tau0))
    assert abs((den0 - math.e).sum() - np.exp(mx[mx >= tau0]).sum()) < 1e-10


def test_merge_single_victim_closed_forms():
    d = 4
    kc, vc = np.array([[1.0, 0, 0, 0]]), np.array([[2.0, 2, 2, 2]])
    # identical direction: u = 1 -> plain average
    K1, V1, _ = O.weighted_merge(kc, vc, np.array([[3.0, 0, 0, 0]]), np.array([[4.0, 4, 4, 4]]),
                                 np.array([1.0]), np.array([0]), np.array([True]))
    np.testing.assert_allclose(K1[0], [2.0, 0, 0, 0], atol=1e-15)
    np.testing.assert_allclose(V1[0], [3.0] * 4, atol=1e-15)
    # orthogonal: u = 0 -> evicted weight 1/(1+e)
    K2, _, _ = O.weighted_merge(kc, vc, np.array([[0.0, 5, 0, 0]]), vc, np.array([0.0]), np.array([0]), np.array([True]))
    w = 1.0 / (1.0 + math.e)
    np.testing.assert_allclose(K2[0], [1 - w, 5 * w, 0, 0], atol=1e-15)


def make_slice(r, P, d, G):
    K, V = r.standard_normal((P, d)), r.standard_normal((P, d))
    Q = r.standard_normal((G, P, d)) * 1.5
    score = sum(O.colsum_scores(Q[g], K) for g in range(G))
    return Q, K, V, score


def test_prefill_compress_slice_properties():
    r = rng(12)
    P, d, S, T, M = 96, 16, 24, 2, 6
    Q, K, V, score = make_slice(r, P, d, 2)
    K, V = O.round_storage(K, "f16"), O.round_storage(V, "f16")
    st = O.prefill_compress_slice(K, V, score, S, T, M, "f16")
    assert st.pos.size == S and np.all(np.diff(st.pos) > 0)
    assert set(range(T)) <= set(st.pos.tolist()) and set(range(P - M, P)) <= set(st.pos.tolist())
    np.testing.assert_array_equal(st.score, score[st.pos])
    assert np.all(O.round_storage(st.K, "f16") == st.K)            # stored values are f16-representable
    # pure eviction: the cache is a bit-identical gather
    st_inf = O.prefill_compress_slice(K, V, score, S, T, M, "f16", tau_override=float("inf"))
    np.testing.assert_array_equal(st_inf.K, K[st_inf.pos])
    np.testing.assert_array_equal(st_inf.V, V[st_inf.pos])
    assert st_inf.tau == st.tau                                     # tau_0 is still the mean of row maxima
    # rows that received nothing are untouched; rows that did are inside the hull of their sources
    untouched = st.log["den"] == math.e
    np.testing.assert_array_equal(st.K[untouched], K[st.pos][untouched])
    assert (~untouched).any() and untouched.any()
    # S >= P keeps everything
    st_all = O.prefill_compress_slice(K, V, score, P + 5, T, M, "f16")
    np.testing.assert_array_equal(st_all.K, K)
    assert st_all.tau == 0.0


# ---------------------------------------------------------------- O-8 decode step
def test_decode_equals_full_attention_when_budget_never_reached():
    r = rng(13)
    P, d, G, steps = 40, 8, 2, 6
    Q, K, V, score = make_slice(r, P, d, G)
    st = O.prefill_compress_slice(K, V, score, P + steps, 1, 4, "f32")
    Kf, Vf = K.copy(), V.copy()
    for t in range(steps):
        q, k, v = r.standard_normal((G, d)), r.standard_normal(d), r.standard_normal(d)
        out, log = O.decode_step_slice(st, q, k, v, P + t, 0.7)
        Kf, Vf = np.vstack([Kf, k]), np.vstack([Vf, v])
        for g in range(G):                                          # independent textbook attention
            p = scipy.special.softmax(Kf @ q[g] / math.sqrt(d))
            np.testing.assert_allclose(out[g], p @ Vf, rtol=1e-12, atol=1e-14)
        assert not log.evicted and st.pos.size == P + t + 1
        np.testing.assert_allclose(out, O.full_attention_step(q, Kf, Vf), rtol=1e-12)


def test_decode_invariants():
    r = rng(14)
    P, d, G, S, T, M, steps = 64, 8, 2, 20, 1, 5, 30
    Q, K, V, score = make_slice(r, P, d, G)
    st = O.prefill_compress_slice(K, V, score, S, T, M, "f32")
    total = st.score.sum()
    for i in range(steps):
        t = P + i
        before = st.score.sum()
        q, k, v = r.standard_normal((G, d)), r.standard_normal(d), r.standard_normal(d)
        K_before, pos_before, score_before = st.K.copy(), st.pos.copy(), st.score.copy()
        out, log = O.decode_step_slice(st, q, k, v, t, 0.7)
        assert st.pos.size == S and log.evicted                     # constant size, one victim per step
        assert set(range(T)) <= set(st.pos.tolist())                # sinks stay
        assert set(range(t - M + 1, t + 1)) <= set(st.pos.tolist())  # the M newest stay
        assert T <= log.victim_pos <= t - M
        # accumulated probabilities: G per step enter, the victim's score leaves
        # (its final score = its old score + this step's probability)
        assert st.score.sum() < before + G + 1e-9
        # out is attention over the pre-eviction cache
        Kall = np.vstack([K_before, k])
        assert out.shape == (G, d)
        p0 = scipy.special.softmax(Kall @ q[0] / math.sqrt(d))
        # victim had the lowest updated score among the eligible slots
        upd = np.append(score_before, 0.0) + sum(
            scipy.special.softmax(Kall @ q[g] / math.sqrt(d)) for g in range(G))
        posall = np.append(pos_before, t)
        elig = (posall >= T) & (posall <= t - M)
        assert upd[posall == log.victim_pos][0] == pytest.approx(upd[elig].min(), rel=1e-12)
        assert abs(upd.sum() - (before + G)) < 1e-9
        if log.merged:
            assert log.mx >= log.tau
        else:
            assert log.mx < log.tau


def test_ema_threshold_closed_form_and_order_equivalence():
    # constant best similarity c: tau_t = c + (1-beta)^t (tau_0 - c)  (geometric EMA)
    d = 4
    beta, c = 0.7, 0.6
    base = np.array([1.0, 0.0, 0.0, 0.0])
    other = np.array([c, math.sqrt(1 - c * c), 0.0, 0.0])            # cosine(base, other) = c
    tau0 = 0.1
    for t_steps in range(1, 6):
        st = O.SliceState(pos=np.array([0, 1]), K=np.vstack([base, other]), V=np.zeros((2, d)),
                          score=np.array([5.0, 0.0]), tau=tau0, S=2, T=1, M=1, dtype="f32")
        taus = []
        for i in range(t_steps):
            # new token = `other` again, huge query weight on slot 0 keeps it safe; victim is pos>=1 oldest
            out, log = O.decode_step_slice(st, np.zeros((1, d)), other, np.zeros(d), 2 + i, beta,
                                           tau_override=float("inf"))
            taus.append(st.tau)
            # similarity of the victim (= other) to the best remaining: other again -> 1.0 unless only base
        # after eviction the victim `other` (old) is compared with {base, new other}: max = 1.0
        c_eff = 1.0
        for i, tv in enumerate(taus, 1):
            assert tv == pytest.approx(c_eff + (1 - beta) ** i * (tau0 - c_eff), rel=1e-12)
    # compare-after-update equals compare-before-update for 0 <= beta < 1:
    # mx >= beta*mx + (1-beta)*tau  <=>  mx >= tau
    r = rng(15)
    for _ in range(1000):
        mx, tau, b = r.uniform(-1, 1), r.uniform(-1, 1), r.uniform(0, 0.99)
        if abs(mx - tau) > 1e-12:
            assert (mx >= b * mx + (1 - b) * tau) == (mx >= tau)
    # beta = 1: threshold equals the current maximum -> always merged ("w.o. EMA threshold")
    st = O.SliceState(pos=np.array([0, 1, 2]), K=r.standard_normal((3, d)), V=r.standard_normal((3, d)),
                      score=np.array([5.0, 0.1, 0.2]), tau=0.99, S=3, T=1, M=1, dtype="f32")
    out, log = O.decode_step_slice(st, r.standard_normal((1, d)), r.standard_normal(d), r.standard_normal(d), 3, 1.0)
    assert log.merged and log.tau == log.mx


def test_decode_merge_single_token_weights():
    d = 4
    r = rng(16)
    K = np.array([[1.0, 0, 0, 0], [0.0, 1, 0, 0], [0.0, 0.6, 0.8, 0]])
    V = r.standard_normal((3, d))
    st = O.SliceState(pos=np.array([0, 1, 2]), K=K.copy(), V=V.copy(), score=np.array([9.0, 0.0, 1.0]),
                      tau=-1.0, S=3, T=1, M=1, dtype="f32")
    knew = np.array([0.0, 0, 0, 1.0])
    out, log = O.decode_step_slice(st, np.zeros((1, d)), knew, np.ones(d), 3, 0.5)
    assert log.victim_pos == 1 and log.nn_pos == 2 and log.mx == pytest.approx(0.6)
    w_e = math.exp(0.6) / (math.exp(0.6) + math.e)
    row = list(st.pos).index(2)
    np.testing.assert_allclose(st.K[row], O.round_storage((1 - w_e) * K[2] + w_e * K[1], "f32"), atol=0)
    np.testing.assert_allclose(st.V[row], O.round_storage((1 - w_e) * V[2] + w_e * V[1], "f32"), atol=0)
    assert st.tau == pytest.approx(0.5 * 0.6 + 0.5 * -1.0)
    assert st.pos.tolist() == [0, 2, 3]


# ---------------------------------------------------------------- budgets with an upper clamp (Eq. 5 + bounds)
def _bisect_budgets(w, tot, lo, cap):
    """Independent statement of the clamped proportional rule: bisection on the monotone total."""
    a, b = 0.0, 1.0
    while np.clip(b * w, lo, cap).sum() < tot and b < 1e307:
        b *= 2.0
    for _ in range(300):
        mid = 0.5 * (a + b)
        if np.clip(mid * w, lo, cap).sum() < tot:
            a = mid
        else:
            b = mid
    return np.clip(b * w, lo, cap)


def test_budgets_with_max_budget_closed_form():
    # Eq. 5 with weights 8 : 1 : 1 (F = 0, ln 8, ln 8): unclamped shares of S_tot = 0.5 * 3 * 1000 = 1500 would be
    # 1200, 150, 150.  A cap of 600 saturates layer 0; the other two share the remaining 900 by weight: 450 each.
    F = np.array([[0.0], [math.log(8.0)], [math.log(8.0)]])
    assert O.layer_budgets(F, 1000, 0.5).tolist() == [1000, 250, 250]          # cap = P binds already
    assert O.layer_budgets(F, 1000, 0.5, max_budget=600).tolist() == [600, 450, 450]
    assert O.layer_budgets(F, 1000, 0.5, max_budget=1200).tolist() == [1200, 150, 150]
    # weights 4 : 2 : 1, S_tot = 700, cap 300: layer 0 saturates, the rest share 400 as 2 : 1 -> 266.67, 133.33
    F = np.array([[0.0], [math.log(2.0)], [math.log(4.0)]])
    S = O.layer_budgets(F, 1000, 0.7 / 3.0, max_budget=300)
    assert S.tolist() == [300, 267, 133]
    # both clamps at once: lower clamp 100 lifts layer 2; the middle layer takes what is left
    S = O.layer_budgets(np.array([[0.0], [math.log(2.0)], [math.log(400.0)]]), 1000, 0.6 / 3.0, min_budget=100,
                        max_budget=300)
    assert S.tolist() == [300, 200, 100]


def test_budgets_with_max_budget_sum_bounds_and_bisection():
    r = rng(61)
    done = 0
    for trial in range(300):
        L = int(r.integers(1, 40))
        H = int(r.integers(1, 5))
        P = int(r.integers(16, 5000))
        rho = float(r.uniform(0.05, 0.9))
        smin = int(r.integers(1, 8))
        tot = math.floor(rho * L * P + 0.5)
        mean = tot / L
        cap = int(min(P, max(smin, math.ceil(mean * float(r.uniform(1.0, 4.0))))))
        F = r.gamma(1.0, size=(L, H)) * float(r.choice([0.01, 1.0, 50.0, 1e4]))
        gamma = float(r.choice([1.0, 10.0, 100.0]))
        hr = int(trial % 4)
        if not (L * smin <= tot <= L * cap):
            continue
        S = O.layer_budgets(F, P, rho, smin, gamma, hr, cap)
        assert S.sum() == tot                                         # sum_l alpha_l = L * rho still holds
        assert S.min() >= smin and S.max() <= cap
        w = np.maximum(O.layer_weights(F, gamma, hr), 1e-300)
        x = _bisect_budgets(w, tot, smin, cap)
        assert np.all(np.abs(S - x) < 1.0 + 1e-6), (S, x)
        for a in range(L):                                            # a larger weight never gets a smaller cache
            for b in range(L):
                if w[a] > w[b]:
                    assert S[a] >= S[b] - 1
        done += 1
    assert done > 150


def test_allocate_budgets_remainders_go_to_the_lower_unit():
    # three equal units share 10: 3.33 each -> floor 3, one left over -> unit 0
    assert O.allocate_budgets(np.ones(3), 10, 1, 10).tolist() == [4, 3, 3]
    assert O.allocate_budgets(np.ones(3), 11, 1, 10).tolist() == [4, 4, 3]
    # a saturated unit never takes a remainder
    assert O.allocate_budgets(np.array([100.0, 1.0, 1.0]), 11, 1, 4).tolist() == [4, 4, 3]


# ---------------------------------------------------------------- per-head and exponential-decay allocation
def test_head_budgets_follow_the_appendix_formula():
    r = rng(62)
    L, H, P, rho = 6, 4, 3000, 0.25
    F = r.uniform(0.0, 1.0, size=(L, H))
    a = scipy.special.softmax(-F.reshape(-1)).reshape(L, H)        # alpha_l^h, sums to one over all (l, h)
    S = O.head_budgets(F, P, rho)
    tot = math.floor(rho * L * H * P + 0.5)
    assert S.shape == (L, H) and S.sum() == tot
    assert np.all(np.abs(S - a * tot) < 1.0)                        # S_l^h = alpha_l^h * S_total
    # S_l = sum_h S_l^h is the per-layer rule's size times the number of heads (alpha_l = sum_h alpha_l^h)
    Sl = O.layer_budgets(F, P, rho)
    assert np.all(np.abs(S.sum(axis=1) - H * Sl) <= H + 1)
    # grouped queries: a KV head's weight is the sum of its query heads' weights
    Sg = O.head_budgets(F, P, rho, group=2)
    ag = a.reshape(L, 2, 2).sum(axis=2)
    totg = math.floor(rho * L * 2 * P + 0.5)
    assert Sg.shape == (L, 2) and Sg.sum() == totg
    assert np.all(np.abs(Sg - ag * totg) < 1.0)
    # equal densities -> every head gets rho * P; one head, one layer -> rho * P
    assert (O.head_budgets(np.full((3, 4), 2.5), 1000, 0.2) == 200).all()
    assert O.head_budgets(np.array([[7.0]]), 1000, 0.3)[0, 0] == 300
    # bounds
    Sc = O.head_budgets(F * 50.0, P, rho, min_budget=16, max_budget=1500)
    assert Sc.min() >= 16 and Sc.max() <= 1500 and Sc.sum() == tot


def test_exp_decay_budgets_closed_form():
    # alpha_l = exp(-F_l): F = 0, ln 2, ln 4 -> 1, 1/2, 1/4 of the prompt; not normalised
    F = np.array([[0.0], [math.log(2.0)], [math.log(4.0)]])
    assert O.exp_decay_budgets(F, 1000).tolist() == [1000, 500, 250]
    assert O.exp_decay_budgets(F, 1000, gamma=2.0).tolist() == [1000, 707, 500]
    assert O.exp_decay_budgets(F, 1000, min_budget=300, max_budget=800).tolist() == [800, 500, 300]
    # several heads: the mean of the per-head factors
    F2 = np.array([[0.0, math.log(4.0)]])
    assert O.exp_decay_budgets(F2, 1000).tolist() == [625]
    # monotone in the density
    r = rng(63)
    Fr = np.sort(r.uniform(0, 3, size=(9, 1)), axis=0)
    assert np.all(np.diff(O.exp_decay_budgets(Fr, 4096)) <= 0)


# ---------------------------------------------------------------- grouped-query score (reading for GQA)
def test_group_score_is_the_sum_over_the_query_heads():
    # Hq = 4, G = 2: KV head 0 owns query heads 0, 1; KV head 1 owns 2, 3
    cs = np.array([[1.0, 2.0, 3.0], [10.0, 20.0, 30.0], [0.5, 0.25, 0.125], [4.0, 4.0, 4.0]])
    assert O.group_score(cs, 0, 2).tolist() == [11.0, 22.0, 33.0]
    assert O.group_score(cs, 1, 2).tolist() == [4.5, 4.25, 4.125]
    assert O.group_score(cs, 2, 1).tolist() == [0.5, 0.25, 0.125]
    # the same sum that the decode step accumulates: two query heads with known probabilities
    d = 2
    st = O.SliceState(pos=np.array([0]), K=np.zeros((1, d)), V=np.zeros((1, d)), score=np.array([0.0]), tau=0.0,
                      S=8, T=0, M=1, dtype="f32")
    O.decode_attend(st, np.zeros((2, d)), np.zeros(d), np.zeros(d), 1)   # zero logits: each head gives 1/2, 1/2
    assert st.score.tolist() == [1.0, 1.0]
    # and the stack uses it
    stack = O.OracleStack(n_layers=1, batch=1, n_q_heads=4, n_kv_heads=2, d_head=2, dtype="f32", prompt_len=3,
                          rho=1.0, n_sink=0, window=1, nm_ratio=3.0, beta=0.7)
    stack.colsum[0, 0] = cs
    assert stack.group_score(0, 0, 1).tolist() == [4.5, 4.25, 4.125]


# ---------------------------------------------------------------- exact ties at decode (readings)
def test_decode_victim_tie_goes_to_the_later_position():
    d = 4
    K = np.eye(4)[:3] * 1.0
    # slots at positions 0 (sink), 1, 2 with bit-equal scores on 1 and 2; zero queries add the same 1/4 to each
    st = O.SliceState(pos=np.array([0, 1, 2]), K=K.copy(), V=np.zeros((3, d)), score=np.array([9.0, 0.5, 0.5]),
                      tau=5.0, S=3, T=1, M=1, dtype="f32")
    out, log = O.decode_step_slice(st, np.zeros((1, d)), np.array([0.0, 0, 0, 1.0]), np.zeros(d), 3, 0.7)
    assert log.evicted and log.victim_pos == 2 and log.runner_up_pos == 1 and log.victim_gap == 0.0
    assert st.pos.tolist() == [0, 1, 3]
    assert O.victim_order(O.SliceState(pos=np.array([0, 1, 2, 3]), K=np.zeros((4, d)), V=np.zeros((4, d)),
                                       score=np.array([0.0, 0.5, 0.5, 0.1]), tau=0.0, S=3, T=1, M=1, dtype="f32"),
                          3) == [2, 1]                                 # pos 0 is a sink, pos 3 is in the window


def test_decode_neighbour_tie_goes_to_the_earlier_position():
    d = 4
    # victim = position 1 (lowest score); positions 0 and 2 hold the same direction (bit-equal cosine 0.6)
    K = np.array([[0.6, 0.8, 0, 0], [1.0, 0, 0, 0], [0.6, 0.8, 0, 0]])
    V = np.arange(12.0).reshape(3, d)
    st = O.SliceState(pos=np.array([0, 1, 2]), K=K.copy(), V=V.copy(), score=np.array([9.0, 0.0, 1.0]),
                      tau=-1.0, S=3, T=1, M=1, dtype="f32")
    out, log = O.decode_step_slice(st, np.zeros((1, d)), np.array([0.0, 0, 0, 1.0]), np.zeros(d), 3, 0.5)
    assert log.victim_pos == 1 and log.nn_pos == 0 and log.nn_runner_pos == 2 and log.nn_gap == 0.0
    assert log.merged
    w_e = math.exp(0.6) / (math.exp(0.6) + math.e)
    np.testing.assert_allclose(st.K[0], O.round_storage((1 - w_e) * K[0] + w_e * K[1], "f32"), atol=0)
    np.testing.assert_array_equal(st.K[1], K[2])                     # the later twin is untouched


# ---------------------------------------------------------------- ablation switches (Section 5.4 tables)
def test_average_merge_policy():
    r = rng(64)
    Lc, Le, d = 5, 30, 8
    Kc, Vc = r.standard_normal((Lc, d)), r.standard_normal((Lc, d))
    Ke, Ve = r.standard_normal((Le, d)), r.standard_normal((Le, d))
    mx, nn = O.nearest_neighbour(O.cosine_matrix(Ke, Kc))
    mask = O.merge_mask(mx, O.initial_threshold(mx))
    Ka, Va, den = O.weighted_merge(Kc, Vc, Ke, Ve, mx, nn, mask, "average")
    for j in range(Lc):
        idx = np.nonzero((nn == j) & mask)[0]
        assert den[j] == 1 + idx.size
        np.testing.assert_allclose(Ka[j], (Kc[j] + Ke[idx].sum(0)) / (1 + idx.size), atol=1e-13)   # plain mean
        np.testing.assert_allclose(Va[j], (Vc[j] + Ve[idx].sum(0)) / (1 + idx.size), atol=1e-13)
    # one victim at decode: the plain average of the two rows, whatever the similarity
    K = np.array([[1.0, 0, 0, 0], [0.0, 1, 0, 0], [0.0, 0.6, 0.8, 0]])
    V = r.standard_normal((3, 4))
    st = O.SliceState(pos=np.array([0, 1, 2]), K=K.copy(), V=V.copy(), score=np.array([9.0, 0.0, 1.0]),
                      tau=-1.0, S=3, T=1, M=1, dtype="f32", policy="average")
    out, log = O.decode_step_slice(st, np.zeros((1, 4)), np.array([0.0, 0, 0, 1.0]), np.ones(4), 3, 0.5)
    assert log.merged and log.nn_pos == 2
    row = list(st.pos).index(2)
    np.testing.assert_allclose(st.K[row], O.round_storage(0.5 * (K[2] + K[1]), "f32"), atol=0)
    np.testing.assert_allclose(st.V[row], O.round_storage(0.5 * (V[2] + V[1]), "f32"), atol=0)


def test_value_feature_uses_cosine_of_the_values():
    r = rng(65)
    P, d, S, T, M = 48, 8, 12, 1, 3
    Q, K, V, score = make_slice(r, P, d, 1)
    sk = O.prefill_compress_slice(K, V, score, S, T, M, "f32", feature="k")
    sv = O.prefill_compress_slice(K, V, score, S, T, M, "f32", feature="v")
    np.testing.assert_array_equal(sk.pos, sv.pos)                  # eviction does not depend on the feature
    ret, ev = sk.log["retained"], sk.log["evicted"]
    Uv = 1.0 - scipy.spatial.distance.cdist(V[ev], V[ret], "cosine")
    np.testing.assert_allclose(sv.log["U"], Uv, atol=1e-12)
    np.testing.assert_array_equal(sv.log["nn"], np.argmax(Uv, axis=1))
    assert abs(sv.tau - Uv.max(axis=1).mean()) < 1e-12
    # swapping the roles of K and V swaps the two results
    sw = O.prefill_compress_slice(V, K, score, S, T, M, "f32", feature="k")
    np.testing.assert_array_equal(sw.K, sv.V)
    np.testing.assert_array_equal(sw.V, sv.K)
    # decode: the neighbour is the best cosine among the values
    st = O.SliceState(pos=np.array([0, 1, 2]), K=np.eye(4)[:3].copy(),
                      V=np.array([[0.0, 1, 0, 0], [1.0, 0, 0, 0], [0.8, 0.6, 0, 0]]),
                      score=np.array([9.0, 0.0, 1.0]), tau=-1.0, S=3, T=1, M=1, dtype="f32", feature="v")
    out, log = O.decode_step_slice(st, np.zeros((1, 4)), np.array([0.0, 0, 0, 1.0]), np.array([0.0, 0, 1, 0]), 3, 0.5)
    assert log.victim_pos == 1 and log.nn_pos == 2 and log.mx == pytest.approx(0.8)


def test_no_ema_threshold_merges_every_victim():
    # beta = 1 ("w.o. EMA-Threshold"): tau_t equals the current maximum, so every evicted token is merged
    r = rng(66)
    P, d, G, S, T, M = 40, 8, 1, 12, 1, 3
    Q, K, V, score = make_slice(r, P, d, G)
    st = O.prefill_compress_slice(K, V, score, S, T, M, "f32")
    for i in range(12):
        out, log = O.decode_step_slice(st, r.standard_normal((G, d)), r.standard_normal(d), r.standard_normal(d),
                                       P + i, 1.0)
        assert log.evicted and log.merged and log.tau == log.mx
    # beta = 0: the threshold never moves from tau_0
    st = O.prefill_compress_slice(K, V, score, S, T, M, "f32")
    tau0 = st.tau
    for i in range(6):
        O.decode_step_slice(st, r.standard_normal((G, d)), r.standard_normal(d), r.standard_normal(d), P + i, 0.0)
        assert st.tau == tau0


def test_window_only_cache_and_zero_keys():
    # N = 0: the cache is the sinks and the window; the victim at decode is the oldest window position
    r = rng(67)
    P, d = 30, 4
    Q, K, V, score = make_slice(r, P, d, 1)
    st = O.prefill_compress_slice(K, V, score, 9, 1, 8, "f32")
    assert st.pos.tolist() == [0] + list(range(22, 30))
    out, log = O.decode_step_slice(st, r.standard_normal((1, d)), r.standard_normal(d), r.standard_normal(d), P, 0.7)
    assert log.victim_pos == 22                                      # only position t - M is outside sinks and window
    # a zero key has similarity 0 to everything and, evicted, merges with weight 1 / (1 + e) if it passes
    K0 = K.copy()
    K0[5] = 0.0
    s0 = O.prefill_compress_slice(K0, V, score, 9, 1, 8, "f32")
    i5 = list(s0.log["evicted"]).index(5)
    assert s0.log["mx"][i5] == 0.0 and s0.log["nn"][i5] == 0


# ---------------------------------------------------------------- ragged batch (per-sequence prompt lengths)
def test_ragged_batch_equals_separate_sequences():
    r = rng(68)
    L, Hq, Hkv, d, Pmax = 2, 4, 2, 8, 40
    lens = [40, 23]
    Qs = [r.standard_normal((2, Hq, Pmax, d)) for _ in range(L)]
    Ks = [r.standard_normal((2, Hkv, Pmax, d)) for _ in range(L)]
    Vs = [r.standard_normal((2, Hkv, Pmax, d)) for _ in range(L)]
    kw = dict(n_layers=L, n_q_heads=Hq, n_kv_heads=Hkv, d_head=d, dtype="f32", rho=0.4, n_sink=1, window=0,
              nm_ratio=3.0, beta=0.7, density_temp=4.0, min_budget=4)
    rag = O.OracleStack(batch=2, prompt_len=Pmax, prompt_lens=lens, **kw)
    for l in range(L):
        rag.layer_stats(l, Qs[l], Ks[l])
    rag.layer_budgets()
    for l in range(L):
        rag.prefill_compress(l, Ks[l], Vs[l])
    dec = [(r.standard_normal((2, Hq, d)), r.standard_normal((2, Hkv, d)), r.standard_normal((2, Hkv, d)))
           for _ in range(3)]
    outs = [[rag.decode_step(l, *dec[s], s) for l in range(L)] for s in range(3)]
    for b, Pb in enumerate(lens):
        one = O.OracleStack(batch=1, prompt_len=Pb, **kw)
        for l in range(L):
            one.layer_stats(l, Qs[l][b:b + 1, :, :Pb], Ks[l][b:b + 1, :, :Pb])
        one.layer_budgets()
        np.testing.assert_array_equal(one.budgets[0], rag.budgets[b])
        assert rag.budgets[b].sum() == Hkv * math.floor(0.4 * L * Pb + 0.5)
        for l in range(L):
            one.prefill_compress(l, Ks[l][b:b + 1, :, :Pb], Vs[l][b:b + 1, :, :Pb])
        for s in range(3):
            for l in range(L):
                res = one.decode_step(l, dec[s][0][b:b + 1], dec[s][1][b:b + 1], dec[s][2][b:b + 1], s)
                for h in range(Hkv):
                    np.testing.assert_array_equal(res[(0, h)][0], outs[s][l][(b, h)][0])
                    assert res[(0, h)][1].victim_pos == outs[s][l][(b, h)][1].victim_pos
                    assert outs[s][l][(b, h)][1].victim_pos < Pb + s + 1
