"""GPU parity: the CUDA path through the C ABI against the float64 oracle, same seeded inputs."""
import dataclasses
import math

import numpy as np
import pytest
import torch

from oracle import d2o_oracle as O
from paper_2406_13035_b200 import binding as B
from paper_2406_13035_b200 import workloads as W

from parity import assert_report, close, np64, run_parity

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _lib(cuda_device):
    from paper_2406_13035_b200 import build
    build.build_library()
    B.load_library()


def small(name="cfg0", **kw):
    return dataclasses.replace(W.CONFIGS[name], **kw)


def test_cfg0_whole_pipeline():
    wl = W.CONFIGS["cfg0"]
    rep = run_parity(wl)
    assert rep.checked_slices == 8 and rep.steps == 16
    assert rep.merges + rep.discards == 8 * 16
    assert_report(rep, wl.dtype)
    print("cfg0", rep.max_err, rep.ties, rep.merges, rep.discards)


@pytest.mark.parametrize("name", ["cfg1", "cfg2", "cfg3", "cfg4"])
def test_scaled_twins(name):
    wl = W.twin(name)
    rep = run_parity(wl)
    assert_report(rep, wl.dtype)
    assert rep.merges > 0 and rep.discards > 0
    print(name, rep.max_err, rep.ties, rep.merges, rep.discards)


@pytest.mark.parametrize("stages,hints", [(2, 1), (3, 0), (9, 1)])
def test_ring_depths_agree(stages, hints):
    wl = small(prompt_len=512, decode_steps=8)
    rep = run_parity(wl, decode_stages=stages, decode_l2_hints=hints)
    assert_report(rep, wl.dtype)


@pytest.mark.parametrize("name,warps", [("cfg1", 4), ("cfg4", 4), ("cfg2", 16), ("cfg3", 16)])
def test_decode_cta_sizes_agree(name, warps):
    wl = W.twin(name)
    rep = run_parity(wl, decode_warps=warps, steps=8)
    assert_report(rep, wl.dtype)


@pytest.mark.parametrize("name,rows", [("cfg1", 64), ("cfg2", 40), ("cfg3", 128), ("cfg0", 8)])
def test_logits_beyond_shared_memory_agree(name, rows):
    # most rows of every slice keep their logits in the L2-resident array instead of shared memory
    wl = W.CONFIGS[name] if name == "cfg0" else W.twin(name)
    rep = run_parity(wl, decode_smem_rows=rows, steps=8)
    assert_report(rep, wl.dtype)


@pytest.mark.parametrize("name,pairs", [("cfg1", 1), ("cfg2", 3), ("cfg3", 2), ("cfg4", 1), ("cfg0", 1)])
def test_long_slice_launch_agrees(name, pairs):
    # the pairs with the largest budgets in a sixteen-warp launch of their own, the rest overlapping it
    wl = dataclasses.replace(W.CONFIGS[name], n_layers=2, decode_steps=8) if name == "cfg0" else W.twin(name)
    rep = run_parity(wl, decode_long_pairs=pairs, steps=8)
    assert_report(rep, wl.dtype)


def test_layer_by_layer_calls_match():
    wl = W.twin("cfg1")
    rep = run_parity(wl, layers_per_call=1, steps=6)
    assert_report(rep, wl.dtype)


@pytest.mark.parametrize("tau", [float("inf"), float("-inf")])
def test_threshold_overrides(tau):
    wl = small(prompt_len=384, decode_steps=6)
    rep = run_parity(wl, ctx_over=dict(tau_override=tau))
    assert_report(rep, wl.dtype)
    if tau > 0:
        assert rep.merges == 0            # pure eviction
    else:
        assert rep.discards == 0          # every victim merged


@pytest.mark.parametrize("T,window,d,dtype,hq,hkv", [(0, 8, 64, "f16", 4, 4), (4, 0, 128, "f32", 4, 2),
                                                     (2, 16, 64, "bf16", 8, 1), (1, 0, 128, "bf16", 8, 4)])
def test_shape_and_hyperparameter_sweep(T, window, d, dtype, hq, hkv):
    wl = dataclasses.replace(W.CONFIGS["cfg0"], name="sweep", n_q_heads=hq, n_kv_heads=hkv, d_head=d, dtype=dtype,
                             prompt_len=333, decode_steps=9, n_sink=T, window=window, rho=0.3, n_layers=2,
                             batch=2, density_temp=50.0, min_budget=max(8, T + 1))
    rep = run_parity(wl)
    assert_report(rep, wl.dtype)


@pytest.mark.parametrize("dtype,d,hq,hkv,warps,smem_rows", [
    ("f16", 128, 4, 2, 0, 0), ("f16", 128, 8, 2, 16, 0), ("f16", 128, 8, 1, 4, 0),
    ("f16", 64, 4, 2, 4, 0), ("f16", 64, 8, 2, 8, 0), ("bf16", 64, 8, 1, 16, 0),
    ("bf16", 64, 8, 2, 0, 0), ("f16", 64, 8, 4, 8, 96), ("bf16", 128, 8, 2, 8, 200),
])
def test_grouped_query_tensor_path_long_slices(dtype, d, hq, hkv, warps, smem_rows):
    # 16-bit caches with 2, 4 or 8 query heads per KV head (the mma.sync decode path, both element types), with
    # slices several ring stages long for every CTA size, also with most logits outside shared memory
    wl = dataclasses.replace(W.CONFIGS["cfg0"], name="gqa", n_q_heads=hq, n_kv_heads=hkv, d_head=d, dtype=dtype,
                             prompt_len=2048, decode_steps=6, n_sink=1, window=0, rho=0.3, n_layers=2, batch=1,
                             density_temp=500.0, min_budget=16, beta=0.7)
    rep = run_parity(wl, decode_warps=warps, decode_smem_rows=smem_rows)
    assert_report(rep, wl.dtype)
    assert rep.merges + rep.discards == rep.checked_slices * 6


@pytest.mark.parametrize("beta", [0.0, 1.0])
def test_ema_extremes(beta):
    # beta = 1 is the ablation's "w.o. EMA-Threshold" (every victim merged); beta = 0 freezes tau at tau_0
    wl = small(prompt_len=320, decode_steps=8, beta=beta)
    rep = run_parity(wl)
    assert_report(rep, wl.dtype)
    if beta == 1.0:
        assert rep.discards == 0 and rep.merges == 8 * 8
    wl = dataclasses.replace(W.twin("cfg2"), beta=beta, decode_steps=6)
    rep = run_parity(wl)
    assert_report(rep, wl.dtype)
    if beta == 1.0:
        assert rep.discards == 0


@pytest.mark.parametrize("name", ["cfg0", "cfg2"])
def test_window_and_sinks_only(name):
    # N = 0: the cache holds the sinks and the recent window only (S = T + M for every layer)
    base = W.CONFIGS["cfg0"] if name == "cfg0" else W.twin("cfg2")
    P = 256
    wl = dataclasses.replace(base, prompt_len=P, decode_steps=6, rho=0.125, window=30, n_sink=2, min_budget=32,
                             max_budget=32, density_temp=1e30, n_layers=min(base.n_layers, 2))
    rep = run_parity(wl)
    assert_report(rep, wl.dtype)
    assert rep.merges + rep.discards == rep.checked_slices * 6


@pytest.mark.parametrize("name", ["cfg0", "cfg1", "cfg2"])
def test_zero_norm_keys(name):
    # a zero key has similarity 0 to everything: as an evicted prompt token, as a retained one (window), as the
    # key of a generated token, and as the victim of a later step
    base = W.CONFIGS["cfg0"] if name == "cfg0" else W.twin(name)
    wl = dataclasses.replace(base, prompt_len=256, decode_steps=10, n_layers=min(base.n_layers, 2), max_budget=0)

    def prompt_hook(l, Q, K, V):
        K = K.clone()
        K[:, :, 7] = 0                    # low score, mid prompt: evicted
        K[:, :, 100] = 0
        K[:, :, 255] = 0                  # in the recent window: retained
        return Q, K, V

    def decode_hook(step, q, k, v):
        if step in (1, 2):
            k = k.clone()
            k[:] = 0
        return q, k, v

    rep = run_parity(wl, prompt_hook=prompt_hook, decode_hook=decode_hook)
    assert_report(rep, wl.dtype)


@pytest.mark.parametrize("name", ["cfg1", "cfg2"])
def test_rows_with_only_negative_similarities(name):
    # every key in the positive orthant except one in the negative orthant: all its cosines are negative, which the
    # tensor-core similarity kernel hands to the fp32 redo path of the reduce kernel
    wl = dataclasses.replace(W.twin(name), n_layers=2, decode_steps=4)
    seen = {"n": 0}

    def prompt_hook(l, Q, K, V):
        K = K.abs()
        K[:, :, 7] = -K[:, :, 7]
        seen["n"] += 1
        return Q, K, V

    rep = run_parity(wl, prompt_hook=prompt_hook)
    assert_report(rep, wl.dtype)
    assert seen["n"] == 2


@pytest.mark.parametrize("name", ["cfg0", "cfg1", "cfg2"])
def test_average_merge_policy(name):
    # the ablation's average merging: a kept token and everything merged into it weigh the same
    wl = small(prompt_len=320, decode_steps=8) if name == "cfg0" else dataclasses.replace(W.twin(name), n_layers=2,
                                                                                            decode_steps=8)
    rep = run_parity(wl, ctx_over=dict(merge_policy=1))
    assert_report(rep, wl.dtype)
    assert rep.merges > 0


@pytest.mark.parametrize("name", ["cfg1", "cfg2", "cfg0"])
def test_per_head_budgets(name):
    # S_l^h = alpha_l^h * S_total: every (layer, KV head) has its own cache size, window and threshold
    wl = dataclasses.replace(W.CONFIGS["cfg0"], n_layers=3, prompt_len=384, decode_steps=8, density_temp=40.0,
                             min_budget=24) if name == "cfg0" else dataclasses.replace(W.twin(name), decode_steps=8)
    rep = run_parity(wl, ctx_over=dict(budget_rule=1))
    assert_report(rep, wl.dtype)
    assert rep.merges + rep.discards > 0


@pytest.mark.parametrize("name", ["cfg1", "cfg2"])
def test_exponential_decay_budgets(name):
    # S_l = exp(-F_l / gamma) * P, not normalised: gamma of the order of the densities keeps the sizes between the clamps
    wl = dataclasses.replace(W.twin(name), decode_steps=6)
    rep = run_parity(wl, ctx_over=dict(budget_rule=2, density_temp=float(wl.prompt_len) / 1.5,
                                       max_budget=wl.prompt_len // 2))
    assert_report(rep, wl.dtype)
    assert rep.merges + rep.discards > 0


@pytest.mark.parametrize("name", ["cfg0", "cfg1", "cfg2"])
def test_value_feature_prompt_stage(name):
    # the ablation's "Feature choice" V: nearest neighbours, tau_0 and merge weights from the cosine of the values
    wl = small(prompt_len=320, decode_steps=0) if name == "cfg0" else dataclasses.replace(W.twin(name), n_layers=2,
                                                                                            decode_steps=0)
    rep = run_parity(wl, ctx_over=dict(sim_feature=1))
    assert_report(rep, wl.dtype)
    assert rep.steps == 0 and rep.gpu_stats.prefill_merged > 0
    from parity import make_ctx
    with pytest.raises(B.D2OError) as e:                  # generation with this switch is not built
        make_ctx(dataclasses.replace(wl, decode_steps=4), sim_feature=1)
    assert e.value.status == 2


@pytest.mark.parametrize("name", ["cfg0", "cfg2"])
def test_streaming_session_shape(name):
    # The multi-turn setting of the paper's appendix (fixed budget 2048 with N = 48 important and M = 2000 recent
    # tokens, no sinks), scaled by 1/16: the prompt is shorter than the budget, so the cache first grows by appending,
    # then every new token evicts one; the cache is almost all window.
    base = W.CONFIGS["cfg0"] if name == "cfg0" else W.twin("cfg2")
    wl = dataclasses.replace(base, n_layers=2, batch=1, prompt_len=64, decode_steps=100, rho=2.0, n_sink=0,
                             window=125, min_budget=128, max_budget=128, density_temp=1e30)
    rep = run_parity(wl)
    assert_report(rep, wl.dtype)
    assert rep.merges + rep.discards == rep.checked_slices * (100 - 64)      # evictions start once 128 rows are held


@pytest.mark.parametrize("name,lens", [("cfg0", [384, 131]), ("cfg1", [512, 77]), ("cfg2", [1024, 389]),
                                       ("cfg2", [300, 1024])])
def test_ragged_batch(name, lens):
    # per-sequence prompt lengths in one padded batch: own column sums, budgets, eviction and token positions
    base = dataclasses.replace(W.CONFIGS["cfg0"], n_layers=2, batch=2, prompt_len=384, density_temp=40.0,
                               min_budget=16) if name == "cfg0" else W.twin(name)
    wl = dataclasses.replace(base, batch=2, decode_steps=6, max_budget=0, min_budget=min(base.min_budget, 16))
    assert wl.prompt_len == max(lens)
    rep = run_parity(wl, prompt_lens=lens)
    # a 77-token prompt has many nearly equal small scores at its end: one Top-N boundary of the 256 slices of the
    # fp16 case is a tie below 1e-6 relative between float32 and float64 (counted, followed)
    assert_report(rep, wl.dtype, max_ties=1 if name == "cfg1" else 0)
    print("ragged", name, lens, rep.ties)
    assert rep.merges + rep.discards == rep.checked_slices * 6


def test_ragged_lengths_are_validated(cuda_device):
    from parity import make_ctx
    wl = small(prompt_len=256, decode_steps=2, batch=2)
    ctx = make_ctx(wl)
    for bad in ([256, 0], [257, 10], [256, 20]):         # 20 positions cannot hold L * min_budget = 8 rows at rho 0.25
        with pytest.raises(B.D2OError) as e:
            ctx.d2o_set_prompt_lens(bad)
        assert e.value.status == 1
    ctx.d2o_set_prompt_lens([256, 100])
    s = W.LayerStream(wl, 0, "cuda:0")
    Q, K, V = s.prompt()
    ctx.d2o_layer_stats(0, Q, K)
    with pytest.raises(B.D2OError) as e:                  # too late: the prompt is being fed
        ctx.d2o_set_prompt_lens([256, 100])
    assert e.value.status == 4
    ctx.close()


def test_more_sinks_than_budget_is_rejected(cuda_device):
    from parity import make_ctx
    wl = small(prompt_len=128, decode_steps=2, n_sink=40, min_budget=8)
    with pytest.raises(B.D2OError) as e:
        make_ctx(wl)
    assert e.value.status == 1            # min_budget must leave room for the sinks and one more token


def test_budget_never_reached_equals_full_attention():
    """With S_l >= prompt + steps nothing is evicted and the output is plain softmax attention."""
    wl = small(prompt_len=200, decode_steps=7, rho=1.035)
    rep = run_parity(wl, ctx_over=dict(max_budget=207))
    assert rep.merges == 0 and rep.discards == 0
    assert_report(rep, wl.dtype)


def test_budgets_large_temperature_gives_uniform_allocation(cuda_device):
    # gamma -> infinity: the uniform allocation of the paper's ablation (alpha_l = rho)
    F = np.random.default_rng(3).gamma(1.0, size=(2, 16, 8)) * 500.0
    bud, win, off, status = B.d2o_budgets_from_density(torch.tensor(F, device=cuda_device), n_kv_heads=2,
                                                       prompt_len=2000, rho=B.f32(0.2), min_budget=1,
                                                       density_temp=B.f32(1e30), head_reduce=0, n_sink=1, window=0,
                                                       nm_ratio=B.f32(3.0))
    assert int(status[0]) == 0
    assert (bud.cpu().numpy() == 400).all()


def test_budgets_pure_function_matches_oracle(cuda_device):
    r = np.random.default_rng(5)
    done = 0
    for trial in range(60):
        Bn, L, H = int(r.integers(1, 4)), int(r.integers(1, 40)), 2 * int(r.integers(1, 5))
        P = int(r.integers(64, 9000))
        rho = B.f32(float(r.uniform(0.05, 1.0)))
        gamma = B.f32(float(r.choice([1.0, 10.0, 1000.0])))
        smin = int(r.integers(1, 12))
        F = r.gamma(1.0, size=(Bn, L, H)) * float(r.choice([0.01, 1.0, 30.0, 3000.0]))
        tot = math.floor(rho * L * P + 0.5)
        # every other trial with an upper clamp between the mean and four times the mean
        cap = 0 if trial % 2 == 0 else int(min(P, max(smin, math.ceil(tot / L * float(r.uniform(1.0, 4.0))))))
        if L * smin > tot or (cap and L * cap < tot):
            continue
        hr = int(trial % 4)                                          # both softmax rules and both reciprocal rules
        nm = B.f32(3.0)
        bud, win, off, status = B.d2o_budgets_from_density(torch.tensor(F, device=cuda_device), n_kv_heads=2,
                                                           prompt_len=P, rho=rho, min_budget=smin, max_budget=cap,
                                                           density_temp=gamma, head_reduce=hr, n_sink=1, window=0,
                                                           nm_ratio=nm)
        bud = bud.cpu().numpy()
        assert int(status[0]) == 0
        for b in range(Bn):
            ref = O.layer_budgets(F[b], P, rho, smin, gamma, hr, cap)
            np.testing.assert_array_equal(bud[b, :, 0], ref)
            np.testing.assert_array_equal(bud[b, :, 1], ref)          # every KV head of a layer gets the layer's size
            for l in range(L):
                assert int(win[b, l, 0]) == O.window_size(int(ref[l]), min(1, int(ref[l])), 0, nm)
        o = off.cpu().numpy()
        run = 0
        for l in range(L):
            for b in range(Bn):
                for h in range(2):
                    assert o[b, l, h] == run
                    run += (bud[b, l, h] + 7) // 8 * 8      # slices start at multiples of 8 rows
        done += 1
    assert done > 30


def test_per_head_and_exponential_decay_budgets_match_oracle(cuda_device):
    r = np.random.default_rng(15)
    done = 0
    for trial in range(40):
        Bn, L, Hkv, G = int(r.integers(1, 3)), int(r.integers(1, 33)), int(r.choice([1, 2, 8, 32])), int(r.choice([1, 2, 4, 8]))
        H = Hkv * G
        P = int(r.integers(64, 9000))
        rho = B.f32(float(r.uniform(0.05, 1.0)))
        gamma = B.f32(float(r.choice([1.0, 10.0, 1000.0])))
        smin = int(r.integers(1, 12))
        F = r.gamma(1.0, size=(Bn, L, H)) * float(r.choice([0.01, 1.0, 30.0, 3000.0]))
        tot = math.floor(rho * (L * Hkv) * P + 0.5)
        cap = 0 if trial % 2 == 0 else int(min(P, max(smin, math.ceil(tot / (L * Hkv) * float(r.uniform(1.0, 4.0))))))
        if L * Hkv * smin > tot or (cap and L * Hkv * cap < tot):
            continue
        kw = dict(n_kv_heads=Hkv, prompt_len=P, rho=rho, min_budget=smin, max_budget=cap, density_temp=gamma,
                  n_sink=1, window=0, nm_ratio=B.f32(3.0))
        bud, _, off, status = B.d2o_budgets_from_density(torch.tensor(F, device=cuda_device), budget_rule=1, **kw)
        assert int(status[0]) == 0
        bud = bud.cpu().numpy()
        for b in range(Bn):
            np.testing.assert_array_equal(bud[b], O.head_budgets(F[b], P, rho, G, smin, gamma, cap))
        o = off.cpu().numpy()
        run = 0
        for l in range(L):
            for b in range(Bn):
                for h in range(Hkv):
                    assert o[b, l, h] == run
                    run += (bud[b, l, h] + 7) // 8 * 8
        bud2, _, _, status = B.d2o_budgets_from_density(torch.tensor(F, device=cuda_device), budget_rule=2, **kw)
        assert int(status[0]) == 0
        bud2 = bud2.cpu().numpy()
        for b in range(Bn):
            ref = O.exp_decay_budgets(F[b], P, smin, gamma, cap)
            for h in range(Hkv):
                np.testing.assert_array_equal(bud2[b, :, h], ref)
        done += 1
    assert done > 20


@pytest.mark.parametrize("dtype,d,G,n_slices,cap,length", [("f16", 128, 1, 6, 700, 513), ("bf16", 128, 4, 3, 4100, 4099),
                                                           ("f32", 64, 2, 5, 64, 0), ("f16", 64, 8, 2, 300, 77)])
def test_full_decode_kernel(cuda_device, dtype, d, G, n_slices, cap, length):
    td = W.TORCH_DTYPES[dtype]
    g = torch.Generator(device=cuda_device).manual_seed(11)
    kc = torch.randn(n_slices, cap, d, generator=g, device=cuda_device).to(td)
    vc = torch.randn(n_slices, cap, d, generator=g, device=cuda_device).to(td)
    q = (2 * torch.randn(n_slices, G, d, generator=g, device=cuda_device)).to(td)
    k = torch.randn(n_slices, d, generator=g, device=cuda_device).to(td)
    v = torch.randn(n_slices, d, generator=g, device=cuda_device).to(td)
    out = torch.empty_like(q)
    kc0, vc0 = kc.clone(), vc.clone()
    B.d2o_full_decode_step(kc, vc, length, q, k, v, out)
    torch.cuda.synchronize()
    assert torch.equal(kc[:, length], k) and torch.equal(vc[:, length], v)          # appended
    assert torch.equal(kc[:, :length], kc0[:, :length]) and torch.equal(kc[:, length + 1:], kc0[:, length + 1:])
    for s in range(n_slices):
        Kf = np.vstack([np64(kc0[s, :length]), np64(k[s])[None]])
        Vf = np.vstack([np64(vc0[s, :length]), np64(v[s])[None]])
        ref = O.full_attention_step(np64(q[s]), Kf, Vf)
        assert close(np64(out[s]), ref, dtype) <= 1.0


def test_out_of_order_calls_are_rejected(cuda_device):
    from parity import make_ctx
    wl = small(prompt_len=128, decode_steps=2)
    ctx = make_ctx(wl)
    s = W.LayerStream(wl, 0, "cuda:0")
    Q, K, V = s.prompt()
    with pytest.raises(B.D2OError) as e:
        ctx.d2o_layer_budgets()
    assert e.value.status == 4
    with pytest.raises(B.D2OError) as e:
        ctx.d2o_prefill_compress(0, K, V)
    assert e.value.status == 4
    ctx.d2o_layer_stats(0, Q, K)
    ctx.d2o_layer_budgets()
    q, k, v = s.decode()
    out = torch.empty_like(q)
    with pytest.raises(B.D2OError) as e:
        ctx.d2o_decode_step(0, 1, q, k, v, out)
    assert e.value.status == 4
    ctx.d2o_prefill_compress(0, K, V)
    ctx.d2o_decode_step(0, 1, q, k, v, out)
    ctx.d2o_decode_step(0, 1, q, k, v, out)
    with pytest.raises(B.D2OError) as e:                      # max_new_tokens = 2
        ctx.d2o_decode_step(0, 1, q, k, v, out)
    assert e.value.status == 4
    assert ctx.d2o_get_stats().error_word == 0


def test_host_buffer_entry_matches_device_entry(cuda_device):
    from parity import make_ctx
    wl = W.twin("cfg2")
    outs = []
    for host in (False, True):
        ctx = make_ctx(wl)
        streams = [W.LayerStream(wl, l, "cuda:0") for l in range(wl.n_layers)]
        kv = []
        for l, s in enumerate(streams):
            Q, K, V = s.prompt()
            ctx.d2o_layer_stats(l, Q, K)
            kv.append((K, V))
        ctx.d2o_layer_budgets()
        for l, (K, V) in enumerate(kv):
            ctx.d2o_prefill_compress(l, K, V)
        res = []
        for step in range(4):
            q, k, v = (torch.stack(x) for x in zip(*[s.decode() for s in streams]))
            if host:
                qh, kh, vh = q.cpu().pin_memory(), k.cpu().pin_memory(), v.cpu().pin_memory()
                oh = torch.empty_like(qh).pin_memory()
                ctx.d2o_decode_step_host(0, wl.n_layers, qh, kh, vh, oh)
                res.append(oh.clone())
            else:
                o = torch.empty_like(q)
                ctx.d2o_decode_step(0, wl.n_layers, q, k, v, o)
                res.append(o.cpu())
        outs.append(torch.stack(res))
        ctx.close()
    assert torch.equal(outs[0], outs[1])
