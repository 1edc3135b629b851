"""The seeded input generator: shapes, determinism, dtype, and the structure the recipe promises."""
import numpy as np
import torch

from paper_2406_13035_b200 import workloads as W


def test_configs_cover_the_five_benchmark_shapes():
    assert set(W.CONFIGS) == {"cfg0", "cfg1", "cfg2", "cfg3", "cfg4", "session"}
    ses = W.CONFIGS["session"]                          # the multi-turn shape: 2048 = 48 important + 2000 recent tokens
    assert ses.max_budget == ses.min_budget == 2048 and ses.window == 2000 and ses.n_sink == 0
    c1 = W.CONFIGS["cfg1"]
    assert (c1.n_layers, c1.n_q_heads, c1.n_kv_heads, c1.d_head, c1.dtype, c1.prompt_len) == (32, 32, 32, 128, "f16", 4096)
    assert W.CONFIGS["cfg2"].group == 4 and W.CONFIGS["cfg3"].prompt_len == 32768
    assert c1.layer_temp(0) == 1.0 and abs(c1.layer_temp(31) - 0.25) < 1e-12


def test_layer_stream_is_deterministic_and_shaped():
    wl = W.twin("cfg2")
    a, b = W.LayerStream(wl, 1), W.LayerStream(wl, 1)
    qa, ka, va = a.prompt()
    qb, kb, vb = b.prompt()
    assert qa.shape == (wl.batch, wl.n_q_heads, wl.prompt_len, wl.d_head)
    assert ka.shape == va.shape == (wl.batch, wl.n_kv_heads, wl.prompt_len, wl.d_head)
    assert qa.dtype == torch.bfloat16
    assert torch.equal(qa, qb) and torch.equal(ka, kb) and torch.equal(va, vb)
    da, db = a.decode(), b.decode()
    assert all(torch.equal(x, y) for x, y in zip(da, db))
    assert da[0].shape == (wl.batch, wl.n_q_heads, wl.d_head) and da[1].shape == (wl.batch, wl.n_kv_heads, wl.d_head)
    q2 = W.LayerStream(wl, 2).prompt()[0]
    assert not torch.equal(q2, qa)


def test_sink_and_ar1_structure():
    wl = W.CONFIGS["cfg0"]
    s = W.LayerStream(wl, 0)
    q, k, v = s.prompt()
    kn = k.double().norm(dim=-1)
    rms = kn.pow(2).mean(dim=-1).sqrt()
    assert torch.all(kn[:, :, 0] > 3.5 * rms)                         # sink key norm ~4x
    eta = q.double() - s.m_q[:, :, None, :].double()
    c = (eta[:, :, 1:] * eta[:, :, :-1]).mean() / (eta * eta).mean()
    assert 0.85 < float(c) < 0.95                                      # AR(1) coefficient 0.9


def test_ar1_blocks_match_recurrence():
    g = torch.Generator().manual_seed(1)
    xi = torch.randn(2, 150, 3, generator=g)
    eta, last = W._ar1(xi, torch.zeros(2, 3))
    ref = torch.zeros(2, 3)
    for i in range(150):
        ref = 0.9 * ref + (1 - 0.81) ** 0.5 * xi[:, i]
        assert torch.allclose(eta[:, i], ref, atol=1e-5)
    assert torch.allclose(last, ref, atol=1e-5)
