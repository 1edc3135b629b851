"""d2o_prefill_compress_layers (several layers per call, up to four side by side on the library's own streams)
against d2o_prefill_compress called layer by layer: the compressed caches, thresholds and the decode steps that
follow must be identical bit for bit."""
import dataclasses

import numpy as np
import pytest
import torch

from paper_2406_13035_b200 import binding as B
from paper_2406_13035_b200 import workloads as W

from parity import make_ctx

pytestmark = [pytest.mark.gpu]


@pytest.fixture(scope="module", autouse=True)
def _lib(cuda_device):
    from paper_2406_13035_b200 import build
    build.build_library()
    B.load_library()


def _same_slice(sa, sb, tag):
    assert sa["len"] == sb["len"] and sa["S"] == sb["S"], tag
    assert np.float32(sa["tau"]).tobytes() == np.float32(sb["tau"]).tobytes(), tag
    for key in ("pos", "score", "rnorm", "K", "V"):
        assert torch.equal(sa[key].view(torch.uint8), sb[key].view(torch.uint8)), (key, tag)


def _run(wl, ranges, steps=4, device="cuda:0"):
    """`ranges`: the (l0, l1) calls of the second context; together they cover every layer once."""
    a, b = make_ctx(wl, device), make_ctx(wl, device)
    streams = [W.LayerStream(wl, l, device) for l in range(wl.n_layers)]
    KV = []
    for l in range(wl.n_layers):
        Q, K, V = streams[l].prompt()
        a.d2o_layer_stats(l, Q, K)
        b.d2o_layer_stats(l, Q, K)
        KV.append((K, V))
    a.d2o_layer_budgets()
    b.d2o_layer_budgets()
    for l in range(wl.n_layers):
        a.d2o_prefill_compress(l, *KV[l])
    for l0, l1 in ranges:
        b.d2o_prefill_compress_layers(l0, l1, [KV[l][0] for l in range(l0, l1)], [KV[l][1] for l in range(l0, l1)])
    # the caller's stream continues behind every lane: decode at once, no synchronisation in between
    outs = []
    for s in range(steps):
        q, k, v = [torch.stack(t) for t in zip(*[st.decode() for st in streams])]
        oa, ob = torch.empty_like(q), torch.empty_like(q)
        a.d2o_decode_step(0, wl.n_layers, q, k, v, oa)
        b.d2o_decode_step(0, wl.n_layers, q, k, v, ob)
        outs.append((oa, ob))
    torch.cuda.synchronize()
    for c in (a, b):
        st = c.d2o_get_stats()
        assert st.error_word == 0, f"device error word {st.error_word} detail {st.error_detail:#x}"
    sa, sb = a.d2o_get_stats(), b.d2o_get_stats()
    assert (sa.prefill_evicted, sa.prefill_merged, sa.merges, sa.discards) == \
           (sb.prefill_evicted, sb.prefill_merged, sb.merges, sb.discards)
    for oa, ob in outs:
        assert torch.equal(oa.view(torch.uint8), ob.view(torch.uint8))
    ta, tb = a.tables(), b.tables()
    for l in range(wl.n_layers):
        for bb in range(wl.batch):
            for h in range(wl.n_kv_heads):
                _same_slice(a.slice_state(l, bb, h, ta), b.slice_state(l, bb, h, tb), (l, bb, h))
    a.close(); b.close()


@pytest.mark.parametrize("name", ["cfg1", "cfg2", "cfg3"])
def test_all_layers_in_one_call(name):
    wl = dataclasses.replace(W.twin(name), decode_steps=4)
    _run(wl, [(0, wl.n_layers)])


def test_more_layers_than_lanes_and_split_calls():
    wl = W.twin("cfg1").scaled(n_layers=11, prompt_div=1, batch=1, steps=4)
    _run(wl, [(0, 7), (7, 8), (8, 11)])


def test_fp32_config_0_shape():
    wl = dataclasses.replace(W.CONFIGS["cfg0"], n_layers=6, decode_steps=4, density_temp=50.0, min_budget=64)
    _run(wl, [(0, 6)])


@pytest.mark.parametrize("name", ["cfg0", "cfg1", "cfg2"])
def test_layer_stats_of_several_layers_in_one_call(name):
    """d2o_layer_stats_layers against layer-by-layer calls: column sums, densities and budgets bit for bit."""
    wl = (dataclasses.replace(W.CONFIGS["cfg0"], n_layers=5, density_temp=50.0, min_budget=64) if name == "cfg0"
          else W.twin(name).scaled(n_layers=5, prompt_div=1, batch=2, steps=2))
    a, b = make_ctx(wl), make_ctx(wl)
    streams = [W.LayerStream(wl, l, "cuda:0") for l in range(wl.n_layers)]
    QK = [s.prompt()[:2] for s in streams]
    for l, (Q, K) in enumerate(QK):
        a.d2o_layer_stats(l, Q, K)
    b.d2o_layer_stats_layers(0, 3, [q for q, _ in QK[:3]], [k for _, k in QK[:3]])
    b.d2o_layer_stats_layers(3, 4, [QK[3][0]], [QK[3][1]])
    b.d2o_layer_stats_layers(4, 5, [QK[4][0]], [QK[4][1]], [None])
    for l in range(wl.n_layers):
        assert torch.equal(a.colsum(l).view(torch.uint8), b.colsum(l).view(torch.uint8)), l
    assert torch.equal(a.density().view(torch.uint8), b.density().view(torch.uint8))
    assert torch.equal(a.d2o_layer_budgets(), b.d2o_layer_budgets())
    for c in (a, b):
        assert c.d2o_get_stats().error_word == 0
    a.close(); b.close()


def test_argument_checks():
    wl = dataclasses.replace(W.twin("cfg1"), decode_steps=2)
    c = make_ctx(wl)
    s = W.LayerStream(wl, 0, "cuda:0")
    Q, K, V = s.prompt()
    with pytest.raises(B.D2OError) as e:                   # budgets first
        c.d2o_prefill_compress_layers(0, 2, [K, K], [V, V])
    assert e.value.status == 4
    with pytest.raises(B.D2OError) as e:
        c.d2o_prefill_compress_layers(2, 2, [], [])
    assert e.value.status == 1
    c.close()
