"""The checked build (libd2o_checked.so, -DD2O_CHECKED): every index a kernel derives from data is compared with
its range before use; a violation sets the error word instead of touching memory.  The whole path must run clean
(error word 0) and match the oracle exactly as the ordinary build does.  This is the library's memory-safety
evidence next to the oracle comparison."""
import dataclasses
import os

import pytest

from paper_2406_13035_b200 import binding as B
from paper_2406_13035_b200 import build
from paper_2406_13035_b200 import workloads as W

from parity import assert_report, run_parity

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _checked_library(cuda_device):
    path = build.build_library(checked=True)
    assert os.path.exists(path)
    B.use_library(path)
    B.load_library()
    yield
    B.use_library(build.LIB)
    build.build_library()
    B.load_library()


@pytest.mark.parametrize("name", ["cfg0", "cfg1", "cfg2", "cfg3", "cfg4"])
def test_checked_build_runs_clean(name):
    wl = W.CONFIGS["cfg0"] if name == "cfg0" else dataclasses.replace(W.twin(name), n_layers=2, decode_steps=8)
    rep = run_parity(wl)                       # asserts error word 0 at the end
    assert_report(rep, wl.dtype)
    assert rep.merges + rep.discards > 0


def test_checked_build_budget_rules_and_fp32_similarity():
    wl = dataclasses.replace(W.twin("cfg2"), n_layers=2, decode_steps=4)
    assert_report(run_parity(wl, ctx_over=dict(budget_rule=1)), wl.dtype)
    assert_report(run_parity(wl, similarity_path=1, stats_path=1), wl.dtype)


def test_checked_build_multi_layer_and_multi_step_entry_points():
    """The several-layers / several-steps calls on the checked build: error word 0, and the same outputs as the
    single calls of the same build."""
    import torch
    from parity import make_ctx
    wl = dataclasses.replace(W.twin("cfg2"), n_layers=3, decode_steps=9)
    a, b = make_ctx(wl), make_ctx(wl)
    streams = [W.LayerStream(wl, l, "cuda:0") for l in range(wl.n_layers)]
    P = [s.prompt() for s in streams]
    for l, (Q, K, V) in enumerate(P):
        a.d2o_layer_stats(l, Q, K)
    b.d2o_layer_stats_layers(0, wl.n_layers, [p[0] for p in P], [p[1] for p in P])
    a.d2o_layer_budgets(); b.d2o_layer_budgets()
    for l, (Q, K, V) in enumerate(P):
        a.d2o_prefill_compress(l, K, V)
    b.d2o_prefill_compress_layers(0, wl.n_layers, [p[1] for p in P], [p[2] for p in P])
    qs, ks, vs = [], [], []
    for _ in range(wl.decode_steps):
        q, k, v = zip(*[s.decode() for s in streams])
        qs.append(torch.stack(q)); ks.append(torch.stack(k)); vs.append(torch.stack(v))
    dq, dk, dv = torch.stack(qs), torch.stack(ks), torch.stack(vs)
    oa, ob = torch.empty_like(dq), torch.empty_like(dq)
    for s in range(wl.decode_steps):
        a.d2o_decode_step(0, wl.n_layers, dq[s], dk[s], dv[s], oa[s])
    b.d2o_decode_steps(0, wl.n_layers, 5, dq[:5], dk[:5], dv[:5], ob[:5])
    hq, hk, hv = dq[5:].cpu().pin_memory(), dk[5:].cpu().pin_memory(), dv[5:].cpu().pin_memory()
    ho = torch.empty_like(hq).pin_memory()
    b.d2o_decode_steps_host(0, wl.n_layers, 4, hq, hk, hv, ho)
    ob[5:] = ho.cuda()
    torch.cuda.synchronize()
    for c in (a, b):
        st = c.d2o_get_stats()
        assert st.error_word == 0, f"device error word {st.error_word} detail {st.error_detail:#x}"
    assert torch.equal(oa.view(torch.uint8), ob.view(torch.uint8))
    a.close(); b.close()
