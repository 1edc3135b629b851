"""d2o_decode_steps (several generated tokens per call, a step's grids chained to the previous step's by a per-slice
step counter) against d2o_decode_step called once per token.

The header promises the same results bit for bit, so two contexts are fed the same seeded tensors: one is stepped
call by call (the path the oracle parity tests cover), the other takes the tokens in one or several multi-step
calls.  Outputs of every step and the final state of every checked slice must be identical.  One case also runs the
oracle beside the chained context's outputs.
"""
import dataclasses

import numpy as np
import pytest
import torch

from paper_2406_13035_b200 import binding as B
from paper_2406_13035_b200 import workloads as W

from parity import close, make_ctx, make_oracle, np64, _lazy64

pytestmark = [pytest.mark.gpu]


@pytest.fixture(scope="module", autouse=True)
def _lib(cuda_device):
    from paper_2406_13035_b200 import build
    build.build_library()
    B.load_library()


def _prepare(wl, n_ctx, device="cuda:0", **over):
    """Contexts after the prompt stage on the same tensors, and the decode inputs of all steps."""
    ctxs = [make_ctx(wl, device, **over) for _ in range(n_ctx)]
    streams = [W.LayerStream(wl, l, device) for l in range(wl.n_layers)]
    KV = []
    for l in range(wl.n_layers):
        Q, K, V = streams[l].prompt()
        for c in ctxs:
            c.d2o_layer_stats(l, Q, K)
        KV.append((K, V))
        del Q
    for c in ctxs:
        c.d2o_layer_budgets()
    for l in range(wl.n_layers):
        for c in ctxs:
            c.d2o_prefill_compress(l, *KV[l])
    qs, ks, vs = [], [], []
    for _ in range(wl.decode_steps):
        q, k, v = zip(*[s.decode() for s in streams])
        qs.append(torch.stack(q)); ks.append(torch.stack(k)); vs.append(torch.stack(v))
    return ctxs, KV, torch.stack(qs).contiguous(), torch.stack(ks).contiguous(), torch.stack(vs).contiguous()


def _same_state(a, b, slices):
    ta, tb = a.tables(), b.tables()
    for x, y in zip(ta, tb):
        assert torch.equal(x, y)
    for l, bb, h in slices:
        sa, sb = a.slice_state(l, bb, h, ta), b.slice_state(l, bb, h, tb)
        assert sa["len"] == sb["len"] and sa["S"] == sb["S"], (l, bb, h)
        assert np.float32(sa["tau"]).tobytes() == np.float32(sb["tau"]).tobytes(), (l, bb, h)
        for key in ("pos", "score", "rnorm", "K", "V"):
            assert torch.equal(sa[key].view(torch.uint8), sb[key].view(torch.uint8)), (key, l, bb, h)


def _all_slices(wl):
    return [(l, b, h) for l in range(wl.n_layers) for b in range(wl.batch) for h in range(wl.n_kv_heads)]


def _run_pair(wl, calls, slices=None, long_pairs=0, **over):
    """`calls`: step counts of the multi-step calls (0 = one single-step call) that together cover wl.decode_steps."""
    (a, b), _, dq, dk, dv = _prepare(wl, 2, **over)
    if long_pairs:
        for c in (a, b):
            c.d2o_set_tuning(0, 1, 0, 0, 0, 0, long_pairs)
    L, n = wl.n_layers, wl.decode_steps
    out_a = torch.empty_like(dq)
    out_b = torch.full_like(dq, float("nan"))
    for s in range(n):
        a.d2o_decode_step(0, L, dq[s], dk[s], dv[s], out_a[s])
    s = 0
    for cnt in calls:
        if cnt == 0:
            b.d2o_decode_step(0, L, dq[s], dk[s], dv[s], out_b[s])
            s += 1
        else:
            b.d2o_decode_steps(0, L, cnt, dq[s:s + cnt], dk[s:s + cnt], dv[s:s + cnt], out_b[s:s + cnt])
            s += cnt
    assert s == n
    torch.cuda.synchronize()
    for c in (a, b):
        st = c.d2o_get_stats()
        assert st.error_word == 0, f"device error word {st.error_word} detail {st.error_detail:#x}"
    assert a.d2o_get_stats().decode_steps == b.d2o_get_stats().decode_steps
    assert torch.equal(out_a.view(torch.uint8), out_b.view(torch.uint8))
    _same_state(a, b, _all_slices(wl) if slices is None else slices)
    a.close(); b.close()


@pytest.mark.parametrize("name", ["cfg0", "cfg1", "cfg2", "cfg3", "cfg4"])
def test_chained_steps_equal_single_steps(name):
    wl = W.CONFIGS["cfg0"] if name == "cfg0" else dataclasses.replace(W.twin(name), decode_steps=24)
    _run_pair(wl, [wl.decode_steps])


def test_chained_and_single_calls_mixed():
    wl = dataclasses.replace(W.twin("cfg2"), decode_steps=20)
    _run_pair(wl, [1, 5, 0, 0, 9, 2, 0])


def test_chained_steps_while_the_cache_still_fills():
    # budgets above the prompt length: the first steps append, the later ones evict
    wl = dataclasses.replace(W.CONFIGS["cfg0"], n_layers=2, batch=2, prompt_len=200, decode_steps=20, rho=1.035,
                             min_budget=8)
    _run_pair(wl, [20], max_budget=207)


def test_chained_steps_with_two_launch_classes():
    # two (layer, sequence) pairs go into a launch of their own; both launches of a step are chained
    wl = dataclasses.replace(W.twin("cfg3"), decode_steps=12)
    _run_pair(wl, [12], long_pairs=2)


def test_chained_steps_on_layer_ranges():
    """Layer ranges are stepped independently of one another: every range in one multi-step call of its own."""
    wl = dataclasses.replace(W.twin("cfg1"), decode_steps=10)
    (a, b), _, dq, dk, dv = _prepare(wl, 2)
    n = wl.decode_steps
    out_a, out_b = torch.empty_like(dq), torch.full_like(dq, float("nan"))
    for s in range(n):
        a.d2o_decode_step(0, wl.n_layers, dq[s], dk[s], dv[s], out_a[s])
    for l0, l1 in ((0, 1), (1, 4)):
        q, k, v = (t[:, l0:l1].contiguous() for t in (dq, dk, dv))
        o = torch.empty_like(q)
        b.d2o_decode_steps(l0, l1, n, q, k, v, o)
        out_b[:, l0:l1] = o
    torch.cuda.synchronize()
    assert b.d2o_get_stats().error_word == 0
    assert torch.equal(out_a.view(torch.uint8), out_b.view(torch.uint8))
    _same_state(a, b, _all_slices(wl))
    a.close(); b.close()


def test_chained_steps_argument_checks():
    wl = dataclasses.replace(W.CONFIGS["cfg0"], decode_steps=4)
    (c,), _, dq, dk, dv = _prepare(wl, 1)
    out = torch.empty_like(dq)
    with pytest.raises(B.D2OError):
        c.d2o_decode_steps(0, 1, 0, dq, dk, dv, out)
    with pytest.raises(B.D2OError):                       # more tokens than max_new_tokens leaves
        c.d2o_decode_steps(0, 1, 5, dq, dk, dv, out)
    c.d2o_decode_steps(0, 1, 4, dq, dk, dv, out)
    with pytest.raises(B.D2OError):
        c.d2o_decode_steps(0, 1, 1, dq, dk, dv, out)
    assert c.d2o_get_stats().error_word == 0
    c.close()


@pytest.mark.slow
def test_chained_steps_full_size_config_1():
    """All 32 layers of the 7B-shaped config (1024 slices), 48 tokens in one call."""
    wl = dataclasses.replace(W.CONFIGS["cfg1"], decode_steps=48)
    r = np.random.default_rng(5)
    picks = sorted({(int(r.integers(wl.n_layers)), 0, int(r.integers(wl.n_kv_heads))) for _ in range(48)})
    _run_pair(wl, [48], slices=picks)


@pytest.mark.parametrize("name,steps", [("cfg0", 16), ("cfg2", 9), ("cfg1", 1)])
def test_pipelined_host_steps_equal_device_steps(name, steps):
    """d2o_decode_steps_host (copies of neighbouring steps beside the kernels, two staging sets): same outputs and
    state as stepping with device tensors."""
    wl = W.CONFIGS["cfg0"] if name == "cfg0" else dataclasses.replace(W.twin(name), decode_steps=steps)
    wl = dataclasses.replace(wl, decode_steps=steps)
    (a, b), _, dq, dk, dv = _prepare(wl, 2)
    L = wl.n_layers
    out_a = torch.empty_like(dq)
    for s in range(steps):
        a.d2o_decode_step(0, L, dq[s], dk[s], dv[s], out_a[s])
    hq, hk, hv = dq.cpu().pin_memory(), dk.cpu().pin_memory(), dv.cpu().pin_memory()
    ho = torch.full_like(hq, float("nan")).pin_memory()
    b.d2o_decode_steps_host(0, L, steps, hq, hk, hv, ho)       # returns when the last copy back has completed
    assert torch.equal(out_a.cpu().view(torch.uint8), ho.view(torch.uint8))
    for c in (a, b):
        assert c.d2o_get_stats().error_word == 0
    _same_state(a, b, _all_slices(wl))
    a.close(); b.close()


def test_chained_outputs_against_the_oracle():
    """Config 0, every slice: the oracle steps beside the outputs of one multi-step call."""
    wl = W.CONFIGS["cfg0"]
    (c,), KV, dq, dk, dv = _prepare(wl, 1)
    out = torch.empty_like(dq)
    c.d2o_decode_steps(0, wl.n_layers, wl.decode_steps, dq, dk, dv, out)
    torch.cuda.synchronize()
    assert c.d2o_get_stats().error_word == 0
    orc = make_oracle(wl, c.cfg)
    streams = [W.LayerStream(wl, l, "cuda:0") for l in range(wl.n_layers)]
    for l in range(wl.n_layers):
        Q, K, _ = streams[l].prompt()
        orc.layer_stats(l, _lazy64(Q.cpu()), _lazy64(K.cpu()))
    orc.layer_budgets()
    assert np.array_equal(orc.budgets, c.tables()[0].numpy())
    for l in range(wl.n_layers):
        K, V = KV[l]
        orc.prefill_compress(l, _lazy64(K.cpu()), _lazy64(V.cpu()))
    G = wl.group
    worst = 0.0
    for s in range(wl.decode_steps):
        for l in range(wl.n_layers):
            ref = orc.decode_step(l, np64(dq[s, l]), np64(dk[s, l]), np64(dv[s, l]), s)
            got = np64(out[s, l])
            for (b, h), (o, _) in ref.items():
                worst = max(worst, close(got[b, h * G:(h + 1) * G], o, wl.dtype))
    assert worst <= 1.0, worst
    c.close()
