"""Failure detection: a device-side wait that runs out is reported, nothing hangs, nothing traps.

The decode kernel waits for stages of cache rows that its copy engine delivers.  The test knob
d2o_set_fault_injection makes one stage never arrive and shortens the wait limit to two
milliseconds: the kernel must come back on its own, leave the slice untouched, and report
D2O_ERR_TIMEOUT through d2o_get_stats; later steps on the same context do nothing; the CUDA context
stays usable for a fresh library context.
"""
import dataclasses
import time

import pytest
import torch

from paper_2406_13035_b200 import binding as B
from paper_2406_13035_b200 import workloads as W

from parity import assert_report, make_ctx, run_parity

pytestmark = pytest.mark.gpu

D2O_ERR_TIMEOUT = 6


def _state(ctx, wl):
    tabs = ctx.tables()
    return [ctx.slice_state(0, 0, h, tabs) for h in range(wl.n_kv_heads)]


def _same(a, b):
    return all(x["len"] == y["len"] and x["tau"] == y["tau"] and torch.equal(x["pos"], y["pos"]) and
               torch.equal(x["score"], y["score"]) and torch.equal(x["K"], y["K"]) and torch.equal(x["V"], y["V"])
               for x, y in zip(a, b))


@pytest.mark.parametrize("name", ["cfg0", "cfg2"])
def test_decode_wait_that_runs_out_is_reported(cuda_device, name):
    from paper_2406_13035_b200 import build
    build.build_library()
    B.load_library()
    base = W.CONFIGS["cfg0"] if name == "cfg0" else W.twin("cfg2")
    # caches of ~200 rows: several stages per pass, so that stage 1 belongs to the key pass
    wl = dataclasses.replace(base, prompt_len=512, decode_steps=4, n_layers=1, batch=1, max_budget=0, rho=0.4)
    ctx = make_ctx(wl)
    s = W.LayerStream(wl, 0, "cuda:0")
    Q, K, V = s.prompt()
    ctx.d2o_layer_stats(0, Q, K)
    ctx.d2o_layer_budgets()
    ctx.d2o_prefill_compress(0, K, V)
    q, k, v = s.decode()
    out = torch.zeros_like(q)
    ctx.d2o_decode_step(0, 1, q, k, v, out)                      # an ordinary step first
    torch.cuda.synchronize()
    assert ctx.d2o_get_stats().error_word == 0
    before = _state(ctx, wl)
    # stage 1 of every slice never arrives; a wait gives up after 2 ms
    ctx.d2o_set_fault_injection(wait_limit_us=2000, producer_stop_stage=1)
    q, k, v = s.decode()
    t0 = time.perf_counter()
    ctx.d2o_decode_step(0, 1, q, k, v, out)
    torch.cuda.synchronize()
    dt = time.perf_counter() - t0
    st = ctx.d2o_get_stats()
    assert st.error_word == D2O_ERR_TIMEOUT, (st.error_word, hex(st.error_detail))
    assert dt < 2.0, f"the step took {dt:.3f} s"
    assert _same(before, _state(ctx, wl))                        # the wait ran out in the key pass: nothing was written
    # later steps on this context do nothing and return at once, with or without the knob
    ctx.d2o_set_fault_injection(0, -1)
    q, k, v = s.decode()
    t0 = time.perf_counter()
    ctx.d2o_decode_step(0, 1, q, k, v, out)
    torch.cuda.synchronize()
    assert time.perf_counter() - t0 < 0.5
    assert ctx.d2o_get_stats().error_word == D2O_ERR_TIMEOUT
    assert _same(before, _state(ctx, wl))
    ctx.close()
    # the CUDA context is intact: a fresh library context passes an ordinary parity run
    small = dataclasses.replace(W.CONFIGS["cfg0"], prompt_len=128, decode_steps=2)
    rep = run_parity(small)
    assert_report(rep, small.dtype)
