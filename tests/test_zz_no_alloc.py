"""The allocation-free entry point against the regular one.

Some users of the library cannot call cudaMalloc while it runs: an inference server whose memory
pool has taken the whole device, or a host application that passes tensors in but keeps its
allocator to itself.  d2o_layer_stats_static serves them with a scratch array that lives inside
the library image.  It runs the library's generic kernels: where d2o_layer_stats runs them too
(fp32 inputs, or a prompt length that is not a multiple of 4) the two must agree bit for bit, and
where d2o_layer_stats takes its tensor-core kernels they must agree within the parity tolerance;
in both cases also on a second call that finds the first call's leftovers in the scratch array.
The results are checked against the CPU oracle as well, and the free device memory must not move
across the call.
This file sorts last on purpose, so that a run which stops at the first failure has already
been through every other test.
"""
import dataclasses

import pytest
import torch

from paper_2406_13035_b200 import binding as B
from paper_2406_13035_b200 import workloads as W

from parity import make_ctx

pytestmark = pytest.mark.gpu


def _regular(wl, Q, K):
    ctx = make_ctx(wl)
    ctx.d2o_layer_stats(0, Q, K)
    cs = ctx.colsum(0).clone()
    F = ctx.density()[:, 0, :].clone()
    torch.cuda.synchronize()
    ctx.close()
    return cs, F


@pytest.mark.parametrize("name,P,same_kernels", [("cfg0", 300, True), ("cfg2", 777, True), ("cfg2", 512, False)])
def test_static_scratch_entry_matches_regular_entry(cuda_device, name, P, same_kernels):
    import numpy as np
    from oracle import d2o_oracle as O
    from paper_2406_13035_b200 import build
    build.build_library()
    B.load_library()
    base = dataclasses.replace(W.CONFIGS[name], n_layers=1, batch=2, prompt_len=P, decode_steps=1, window=8,
                               max_budget=0)
    for call in range(2):                               # the second call reuses the scratch of the first
        wl = dataclasses.replace(base, seed=base.seed + call)
        Q, K, _ = W.LayerStream(wl, 0, "cuda:0").prompt()
        ref_cs, ref_F = _regular(wl, Q, K)
        cs = torch.full((wl.batch, wl.n_q_heads, P), float("nan"), dtype=torch.float32, device=cuda_device)
        F = torch.full((wl.batch, wl.n_q_heads), float("nan"), dtype=torch.float64, device=cuda_device)
        torch.cuda.synchronize()
        free_before, _ = torch.cuda.mem_get_info()
        B.d2o_layer_stats_static(Q, K, cs, F)
        torch.cuda.synchronize()
        free_after, _ = torch.cuda.mem_get_info()
        assert free_after == free_before                 # nothing was allocated or freed on the device
        torch.testing.assert_close(cs, ref_cs, rtol=2e-4, atol=0)
        torch.testing.assert_close(F, ref_F, rtol=2e-4, atol=0)
        if same_kernels:                                 # same kernels in the same order: bit-identical
            assert torch.equal(cs, ref_cs) and torch.equal(F, ref_F)
        # against the oracle, on two heads of the second sequence
        Qc, Kc = Q.cpu().double().numpy(), K.cpu().double().numpy()
        for hq in (0, wl.n_q_heads - 1):
            s_ref = O.colsum_scores(Qc[1, hq], Kc[1, hq // wl.group])
            got = cs[1, hq].cpu().double().numpy()
            assert np.max(np.abs(got - s_ref) / np.maximum(np.abs(s_ref), 1e-6)) < 2e-4
            assert abs(float(F[1, hq]) - O.attention_density(s_ref)) <= 2e-4 * O.attention_density(s_ref)


def test_static_scratch_entry_rejects_oversize(cuda_device):
    B.load_library()
    P = B.STATIC_LSE_FLOATS // 8 + 1                    # 1 x 8 heads x P floats: one row too many
    Q = torch.zeros(1, 8, P, 64, dtype=torch.float16, device=cuda_device)
    K = torch.zeros(1, 8, P, 64, dtype=torch.float16, device=cuda_device)
    cs = torch.zeros(1, 8, P, dtype=torch.float32, device=cuda_device)
    F = torch.zeros(1, 8, dtype=torch.float64, device=cuda_device)
    with pytest.raises(B.D2OError) as e:
        B.d2o_layer_stats_static(Q, K, cs, F)
    assert e.value.status == 7
    # more (sequence, head) pairs than a grid has rows
    Q = torch.zeros(1, 65536, 4, 64, dtype=torch.float16, device=cuda_device)
    K = torch.zeros(1, 65536, 4, 64, dtype=torch.float16, device=cuda_device)
    cs = torch.zeros(1, 65536, 4, dtype=torch.float32, device=cuda_device)
    F = torch.zeros(1, 65536, dtype=torch.float64, device=cuda_device)
    with pytest.raises(B.D2OError) as e:
        B.d2o_layer_stats_static(Q, K, cs, F)
    assert e.value.status == 7
