"""Parity at the full sizes of the benchmark configurations, on sampled slices.

The GPU runs the whole workload through the C ABI in the launch configuration bench.py times
(every layer, every sequence, all layers per decode call); the float64 oracle follows a seeded
sample of (layer, sequence, KV head) slices stage by stage: column sums and densities of their
query heads, the budget function on the GPU's full density array, prompt-stage compression, and
the decode steps.  The number of decode steps is bounded for the larger configs so that the
whole file stays within a few minutes; the prompt stage always runs at full length.
"""
import dataclasses

import numpy as np
import pytest

from paper_2406_13035_b200 import binding as B
from paper_2406_13035_b200 import workloads as W

from parity import assert_report, run_parity

pytestmark = [pytest.mark.gpu, pytest.mark.slow]


@pytest.fixture(scope="module", autouse=True)
def _lib(cuda_device):
    from paper_2406_13035_b200 import build
    build.build_library()
    B.load_library()


def sample_slices(wl, n, seed):
    r = np.random.default_rng(seed)
    out = set()
    while len(out) < n:
        out.add((int(r.integers(wl.n_layers)), int(r.integers(wl.batch)), int(r.integers(wl.n_kv_heads))))
    return sorted(out)


@pytest.mark.parametrize("name,n_slices,steps,batch", [
    ("cfg1", 8, 256, None),      # Llama-2-7B-shaped, all 256 decode steps
    ("cfg2", 6, 48, None),       # Llama-3-8B-shaped GQA, batch 16, prompt 8192
    ("cfg3", 2, 32, None),       # prompt 32768
    ("cfg4", 8, 64, 8),          # serving sweep, batch 8
    ("cfg4", 6, 48, 1),          # serving sweep, batch 1
    ("cfg4", 6, 24, 32),         # serving sweep, batch 32
])
def test_full_size_sampled_slices(name, n_slices, steps, batch):
    wl = W.CONFIGS[name]
    if batch is not None:
        wl = dataclasses.replace(wl, batch=batch)
    slices = sample_slices(wl, n_slices, seed=20240613 + len(name) + wl.prompt_len)
    rep = run_parity(wl, slices=slices, steps=steps)
    assert rep.checked_slices == n_slices and rep.steps == steps
    assert_report(rep, wl.dtype)
    assert rep.merges + rep.discards > 0
    print(name, "slices", slices, rep.max_err, rep.ties, "merges", rep.merges, "discards", rep.discards,
          "storage flips", rep.storage_flips)
