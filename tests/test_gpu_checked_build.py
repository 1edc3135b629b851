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
