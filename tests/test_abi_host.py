"""Host-side checks that need no GPU: the shared object loads, exports every symbol the header
declares, and rejects bad arguments with status codes before touching the device."""
import ctypes as C
import os
import re

import pytest

from paper_2406_13035_b200 import binding as B
from paper_2406_13035_b200 import build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build_library()
    return B.load_library()


def header_functions():
    text = open(os.path.join(ROOT, "include", "d2o.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(d2o_[a-z_0-9]+)\s*\(", text)))


def test_exports_match_header(lib):
    names = header_functions()
    assert "d2o_layer_budgets" in names and "d2o_prefill_compress" in names and "d2o_decode_step" in names
    for n in names:
        assert hasattr(lib, n), f"{n} declared in d2o.h but not exported"
    assert sorted(B.EXPORTS) == names


def good(**kw):
    base = dict(n_layers=4, batch=2, n_q_heads=8, n_kv_heads=2, d_head=128, dtype="bf16", prompt_len=512,
                max_new_tokens=16, rho=0.25)
    base.update(kw)
    return B.make_config(**base)


def test_workspace_size_and_validation(lib):
    sb, xb = B.d2o_workspace_size(good())
    assert sb > 0 and xb > 0 and sb % 256 == 0
    # K and V pools dominate: B * Hkv * round(rho*L*P) rows of d elements, twice
    rows = 2 * 2 * round(0.25 * 4 * 512)
    assert sb >= 2 * rows * 128 * 2
    sb2, _ = B.d2o_workspace_size(good(rho=0.5))
    assert sb2 > sb
    bad = [dict(n_q_heads=7), dict(d_head=96), dict(dtype="f32", d_head=32), dict(rho=0.0), dict(rho=float("nan")),
           dict(beta=1.5), dict(n_layers=0), dict(prompt_len=0), dict(min_budget=0), dict(min_budget=1, n_sink=4),
           dict(rho=2.0), dict(density_temp=0.0), dict(head_reduce=7), dict(n_q_heads=24, n_kv_heads=8),
           dict(max_budget=4096), dict(budget_rule=3), dict(sim_feature=2), dict(merge_policy=-1)]
    for kw in bad:
        with pytest.raises(B.D2OError) as ei:
            B.d2o_workspace_size(good(**kw))
        assert ei.value.status in (1, 2), kw
    a, b = C.c_size_t(), C.c_size_t()
    assert lib.d2o_workspace_size(None, C.byref(a), C.byref(b)) == 1
    assert lib.d2o_workspace_size(C.byref(good()), None, None) == 1


def test_null_and_misaligned_arguments(lib):
    cfg = good()
    h = C.c_void_p()
    assert lib.d2o_create(C.byref(cfg), None, 0, None, 0, None, C.byref(h)) == 1
    assert lib.d2o_create(C.byref(cfg), 256 + 8, 1 << 40, 512, 1 << 40, None, C.byref(h)) == 3    # misaligned
    assert lib.d2o_create(C.byref(cfg), 256, 16, 512, 16, None, C.byref(h)) == 3                  # too small
    assert lib.d2o_layer_stats(None, 0, None, None, None, None) == 1
    assert lib.d2o_layer_budgets(None, None, None) == 1
    assert lib.d2o_prefill_compress(None, 0, None, None, None) == 1
    assert lib.d2o_decode_step(None, 0, 1, None, None, None, None, None) == 1
    assert lib.d2o_full_decode_step(1, 96, 1, 1, 16, 0, 16, 16, 16, 16, 16, 16, None) == 2
    assert lib.d2o_full_decode_step(1, 128, 1, 1, 16, 16, 16, 16, 16, 16, 16, 16, None) == 1     # len >= capacity
    assert lib.d2o_full_decode_step(1, 128, 1, 1, 16, 0, 8, 16, 16, 16, 16, 16, None) == 1       # misaligned cache
    assert lib.d2o_budgets_from_density(None, 1, 1, 1, 1, 16, 0.5, 1, 0, 1.0, 0, 0, 1, 0, 3.0, None, None, None,
                                        None, None) == 1
    assert lib.d2o_status_string(0) == b"ok" and b"order" in lib.d2o_status_string(4)
    lib.d2o_destroy(None)


def test_missing_library_fails_loudly(monkeypatch, tmp_path):
    monkeypatch.setattr(B, "_lib", None)
    monkeypatch.setattr(B, "LIB_PATH", str(tmp_path / "nope.so"))
    with pytest.raises(B.D2OError):
        B.load_library()
