"""ctypes binding of libd2o.so: same names as include/d2o.h, argument marshalling only.

PyTorch is used for device memory and streams; every step of the path runs in the library's
CUDA kernels.  There is no CPU fallback: if the shared object is missing or a call fails, an
exception is raised.
"""
from __future__ import annotations

import ctypes as C
import math
import os
from typing import Optional

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libd2o.so")

D2O_F32, D2O_F16, D2O_BF16 = 0, 1, 2
DTYPE_CODE = {"f32": D2O_F32, "f16": D2O_F16, "bf16": D2O_BF16,
              torch.float32: D2O_F32, torch.float16: D2O_F16, torch.bfloat16: D2O_BF16}
TORCH_DTYPE = {D2O_F32: torch.float32, D2O_F16: torch.float16, D2O_BF16: torch.bfloat16}

EXPORTS = [
    "d2o_status_string", "d2o_last_cuda_error", "d2o_workspace_size", "d2o_create", "d2o_destroy",
    "d2o_layer_stats", "d2o_layer_stats_layers", "d2o_layer_budgets", "d2o_budgets_from_density", "d2o_prefill_compress",
    "d2o_prefill_compress_layers", "d2o_decode_step", "d2o_decode_steps", "d2o_decode_step_host", "d2o_decode_steps_host", "d2o_full_decode_step", "d2o_get_view", "d2o_get_stats",
    "d2o_set_tuning", "d2o_layer_stats_static", "d2o_set_fault_injection", "d2o_set_prompt_lens",
]
STATIC_LSE_FLOATS = 1 << 20      # D2O_STATIC_LSE_FLOATS of include/d2o.h


class D2OConfig(C.Structure):
    _fields_ = [("n_layers", C.c_int32), ("batch", C.c_int32), ("n_q_heads", C.c_int32),
                ("n_kv_heads", C.c_int32), ("d_head", C.c_int32), ("dtype", C.c_int32),
                ("prompt_len", C.c_int32), ("max_new_tokens", C.c_int32), ("rho", C.c_float),
                ("n_sink", C.c_int32), ("window", C.c_int32), ("nm_ratio", C.c_float), ("beta", C.c_float),
                ("tau_override", C.c_float), ("density_temp", C.c_float), ("min_budget", C.c_int32),
                ("max_budget", C.c_int32), ("head_reduce", C.c_int32), ("budget_rule", C.c_int32),
                ("sim_feature", C.c_int32), ("merge_policy", C.c_int32)]


class D2OView(C.Structure):
    _fields_ = [("colsum", C.c_void_p), ("density", C.c_void_p), ("budgets", C.c_void_p),
                ("windows", C.c_void_p), ("row_off", C.c_void_p), ("k_cache", C.c_void_p),
                ("v_cache", C.c_void_p), ("pos", C.c_void_p), ("score", C.c_void_p), ("rnorm", C.c_void_p),
                ("len", C.c_void_p), ("tau", C.c_void_p), ("evict_idx", C.c_void_p), ("evict_mx", C.c_void_p),
                ("evict_nn", C.c_void_p), ("pool_rows", C.c_int64)]


class D2OStats(C.Structure):
    _fields_ = [("decode_steps", C.c_uint64), ("evictions", C.c_uint64), ("merges", C.c_uint64),
                ("discards", C.c_uint64), ("prefill_evicted", C.c_uint64), ("prefill_merged", C.c_uint64),
                ("error_word", C.c_uint32), ("error_detail", C.c_uint32), ("decode_launches", C.c_uint64),
                ("guess_misses", C.c_uint64)]


class D2OError(RuntimeError):
    def __init__(self, status: int, what: str):
        self.status = status
        super().__init__(what)


_lib = None


def use_library(path: str):
    """Selects the shared object the binding loads next (libd2o.so, or the checked build libd2o_checked.so)."""
    global _lib, LIB_PATH
    _lib, LIB_PATH = None, path


def load_library() -> C.CDLL:
    """Loads libd2o.so (built by paper_2406_13035_b200.build).  Raises if it is missing."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise D2OError(-1, f"{LIB_PATH} not found: run `python -m paper_2406_13035_b200.build` "
                           "(there is no CPU fallback)")
    lib = C.CDLL(LIB_PATH)
    vp, i32, f32 = C.c_void_p, C.c_int32, C.c_float
    lib.d2o_status_string.restype = C.c_char_p
    lib.d2o_status_string.argtypes = [C.c_int]
    lib.d2o_last_cuda_error.restype = C.c_char_p
    lib.d2o_workspace_size.argtypes = [C.POINTER(D2OConfig), C.POINTER(C.c_size_t), C.POINTER(C.c_size_t)]
    lib.d2o_create.argtypes = [C.POINTER(D2OConfig), vp, C.c_size_t, vp, C.c_size_t, vp, C.POINTER(vp)]
    lib.d2o_destroy.argtypes = [vp]
    lib.d2o_destroy.restype = None
    lib.d2o_layer_stats.argtypes = [vp, i32, vp, vp, vp, vp]
    lib.d2o_layer_stats_layers.argtypes = [vp, i32, i32, C.POINTER(vp), C.POINTER(vp), C.POINTER(vp), vp]
    lib.d2o_layer_budgets.argtypes = [vp, vp, vp]
    lib.d2o_budgets_from_density.argtypes = [vp, i32, i32, i32, i32, i32, f32, i32, i32, f32, i32, i32, i32, i32, f32,
                                             vp, vp, vp, vp, vp]
    lib.d2o_prefill_compress.argtypes = [vp, i32, vp, vp, vp]
    lib.d2o_prefill_compress_layers.argtypes = [vp, i32, i32, C.POINTER(vp), C.POINTER(vp), vp]
    lib.d2o_decode_step.argtypes = [vp, i32, i32, vp, vp, vp, vp, vp]
    lib.d2o_decode_step_host.argtypes = [vp, i32, i32, vp, vp, vp, vp, vp]
    lib.d2o_decode_steps.argtypes = [vp, i32, i32, i32, vp, vp, vp, vp, vp]
    lib.d2o_decode_steps_host.argtypes = [vp, i32, i32, i32, vp, vp, vp, vp, vp]
    lib.d2o_full_decode_step.argtypes = [i32, i32, i32, i32, i32, i32, vp, vp, vp, vp, vp, vp, vp]
    lib.d2o_get_view.argtypes = [vp, i32, C.POINTER(D2OView)]
    lib.d2o_get_stats.argtypes = [vp, C.POINTER(D2OStats), vp]
    lib.d2o_set_tuning.argtypes = [vp, i32, i32, i32, i32, i32, i32, i32]
    lib.d2o_layer_stats_static.argtypes = [i32, i32, i32, i32, i32, i32, vp, vp, vp, vp, vp]
    lib.d2o_set_fault_injection.argtypes = [vp, i32, i32]
    lib.d2o_set_prompt_lens.argtypes = [vp, vp, vp]
    for name in EXPORTS:
        if name not in ("d2o_status_string", "d2o_last_cuda_error", "d2o_destroy"):
            getattr(lib, name).restype = C.c_int
    _lib = lib
    return lib


def _check(status: int, what: str):
    if status != 0:
        lib = load_library()
        msg = lib.d2o_status_string(status).decode()
        if status == 5:
            msg += ": " + lib.d2o_last_cuda_error().decode()
        raise D2OError(status, f"{what}: {msg}")


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    if t is None:
        return None
    assert t.is_contiguous(), "tensors must be contiguous"
    return t.data_ptr()


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def f32(x: float) -> float:
    """The value a C float argument will hold (so that a float64 checker can use the same number)."""
    return float(torch.tensor(x, dtype=torch.float32).item())


def make_config(*, n_layers, batch, n_q_heads, n_kv_heads, d_head, dtype, prompt_len, max_new_tokens, rho,
                n_sink=1, window=0, nm_ratio=3.0, beta=0.7, tau_override=float("nan"), density_temp=1.0,
                min_budget=8, max_budget=0, head_reduce=0, budget_rule=0, sim_feature=0, merge_policy=0) -> D2OConfig:
    return D2OConfig(n_layers, batch, n_q_heads, n_kv_heads, d_head, DTYPE_CODE[dtype], prompt_len, max_new_tokens,
                     rho, n_sink, window, nm_ratio, beta, tau_override, density_temp, min_budget, max_budget,
                     head_reduce, budget_rule, sim_feature, merge_policy)


def d2o_workspace_size(cfg: D2OConfig):
    a, b = C.c_size_t(), C.c_size_t()
    _check(load_library().d2o_workspace_size(C.byref(cfg), C.byref(a), C.byref(b)), "d2o_workspace_size")
    return a.value, b.value


class D2OContext:
    """Owns the device buffers (torch) and the d2o_ctx handle; methods mirror the C entry points."""

    def __init__(self, cfg: D2OConfig, device="cuda:0"):
        self.lib = load_library()
        self.cfg = cfg
        self.device = torch.device(device)
        sb, xb = d2o_workspace_size(cfg)
        self.state = torch.empty(sb + 256, dtype=torch.uint8, device=self.device)
        self.scratch = torch.empty(xb + 256, dtype=torch.uint8, device=self.device)
        sp = (self.state.data_ptr() + 255) // 256 * 256
        xp = (self.scratch.data_ptr() + 255) // 256 * 256
        self._state_off = sp - self.state.data_ptr()
        self._scratch_off = xp - self.scratch.data_ptr()
        h = C.c_void_p()
        with torch.cuda.device(self.device):
            _check(self.lib.d2o_create(C.byref(cfg), sp, sb, xp, xb, _stream(), C.byref(h)), "d2o_create")
        self.handle = h
        self.tdtype = TORCH_DTYPE[cfg.dtype]
        self.budgets_host = None

    def close(self):
        if self.handle:
            self.lib.d2o_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # ---- the path
    def d2o_set_prompt_lens(self, lens):
        t = torch.as_tensor(lens, dtype=torch.int32).contiguous()
        assert t.numel() == self.cfg.batch and t.device.type == "cpu"
        _check(self.lib.d2o_set_prompt_lens(self.handle, t.data_ptr(), _stream()), "d2o_set_prompt_lens")

    def d2o_layer_stats(self, layer: int, Q: torch.Tensor, K: torch.Tensor, lse: Optional[torch.Tensor] = None):
        _check(self.lib.d2o_layer_stats(self.handle, layer, _ptr(Q), _ptr(K), _ptr(lse), _stream()), "d2o_layer_stats")

    def d2o_layer_stats_layers(self, l0: int, l1: int, Qs, Ks, lses=None):
        """`Qs`, `Ks` (and `lses`, entries may be None): one device tensor per layer of [l0, l1)."""
        n = l1 - l0
        assert len(Qs) == n and len(Ks) == n and (lses is None or len(lses) == n)
        qa = (C.c_void_p * n)(*[_ptr(t) for t in Qs])
        ka = (C.c_void_p * n)(*[_ptr(t) for t in Ks])
        la = None if lses is None else (C.c_void_p * n)(*[_ptr(t) for t in lses])
        _check(self.lib.d2o_layer_stats_layers(self.handle, l0, l1, qa, ka, la, _stream()), "d2o_layer_stats_layers")

    def d2o_layer_budgets(self) -> torch.Tensor:
        out = torch.empty(self.cfg.batch, self.cfg.n_layers, self.cfg.n_kv_heads, dtype=torch.int32)
        _check(self.lib.d2o_layer_budgets(self.handle, out.data_ptr(), _stream()), "d2o_layer_budgets")
        self.budgets_host = out
        return out

    def d2o_prefill_compress(self, layer: int, K: torch.Tensor, V: torch.Tensor):
        _check(self.lib.d2o_prefill_compress(self.handle, layer, _ptr(K), _ptr(V), _stream()), "d2o_prefill_compress")

    def d2o_prefill_compress_layers(self, l0: int, l1: int, Ks, Vs):
        """`Ks`, `Vs`: one device tensor per layer of [l0, l1)."""
        n = l1 - l0
        assert len(Ks) == n and len(Vs) == n
        ka = (C.c_void_p * n)(*[_ptr(t) for t in Ks])
        va = (C.c_void_p * n)(*[_ptr(t) for t in Vs])
        _check(self.lib.d2o_prefill_compress_layers(self.handle, l0, l1, ka, va, _stream()),
               "d2o_prefill_compress_layers")

    def d2o_decode_step(self, l0: int, l1: int, q, k, v, out):
        _check(self.lib.d2o_decode_step(self.handle, l0, l1, _ptr(q), _ptr(k), _ptr(v), _ptr(out), _stream()),
               "d2o_decode_step")

    def d2o_decode_steps(self, l0: int, l1: int, n_steps: int, q, k, v, out):
        _check(self.lib.d2o_decode_steps(self.handle, l0, l1, n_steps, _ptr(q), _ptr(k), _ptr(v), _ptr(out), _stream()),
               "d2o_decode_steps")

    def d2o_decode_step_host(self, l0: int, l1: int, q, k, v, out):
        for t in (q, k, v, out):
            assert t.device.type == "cpu"
        _check(self.lib.d2o_decode_step_host(self.handle, l0, l1, _ptr(q), _ptr(k), _ptr(v), _ptr(out), _stream()),
               "d2o_decode_step_host")

    def d2o_decode_steps_host(self, l0: int, l1: int, n_steps: int, q, k, v, out):
        for t in (q, k, v, out):
            assert t.device.type == "cpu"
        _check(self.lib.d2o_decode_steps_host(self.handle, l0, l1, n_steps, _ptr(q), _ptr(k), _ptr(v), _ptr(out),
                                              _stream()), "d2o_decode_steps_host")

    def d2o_set_tuning(self, decode_stages: int = 0, decode_l2_hints: int = 1, similarity_path: int = 0,
                       stats_path: int = 0, decode_warps: int = 0, decode_smem_rows: int = 0,
                       decode_long_pairs: int = 0):
        _check(self.lib.d2o_set_tuning(self.handle, decode_stages, decode_l2_hints, similarity_path, stats_path,
                                       decode_warps, decode_smem_rows, decode_long_pairs), "d2o_set_tuning")

    def d2o_set_fault_injection(self, wait_limit_us: int = 0, producer_stop_stage: int = -1):
        _check(self.lib.d2o_set_fault_injection(self.handle, wait_limit_us, producer_stop_stage),
               "d2o_set_fault_injection")

    def d2o_get_stats(self) -> D2OStats:
        s = D2OStats()
        _check(self.lib.d2o_get_stats(self.handle, C.byref(s), _stream()), "d2o_get_stats")
        return s

    # ---- inspection (device views as torch tensors; no copies)
    def _view(self, layer: int) -> D2OView:
        v = D2OView()
        _check(self.lib.d2o_get_view(self.handle, layer, C.byref(v)), "d2o_get_view")
        return v

    def _wrap(self, ptr: int, nbytes: int, dtype, shape):
        base = self.state.data_ptr()
        if base <= ptr < base + self.state.numel():
            buf = self.state
        else:
            buf, base = self.scratch, self.scratch.data_ptr()
        off = ptr - base
        return buf[off:off + nbytes].view(dtype).view(*shape)

    def colsum(self, layer: int) -> torch.Tensor:
        c = self.cfg
        v = self._view(layer)
        return self._wrap(v.colsum, c.batch * c.n_q_heads * c.prompt_len * 4, torch.float32,
                          (c.batch, c.n_q_heads, c.prompt_len))

    def density(self) -> torch.Tensor:
        c = self.cfg
        v = self._view(0)
        return self._wrap(v.density, c.batch * c.n_layers * c.n_q_heads * 8, torch.float64,
                          (c.batch, c.n_layers, c.n_q_heads))

    def tables(self):
        """(budgets, windows, row_off), each [B, L, Hkv], as host tensors."""
        c = self.cfg
        v = self._view(0)
        shape = (c.batch, c.n_layers, c.n_kv_heads)
        n = c.batch * c.n_layers * c.n_kv_heads
        b = self._wrap(v.budgets, n * 4, torch.int32, shape).cpu()
        w = self._wrap(v.windows, n * 4, torch.int32, shape).cpu()
        o = self._wrap(v.row_off, n * 8, torch.int64, shape).cpu()
        return b, w, o

    def slice_state(self, layer: int, b: int, h: int, tables=None):
        """Host copy of one slice's cache: dict(pos, score, rnorm, K, V, len, tau)."""
        c = self.cfg
        v = self._view(layer)
        bud, win, off = tables if tables is not None else self.tables()
        S = int(bud[b, layer, h])
        r0 = int(off[b, layer, h])
        esz = 4 if c.dtype == D2O_F32 else 2
        rows = v.pool_rows
        sidx = (layer * c.batch + b) * c.n_kv_heads + h
        nsl = c.n_layers * c.batch * c.n_kv_heads
        ln = int(self._wrap(v.len, nsl * 4, torch.int32, (nsl,))[sidx].item())
        tau = float(self._wrap(v.tau, nsl * 4, torch.float32, (nsl,))[sidx].item())
        pos = self._wrap(v.pos, rows * 4, torch.int32, (rows,))[r0:r0 + ln].cpu()
        score = self._wrap(v.score, rows * 4, torch.float32, (rows,))[r0:r0 + ln].cpu()
        rnorm = self._wrap(v.rnorm, rows * 4, torch.float32, (rows,))[r0:r0 + ln].cpu()
        K = self._wrap(v.k_cache, rows * c.d_head * esz, self.tdtype, (rows, c.d_head))[r0:r0 + ln].cpu()
        V = self._wrap(v.v_cache, rows * c.d_head * esz, self.tdtype, (rows, c.d_head))[r0:r0 + ln].cpu()
        return dict(pos=pos, score=score, rnorm=rnorm, K=K, V=V, len=ln, tau=tau, S=S, M=int(win[b, layer, h]))

    def evict_lists(self, b: int, h: int, Le: int):
        """Scratch of the layer compressed last: evicted positions, Max(U[i,:]) and Argmax slot."""
        c = self.cfg
        v = self._view(0)
        n = c.batch * c.n_kv_heads * c.prompt_len
        sl = b * c.n_kv_heads + h
        idx = self._wrap(v.evict_idx, n * 4, torch.int32, (c.batch * c.n_kv_heads, c.prompt_len))[sl, :Le].cpu()
        mx = self._wrap(v.evict_mx, n * 4, torch.float32, (c.batch * c.n_kv_heads, c.prompt_len))[sl, :Le].cpu()
        nn = self._wrap(v.evict_nn, n * 4, torch.int32, (c.batch * c.n_kv_heads, c.prompt_len))[sl, :Le].cpu()
        return idx, mx, nn


def d2o_budgets_from_density(density: torch.Tensor, *, n_kv_heads: int, prompt_len: int, rho: float,
                             min_budget: int, max_budget: int = 0, density_temp: float = 1.0, head_reduce: int = 0,
                             budget_rule: int = 0, n_sink: int = 1, window: int = 0, nm_ratio: float = 3.0):
    """density: CUDA float64 [B, L, H] -> (budgets, windows, row_off) CUDA tensors [B, L, Hkv]."""
    lib = load_library()
    B, L, H = density.shape
    dev = density.device
    budgets = torch.zeros(B, L, n_kv_heads, dtype=torch.int32, device=dev)
    windows = torch.zeros(B, L, n_kv_heads, dtype=torch.int32, device=dev)
    row_off = torch.zeros(B, L, n_kv_heads, dtype=torch.int64, device=dev)
    status = torch.zeros(4, dtype=torch.int32, device=dev)
    _check(lib.d2o_budgets_from_density(_ptr(density), B, L, H, n_kv_heads, prompt_len, rho, min_budget, max_budget,
                                        density_temp, head_reduce, budget_rule, n_sink, window, nm_ratio, _ptr(budgets),
                                        _ptr(windows), _ptr(row_off), _ptr(status), _stream()),
           "d2o_budgets_from_density")
    return budgets, windows, row_off, status


def d2o_full_decode_step(k_cache: torch.Tensor, v_cache: torch.Tensor, length: int, q: torch.Tensor,
                         k: torch.Tensor, v: torch.Tensor, out: torch.Tensor):
    """k_cache/v_cache [n_slices, capacity, d]; q/out [n_slices, G, d]; k/v [n_slices, d]."""
    lib = load_library()
    n_slices, capacity, d = k_cache.shape
    G = q.shape[1]
    _check(lib.d2o_full_decode_step(DTYPE_CODE[k_cache.dtype], d, n_slices, G, capacity, length, _ptr(k_cache),
                                    _ptr(v_cache), _ptr(q), _ptr(k), _ptr(v), _ptr(out), _stream()),
           "d2o_full_decode_step")


def d2o_layer_stats_static(Q: torch.Tensor, K: torch.Tensor, colsum: torch.Tensor, density: torch.Tensor):
    """Allocation-free column sums and densities of one layer's prompt attention.

    For callers that must not allocate device memory while the library works (a serving process
    whose pool owns the whole GPU, a plugin without an allocator): the library's only scratch is
    a fixed 4 MiB array inside its own image.  The caller provides every tensor, outputs included:
    Q [B, Hq, P, d], K [B, Hkv, P, d], colsum float32 [B, Hq, P], density float64 [B, Hq].
    Raises D2OError (status 7) if B * Hq * P exceeds STATIC_LSE_FLOATS.  Calls that overlap on the
    GPU share the scratch array and race; make the first call on a device outside stream capture."""
    lib = load_library()
    B, Hq, P, d = Q.shape
    Hkv = K.shape[1]
    assert colsum.dtype == torch.float32 and tuple(colsum.shape) == (B, Hq, P)
    assert density.dtype == torch.float64 and tuple(density.shape) == (B, Hq)
    _check(lib.d2o_layer_stats_static(DTYPE_CODE[Q.dtype], d, B, Hq, Hkv, P, _ptr(Q), _ptr(K), _ptr(colsum),
                                      _ptr(density), _stream()), "d2o_layer_stats_static")
