"""Seeded synthetic attention tensors for the D2O hot path.

This module only *draws inputs*.  It contains none of the method's arithmetic
(no softmax, no scores, no selection, no similarity, no merging) and imports
neither the CUDA binding nor the CPU oracle, so both sides can be fed from it.

The tensors stand in for the Llama-2-7B / Llama-3-8B / Mistral-7B long-context
attention workloads the paper evaluates on (Section 5.1): same head counts, head
dimension, dtype, prompt length and cache ratio, with a structure that produces
the attention patterns the method relies on (one attention sink, a few "heavy"
tokens that attract most queries, low-rank clustered keys so that evicted keys
have near neighbours among the retained ones).

Recipe, per (layer, batch element, KV head):
  * mean query direction ``m`` ~ N(0, I_d), scaled to ``|m| = 0.5 * sqrt(d)``;
  * keys ``k_j = W z_j + 0.3 * eps_j`` with ``W`` a ``d x r`` Gaussian / sqrt(r),
    ``z_j ~ N(0, I_r)``, ``eps_j ~ N(0, I_d)``;
  * position 0 is the sink: ``k_0 = 4 * rms|k| * m / |m|``;
  * a seeded fraction of positions is "heavy":
    ``k_j <- |k_j| * normalize(m/|m| + 0.5 * k_j/|k_j|)``;
  * queries follow an AR(1) process around the mean query,
    ``q_i = m_g + eta_i``, ``eta_i = 0.9 eta_{i-1} + sqrt(1 - 0.81) xi_i``;
    the ``G`` query heads of a group use ``m_g = m + N(0, 0.1^2)``;
    every query of layer ``l`` is divided by the layer temperature ``temp_l``;
  * values ``v_j ~ N(0, I_d)``;
  * decode-time ``q`` continues the AR(1) process and decode-time ``k, v`` are
    drawn from the same key / value recipe.
Everything is produced in float32 and rounded once to the storage dtype.
"""
from __future__ import annotations

import dataclasses
import math
from typing import Dict, Optional, Tuple

import torch

TORCH_DTYPES = {"f32": torch.float32, "f16": torch.float16, "bf16": torch.bfloat16}


@dataclasses.dataclass(frozen=True)
class Workload:
    """Shape, hyper-parameters and generator settings of one benchmark config."""

    name: str
    batch: int
    n_layers: int
    n_q_heads: int
    n_kv_heads: int
    d_head: int
    dtype: str            # "f32" | "f16" | "bf16"
    prompt_len: int
    decode_steps: int
    rho: float            # global cache ratio
    n_sink: int = 1       # T
    window: int = 0       # M; 0 -> derived per layer from nm_ratio
    nm_ratio: float = 3.0
    beta: float = 0.7
    density_temp: float = 1.0
    min_budget: int = 8
    max_budget: int = 0       # upper clamp of S_l; 0 = prompt length
    rank: int = 8
    heavy_frac: float = 0.05
    temp_first: float = 1.0   # softmax temperature of layer 0
    temp_last: float = 1.0    # softmax temperature of the last layer
    seed: int = 2406130

    @property
    def group(self) -> int:
        return self.n_q_heads // self.n_kv_heads

    def layer_temp(self, layer: int) -> float:
        if self.n_layers == 1:
            return self.temp_first
        f = layer / (self.n_layers - 1)
        return self.temp_first + (self.temp_last - self.temp_first) * f

    def scaled(self, *, n_layers: int, prompt_div: int, batch: int, steps: int,
               name: Optional[str] = None) -> "Workload":
        """A small twin: same heads / GQA / dtype / ratio / window rule."""
        window = self.window
        if window > 0:
            window = max(4, window // prompt_div)
        return dataclasses.replace(
            self, name=name or (self.name + "_twin"), n_layers=n_layers,
            prompt_len=self.prompt_len // prompt_div, batch=min(self.batch, batch),
            decode_steps=steps, window=window, max_budget=self.max_budget // prompt_div)


# The five configurations named by the benchmark definition.  ``density_temp``
# (gamma in exp(-F/gamma)) is 1 for the single-layer config.  For the stacks it is set
# from the spread of the densities this generator produces: the sink token collects most
# of every row, so F is close to P - 1 in every layer and differs between the first and the
# last layer by about 5 (P = 4096), 13 (P = 8192), 170 (P = 32768) and 1.4 (P = 2048);
# gamma of that order gives budgets that differ by a factor of three to five.
CONFIGS: Dict[str, Workload] = {
    "cfg0": Workload("cfg0", batch=1, n_layers=1, n_q_heads=8, n_kv_heads=8, d_head=64,
                     dtype="f32", prompt_len=1024, decode_steps=16, rho=0.25, window=32,
                     beta=0.9, rank=8, heavy_frac=0.05, seed=2406130),
    "cfg1": Workload("cfg1", batch=1, n_layers=32, n_q_heads=32, n_kv_heads=32, d_head=128,
                     dtype="f16", prompt_len=4096, decode_steps=256, rho=0.20,
                     beta=0.7, rank=8, heavy_frac=0.05, temp_first=1.0, temp_last=0.25,
                     density_temp=8.0, max_budget=2048, seed=2406131),
    "cfg2": Workload("cfg2", batch=16, n_layers=32, n_q_heads=32, n_kv_heads=8, d_head=128,
                     dtype="bf16", prompt_len=8192, decode_steps=512, rho=0.10, window=64,
                     beta=0.7, rank=16, heavy_frac=0.02, temp_first=1.0, temp_last=0.25,
                     density_temp=10.0, max_budget=4096, seed=2406132),
    "cfg3": Workload("cfg3", batch=4, n_layers=32, n_q_heads=32, n_kv_heads=8, d_head=128,
                     dtype="bf16", prompt_len=32768, decode_steps=256, rho=0.05,
                     beta=0.7, rank=8, heavy_frac=0.05, temp_first=1.0, temp_last=0.25,
                     density_temp=120.0, max_budget=6144, seed=2406133),
    "cfg4": Workload("cfg4", batch=8, n_layers=32, n_q_heads=32, n_kv_heads=32, d_head=128,
                     dtype="f16", prompt_len=2048, decode_steps=1024, rho=0.20,
                     beta=0.7, rank=8, heavy_frac=0.05, temp_first=1.0, temp_last=0.25,
                     density_temp=3.0, max_budget=1024, seed=2406134),
}


# Not one of the five benchmark configurations: the steady state of the paper's multi-turn (streaming) setting,
# appendix "Generated Samples of Multi-turn Conversations": every layer holds a fixed budget of 2048 tokens, of which
# N = 48 are important tokens and M = 2000 the recent window (no sinks: 48 + 2000 = 2048).  The "prompt" is the 2048
# tokens the conversation has accumulated, so nothing is evicted at the prompt stage and every generated token
# evicts one.  Llama-2-7B-shaped heads, four sessions.
CONFIGS["session"] = Workload("session", batch=4, n_layers=32, n_q_heads=32, n_kv_heads=32, d_head=128,
                              dtype="f16", prompt_len=2048, decode_steps=256, rho=1.0, n_sink=0, window=2000,
                              beta=0.7, rank=8, heavy_frac=0.05, temp_first=1.0, temp_last=0.25,
                              density_temp=1e30, min_budget=2048, max_budget=2048, seed=2406135)


def twin(name: str) -> Workload:
    """Scaled twin used by the whole-pipeline parity tests (4 layers, P/8, B<=2)."""
    return CONFIGS[name].scaled(n_layers=4, prompt_div=8, batch=2, steps=16)


def _gen(seed: int, *keys: int, device: str = "cpu") -> torch.Generator:
    g = torch.Generator(device=device)
    s = seed
    for k in keys:
        s = (s * 1000003 + 7919 * (k + 1)) % (2 ** 62)
    g.manual_seed(s)
    return g


def _ar1(noise: torch.Tensor, eta0: torch.Tensor, coef: float = 0.9) -> Tuple[torch.Tensor, torch.Tensor]:
    """AR(1) filter along dim -2: eta_i = coef*eta_{i-1} + sqrt(1-coef^2)*noise_i.

    Evaluated block by block with a lower-triangular Toeplitz matrix so that long
    prompts need no per-position Python loop.  Returns (eta, last eta)."""
    n = noise.shape[-2]
    blk = 64
    c = math.sqrt(1.0 - coef * coef)
    idx = torch.arange(blk, device=noise.device)
    diff = (idx[:, None] - idx[None, :]).clamp(min=0).to(torch.float32)
    tri = (idx[:, None] >= idx[None, :]).to(torch.float32)
    A = tri * torch.pow(torch.tensor(coef, device=noise.device), diff) * c      # [blk, blk]
    carry = torch.pow(torch.tensor(coef, device=noise.device), (idx + 1).to(torch.float32))  # [blk]
    out = torch.empty_like(noise)
    prev = eta0
    for s in range(0, n, blk):
        e = min(s + blk, n)
        m = e - s
        seg = torch.matmul(A[:m, :m], noise[..., s:e, :]) + carry[:m, None] * prev[..., None, :]
        out[..., s:e, :] = seg
        prev = seg[..., m - 1, :]
    return out, prev


class LayerStream:
    """Generator state of one layer: prompt tensors, then one (q, k, v) per decode step.

    All tensors are created on ``device`` from a ``torch.Generator`` seeded by
    (workload seed, layer, purpose), so a given (workload, layer, device type)
    always yields the same values."""

    def __init__(self, wl: Workload, layer: int, device: str = "cpu"):
        self.wl, self.layer, self.device = wl, layer, device
        B, Hkv, G, d, r = wl.batch, wl.n_kv_heads, wl.group, wl.d_head, wl.rank
        g = _gen(wl.seed, layer, 0, device=device)
        m = torch.randn(B, Hkv, d, generator=g, device=device)
        m = m * (0.5 * math.sqrt(d) / m.norm(dim=-1, keepdim=True))
        self.m_hat = m / m.norm(dim=-1, keepdim=True)                      # [B,Hkv,d]
        self.W = torch.randn(B, Hkv, d, r, generator=g, device=device) / math.sqrt(r)
        mg = m[:, :, None, :] + 0.1 * torch.randn(B, Hkv, G, d, generator=g, device=device)
        self.m_q = mg.reshape(B, Hkv * G, d)                               # [B,Hq,d]
        self.eta = torch.zeros(B, Hkv * G, d, device=device)
        self.temp = wl.layer_temp(layer)
        self.tdtype = TORCH_DTYPES[wl.dtype]
        self._step = 0

    def _keys(self, n: int, g: torch.Generator) -> torch.Tensor:
        wl = self.wl
        B, Hkv, d, r = wl.batch, wl.n_kv_heads, wl.d_head, wl.rank
        z = torch.randn(B, Hkv, n, r, generator=g, device=self.device)
        eps = torch.randn(B, Hkv, n, d, generator=g, device=self.device)
        k = torch.matmul(z, self.W.transpose(-1, -2)) + 0.3 * eps          # [B,Hkv,n,d]
        heavy = torch.rand(B, Hkv, n, generator=g, device=self.device) < wl.heavy_frac
        kn = k.norm(dim=-1, keepdim=True)
        hv = self.m_hat[:, :, None, :] + 0.5 * k / kn
        hv = kn * hv / hv.norm(dim=-1, keepdim=True)
        return torch.where(heavy[..., None], hv, k)

    def prompt(self) -> Tuple[torch.Tensor, torch.Tensor, torch.Tensor]:
        """Q [B,Hq,P,d], K [B,Hkv,P,d], V [B,Hkv,P,d] in the storage dtype."""
        wl = self.wl
        B, Hq, Hkv, d, P = wl.batch, wl.n_q_heads, wl.n_kv_heads, wl.d_head, wl.prompt_len
        g = _gen(wl.seed, self.layer, 1, device=self.device)
        k = self._keys(P, g)
        rms = k.norm(dim=-1).pow(2).mean(dim=-1).sqrt()                    # [B,Hkv]
        k[:, :, 0, :] = 4.0 * rms[..., None] * self.m_hat
        v = torch.randn(B, Hkv, P, d, generator=g, device=self.device)
        xi = torch.randn(B, Hq, P, d, generator=g, device=self.device)
        eta, self.eta = _ar1(xi, self.eta)
        q = (self.m_q[:, :, None, :] + eta) / self.temp
        return q.to(self.tdtype), k.to(self.tdtype), v.to(self.tdtype)

    def decode(self) -> Tuple[torch.Tensor, torch.Tensor, torch.Tensor]:
        """Next token: q [B,Hq,d], k [B,Hkv,d], v [B,Hkv,d] in the storage dtype."""
        wl = self.wl
        B, Hq, Hkv, d = wl.batch, wl.n_q_heads, wl.n_kv_heads, wl.d_head
        g = _gen(wl.seed, self.layer, 2, self._step, device=self.device)
        self._step += 1
        k = self._keys(1, g)[:, :, 0, :]
        v = torch.randn(B, Hkv, d, generator=g, device=self.device)
        xi = torch.randn(B, Hq, d, generator=g, device=self.device)
        self.eta = 0.9 * self.eta + math.sqrt(1.0 - 0.81) * xi
        q = (self.m_q + self.eta) / self.temp
        return q.to(self.tdtype), k.to(self.tdtype), v.to(self.tdtype)
