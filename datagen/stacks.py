"""Seeded synthetic MoE stacks and token streams (inputs only, no method arithmetic).

The five stack shapes are the benchmark configurations of this repository:
public MoE model *shapes* with random weights, a router chain with planted
layer-to-layer correlation and an AR(1) token stream with planted
token-to-token correlation.  They stand in for the trained checkpoints and the
text datasets of the paper's evaluation (Tables 1-2), which are not available.

Recipe
  expert weights   N(0, 0.02) (0.02 is the standard deviation), one random
                   stream per (layer, expert, matrix), rounded RNE to the
                   storage dtype; fp8: per-output-channel scale = amax/448
                   stored as bf16, then saturating RNE e4m3.
  router weights   W_0 ~ N(0, 0.02); W_{l+1} = c W_l + sqrt(1-c^2) N(0, 0.02),
                   chain kept in fp32, each layer rounded to the router dtype.
  token inputs     per sequence b: n_t = sqrt(H) g_t/||g_t||_2 (unit RMS),
                   x_0 = n_0, x_t = rho x_{t-1} + sqrt(1-rho^2) n_t.
"""
from __future__ import annotations

import dataclasses
import math

import torch

from . import rng

SEED_WEIGHTS = 0
SEED_TOKENS = 1
SEED_TRACES = 2

_TAG_EXPERT, _TAG_SHARED, _TAG_ROUTER, _TAG_TOKEN, _TAG_TRACE = 11, 12, 13, 14, 15
_MAT = {"gate": 0, "up": 1, "down": 2}

SIGMA = 0.02
FP8_MAX = 448.0


@dataclasses.dataclass(frozen=True)
class StackConfig:
    name: str
    n_layers: int
    n_experts: int
    top_k: int
    n_shared: int
    hidden: int
    inter: int
    dtype: str              # "f32" | "bf16" | "fp8"
    router_c: float         # layer-to-layer router correlation
    router_s: float         # weight of the fresh noise in the router chain
    rho: float              # AR(1) coefficient of the token stream
    tokens: int
    batches: tuple
    profile_tokens: int
    cache_slots: int = 0    # 0: every expert resident in HBM
    residual_scale: float = 0.1
    rms_eps: float = 1e-6

    @property
    def router_dtype(self) -> str:
        return "f32" if self.dtype == "f32" else "bf16"

    @property
    def weight_bytes(self) -> int:
        return {"f32": 4, "bf16": 2, "fp8": 1}[self.dtype]

    @property
    def expert_bytes(self) -> int:
        n = 3 * self.hidden * self.inter * self.weight_bytes
        if self.dtype == "fp8":
            n += 2 * (2 * self.inter + self.hidden)
        return n

    @property
    def router_bytes(self) -> int:
        return self.n_experts * self.hidden * (4 if self.dtype == "f32" else 2)

    def scaled(self, **kw) -> "StackConfig":
        return dataclasses.replace(self, **kw)


CONFIGS = {
    "C0": StackConfig("C0-tiny-f32", 4, 8, 2, 0, 256, 512, "f32", 0.8, 0.6, 0.9, 64, (1,), 16),
    "C1": StackConfig("C1-mixtral-bf16", 32, 8, 2, 0, 4096, 14336, "bf16", 0.8, 0.6, 0.9, 256,
                      (1, 4), 64),
    "C2": StackConfig("C2-dsv2lite-bf16", 26, 64, 6, 2, 2048, 1408, "bf16", 0.8, 0.6, 0.9, 512,
                      (1, 8), 64),
    "C3": StackConfig("C3-qwen3-30b-bf16-offload", 48, 128, 8, 0, 2048, 768, "bf16", 0.7,
                      math.sqrt(1 - 0.49), 0.85, 512, (1, 16), 64, cache_slots=48 * 128 // 4),
    "C4": StackConfig("C4-qwen3-235b-fp8-offload", 94, 128, 8, 0, 4096, 1536, "fp8", 0.7,
                      math.sqrt(1 - 0.49), 0.85, 1024, (1, 32), 64,
                      cache_slots=(96 * 10**9) // (3 * 4096 * 1536 + 2 * (2 * 1536 + 4096))),
}

_TORCH_DT = {"f32": torch.float32, "bf16": torch.bfloat16}


def _normal_matrix(rows, cols, key, device):
    return rng.normal(rows * cols, key, device).view(rows, cols)


def quantize_fp8(w: torch.Tensor):
    """Per-output-channel (row) scale amax/448 as bf16, then saturating RNE e4m3."""
    amax = w.abs().amax(dim=1).clamp_min(1e-12)
    scale = (amax / FP8_MAX).to(torch.bfloat16)
    q = (w / scale.to(torch.float32)[:, None]).clamp(-FP8_MAX, FP8_MAX).to(torch.float8_e4m3fn)
    return q, scale


def expert_weights(cfg: StackConfig, layer: int, expert: int, shared: bool = False,
                   device="cpu") -> dict:
    """gate [I][H], up [I][H], down [H][I] in the storage dtype (+ *_scale for fp8)."""
    out = {}
    tag = _TAG_SHARED if shared else _TAG_EXPERT
    for name, m in _MAT.items():
        rows, cols = (cfg.hidden, cfg.inter) if name == "down" else (cfg.inter, cfg.hidden)
        key = rng.stream_key(SEED_WEIGHTS, tag, layer, expert, m)
        w = torch.mul(_normal_matrix(rows, cols, key, device), SIGMA)
        if cfg.dtype == "fp8":
            out[name], out[name + "_scale"] = quantize_fp8(w)
        else:
            out[name] = w.to(_TORCH_DT[cfg.dtype])
    return out


def router_weights(cfg: StackConfig) -> list:
    """Per-layer router matrices [E][H] in the router dtype, generated on the CPU."""
    ws = []
    w = None
    for layer in range(cfg.n_layers):
        key = rng.stream_key(SEED_WEIGHTS, _TAG_ROUTER, layer)
        fresh = torch.mul(_normal_matrix(cfg.n_experts, cfg.hidden, key, "cpu"), SIGMA)
        w = fresh if w is None else torch.add(torch.mul(w, cfg.router_c),
                                              torch.mul(fresh, cfg.router_s))
        ws.append(w.to(_TORCH_DT[cfg.router_dtype]).contiguous())
    return ws


def token_inputs(cfg: StackConfig, batch: int, tokens: int) -> torch.Tensor:
    """Stack inputs h_0(t) as fp32 [tokens][batch][H], generated on the CPU in float64."""
    out = torch.empty(tokens, batch, cfg.hidden, dtype=torch.float32)
    a, b = cfg.rho, math.sqrt(1.0 - cfg.rho * cfg.rho)
    for s in range(batch):
        key = rng.stream_key(SEED_TOKENS, _TAG_TOKEN, s)
        g = rng.normal(tokens * cfg.hidden, key).view(tokens, cfg.hidden).to(torch.float64)
        n = g * (math.sqrt(cfg.hidden) / g.norm(dim=1, keepdim=True))
        x = n[0]
        out[0, s] = x.to(torch.float32)
        for t in range(1, tokens):
            x = a * x + b * n[t]
            out[t, s] = x.to(torch.float32)
    return out


def planted_pair_trace(n_experts: int, q: float, tokens: int, stream: int = 0):
    """Routing-only K=1 trace for one layer pair with a planted transition.

    Layer-i expert e_t is uniform; the layer-(i+1) expert is pi(e_t) with
    probability q, otherwise uniform over the other E-1 experts.  Returns
    (e [tokens], f [tokens], pi [E]) as int64 CPU tensors; pi is a fixed
    derangement-free shift-and-scramble permutation.
    """
    key_e = rng.stream_key(SEED_TRACES, _TAG_TRACE, stream, 0)
    key_u = rng.stream_key(SEED_TRACES, _TAG_TRACE, stream, 1)
    key_o = rng.stream_key(SEED_TRACES, _TAG_TRACE, stream, 2)
    key_p = rng.stream_key(SEED_TRACES, _TAG_TRACE, stream, 3)
    pi = torch.argsort(rng.uniform_bits(n_experts, key_p))
    e = rng.uniform_int(tokens, n_experts, key_e)
    follow = rng.uniform01(tokens, key_u) < q
    other = rng.uniform_int(tokens, n_experts - 1, key_o)
    target = pi[e]
    other = other + (other >= target).to(torch.int64)   # uniform over ids != target
    f = torch.where(follow, target, other)
    return e, f, pi


def random_topk_trace(n_experts: int, top_k: int, tokens: int, layers: int, batch: int = 1,
                      stream: int = 0) -> torch.Tensor:
    """Independent uniform routing: int32 [tokens][layers][batch][K], ids ascending."""
    key = rng.stream_key(SEED_TRACES, _TAG_TRACE, stream, 7)
    n = tokens * layers * batch
    r = rng.uniform_bits(n * n_experts, key).view(n, n_experts)
    ids = torch.argsort(r, dim=1)[:, :top_k]
    ids = torch.sort(ids, dim=1).values
    return ids.view(tokens, layers, batch, top_k).to(torch.int32)
