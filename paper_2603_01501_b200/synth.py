"""Seeded synthetic gradient lists shaped like LLM policy gradients.

This module only *produces inputs*: random tensors with a prescribed cosine to
a stored direction.  It contains none of the method's arithmetic (no regime
rule, no coefficient, no in-place update) and is the one module that both the
CUDA path's callers and the CPU checker's callers may use.

Real policy gradients (App. C: Qwen3 / Llama policies trained with VERL) need
models, data and a rollout engine; the lists below stand in for them with the
same tensor-size mix: one huge embedding, large MLP matrices, medium attention
matrices, and hundreds of tiny norm/bias vectors, each tensor its own
allocation as ``.grad`` tensors are.
"""
from __future__ import annotations

import math
import random
from dataclasses import dataclass
from typing import Dict, List, Optional, Sequence, Tuple

import torch


@dataclass(frozen=True)
class DecoderDims:
    hidden: int
    layers: int
    q_heads: int
    kv_heads: int
    head_dim: int
    intermediate: int
    vocab: int
    tied: bool
    qkv_bias: bool = True


DIMS: Dict[str, DecoderDims] = {
    # name            hidden layers q  kv hd   inter  vocab  tied
    "1.5b": DecoderDims(1536, 28, 12, 2, 128, 8960, 151936, True),
    "7b": DecoderDims(3584, 28, 28, 4, 128, 18944, 152064, False),
    "14b": DecoderDims(5120, 48, 40, 8, 128, 13824, 152064, False),
    # scaled-down lists with the same structure, for cases a CPU checks in seconds;
    # odd sizes on purpose so tensor tails are ragged
    # a 0.25 B list (1-2 GB per buffer): larger than L2, small enough for profiler captures
    "0.25b": DecoderDims(1024, 12, 8, 2, 128, 4096, 32000, False),
    # one flat vector of 2^20 elements (a single "tensor"): the small, launch-bound case
    "flat_1m": DecoderDims(0, 0, 0, 0, 0, 0, 0, True),
    "mini": DecoderDims(96, 3, 3, 1, 32, 250, 1021, True),
    "small": DecoderDims(384, 6, 6, 2, 64, 1030, 15013, False),
}


def decoder_tensor_list(dims: DecoderDims) -> List[Tuple[str, int]]:
    """(name, numel) of every trainable tensor of a decoder-only transformer
    with grouped-query attention, SwiGLU MLP and RMSNorm, in module order."""
    if dims.hidden == 0:
        return [("flat", 1 << 20)]
    h, qd, kvd = dims.hidden, dims.q_heads * dims.head_dim, dims.kv_heads * dims.head_dim
    out: List[Tuple[str, int]] = [("embed", dims.vocab * h)]
    for l in range(dims.layers):
        p = f"layers.{l}."
        out.append((p + "input_norm", h))
        out.append((p + "q_proj.weight", qd * h))
        if dims.qkv_bias:
            out.append((p + "q_proj.bias", qd))
        out.append((p + "k_proj.weight", kvd * h))
        if dims.qkv_bias:
            out.append((p + "k_proj.bias", kvd))
        out.append((p + "v_proj.weight", kvd * h))
        if dims.qkv_bias:
            out.append((p + "v_proj.bias", kvd))
        out.append((p + "o_proj.weight", h * qd))
        out.append((p + "post_attn_norm", h))
        out.append((p + "gate_proj.weight", dims.intermediate * h))
        out.append((p + "up_proj.weight", dims.intermediate * h))
        out.append((p + "down_proj.weight", h * dims.intermediate))
    out.append(("final_norm", h))
    if not dims.tied:
        out.append(("lm_head", dims.vocab * h))
    return out


def list_numel(shapes: Sequence[Tuple[str, int]]) -> int:
    return sum(n for _, n in shapes)


def per_tensor_scales(config_id: int, count: int) -> List[float]:
    """sigma_i = 10^U(-4,-1): log-uniform per-tensor gradient scales, from a
    Mersenne-Twister stream seeded by the config number."""
    rng = random.Random(1000003 * config_id + 17)
    return [10.0 ** rng.uniform(-4.0, -1.0) for _ in range(count)]


def _gen(device, seed: int) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(seed)
    return g


def tensor_seed(config_id: int, index: int, stream: int) -> int:
    return config_id * 10**9 + index * 2 + stream


def flat_pair_with_cosine(n: int, rho: float, s: float = 1.0, seed: int = 0,
                          device="cpu") -> Tuple[torch.Tensor, torch.Tensor]:
    """One float32 pair (g, d) of length n whose cosine is rho by construction:
    d ~ N(0,1); noise ~ N(0,1) made orthogonal to d and normalised;
    g = s (rho d/|d| + sqrt(1-rho^2) noise/|noise|), built in float64 and
    rounded once to float32."""
    d = torch.randn(n, generator=_gen(device, seed * 2), device=device, dtype=torch.float64)
    z = torch.randn(n, generator=_gen(device, seed * 2 + 1), device=device, dtype=torch.float64)
    z = z - (torch.dot(z, d) / torch.dot(d, d)) * d
    z = z / z.norm()
    g = s * (rho * d / d.norm() + math.sqrt(1.0 - rho * rho) * z)
    return g.to(torch.float32), d.to(torch.float32)


def gaussian_tensor_pair(numel: int, sigma: float, rho: float, config_id: int, index: int,
                         g_dtype: torch.dtype, device) -> Tuple[torch.Tensor, torch.Tensor]:
    """d = sigma z, g = rho d + sqrt(1-rho^2) sigma w with z, w iid N(0,1):
    expected cosine rho, realised cosine rho +- O(numel^-1/2).  g is rounded to
    g_dtype from the float32 construction; d stays float32."""
    z = torch.randn(numel, generator=_gen(device, tensor_seed(config_id, index, 0)),
                    device=device, dtype=torch.float32)
    d = z.mul_(sigma)
    w = torch.randn(numel, generator=_gen(device, tensor_seed(config_id, index, 1)),
                    device=device, dtype=torch.float32)
    g = w.mul_(math.sqrt(1.0 - rho * rho) * sigma).add_(d, alpha=rho)
    if g_dtype != torch.float32:
        g = g.to(g_dtype)
    return g, d


def gradient_list(shapes: Sequence[Tuple[str, int]], rho: float, config_id: int,
                  g_dtype: torch.dtype = torch.float32, device="cpu",
                  indices: Optional[Sequence[int]] = None):
    """Lists (g_i), (d_i), one separately allocated tensor per parameter.
    `indices` restricts generation to some tensors of the list (same values as
    in the full list), so a checker can regenerate them one by one."""
    sig = per_tensor_scales(config_id, len(shapes))
    idx = range(len(shapes)) if indices is None else indices
    gs, ds = [], []
    for i in idx:
        g, d = gaussian_tensor_pair(shapes[i][1], sig[i], rho, config_id, i, g_dtype, device)
        gs.append(g)
        ds.append(d)
    return gs, ds


class StalenessProcess:
    """Exogenous gradient sequence for a staleness run on one tensor list.

    g_1 = e_1;  g_t = rho m_t + sqrt(1-rho^2) e_t, where e_t is a fresh
    per-tensor Gaussian draw (scales sigma_i) and m_t is the sum of the last
    min(k, t-1) gradients rescaled to the norm of e_t.  For k = 1 and equal
    norms this is the AR(1) recursion g_t = rho g_{t-1} + sqrt(1-rho^2) e_t.
    The window k models drift accumulated over the last k updates by a policy
    that lags k steps behind.  Gradients do not depend on what the controller
    does with them.
    """

    def __init__(self, shapes: Sequence[Tuple[str, int]], rho: float, k: int, config_id: int,
                 run_id: int, device="cpu"):
        self.shapes = list(shapes)
        self.rho, self.k, self.device = float(rho), int(k), device
        self.config_id, self.run_id = config_id, run_id
        self.sigma = per_tensor_scales(config_id, len(shapes))
        self.window: List[List[torch.Tensor]] = []   # most recent last
        self.t = 0

    def _noise(self, t: int) -> List[torch.Tensor]:
        out = []
        for i, (_, n) in enumerate(self.shapes):
            seed = tensor_seed(self.config_id, i, 0) + 7919 * (self.run_id * 100003 + t)
            e = torch.randn(n, generator=_gen(self.device, seed), device=self.device,
                            dtype=torch.float32)
            out.append(e.mul_(self.sigma[i]))
        return out

    @staticmethod
    def _norm(ts: List[torch.Tensor]) -> float:
        return math.sqrt(sum(float(torch.sum(t.double() ** 2)) for t in ts))

    def next(self) -> List[torch.Tensor]:
        """Returns g_t as a new list of float32 tensors (the caller may modify them)."""
        self.t += 1
        e = self._noise(self.t)
        if not self.window or self.rho == 0.0:
            g = e
        else:
            m = [torch.zeros_like(x) for x in e]
            for past in self.window:
                for acc, p in zip(m, past):
                    acc.add_(p)
            scale = self._norm(e) / max(self._norm(m), 1e-300)
            c = math.sqrt(1.0 - self.rho ** 2)
            g = [ei.mul_(c).add_(mi, alpha=self.rho * scale) for ei, mi in zip(e, m)]
        self.window.append([x.clone() for x in g])
        if len(self.window) > self.k:
            self.window.pop(0)
        return g


def refresh_gradient_list(g_list: Sequence[torch.Tensor], d_list: Sequence[torch.Tensor],
                          sigma: Sequence[float], rho: float, gen: torch.Generator,
                          scratch: torch.Tensor) -> None:
    """Overwrites every g_i with a fresh gradient whose expected cosine to the
    current stored direction is rho: g_i = rho d_i + sqrt(1-rho^2) sigma_i w,
    w ~ N(0,1) (one AR(1) step of the staleness process).  `scratch` is a
    float32 work buffer at least as long as the largest tensor."""
    c = math.sqrt(1.0 - rho * rho)
    for g, d, s in zip(g_list, d_list, sigma):
        w = scratch[: g.numel()]
        w.normal_(generator=gen)
        w.mul_(c * s).add_(d, alpha=rho)
        g.copy_(w)


WORKLOADS = {
    # name: (dims key, g dtype, rho, config id)  -- the decoder-shaped lists of the benchmark
    "cfg1_flat_f32": ("flat_1m", torch.float32, 0.9, 1),
    "cfg2_1.5b_f32": ("1.5b", torch.float32, 0.8, 2),
    "cfg3_7b_bf16": ("7b", torch.bfloat16, 0.95, 3),
    "cfg5_14b_f32": ("14b", torch.float32, 0.9, 5),
    "prof_0.25b_f32": ("0.25b", torch.float32, 0.9, 5),
    "prof_0.25b_bf16": ("0.25b", torch.bfloat16, 0.95, 3),
    "prof_0.25b_bf16_dbf16": ("0.25b", torch.bfloat16, 0.95, 3),
    "cfg3_7b_bf16_dbf16": ("7b", torch.bfloat16, 0.95, 3),     # same list, bfloat16 snapshot
    "small_f32": ("small", torch.float32, 0.9, 2),
    "small_bf16": ("small", torch.bfloat16, 0.95, 3),
}

# element type of the stored direction where it is not float32
WORKLOAD_D_DTYPE = {"cfg3_7b_bf16_dbf16": torch.bfloat16, "prof_0.25b_bf16_dbf16": torch.bfloat16}
