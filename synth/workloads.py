"""Synthetic MoE-layer workloads shaped like the paper's on-device model classes.

Shapes only: E = 8 experts with 2 active per token (Section 3.1), SwiGLU experts,
optionally weight-decomposed (Eq. 1), uneven or Zipf-skewed expert load.  The
tensors come from `synth.rng`; nothing here computes any part of the layer.

Layouts handed out (the mathematical, row-vector convention y = x @ W):
  x        [T, d]                fp32 or bf16
  w_router [d, E]  bf16          b_router [E] fp32 or None
  w_gate, w_up [E, d, f] bf16    w_down [E, f, d] bf16
  WD factors: gL,uL [E, d, r]; gR,uR [E, r, f]; dL [E, f, r]; dR [E, r, d]  (bf16)
"""
from __future__ import annotations

import math
from dataclasses import dataclass, replace

import numpy as np
import torch

from . import rng

BASE_SEED = 20250300


@dataclass(frozen=True)
class LayerShape:
    name: str
    cfg_id: int
    d_model: int
    d_ff: int
    n_experts: int = 8
    top_k: int = 2
    wd_rank: int = 0            # 0 = dense experts
    x_dtype: str = "bf16"       # "f32" | "bf16"
    bias: str = "none"          # "none" | "normal" (sigma 0.5) | "zipf" (alpha 1.2)

    def with_(self, **kw) -> "LayerShape":
        return replace(self, **kw)

    @property
    def expert_elems(self) -> int:
        if self.wd_rank:
            return 3 * self.wd_rank * (self.d_model + self.d_ff)
        return 3 * self.d_model * self.d_ff


TINY = LayerShape("tiny", 1, 256, 512, x_dtype="f32")
WEARABLE = LayerShape("wearable", 2, 1024, 2816)
PHONE = LayerShape("phone", 3, 2048, 5632, bias="normal")
PHONE_WD128 = LayerShape("phone-wd-r128", 4, 2048, 5632, wd_rank=128)
PHONE_WD1024 = LayerShape("phone-wd-r1024", 4, 2048, 5632, wd_rank=1024)
PHONE_OFFLOAD = LayerShape("phone-offload", 5, 2048, 5632, n_experts=16, bias="zipf")

SHAPES = {s.name: s for s in (TINY, WEARABLE, PHONE, PHONE_WD128, PHONE_WD1024, PHONE_OFFLOAD)}

_TDTYPE = {"f32": torch.float32, "bf16": torch.bfloat16}


def _seed(shape: LayerShape, tensor_id: int, layer: int = 0) -> int:
    return BASE_SEED + 1000 * shape.cfg_id + tensor_id + 100000 * layer


def make_x(shape: LayerShape, T: int, device="cpu", layer: int = 0, step: int = 0) -> torch.Tensor:
    return rng.normal(_seed(shape, 1, layer) + 7919 * step, (T, shape.d_model), 1.0,
                      _TDTYPE[shape.x_dtype], device)


def make_router(shape: LayerShape, device="cpu", layer: int = 0):
    d, E = shape.d_model, shape.n_experts
    w_router = rng.normal(_seed(shape, 2, layer), (d, E), d ** -0.5, torch.bfloat16, device)
    if shape.bias == "none":
        b = None
    elif shape.bias == "normal":
        b = rng.normal(_seed(shape, 3, layer), (E,), 0.5, torch.float32, device)
    elif shape.bias == "zipf":
        # exp(b[e]) proportional to rank(e)^-1.2 with a seeded rank assignment per layer
        rank = rng.permutation(_seed(shape, 3, layer), E).to(torch.float64) + 1.0
        b = (-1.2 * torch.log(rank)).to(torch.float32).to(device)
    else:
        raise ValueError(shape.bias)
    return w_router, b


def make_experts(shape: LayerShape, device="cpu", layer: int = 0) -> dict:
    d, f, E, r = shape.d_model, shape.d_ff, shape.n_experts, shape.wd_rank
    bf = torch.bfloat16
    if r == 0:
        return {
            "w_gate": rng.normal(_seed(shape, 10, layer), (E, d, f), d ** -0.5, bf, device),
            "w_up": rng.normal(_seed(shape, 11, layer), (E, d, f), d ** -0.5, bf, device),
            "w_down": rng.normal(_seed(shape, 12, layer), (E, f, d), f ** -0.5, bf, device),
        }
    return {
        "gL": rng.normal(_seed(shape, 20, layer), (E, d, r), d ** -0.5, bf, device),
        "gR": rng.normal(_seed(shape, 21, layer), (E, r, f), r ** -0.5, bf, device),
        "uL": rng.normal(_seed(shape, 22, layer), (E, d, r), d ** -0.5, bf, device),
        "uR": rng.normal(_seed(shape, 23, layer), (E, r, f), r ** -0.5, bf, device),
        "dL": rng.normal(_seed(shape, 24, layer), (E, f, r), f ** -0.5, bf, device),
        "dR": rng.normal(_seed(shape, 25, layer), (E, r, d), r ** -0.5, bf, device),
    }


def make_layer(shape: LayerShape, T: int, device="cpu", layer: int = 0) -> dict:
    w_router, b_router = make_router(shape, device, layer)
    out = {"x": make_x(shape, T, device, layer), "w_router": w_router, "b_router": b_router}
    out.update(make_experts(shape, device, layer))
    return out


def to_host_bits(t: torch.Tensor | None):
    """Torch tensor -> numpy array a CPU checker can widen exactly:
    bf16 becomes its uint16 bit pattern, fp32/int tensors stay as they are."""
    if t is None:
        return None
    t = t.detach().cpu().contiguous()
    if t.dtype == torch.bfloat16:
        return t.view(torch.int16).numpy().view(np.uint16)
    return t.numpy()


def sticky_routing_trace(seed: int, steps: int, n_experts: int, top_k: int, p_stay: float) -> np.ndarray:
    """Synthetic decode routing trace [steps, top_k]: with probability p_stay a step
    keeps the previous expert set, otherwise one member is replaced by a uniformly
    drawn expert outside the set.  Stands in for routing on real text (Table 3)."""
    u = rng.uniform01(seed, torch.arange(3 * steps, dtype=torch.int64)).numpy()
    cur = list(range(top_k))
    trace = np.zeros((steps, top_k), dtype=np.int32)
    for s in range(steps):
        if s > 0 and u[3 * s] >= p_stay:
            out_pos = int(u[3 * s + 1] * top_k) % top_k
            others = [e for e in range(n_experts) if e not in cur]
            cur[out_pos] = others[int(u[3 * s + 2] * len(others)) % len(others)]
        trace[s] = cur
    return trace


def zipf_mass(alpha: float, n: int, top: int) -> float:
    w = [i ** -alpha for i in range(1, n + 1)]
    return sum(w[:top]) / sum(w)


def expert_bytes(shape: LayerShape) -> int:
    return 2 * shape.expert_elems


def describe(shape: LayerShape) -> str:
    kind = f"WD r={shape.wd_rank}" if shape.wd_rank else "dense"
    return (f"{shape.name}: d={shape.d_model} f={shape.d_ff} E={shape.n_experts} k={shape.top_k} "
            f"{kind} x={shape.x_dtype} bias={shape.bias} "
            f"({expert_bytes(shape) / 1e6:.2f} MB/expert)")



