"""Seeded synthetic inputs for the fused FP8 MoE layer.

This module only *prepares inputs*: random draws, casts and the input-side
block quantisation that the workload description prescribes (activations per
token per 128 columns, weights per 128x128 block, scale = amax/448).  It holds
none of the layer's own arithmetic (routing, GEMMs, SwiGLU, re-quantisation,
combine), imports neither the CUDA binding nor the CPU oracle, and serves both.

The five benchmark workloads stand in for the FlashInfer-Bench Fused-MoE
contest workloads the paper measured on (DeepSeek-V3 layer shapes); none of
the contest's own items is reproduced here.
"""
from __future__ import annotations

from dataclasses import dataclass, replace

import numpy as np
import torch

QBLOCK = 128
FP8_MAX = 448.0


@dataclass(frozen=True)
class LayerDims:
    """Shape of one MoE layer (defaults: DeepSeek-V3)."""

    hidden: int = 7168
    intermediate: int = 2048
    num_experts: int = 256
    num_local_experts: int = 32
    n_group: int = 8
    topk_group: int = 4
    top_k: int = 8


@dataclass(frozen=True)
class Workload:
    name: str
    tokens: int
    dims: LayerDims
    seed: int
    local_expert_offset: int = 0
    scaling_factor: float = 2.5
    skew: bool = False


DSV3 = LayerDims()

#: The five benchmark configurations (T, local experts, seed, routing skew).
CONFIGS = (
    Workload("dsv3_T8_E32", 8, DSV3, seed=0),
    Workload("dsv3_T64_E32", 64, DSV3, seed=1),
    Workload("dsv3_T1024_E32", 1024, DSV3, seed=2),
    Workload("dsv3_T8192_E32_skew", 8192, DSV3, seed=3, skew=True),
    Workload("dsv3_T16384_E256", 16384, replace(DSV3, num_local_experts=256), seed=4),
)

#: Local expert ids that receive the +3.0 routing-bias boost in the skewed workload.
SKEW_HOT_EXPERTS = (3, 11, 17, 26)


def _quant_rows_128(x: torch.Tensor):
    """x [R, C] fp32 -> (e4m3 [R, C], scale fp32 [R, C/128]); scale = amax/448."""
    R, C = x.shape
    xb = x.view(R, C // QBLOCK, QBLOCK)
    amax = xb.abs().amax(dim=-1)
    scale = torch.where(amax == 0, torch.ones_like(amax), amax / FP8_MAX)
    q = (xb / scale.unsqueeze(-1)).to(torch.float8_e4m3fn).view(R, C)
    return q, scale.contiguous()


def _quant_blocks_128x128(w: torch.Tensor):
    """w [N, K] fp32 -> (e4m3 [N, K], scale fp32 [N/128, K/128])."""
    N, K = w.shape
    wb = w.view(N // QBLOCK, QBLOCK, K // QBLOCK, QBLOCK)
    amax = wb.abs().amax(dim=(1, 3))
    scale = torch.where(amax == 0, torch.ones_like(amax), amax / FP8_MAX)
    q = (wb / scale[:, None, :, None]).to(torch.float8_e4m3fn).view(N, K)
    return q, scale.contiguous()


def make_inputs(wl: Workload, device: str | torch.device = "cpu") -> dict:
    """Draw one workload.  Order of draws is fixed: hidden, logits, bias, then
    the experts one at a time (w13 then w2), so memory stays bounded.

    Returns torch tensors on `device`:
      hidden_fp8 [T,H] float8_e4m3fn, hidden_scale [T,H/128] fp32,
      router_logits [T,E] fp32 (multiples of 1/64), routing_bias [E] bf16,
      w13 [E_loc,2I,H] fp8, w13_scale [E_loc,2I/128,H/128] fp32,
      w2 [E_loc,H,I] fp8,  w2_scale [E_loc,H/128,I/128] fp32,
    plus the scalars local_expert_offset and scaling_factor.
    """
    d = wl.dims
    dev = torch.device(device)
    g = torch.Generator(device=dev)
    g.manual_seed(wl.seed)
    T, H, I, E, EL = wl.tokens, d.hidden, d.intermediate, d.num_experts, d.num_local_experts

    hidden = torch.randn(T, H, generator=g, device=dev, dtype=torch.float32)
    hidden = hidden.to(torch.bfloat16).to(torch.float32)
    if T > 0:
        hidden_fp8, hidden_scale = _quant_rows_128(hidden)
    else:
        hidden_fp8 = torch.empty(0, H, device=dev, dtype=torch.float8_e4m3fn)
        hidden_scale = torch.empty(0, H // QBLOCK, device=dev, dtype=torch.float32)
    del hidden

    logits = torch.round(torch.randn(T, E, generator=g, device=dev, dtype=torch.float32) * 64.0) / 64.0

    bias = 0.1 * torch.randn(E, generator=g, device=dev, dtype=torch.float32)
    if wl.skew:
        hot = [wl.local_expert_offset + e for e in SKEW_HOT_EXPERTS if e < EL]
        rest = [e for e in range(E) if e not in hot]
        perm = torch.randperm(len(rest), generator=g, device=dev)
        rank = torch.empty(len(rest), device=dev, dtype=torch.float32)
        rank[perm] = torch.arange(1, len(rest) + 1, device=dev, dtype=torch.float32)
        boost = torch.zeros(E, device=dev, dtype=torch.float32)
        boost[torch.tensor(hot, device=dev, dtype=torch.long)] = 3.0
        boost[torch.tensor(rest, device=dev, dtype=torch.long)] = rank.pow(-1.1)
        bias = bias + boost
    bias = bias.to(torch.bfloat16)

    w13 = torch.empty(EL, 2 * I, H, device=dev, dtype=torch.float8_e4m3fn)
    w13_scale = torch.empty(EL, 2 * I // QBLOCK, H // QBLOCK, device=dev, dtype=torch.float32)
    w2 = torch.empty(EL, H, I, device=dev, dtype=torch.float8_e4m3fn)
    w2_scale = torch.empty(EL, H // QBLOCK, I // QBLOCK, device=dev, dtype=torch.float32)
    for e in range(EL):
        a = 0.02 * torch.randn(2 * I, H, generator=g, device=dev, dtype=torch.float32)
        w13[e], w13_scale[e] = _quant_blocks_128x128(a)
        b = 0.02 * torch.randn(H, I, generator=g, device=dev, dtype=torch.float32)
        w2[e], w2_scale[e] = _quant_blocks_128x128(b)
        del a, b

    return {
        "hidden_fp8": hidden_fp8,
        "hidden_scale": hidden_scale,
        "router_logits": logits,
        "routing_bias": bias,
        "w13": w13,
        "w13_scale": w13_scale,
        "w2": w2,
        "w2_scale": w2_scale,
        "local_expert_offset": wl.local_expert_offset,
        "scaling_factor": wl.scaling_factor,
    }


def make_router_inputs(wl: Workload, device: str | torch.device = "cpu") -> dict:
    """Inputs of the layer when it starts from hidden states: the bf16 hidden states whose quantisation
    make_inputs returns as hidden_fp8 / hidden_scale (same generator, same first draw), and a router weight
    [E, H] bf16 drawn N(0, 1/H) so that the logits have about unit variance."""
    d = wl.dims
    dev = torch.device(device)
    g = torch.Generator(device=dev)
    g.manual_seed(wl.seed)
    hidden = torch.randn(wl.tokens, d.hidden, generator=g, device=dev, dtype=torch.float32).to(torch.bfloat16)
    g2 = torch.Generator(device=dev)
    g2.manual_seed(wl.seed + 500009)
    w = torch.randn(d.num_experts, d.hidden, generator=g2, device=dev, dtype=torch.float32) / (d.hidden ** 0.5)
    return {"hidden_bf16": hidden, "router_weight": w.to(torch.bfloat16)}


def make_activations(wl: Workload, seed: int, device: str | torch.device = "cpu") -> dict:
    """A fresh set of per-step activations (hidden + logits) for the same layer,
    used to rotate inputs between timed iterations."""
    d = wl.dims
    dev = torch.device(device)
    g = torch.Generator(device=dev)
    g.manual_seed(seed)
    hidden = torch.randn(wl.tokens, d.hidden, generator=g, device=dev, dtype=torch.float32)
    hidden = hidden.to(torch.bfloat16).to(torch.float32)
    hidden_fp8, hidden_scale = _quant_rows_128(hidden)
    logits = torch.round(torch.randn(wl.tokens, d.num_experts, generator=g, device=dev) * 64.0) / 64.0
    return {"hidden_fp8": hidden_fp8, "hidden_scale": hidden_scale, "router_logits": logits}


def tiny_workload(tokens: int = 5, hidden: int = 256, intermediate: int = 128, num_experts: int = 16,
                  num_local_experts: int = 16, n_group: int = 4, topk_group: int = 2, top_k: int = 2,
                  seed: int = 123, offset: int = 0, scaling: float = 2.5) -> Workload:
    """A miniature layer for brute-force checks."""
    dims = LayerDims(hidden, intermediate, num_experts, num_local_experts, n_group, topk_group, top_k)
    return Workload(f"tiny_T{tokens}", tokens, dims, seed, offset, scaling)


def to_host(inp: dict) -> dict:
    """Byte-identical numpy copies: fp8 tensors as uint8 codes, bf16 as uint16 bits."""
    out = {}
    for k, v in inp.items():
        if not torch.is_tensor(v):
            out[k] = v
        elif v.dtype == torch.float8_e4m3fn:
            out[k] = v.view(torch.uint8).cpu().numpy()
        elif v.dtype == torch.bfloat16:
            out[k] = v.view(torch.int16).cpu().numpy().view(np.uint16)
        else:
            out[k] = v.cpu().numpy()
    return out
