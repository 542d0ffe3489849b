"""Expert-parallel use of the layer: what `local_expert_offset` and "32 local
experts of 256" encode.  Every rank holds the weights of a contiguous slice of
the experts and its own batch of tokens (data parallel).  One forward is

  1. all-gather of the ranks' tokens (FP8 codes, 128-wide scales, router logits),
  2. the fused forward on ALL tokens with this rank's expert slice (routes to
     experts of other ranks are dropped after normalisation, so every rank
     produces a partial output for every token),
  3. reduce-scatter (sum) of the partial outputs: each rank receives the full
     result for its own tokens.

The exchange steps are plain collectives of `torch.distributed` (NCCL over
NVLink on GPUs; any backend works, the host logic is the same); the layer
itself runs in the CUDA library through the callable given at construction.
Ranks may hold different numbers of tokens (including none).
"""
from __future__ import annotations

from typing import Callable

import torch
import torch.distributed as dist


class ExpertParallelMoe:
    """local_forward(hidden_fp8_u8 [T,H], hidden_scale [T,H/128], router_logits [T,E], local_expert_offset)
    -> bf16 [T,H] partial output of this rank's experts for all T gathered tokens."""

    def __init__(self, local_forward: Callable, hidden: int, num_experts: int, num_local_experts: int, group=None):
        if not dist.is_initialized():
            raise RuntimeError("ExpertParallelMoe needs an initialised torch.distributed process group")
        self.group = group
        self.world = dist.get_world_size(group)
        self.rank = dist.get_rank(group)
        if num_local_experts * self.world != num_experts:
            raise ValueError(f"{self.world} ranks x {num_local_experts} local experts do not cover {num_experts} experts")
        self.local_forward = local_forward
        self.hidden, self.num_experts, self.num_local_experts = hidden, num_experts, num_local_experts
        self.local_expert_offset = self.rank * num_local_experts

    # -- collectives ---------------------------------------------------------------------------------
    def _gather_counts(self, n: int, device) -> list[int]:
        mine = torch.tensor([n], dtype=torch.int64, device=device)
        every = torch.empty(self.world, dtype=torch.int64, device=device)
        dist.all_gather_into_tensor(every, mine, group=self.group)
        return [int(v) for v in every.tolist()]

    def _all_gather_rows(self, x: torch.Tensor, counts: list[int], pad_to: int) -> torch.Tensor:
        """Ragged all-gather along dim 0: every rank contributes counts[r] rows; -> the concatenation."""
        padded = x.new_zeros((pad_to,) + tuple(x.shape[1:]))
        padded[: x.shape[0]] = x
        every = x.new_empty((self.world * pad_to,) + tuple(x.shape[1:]))
        dist.all_gather_into_tensor(every, padded, group=self.group)
        every = every.view((self.world, pad_to) + tuple(x.shape[1:]))
        return torch.cat([every[r, : counts[r]] for r in range(self.world)], dim=0)

    def _reduce_scatter_rows(self, partial: torch.Tensor, counts: list[int], pad_to: int) -> torch.Tensor:
        """Sum over ranks of the fp32 partial outputs [sum(counts), H]; this rank gets its own rows."""
        H = partial.shape[1]
        padded = partial.new_zeros(self.world, pad_to, H)
        start = 0
        for r in range(self.world):
            padded[r, : counts[r]] = partial[start:start + counts[r]]
            start += counts[r]
        mine = partial.new_empty(pad_to, H)
        if dist.get_backend(self.group) == "nccl":
            dist.reduce_scatter_tensor(mine, padded.view(self.world * pad_to, H), op=dist.ReduceOp.SUM, group=self.group)
        else:  # backends without a reduce-scatter: all-reduce, then keep this rank's slice
            dist.all_reduce(padded, op=dist.ReduceOp.SUM, group=self.group)
            mine = padded[self.rank]
        return mine[: counts[self.rank]]

    # -- one layer forward ---------------------------------------------------------------------------
    def forward(self, hidden_fp8: torch.Tensor, hidden_scale: torch.Tensor, router_logits: torch.Tensor) -> torch.Tensor:
        """This rank's tokens in (hidden_fp8 [T_r,H] as float8_e4m3fn or uint8 codes, hidden_scale [T_r,H/128] fp32,
        router_logits [T_r,E] fp32) -> bf16 [T_r,H], the full layer output for those tokens."""
        codes = hidden_fp8.view(torch.uint8) if hidden_fp8.dtype != torch.uint8 else hidden_fp8
        n = codes.shape[0]
        counts = self._gather_counts(n, codes.device)
        total, pad_to = sum(counts), max(max(counts), 1)
        if total == 0:
            return torch.empty(0, self.hidden, dtype=torch.bfloat16, device=codes.device)
        all_codes = self._all_gather_rows(codes, counts, pad_to)
        all_scale = self._all_gather_rows(hidden_scale, counts, pad_to)
        all_logits = self._all_gather_rows(router_logits, counts, pad_to)
        partial = self.local_forward(all_codes, all_scale, all_logits, self.local_expert_offset)
        mine = self._reduce_scatter_rows(partial.to(torch.float32), counts, pad_to)
        return mine.to(torch.bfloat16)


def cuda_local_forward(engine, weights: dict) -> Callable:
    """local_forward for ExpertParallelMoe that runs the CUDA library: `engine` is a binding.MoeFp8 sized for
    the gathered token count, `weights` holds this rank's routing_bias, w13, w13_scale, w2, w2_scale and
    scaling_factor (device tensors, as synthetic.make_inputs lays them out)."""

    def run(codes, scale, logits, local_expert_offset):
        inp = dict(weights, hidden_fp8=codes.contiguous(), hidden_scale=scale.contiguous(),
                   router_logits=logits.contiguous(), local_expert_offset=local_expert_offset)
        return engine.forward(inp)

    return run
