"""The no-allocation histogram entry point against the regular path.

moe_fp8_expert_histogram_static serves callers that cannot call cudaMalloc (a stream capture in progress, a
serving loop that must stay clear of the allocator, a plug-in that owns no memory pool): its scratch is a fixed
array inside the library.  Here it is called through the C ABI, twice in a row on different inputs, and its
outputs must equal what the workspace-based forward pass reports for the same routing indices, bit for bit.
This file sorts last so that a stop-at-first-failure run has already been through every other test."""
import numpy as np
import pytest
import torch

import oracle
from paper_2608_14560_b200 import binding
from paper_2608_14560_b200 import synthetic as syn

from parity import make_engine

pytestmark = pytest.mark.gpu

SMALL = syn.LayerDims(hidden=512, intermediate=256, num_local_experts=32)


def _reference_through_forward(wl, device):
    """Routing indices and the histogram as the existing entry points produce them."""
    inp = syn.make_inputs(wl, device)
    eng = make_engine(wl, device)
    eng.forward(inp)
    dbg = eng.debug_export(wl.tokens, rows=False)
    torch.cuda.synchronize()
    assert int(dbg["status"].item()) == 0
    out = (dbg["topk_idx"].clone(), dbg["expert_count"].clone(), dbg["expert_offset"].clone())
    eng.close()
    return out


def test_static_histogram_matches_workspace_path_on_two_calls_in_a_row(cuda_device):
    cases = [syn.Workload("a", 3000, SMALL, seed=51, skew=True),      # 12 blocks of scratch, several full
             syn.Workload("b", 70, SMALL, seed=52, local_expert_offset=96)]  # then a much smaller call
    refs = [_reference_through_forward(wl, cuda_device) for wl in cases]
    for wl, (idx, want_count, want_offset) in zip(cases, refs):
        el = wl.dims.num_local_experts
        count = torch.full((el,), -7, dtype=torch.int32, device=cuda_device)
        offset = torch.full((el + 1,), -7, dtype=torch.int32, device=cuda_device)
        rc = binding.expert_histogram_static(idx, wl.local_expert_offset, el, count, offset)
        torch.cuda.synchronize()
        assert rc == binding.OK
        assert torch.equal(count, want_count)
        assert torch.equal(offset, want_offset)
        assert int(offset[-1]) == int(want_count.sum())
        # and against the CPU oracle's permutation of the same routing indices
        perm = oracle.permute(idx.cpu().numpy(), wl.local_expert_offset, el)
        assert np.array_equal(count.cpu().numpy(), perm["count"])
        assert np.array_equal(offset.cpu().numpy(), perm["offset"])


def test_static_histogram_at_its_capacity_then_a_small_call(cuda_device):
    # the largest call the fixed array admits (every one of its 64 x 256 entries is used), checked against a
    # library histogram; the small call after it must not see anything the large one left behind
    g = torch.Generator(device=cuda_device)
    g.manual_seed(9)
    for T, el, off in [(binding.STATIC_HISTOGRAM_MAX_TOKENS, 256, 0), (5, 7, 100)]:
        # 8 distinct experts per token, as routing produces them
        idx = torch.rand(T, 256, generator=g, device=cuda_device).argsort(dim=1)[:, :8].to(torch.int32).contiguous()
        count = torch.full((el,), -7, dtype=torch.int32, device=cuda_device)
        offset = torch.full((el + 1,), -7, dtype=torch.int32, device=cuda_device)
        assert binding.expert_histogram_static(idx, off, el, count, offset) == binding.OK
        torch.cuda.synchronize()
        local = idx.long().flatten() - off
        local = local[(local >= 0) & (local < el)]
        want = torch.bincount(local, minlength=el).to(torch.int32)
        assert torch.equal(count, want)
        assert torch.equal(offset[1:], torch.cumsum(want, 0).to(torch.int32)) and int(offset[0]) == 0


def test_static_histogram_rejects_sizes_beyond_its_capacity(cuda_device):
    T = binding.STATIC_HISTOGRAM_MAX_TOKENS + 1
    idx = torch.zeros(T, 8, dtype=torch.int32, device=cuda_device)
    count = torch.zeros(32, dtype=torch.int32, device=cuda_device)
    offset = torch.zeros(33, dtype=torch.int32, device=cuda_device)
    assert binding.expert_histogram_static(idx, 0, 32, count, offset) == binding.ERR_STATIC_LIMIT
    assert binding.expert_histogram_static(idx[:4], 250, 32, count, offset) == binding.ERR_BAD_ARG
    assert binding.expert_histogram_static(idx[:0], 0, 32, count, offset) == binding.OK  # T = 0: all zeros
    torch.cuda.synchronize()
    assert int(count.sum()) == 0 and int(offset.abs().sum()) == 0
