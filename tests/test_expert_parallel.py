"""Expert-parallel wrapper: the exchange steps around the layer (all-gather of tokens, reduce-scatter of the
partial outputs).  The host logic runs here as two gloo ranks on CPU with the CPU oracle standing in for the
local forward; on a GPU the kernel side of it (a forward per expert slice, partial outputs summed) is checked on
one device, and the collectives themselves with a one-rank NCCL group."""
import dataclasses
import os
import socket
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)
sys.path.insert(0, os.path.join(ROOT, "tests"))

import oracle  # noqa: E402
from paper_2608_14560_b200 import synthetic as syn  # noqa: E402
from paper_2608_14560_b200.expert_parallel import ExpertParallelMoe, cuda_local_forward  # noqa: E402

TINY = syn.LayerDims(hidden=256, intermediate=128, num_experts=16, num_local_experts=16, n_group=4, topk_group=2, top_k=2)


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _oracle_local_forward(host_weights, dims, el):
    """local_forward for the wrapper that evaluates this rank's expert slice with the CPU oracle."""

    def run(codes, scale, logits, off):
        inp = dict(host_weights, hidden_fp8=codes.numpy(), hidden_scale=scale.numpy(), router_logits=logits.numpy(),
                   local_expert_offset=off,
                   w13=host_weights["w13"][off:off + el], w13_scale=host_weights["w13_scale"][off:off + el],
                   w2=host_weights["w2"][off:off + el], w2_scale=host_weights["w2_scale"][off:off + el])
        bits = oracle.forward(inp, dims.n_group, dims.topk_group, dims.top_k)["out"]
        return torch.from_numpy(bits.view(np.int16)).view(torch.bfloat16)

    return run


def _ep_worker(rank, world, port, counts, q):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        wl = syn.Workload("ep", sum(counts), TINY, seed=7)
        inp = syn.make_inputs(wl)                      # every rank draws the same layer and the same tokens
        host = syn.to_host(inp)
        lo = sum(counts[:rank])
        mine = slice(lo, lo + counts[rank])
        el = TINY.num_experts // world
        ep = ExpertParallelMoe(_oracle_local_forward(host, TINY, el), TINY.hidden, TINY.num_experts, el)
        assert ep.local_expert_offset == rank * el
        out = ep.forward(inp["hidden_fp8"][mine], inp["hidden_scale"][mine], inp["router_logits"][mine])
        # the same tokens through the single-rank layer with every expert local
        ref = oracle.forward(host, TINY.n_group, TINY.topk_group, TINY.top_k, tokens=np.arange(lo, lo + counts[rank]))["out"]
        q.put((rank, out.view(torch.int16).numpy().view(np.uint16), ref))
        dist.barrier()
    finally:
        dist.destroy_process_group()


@pytest.mark.parametrize("counts", [(3, 5), (6, 0)])
def test_two_ranks_over_gloo_equal_the_single_rank_layer(counts):
    from parity import bf16_bits_to_f32
    world, port = 2, _free_port()
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_ep_worker, args=(r, world, port, counts, q)) for r in range(world)]
    for p in procs:
        p.start()
    got = sorted((q.get(timeout=180) for _ in range(world)), key=lambda x: x[0])
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, out, ref in got:
        assert out.shape == (counts[rank], TINY.hidden)
        g, r = bf16_bits_to_f32(out).astype(np.float64), bf16_bits_to_f32(ref).astype(np.float64)
        # partial outputs are rounded to bf16 before they are summed: a few bf16 ulps of the larger partials
        assert np.all(np.abs(g - r) <= 2e-2 * np.abs(r) + 2e-3), f"rank {rank}: max diff {np.abs(g - r).max()}"


def test_wrapper_rejects_a_slice_size_that_does_not_cover_the_experts():
    port = _free_port()
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=0, world_size=1)
    try:
        with pytest.raises(ValueError):
            ExpertParallelMoe(lambda *a: None, 256, 16, 8)
        ep = ExpertParallelMoe(lambda c, s, l, off: torch.zeros(c.shape[0], 256, dtype=torch.bfloat16), 256, 16, 16)
        out = ep.forward(torch.zeros(0, 256, dtype=torch.uint8), torch.zeros(0, 2), torch.zeros(0, 16))
        assert out.shape == (0, 256)
    finally:
        dist.destroy_process_group()


@pytest.mark.gpu
def test_expert_slices_on_one_gpu_sum_to_the_all_local_layer(cuda_device):
    """Eight expert slices of 32 (the offsets an 8-way expert-parallel job uses) run one after another on one
    device; their partial outputs, summed as the reduce-scatter would, against the oracle with all 256 local."""
    from parity import check_output, make_engine, oracle_forward_parallel
    dims = syn.LayerDims(hidden=512, intermediate=256, num_local_experts=256)
    wl = syn.Workload("ep_gpu", 200, dims, seed=17)
    inp = syn.make_inputs(wl, cuda_device)
    shard = dataclasses.replace(dims, num_local_experts=32)
    eng = make_engine(syn.Workload("s", 200, shard, 0), cuda_device)
    total = torch.zeros(200, 512, dtype=torch.float32, device=cuda_device)
    for r in range(8):
        sl = slice(32 * r, 32 * r + 32)
        w = {"routing_bias": inp["routing_bias"], "scaling_factor": inp["scaling_factor"],
             "w13": inp["w13"][sl].contiguous(), "w13_scale": inp["w13_scale"][sl].contiguous(),
             "w2": inp["w2"][sl].contiguous(), "w2_scale": inp["w2_scale"][sl].contiguous()}
        run = cuda_local_forward(eng, w)
        total += run(inp["hidden_fp8"], inp["hidden_scale"], inp["router_logits"], 32 * r).float()
    torch.cuda.synchronize()
    assert eng.status() == 0
    eng.close()
    ref = oracle_forward_parallel(syn.to_host(inp), dims, np.arange(200, dtype=np.int32))
    gpu = total.to(torch.bfloat16).view(torch.int16).cpu().numpy().view(np.uint16)
    check_output(gpu, ref)


@pytest.mark.gpu
def test_one_rank_nccl_group_runs_the_collectives_on_the_gpu(cuda_device):
    from parity import check_output, make_engine, oracle_forward_parallel
    dims = syn.LayerDims(hidden=512, intermediate=256, num_local_experts=256)
    wl = syn.Workload("ep_nccl", 96, dims, seed=18)
    inp = syn.make_inputs(wl, cuda_device)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(_free_port()))
    os.environ.setdefault("NCCL_NVLS_ENABLE", "0")
    torch.cuda.set_device(cuda_device)
    dist.init_process_group("nccl", rank=0, world_size=1, device_id=cuda_device)
    try:
        eng = make_engine(wl, cuda_device)
        w = {k: inp[k] for k in ("routing_bias", "scaling_factor", "w13", "w13_scale", "w2", "w2_scale")}
        ep = ExpertParallelMoe(cuda_local_forward(eng, w), dims.hidden, dims.num_experts, 256)
        out = ep.forward(inp["hidden_fp8"], inp["hidden_scale"], inp["router_logits"])
        torch.cuda.synchronize()
        assert eng.status() == 0
        eng.close()
    finally:
        dist.destroy_process_group()
    ref = oracle_forward_parallel(syn.to_host(inp), dims, np.arange(96, dtype=np.int32))
    check_output(out.view(torch.int16).cpu().numpy().view(np.uint16), ref)
