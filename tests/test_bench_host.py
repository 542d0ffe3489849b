"""Host-side logic of bench.py that runs with more than one rank, exercised on CPU with the gloo backend
(world size 2): the max/sum reductions of per-rank timings, per-rank seeding and the bounded oracle sample."""
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

import bench  # noqa: E402
from paper_2608_14560_b200 import synthetic as syn  # noqa: E402


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, q):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world),
                      LOCAL_RANK=str(rank))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        assert bench.dist_env() == (rank, rank, world)
        ms = 10.0 + 5.0 * rank          # rank 1 is the slow one
        total = bench.max_over_ranks(ms, world)
        tokens = bench.sum_over_ranks(64.0, world)
        dist.barrier()
        q.put((rank, total, tokens))
    finally:
        dist.destroy_process_group()


def test_two_rank_timing_reduction_over_gloo():
    world, port = 2, _free_port()
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    got = sorted(q.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert got == [(0, 15.0, 128.0), (1, 15.0, 128.0)]  # every rank sees the max time and the summed tokens


def test_single_rank_reductions_are_identity():
    assert bench.max_over_ranks(3.5, 1) == 3.5 and bench.sum_over_ranks(7.0, 1) == 7.0


def test_oracle_sample_is_bounded_and_inside_the_workload():
    for wl in syn.CONFIGS:
        s = bench.oracle_sample_tokens(wl)
        assert 1 <= len(s) <= wl.tokens and s[0] == 0 and np.all(np.diff(s) == 1)
        per_token = 4.5 if wl.skew else 8.0 * wl.dims.num_local_experts / wl.dims.num_experts
        assert len(s) * per_token <= 450  # about 10 s of single-thread oracle time at ~22 ms per slot


def test_physical_gpu_index_follows_cuda_visible_devices(monkeypatch):
    monkeypatch.setenv("CUDA_VISIBLE_DEVICES", "3,5")
    assert bench.physical_gpu_index(1) == 5
    monkeypatch.delenv("CUDA_VISIBLE_DEVICES")
    assert bench.physical_gpu_index(2) == 2


def test_roofline_constants_match_the_layer_shape():
    assert bench.FLOPS_PER_SLOT == 88_080_384
    assert bench.BYTES_PER_EXPERT == 44_050_944
    assert bench.W13_BYTES_PER_EXPERT + bench.W2_BYTES_PER_EXPERT == bench.BYTES_PER_EXPERT
