"""GPU parity: the CUDA path, called through the C ABI, against the CPU oracle
on the same seeded inputs.  Routing indices and the permutation are compared
bit for bit, the bf16 output with the tolerance of the workload definition."""
import dataclasses

import numpy as np
import pytest
import torch

import oracle
from paper_2608_14560_b200 import MoeFp8, MoeFp8Error
from paper_2608_14560_b200 import synthetic as syn

from parity import check_output, make_engine, run_and_compare

pytestmark = pytest.mark.gpu

SMALL = syn.LayerDims(hidden=512, intermediate=256, num_local_experts=32)


def _wl(tokens, dims=SMALL, seed=0, **kw):
    return syn.Workload(f"t{tokens}", tokens, dims, seed, **kw)


# ---- small layer, every token compared ------------------------------------
@pytest.mark.parametrize("tokens", [1, 7, 32, 33, 130, 512, 513, 1000])  # 512|513: launch-scheme boundary
def test_small_layer_all_tokens(cuda_device, tokens):
    st = run_and_compare(_wl(tokens, seed=tokens), cuda_device)
    assert st["frac"] >= 0.995


def test_small_layer_skewed_many_tiles_per_expert(cuda_device):
    # hot experts receive every token: several 128-row tiles per expert plus a ragged tail
    st = run_and_compare(_wl(1111, seed=9, skew=True), cuda_device)
    assert st["S"] > 4 * 1111


def test_all_experts_local(cuda_device):
    dims = dataclasses.replace(SMALL, num_local_experts=256)
    st = run_and_compare(_wl(333, dims, seed=5), cuda_device)
    assert st["S"] == 333 * 8


@pytest.mark.parametrize("off,eloc", [(32, 32), (224, 32), (5, 3), (0, 1)])
def test_local_expert_offsets(cuda_device, off, eloc):
    dims = dataclasses.replace(SMALL, num_local_experts=eloc)
    run_and_compare(_wl(200, dims, seed=off + eloc, local_expert_offset=off), cuda_device)


@pytest.mark.parametrize("tokens,eloc,off", [(9, 256, 0), (60, 256, 0), (80, 3, 5), (33, 1, 0), (70, 1, 7)])
def test_fused_small_batch_kernel_with_many_and_with_few_local_experts(cuda_device, tokens, eloc, off):
    # all experts local: a couple of hundred one- or two-row tiles; one local expert: every local row in one
    # expert, i.e. up to three sub-tiles of the same weights
    dims = dataclasses.replace(SMALL, num_local_experts=eloc)
    wl = _wl(tokens, dims, seed=300 + tokens + eloc, local_expert_offset=off)
    inp = syn.make_inputs(wl, cuda_device)
    eng = make_engine(wl, cuda_device)
    got = eng.forward(inp).clone()
    assert eng.last_launch_count() <= 2
    eng.set_small_batch_fusion(False)
    want = eng.forward(inp).clone()
    torch.cuda.synchronize()
    assert eng.status() == 0 and eng.last_launch_count() == 5
    assert torch.equal(got.view(torch.int16), want.view(torch.int16))
    eng.set_small_batch_fusion(True)
    run_and_compare(wl, cuda_device, inp=inp, eng=eng)
    eng.close()


def test_scale_layout_and_gate_order_flags(cuda_device):
    wl = _wl(97, seed=3)
    inp = syn.make_inputs(wl, cuda_device)
    inp_t = dict(inp, hidden_scale=inp["hidden_scale"].t().contiguous())
    run_and_compare(wl, cuda_device, inp=inp_t, hidden_scale_layout=1)
    I = wl.dims.intermediate
    inp_s = dict(inp, w13=torch.cat([inp["w13"][:, I:], inp["w13"][:, :I]], 1).contiguous(),
                 w13_scale=torch.cat([inp["w13_scale"][:, I // 128:], inp["w13_scale"][:, :I // 128]], 1).contiguous())
    run_and_compare(wl, cuda_device, inp=inp_s, gate_first=False)


# ---- degenerate cases -------------------------------------------------------
def test_zero_tokens_and_argument_errors(cuda_device):
    wl = _wl(0)
    inp = syn.make_inputs(wl, cuda_device)
    eng = make_engine(wl, cuda_device, max_tokens=16)
    out = eng.forward(inp)
    assert out.shape == (0, 512) and eng.last_launch_count() == 0
    big = syn.make_inputs(_wl(17), cuda_device)
    with pytest.raises(MoeFp8Error) as ei:
        eng.forward(big)  # T > max_tokens
    assert ei.value.rc == -1
    with pytest.raises(MoeFp8Error):
        eng.forward(dict(syn.make_inputs(_wl(4), cuda_device), local_expert_offset=250))
    with pytest.raises(MoeFp8Error):
        MoeFp8(hidden=500, device=cuda_device)
    eng.close()


def test_no_token_routes_locally(cuda_device):
    wl = _wl(64, seed=1)
    inp = syn.make_inputs(wl, cuda_device)
    inp["router_logits"][:, :32] = -20.0  # local experts (group 0) never win
    st = run_and_compare(wl, cuda_device, inp=inp)
    assert st["S"] == 0


def test_every_token_on_the_same_experts(cuda_device):
    wl = _wl(300, seed=2)
    inp = syn.make_inputs(wl, cuda_device)
    inp["router_logits"][:] = -8.0
    inp["router_logits"][:, [1, 2, 3, 4, 40, 41, 80, 120]] = 6.0
    st = run_and_compare(wl, cuda_device, inp=inp)
    assert st["S"] == 4 * 300 and st["active"] == 4


def test_exact_score_ties_break_to_smaller_index(cuda_device):
    wl = _wl(50, seed=4)
    inp = syn.make_inputs(wl, cuda_device)
    inp["router_logits"][:] = 0.25
    inp["routing_bias"][:] = 0
    run_and_compare(wl, cuda_device, inp=inp)
    inp["router_logits"][:, 128:] = 0.5  # ties inside and across groups 4..7
    run_and_compare(wl, cuda_device, inp=inp)


def test_run_to_run_determinism_and_workspace_reuse(cuda_device):
    wl = _wl(500, seed=6)
    inp = syn.make_inputs(wl, cuda_device)
    eng = make_engine(wl, cuda_device, max_tokens=600)
    a = eng.forward(inp).clone()
    other = syn.make_inputs(_wl(77, seed=8), cuda_device)
    eng.forward(other)  # different T in between: stale scratch must not leak
    b = eng.forward(inp).clone()
    torch.cuda.synchronize()
    assert torch.equal(a.view(torch.int16), b.view(torch.int16))
    run_and_compare(_wl(77, seed=8), cuda_device, inp=other, eng=eng)
    eng.close()


def test_many_batch_sizes_back_to_back_on_one_handle(cuda_device):
    # 600 forwards in random order over batch sizes on both sides of every launch-scheme boundary: the counters
    # and scratch a forward leaves behind must never change the next one (bit-identical outputs, clean status)
    sizes = [1, 8, 32, 33, 128, 129, 512, 513, 700, 2048, 2049]
    inputs = {T: syn.make_inputs(_wl(T, seed=300 + T, skew=(T % 3 == 0)), cuda_device) for T in sizes}
    eng = make_engine(_wl(max(sizes)), cuda_device)
    want = {T: eng.forward(inputs[T]).clone() for T in sizes}
    torch.cuda.synchronize()
    assert eng.status() == 0
    order = np.random.default_rng(5).choice(len(sizes), 600)
    for i, k in enumerate(order):
        T = sizes[k]
        got = eng.forward(inputs[T])
        if i % 20 == 19:
            assert torch.equal(got.view(torch.int16), want[T].view(torch.int16)), f"forward {i}, T={T}"
            assert eng.status() == 0
    run_and_compare(_wl(129, seed=300 + 129, skew=True), cuda_device, inp=inputs[129], eng=eng)
    eng.close()


def test_host_entry_point_matches_device_entry_point(cuda_device):
    wl = _wl(260, seed=12)
    inp = syn.make_inputs(wl, cuda_device)
    eng = make_engine(wl, cuda_device)
    ref = eng.forward(inp).cpu()
    host_act = {k: inp[k].cpu().pin_memory() for k in ("hidden_fp8", "hidden_scale", "router_logits")}
    host_out = torch.empty(wl.tokens, 512, dtype=torch.bfloat16).pin_memory()
    eng.forward_host(host_act, inp, host_out)
    assert torch.equal(ref.view(torch.int16), host_out.view(torch.int16))
    eng.close()


def test_forward_on_a_side_stream_and_after_a_change_of_weights(cuda_device):
    # the forward is enqueued on the caller's current stream; the TMA descriptors of the weights are cached
    # per pointer pair and must be rebuilt when other weight tensors are passed
    wl = _wl(150, seed=21)
    inp_a = syn.make_inputs(wl, cuda_device)
    inp_b = syn.make_inputs(_wl(150, seed=22), cuda_device)
    fresh = make_engine(wl, cuda_device)
    want_b = fresh.forward(inp_b).clone()
    fresh.close()
    eng = make_engine(wl, cuda_device)
    side = torch.cuda.Stream(device=cuda_device)
    side.wait_stream(torch.cuda.current_stream(cuda_device))
    with torch.cuda.stream(side):
        eng.forward(inp_a)
        got_b = eng.forward(inp_b).clone()
    side.synchronize()
    assert eng.status() == 0
    assert torch.equal(want_b.view(torch.int16), got_b.view(torch.int16))
    run_and_compare(wl, cuda_device, inp=inp_a, eng=eng)
    eng.close()


# ---- the five benchmark workloads at full size -----------------------------
def _sample(T, n, seed):
    if T <= n:
        return None
    return np.sort(np.random.default_rng(seed).choice(T, n, replace=False)).astype(np.int32)


# Output: every token up to T = 1024, else 256 random tokens.  Per-slot rows (re-quantised intermediate and
# down-projection row): on the large workloads every row of the first and the last row tile of the largest
# expert segment, of the smallest non-empty segment and of the first tile of a median one -- whole tiles at the
# full K depth, on CTAs that have walked many tiles before them.
@pytest.mark.parametrize("cfg,n_sample,rows", [(0, 8, True), (1, 64, True), (2, 1024, "tiles"), (3, 256, "tiles")])
def test_benchmark_workloads_32_local_experts(cuda_device, cfg, n_sample, rows):
    wl = syn.CONFIGS[cfg]
    st = run_and_compare(wl, cuda_device, sample_tokens=_sample(wl.tokens, n_sample, cfg), check_rows=rows)
    print(wl.name, st)


@pytest.mark.parametrize("tokens,n_sample,rows", [(7, 7, True), (54, 54, True), (14107, 256, "tiles")])
def test_token_counts_quoted_in_the_paper(cuda_device, tokens, n_sample, rows):
    # the paper's table of workload regimes (short / median / long) quotes one latency each for T = 7, 54 and
    # 14107 tokens with 32 local experts
    base = syn.CONFIGS[1]
    wl = syn.Workload(f"dsv3_T{tokens}_E32", tokens, base.dims, base.seed, base.local_expert_offset,
                      base.scaling_factor, base.skew)
    st = run_and_compare(wl, cuda_device, sample_tokens=_sample(tokens, n_sample, tokens), check_rows=rows)
    print(wl.name, st)


def test_benchmark_workload_all_256_experts_local(cuda_device):
    wl = syn.CONFIGS[4]
    st = run_and_compare(wl, cuda_device, sample_tokens=_sample(wl.tokens, 256, 4), check_rows="tiles")
    assert st["S"] == wl.tokens * 8
    print(wl.name, st)


def test_routing_on_logits_far_outside_the_unit_range(cuda_device):
    # the fixed-operation sigmoid on its clamped tails and at large |logit|: indices and weights of the
    # kernel must equal the oracle's bit for bit there too, not only on N(0,1) logits
    wl = _wl(256, seed=31)
    inp = syn.make_inputs(wl, cuda_device)
    g = torch.Generator(device=cuda_device)
    g.manual_seed(77)
    mags = torch.tensor([8.0, 20.0, 87.0, 88.0, 100.0, 1e4, 0.015625, 3.0], device=cuda_device)
    pick = torch.randint(0, len(mags), inp["router_logits"].shape, generator=g, device=cuda_device)
    sign = torch.randint(0, 2, inp["router_logits"].shape, generator=g, device=cuda_device) * 2.0 - 1.0
    inp["router_logits"] = (mags[pick] * sign).contiguous()
    run_and_compare(wl, cuda_device, inp=inp)
    # a dense sweep of the benchmark's 1/64 grid over [-32, 32] and of large magnitudes, one value per expert column
    T = 4096 // 256 * 2
    grid = (torch.arange(-2048, 2048, device=cuda_device, dtype=torch.float32) / 64.0).view(-1, 256)
    big = (torch.arange(-2048, 2048, device=cuda_device, dtype=torch.float32) / 16.0).view(-1, 256)
    wl2 = _wl(T, seed=32)
    inp2 = syn.make_inputs(wl2, cuda_device)
    inp2["router_logits"] = torch.cat([grid, big]).contiguous()
    run_and_compare(wl2, cuda_device, inp=inp2)


def test_device_sigmoid_bits_equal_the_oracle(cuda_device):
    # every point of the benchmark's logit grid (k/64, |k| <= 2048), the clamp boundaries and 2^20 random
    # floats over the whole finite range: the kernel's sigmoid and the oracle's agree in every bit
    from paper_2608_14560_b200 import binding
    rng = np.random.default_rng(11)
    grid = (np.arange(-2048, 2049) / 64.0).astype(np.float32)
    edge = np.float32([0.0, -0.0, 87.0, -87.0, 88.0, -88.0, 88.5, -88.5, 100.0, -100.0, 1e4, -1e4, 3e38, -3e38,
                       1e-30, -1e-30, 1e-45, 0.34657359, -0.34657359])
    rnd_bits = rng.integers(0, 1 << 32, 1 << 20, dtype=np.uint64).astype(np.uint32)
    rnd = rnd_bits.view(np.float32)
    rnd = rnd[np.isfinite(rnd)]
    mid = (rng.standard_normal(1 << 18) * 6.0).astype(np.float32)
    x = np.concatenate([grid, edge, rnd, mid]).astype(np.float32)
    got = binding.debug_sigmoid(torch.from_numpy(x).to(cuda_device)).cpu().numpy()
    want = oracle.sigmoid(x)
    assert np.array_equal(got.view(np.uint32), want.view(np.uint32)), \
        f"{(got.view(np.uint32) != want.view(np.uint32)).sum()} of {x.size} sigmoid values differ"


def test_a_wait_that_runs_out_is_reported_and_the_handle_stays_usable(cuda_device):
    # The copy producer of GEMM1 is told to stop before its third pipeline stage and every wait limit is
    # shortened to 2^20 clocks: the consumers' waits give up, the kernel returns with a time-out code in the
    # status word (nothing traps, nothing spins without a bound), and the next forward on the same handle,
    # with the hook off again, is bit-identical to a forward on a fresh handle.
    wl = _wl(300, seed=41)
    inp = syn.make_inputs(wl, cuda_device)
    fresh = make_engine(wl, cuda_device)
    want = fresh.forward(inp).clone()
    torch.cuda.synchronize()
    fresh.close()
    eng = make_engine(wl, cuda_device)
    eng.debug_set_fault(skip_iteration=2, wait_clocks=1 << 20)
    eng.forward(inp)
    torch.cuda.synchronize()
    assert 1 <= eng.status() <= 5, f"expected a time-out code, got {eng.status()}"
    eng.debug_set_fault(-1, 0)
    got = eng.forward(inp).clone()
    torch.cuda.synchronize()
    assert eng.status() == 0
    assert torch.equal(got.view(torch.int16), want.view(torch.int16))
    run_and_compare(wl, cuda_device, inp=inp, eng=eng)
    eng.close()


# ---- the layer started from bf16 hidden states (router projection + input quantisation in front) ----------
def _from_hidden_case(wl, device, sample_tokens=None, **kw):
    d = wl.dims
    inp = syn.make_inputs(wl, device)
    r = syn.make_router_inputs(wl, device)
    eng = make_engine(wl, device, **kw)
    out = eng.forward_from_hidden({**inp, **r})
    fed = eng.debug_export_inputs(wl.tokens)
    dbg = eng.debug_export(wl.tokens, rows=False)
    torch.cuda.synchronize()
    assert int(dbg["status"].item()) == 0
    host = syn.to_host({**inp, **r})
    # projection and quantisation: bit for bit (the summation order of the projection is part of its definition)
    logits = oracle.router_logits(host["hidden_bf16"], host["router_weight"])
    assert np.array_equal(fed["router_logits"].cpu().numpy().view(np.uint32), logits.view(np.uint32)), \
        "router logits differ from the oracle's fixed-order sum"
    q, s = oracle.quantize_rows(host["hidden_bf16"])
    assert np.array_equal(fed["hidden_fp8"].cpu().numpy(), q)
    gs = fed["hidden_scale"].cpu().numpy()
    assert np.array_equal(gs.T if eng.cfg.hidden_scale_layout else gs, s)
    # routing from those logits: indices and weights bit for bit
    ridx, rw = oracle.route(logits, host["routing_bias"], d.n_group, d.topk_group, d.top_k, float(inp["scaling_factor"]))
    assert np.array_equal(dbg["topk_idx"].cpu().numpy(), ridx)
    assert np.array_equal(dbg["topk_w"].cpu().numpy(), rw)
    # output
    tokens = np.arange(wl.tokens, dtype=np.int32) if sample_tokens is None else sample_tokens
    full = dict(host, hidden_fp8=q, hidden_scale=s, router_logits=logits)
    from parity import oracle_forward_parallel
    ref = oracle_forward_parallel(full, d, tokens)
    gpu = out.view(torch.int16).cpu().numpy().view(np.uint16)[tokens]
    check_output(gpu, ref)
    eng.close()
    return int(((ridx >= wl.local_expert_offset) & (ridx < wl.local_expert_offset + d.num_local_experts)).sum())


@pytest.mark.parametrize("tokens", [1, 8, 33, 128, 129, 700])  # 128 | 129: the two projection tile shapes
def test_from_hidden_small_layer(cuda_device, tokens):
    _from_hidden_case(_wl(tokens, seed=60 + tokens), cuda_device)


def test_from_hidden_transposed_scale_layout(cuda_device):
    _from_hidden_case(_wl(77, seed=59), cuda_device, hidden_scale_layout=1)


@pytest.mark.parametrize("cfg,n_sample", [(1, 64), (2, 128)])
def test_from_hidden_benchmark_shapes(cuda_device, cfg, n_sample):
    wl = syn.CONFIGS[cfg]
    S = _from_hidden_case(wl, cuda_device, sample_tokens=_sample(wl.tokens, n_sample, cfg))
    assert S > 0


# ---- batches of at most 4 tokens: GEMM1's K range of every tile cut over several CTAs ------------------------
@pytest.mark.parametrize("tokens,eloc,off,seed", [(1, 32, 0, 3), (2, 32, 0, 1), (3, 32, 0, 2), (4, 32, 0, 0), (4, 1, 7, 5),
                                                  (4, 3, 5, 6), (4, 256, 0, 7), (1, 256, 0, 8)])
def test_k_split_of_very_small_batches_is_bit_identical(cuda_device, tokens, eloc, off, seed):
    # few tiles (the split is used) and, with all 256 experts local, many tiles (it is not); the full-size layer
    # has 56 K-blocks per GEMM1 tile, i.e. parts of 7 to 28 K-blocks
    dims = dataclasses.replace(syn.CONFIGS[0].dims, num_local_experts=eloc) if eloc <= 32 else dataclasses.replace(SMALL, num_local_experts=eloc)
    wl = syn.Workload(f"k{tokens}", tokens, dims, 700 + seed, local_expert_offset=off)
    inp = syn.make_inputs(wl, cuda_device)
    eng = make_engine(wl, cuda_device)
    eng.debug_set_k_split(False)
    want = eng.forward(inp).clone()
    eng.debug_set_k_split(True)
    for _ in range(3):  # the part counters of one forward must not disturb the next
        got = eng.forward(inp).clone()
    torch.cuda.synchronize()
    assert eng.status() == 0 and eng.last_launch_count() == 1
    assert torch.equal(got.view(torch.int16), want.view(torch.int16))
    run_and_compare(wl, cuda_device, inp=inp, eng=eng)
    eng.close()


# ---- row tiles of at most 32 rows inside the large-tile GEMM kernels: weights on the M side of the MMAs ------
@pytest.mark.parametrize("tokens,kw", [(100, {}), (200, {"skew": True}), (700, {}), (1111, {"skew": True}),
                                       (3000, {"local_expert_offset": 160})])
def test_short_row_tiles_are_bit_identical_to_full_row_tiles(cuda_device, tokens, kw):
    # the same forward with every row tile worked on as a full 128-row tile (hook off) and with the short ones
    # (an expert's last tile of at most 32 rows) taken the other way round, full and short tiles interleaved
    # in every CTA's work list
    wl = _wl(tokens, seed=500 + tokens, **kw)
    inp = syn.make_inputs(wl, cuda_device)
    eng = make_engine(wl, cuda_device)
    eng.debug_set_short_tiles(0)
    want = eng.forward(inp).clone()
    eng.debug_set_short_tiles(1)
    got = eng.forward(inp).clone()
    torch.cuda.synchronize()
    assert eng.status() == 0
    assert torch.equal(got.view(torch.int16), want.view(torch.int16))
    dbg = eng.debug_export(tokens, rows=False)
    counts = dbg["expert_count"].cpu().numpy()
    assert ((counts % 128 > 0) & (counts % 128 <= 32)).any(), "no short row tile in this workload"
    run_and_compare(wl, cuda_device, inp=inp, eng=eng)
    eng.close()


# ---- batches of at most 80 tokens: gather, both GEMMs and the combine as one kernel; up to 16 tokens that ----
# ---- kernel also routes and permutes (every CTA for itself), and the forward is a single launch -------------
@pytest.mark.parametrize("tokens,kw", [(1, {}), (5, {}), (12, {}), (13, {}), (16, {"local_expert_offset": 64}),
                                       (17, {}), (32, {}), (23, {"skew": True}), (33, {}), (64, {"skew": True}),
                                       (80, {}), (80, {"skew": True, "local_expert_offset": 32})])
def test_fused_small_batch_kernel_is_bit_identical_to_the_separate_kernels(cuda_device, tokens, kw):
    wl = _wl(tokens, seed=80 + tokens, **kw)
    inp = syn.make_inputs(wl, cuda_device)
    eng = make_engine(wl, cuda_device)
    eng.set_small_batch_fusion(False)
    want = eng.forward(inp).clone()
    n_sep = eng.last_launch_count()
    eng.set_small_batch_fusion(True)
    got = eng.forward(inp).clone()
    torch.cuda.synchronize()
    assert eng.status() == 0
    assert eng.last_launch_count() == (1 if tokens <= 16 else 2) and n_sep == 5
    assert torch.equal(got.view(torch.int16), want.view(torch.int16))
    run_and_compare(wl, cuda_device, inp=inp, eng=eng)
    eng.close()


def test_fused_small_batch_kernel_transposed_scales_and_full_size_layer(cuda_device):
    wl = _wl(19, seed=90)
    inp = syn.make_inputs(wl, cuda_device)
    run_and_compare(wl, cuda_device, inp=dict(inp, hidden_scale=inp["hidden_scale"].t().contiguous()), hidden_scale_layout=1)
    base = syn.CONFIGS[0]
    for tokens in (1, 16, 32, 64):
        wl = syn.Workload(f"dsv3_T{tokens}_E32", tokens, base.dims, base.seed + tokens)
        inp = syn.make_inputs(wl, cuda_device)
        eng = make_engine(wl, cuda_device)
        eng.set_small_batch_fusion(False)
        want = eng.forward(inp).clone()
        eng.set_small_batch_fusion(True)
        for _ in range(3):  # counters left by one forward must not disturb the next
            got = eng.forward(inp).clone()
        torch.cuda.synchronize()
        assert eng.status() == 0
        assert torch.equal(got.view(torch.int16), want.view(torch.int16))
        run_and_compare(wl, cuda_device, inp=inp, eng=eng)
        eng.close()


@pytest.mark.parametrize("tokens,kw", [(200, {"skew": True}), (256, {}), (130, {"skew": True, "local_expert_offset": 96})])
def test_fused_kernel_with_a_raised_limit_cuts_experts_into_sub_tiles(cuda_device, tokens, kw):
    # beyond the default limit the caller may still ask for the fused kernel (up to 256 tokens): experts with
    # more than 32 rows are then worked on as several sub-tiles of 32 rows
    wl = _wl(tokens, seed=170 + tokens, **kw)
    inp = syn.make_inputs(wl, cuda_device)
    eng = make_engine(wl, cuda_device)
    want = eng.forward(inp).clone()
    assert eng.last_launch_count() == 5
    eng.set_small_batch_fusion(256)
    got = eng.forward(inp).clone()
    torch.cuda.synchronize()
    assert eng.status() == 0 and eng.last_launch_count() == 2
    assert torch.equal(got.view(torch.int16), want.view(torch.int16))
    dbg = run_and_compare(wl, cuda_device, inp=inp, eng=eng)
    eng.close()


@pytest.mark.parametrize("tokens,launches,eloc", [(16, 1, 32), (48, 2, 32), (3, 1, 256)])  # 3 tokens: K split
def test_a_wait_that_runs_out_in_the_fused_small_batch_kernel(cuda_device, tokens, launches, eloc):
    wl = _wl(tokens, dataclasses.replace(SMALL, num_local_experts=eloc), seed=43)
    inp = syn.make_inputs(wl, cuda_device)
    eng = make_engine(wl, cuda_device)
    want = eng.forward(inp).clone()
    torch.cuda.synchronize()
    assert eng.status() == 0 and eng.last_launch_count() == launches
    eng.debug_set_fault(skip_iteration=1, wait_clocks=1 << 20)
    eng.forward(inp)
    torch.cuda.synchronize()
    assert eng.status() in (1, 2, 3, 4, 5, 8), f"expected a time-out code, got {eng.status()}"
    eng.debug_set_fault(-1, 0)
    # the aborted call left its counters half counted; the calls after it alternate between the two counter
    # sets, each zeroing the other one, so all of them must be right
    for _ in range(4):
        got = eng.forward(inp).clone()
        torch.cuda.synchronize()
        assert eng.status() == 0
        assert torch.equal(got.view(torch.int16), want.view(torch.int16))
    eng.close()


def test_small_batches_of_changing_size_share_the_alternating_counters(cuda_device):
    # one handle, batch sizes on both sides of every launch scheme (one launch, routing kernel + fused kernel,
    # separate kernels) in turn: what one forward leaves in the workspace must not reach the next
    sizes = [7, 30, 3, 90, 16, 17, 1, 80, 12, 81, 9, 40]
    base = _wl(max(sizes), seed=47)
    inp = syn.make_inputs(base, cuda_device)
    eng = make_engine(base, cuda_device)
    ref = make_engine(base, cuda_device)
    ref.set_small_batch_fusion(False)
    for t in sizes:
        part = dict(inp, hidden_fp8=inp["hidden_fp8"][:t].contiguous(), hidden_scale=inp["hidden_scale"][:t].contiguous(),
                    router_logits=inp["router_logits"][:t].contiguous())
        got = eng.forward(part).clone()
        want = ref.forward(part).clone()
        torch.cuda.synchronize()
        assert eng.status() == 0 and ref.status() == 0
        assert eng.last_launch_count() == (1 if t <= 16 else 2 if t <= 80 else 5), t
        assert torch.equal(got.view(torch.int16), want.view(torch.int16)), t
    eng.close()
    ref.close()


def test_every_token_count_of_the_bench_sweep(cuda_device):
    # the token counts bench.py times on the 32-local-expert layer (the paper's three batch-size regimes), one
    # set of weights: routing and permutation on all tokens, the output on up to 48 sampled tokens each
    import bench
    base = syn.CONFIGS[1]
    ts = sorted(bench.SWEEP_TOKENS)
    big = syn.Workload("sweep", ts[-1], base.dims, base.seed)
    inp = syn.make_inputs(big, cuda_device)
    eng = make_engine(big, cuda_device, poison=False)
    for t in ts:
        wl = syn.Workload(f"dsv3_T{t}_E32", t, base.dims, base.seed)
        sub = {k: (v[:t] if k in ("hidden_fp8", "hidden_scale", "router_logits") else v) for k, v in inp.items()}
        st = run_and_compare(wl, cuda_device, inp=sub, sample_tokens=_sample(t, 48, t), check_rows=False, eng=eng)
        assert st["frac"] >= 0.995
    eng.close()


@pytest.mark.parametrize("tokens", [300, 40, 9])  # separate kernels | fused behind the routing kernel | one launch
def test_pipelined_host_entry_point_matches_device_entry_point(cuda_device, tokens):
    # five steps through moe_fp8_forward_host_async with three different batches in rotation (two staging sets
    # alternate inside the library): every step's host result equals the device-buffer forward of its batch
    wl = _wl(tokens, seed=13)
    batches = [syn.make_inputs(_wl(tokens, seed=13 + i), cuda_device) for i in range(3)]
    weights = batches[0]
    eng = make_engine(wl, cuda_device)
    want = []
    for b in batches:
        want.append(eng.forward({**weights, **{k: b[k] for k in ("hidden_fp8", "hidden_scale", "router_logits")}}).cpu())
    host_acts = [{k: b[k].cpu().pin_memory() for k in ("hidden_fp8", "hidden_scale", "router_logits")} for b in batches]
    host_outs = [torch.empty(tokens, 512, dtype=torch.bfloat16).pin_memory() for _ in range(5)]
    for i in range(5):
        eng.forward_host_async(host_acts[i % 3], weights, host_outs[i])
    eng.host_sync()
    assert eng.status() == 0
    for i in range(5):
        assert torch.equal(host_outs[i].view(torch.int16), want[i % 3].view(torch.int16)), f"step {i}"
    eng.close()


def test_a_batch_of_65536_tokens(cuda_device):
    # four times the largest benchmark batch: 528 352 padded rows, byte offsets beyond 2^32 in every row buffer
    base = syn.CONFIGS[1]
    wl = syn.Workload("dsv3_T65536_E32", 65536, base.dims, seed=65)
    st = run_and_compare(wl, cuda_device, sample_tokens=_sample(65536, 96, 65), check_rows="tiles", poison=False)
    assert st["S"] > 30000
