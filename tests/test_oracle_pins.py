"""Pins for the CPU oracle: each part is checked against something other than
its own formula (library conversions, fp64 library routines, closed forms,
hand-worked values, brute force, invariants).  No GPU."""
import math
import os

import numpy as np
import pytest
import torch

import oracle
from paper_2608_14560_b200 import synthetic as syn

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


# --------------------------------------------------------------------------
# number formats
# --------------------------------------------------------------------------
def test_e4m3_decode_all_codes_vs_torch():
    codes = np.arange(256, dtype=np.uint8)
    mine = oracle.e4m3_decode(codes)
    ref = torch.from_numpy(codes).view(torch.float8_e4m3fn).to(torch.float32).numpy()
    assert np.array_equal(np.isnan(mine), np.isnan(ref))
    ok = ~np.isnan(ref)
    assert np.array_equal(mine[ok].view(np.uint32), ref[ok].view(np.uint32))
    assert mine[0x7E] == 448.0 and mine[0x08] == 2.0 ** -6 and mine[0x01] == 2.0 ** -9


def test_e4m3_encode_vs_torch_values_midpoints_boundary():
    codes = np.array([c for c in range(256) if (c & 0x7F) != 0x7F], dtype=np.uint8)
    vals = torch.from_numpy(codes).view(torch.float8_e4m3fn).to(torch.float32).numpy()
    pos = np.sort(vals[vals >= 0])
    mids = (pos[:-1] + pos[1:]) / 2  # exact in fp32
    eps = np.concatenate([np.nextafter(mids, np.float32(np.inf)), np.nextafter(mids, np.float32(-np.inf))])
    rng = np.random.default_rng(0)
    rnd = (rng.standard_normal(20000) * rng.choice([1e-3, 0.05, 1.0, 30.0, 150.0], 20000)).astype(np.float32)
    rnd = rnd[np.abs(rnd) <= 464.0]
    x = np.concatenate([vals, mids, -mids, eps, -eps, rnd, np.float32([448.0, 449.0, 463.9, 464.0, -464.0, 0.0, -0.0])])
    x = x.astype(np.float32)
    mine = oracle.e4m3_encode(x)
    ref = torch.from_numpy(x).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    assert np.array_equal(mine, ref)
    # round trip of every finite code
    assert np.array_equal(oracle.e4m3_encode(vals), codes)
    # the oracle's own rule above the library's range: saturate to +-448
    assert oracle.e4m3_encode(np.float32([465.0, 1e6, -500.0, np.inf])).tolist() == [0x7E, 0x7E, 0xFE, 0x7E]


def test_bf16_vs_torch():
    rng = np.random.default_rng(1)
    x = np.concatenate([rng.standard_normal(50000).astype(np.float32) * 10,
                        np.float32([0.0, -0.0, 1.0, 1.00390625, 1.01171875, 3.0e38, 1e-40])])
    # exact ties between two bf16 neighbours
    base = (rng.integers(0x3000, 0x4800, 2000).astype(np.uint32) << 16) | 0x8000
    x = np.concatenate([x, base.view(np.float32)])
    mine = oracle.bf16_encode(x)
    ref = torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(mine, ref)
    assert np.array_equal(oracle.bf16_decode(ref), torch.from_numpy(x).to(torch.bfloat16).to(torch.float32).numpy())


def _ulp_diff(a32, ref64):
    a32 = a32.astype(np.float32)
    ulp = np.spacing(np.abs(ref64).astype(np.float32)).astype(np.float64)
    return np.abs(a32.astype(np.float64) - ref64) / ulp


def test_expdet_and_sigmoid_within_2ulp_of_fp64_library():
    grid = (np.arange(-2048, 2049) / 64.0).astype(np.float32)  # the logit grid of the workloads
    rng = np.random.default_rng(2)
    rnd = (rng.uniform(-80, 80, 20000)).astype(np.float32)
    x = np.concatenate([grid, rnd])
    e = oracle.expdet(x)
    assert _ulp_diff(e, np.exp(x.astype(np.float64))).max() <= 2.0
    s = oracle.sigmoid(x)
    ref = 1.0 / (1.0 + np.exp(-x.astype(np.float64)))
    assert _ulp_diff(s, ref).max() <= 2.5
    assert oracle.sigmoid(np.float32([0.0]))[0] == 0.5
    # clamped tails stay finite and monotone
    t = oracle.expdet(np.float32([-1000.0, -87.0, 88.0, 1000.0]))
    assert t[0] == t[1] > 0 and t[2] == t[3] and np.isfinite(t).all()


# --------------------------------------------------------------------------
# routing
# --------------------------------------------------------------------------
def _bf16_bits(x):
    return torch.tensor(x, dtype=torch.float32).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)


def test_routing_hand_worked_miniature():
    for line in open(os.path.join(GOLDEN, "routing_miniature.txt")):
        if line.startswith("#") or not line.strip():
            continue
        _, lg, bias, idx, w = [f.strip() for f in line.split("|")]
        lg = np.float32(lg.split())[None, :]
        bias = _bf16_bits([float(v) for v in bias.split()])
        gi, gw = oracle.route(lg, bias, n_group=4, topk_group=2, top_k=2, scaling=2.5)
        assert gi[0].tolist() == [int(v) for v in idx.split()]
        assert np.allclose(gw[0], [float(v) for v in w.split()], rtol=0, atol=1e-6)


def test_routing_closed_form_uniform_logits():
    for c in (-3.0, 0.0, 1.25):
        lg = np.full((3, 256), c, np.float32)
        idx, w = oracle.route(lg, np.zeros(256, np.uint16), 8, 4, 8, 2.5)
        assert np.array_equal(idx, np.tile(np.arange(8, dtype=np.int32), (3, 1)))  # all ties -> smallest indices
        if c == 0.0:  # sigmoid 0.5: every sum is exact
            assert np.all(w == np.float32(0.3125))
        assert np.abs(w - np.float32(0.3125)).max() <= 2 * np.spacing(np.float32(0.3125))


def test_routing_closed_form_planted_winners():
    rng = np.random.default_rng(3)
    for _ in range(20):
        lg = np.full((1, 256), -4.0, np.float32)
        groups = rng.choice(8, 4, replace=False)
        # two planted experts in each of 4 groups, distinct large logits
        planted = np.concatenate([g * 32 + rng.choice(32, 2, replace=False) for g in groups])
        vals = rng.permutation(np.arange(8)) * 0.25 + 2.0
        lg[0, planted] = vals.astype(np.float32)
        idx, w = oracle.route(lg, np.zeros(256, np.uint16), 8, 4, 8, 2.5)
        order = planted[np.argsort(-vals)]
        assert idx[0].tolist() == order.tolist()
        s = 1.0 / (1.0 + np.exp(-np.sort(vals)[::-1]))
        assert np.allclose(w[0], 2.5 * s / s.sum(), rtol=2e-6)


def _route_by_full_sort(sig, bias_f32, G, KG, K):
    """Selection by library sorts on given scores (ties -> smaller index)."""
    T, E = sig.shape
    per = E // G
    b = (sig + bias_f32[None, :]).astype(np.float32)
    out = np.empty((T, K), np.int32)
    for t in range(T):
        bt = b[t]
        gs = np.empty(G, np.float32)
        for g in range(G):
            top2 = np.sort(bt[g * per:(g + 1) * per])[-2:]
            gs[g] = np.float32(top2[1]) + np.float32(top2[0])
        kept = np.lexsort((np.arange(G), -gs))[:KG]
        cand = np.concatenate([np.arange(g * per, (g + 1) * per) for g in sorted(kept)])
        order = cand[np.lexsort((cand, -bt[cand]))]
        out[t] = order[:K]
    return out


@pytest.mark.parametrize("seed,skew", [(0, False), (5, True)])
def test_routing_bruteforce_sort_and_invariants(seed, skew):
    wl = syn.Workload("r", 300, syn.LayerDims(hidden=128, intermediate=128, num_local_experts=1), seed, skew=skew)
    d = wl.dims
    g = torch.Generator().manual_seed(seed)
    lg = (torch.round(torch.randn(wl.tokens, 256, generator=g) * 64) / 64).numpy()
    bias = (0.1 * torch.randn(256, generator=g))
    if skew:
        bias[[3, 11, 17, 26]] += 3.0
    bias_bits = bias.to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    bias_f = bias.to(torch.bfloat16).to(torch.float32).numpy()
    idx, w, sig = oracle.route(lg, bias_bits, d.n_group, d.topk_group, d.top_k, 2.5, want_sig=True)
    # selection logic vs library sorts on the same scores
    assert np.array_equal(idx, _route_by_full_sort(sig, bias_f, 8, 4, 8))
    # invariants: distinct experts, at most 4 groups, weights sum to the scaling factor
    for t in range(wl.tokens):
        assert len(set(idx[t].tolist())) == 8
        assert len(set((idx[t] // 32).tolist())) <= 4
    assert np.abs(w.astype(np.float64).sum(1) - 2.5).max() <= 4 * np.spacing(np.float32(2.5))
    # weights follow the unbiased sigmoid (fp64 library value)
    s64 = 1.0 / (1.0 + np.exp(-np.take_along_axis(lg.astype(np.float64), idx.astype(np.int64), 1)))
    assert np.allclose(w, 2.5 * s64 / s64.sum(1, keepdims=True), rtol=3e-6)
    # the 8th selected biased score is positive, so "discarded groups score 0" and "are not candidates" agree
    b_sel = np.take_along_axis(sig + bias_f[None], idx.astype(np.int64), 1)
    assert b_sel.min() > 0


# --------------------------------------------------------------------------
# permutation
# --------------------------------------------------------------------------
@pytest.mark.parametrize("off,eloc", [(0, 32), (32, 32), (224, 32), (0, 256), (7, 3)])
def test_permutation_bijection_and_stable_sort(off, eloc):
    rng = np.random.default_rng(off + eloc)
    T, K = 257, 8
    idx = np.stack([rng.choice(256, K, replace=False) for _ in range(T)]).astype(np.int32)
    p = oracle.permute(idx, off, eloc)
    flat = idx.ravel()
    local = np.nonzero((flat >= off) & (flat < off + eloc))[0]
    assert p["S"] == local.size == p["count"].sum() == p["offset"][-1]
    # library stable sort of the local slots by expert
    ref = local[np.argsort(flat[local], kind="stable")]
    assert np.array_equal(p["row_to_slot"], ref.astype(np.int32))
    assert np.array_equal(p["count"], np.bincount(flat[local] - off, minlength=eloc))
    assert np.array_equal(p["offset"], np.concatenate([[0], np.cumsum(p["count"])]))
    # bijection between local slots and rows; dropped slots are -1
    s2r = p["slot_to_row"]
    assert np.array_equal(np.sort(s2r[local]), np.arange(local.size))
    assert np.all(np.delete(s2r, local) == -1)
    assert np.array_equal(p["row_to_slot"][s2r[local]], local)


def test_permutation_degenerate_cases():
    p = oracle.permute(np.zeros((0, 8), np.int32), 0, 32)
    assert p["S"] == 0 and p["count"].sum() == 0
    idx = np.tile(np.arange(8, dtype=np.int32), (5, 1))  # every token on the same experts
    p = oracle.permute(idx, 0, 4)
    assert p["count"].tolist() == [5, 5, 5, 5] and p["row_to_slot"][:5].tolist() == [0, 8, 16, 24, 32]
    p = oracle.permute(idx, 100, 32)  # nothing local
    assert p["S"] == 0 and np.all(p["slot_to_row"] == -1)


# --------------------------------------------------------------------------
# expert MLP and combine
# --------------------------------------------------------------------------
def _dq(codes):
    return torch.from_numpy(np.ascontiguousarray(codes)).view(torch.float8_e4m3fn).to(torch.float64)


def _expand(scale, n, k):
    return torch.from_numpy(scale).to(torch.float64).repeat_interleave(128, 0).repeat_interleave(128, 1)[:n, :k]


def _mlp_fp64_library(x_q, x_s, w13, w13_s, w2, w2_s):
    """Single-expert closed form with library routines only: fp64 matmul on the
    dequantised tensors, torch's float8 cast for the re-quantisation."""
    H, I = x_q.shape[0], w2.shape[1]
    x = _dq(x_q) * torch.from_numpy(x_s).to(torch.float64).repeat_interleave(128)
    W13 = _dq(w13) * _expand(w13_s, 2 * I, H)
    W2 = _dq(w2) * _expand(w2_s, H, I)
    h = W13 @ x
    g, u = h[:I], h[I:]
    c = (torch.nn.functional.silu(g) * u).to(torch.float32)
    cb = c.view(-1, 128)
    amax = cb.abs().amax(1)
    sc = torch.where(amax == 0, torch.ones_like(amax), amax / 448.0)
    q = (cb / sc[:, None]).to(torch.float8_e4m3fn)
    cdq = (q.to(torch.float64) * sc[:, None].to(torch.float64)).view(-1)
    return (W2 @ cdq).numpy(), q.view(torch.uint8).view(-1).numpy(), sc.numpy()


@pytest.mark.parametrize("H,I,seed", [(256, 128, 0), (384, 256, 1)])
def test_mlp_row_vs_fp64_library(H, I, seed):
    wl = syn.tiny_workload(tokens=3, hidden=H, intermediate=I, num_experts=4, num_local_experts=4,
                           n_group=2, topk_group=1, top_k=1, seed=seed)
    # larger weights so the SwiGLU output is far from the FP8 subnormal range
    inp = syn.to_host(syn.make_inputs(wl))
    for t in range(3):
        e = t % 4
        args = (inp["hidden_fp8"][t], inp["hidden_scale"][t], inp["w13"][e], inp["w13_scale"][e],
                inp["w2"][e], inp["w2_scale"][e])
        y, cq, cs = oracle.mlp_row(*args)
        y64, q64, s64 = _mlp_fp64_library(*args)
        assert np.allclose(cs, s64, rtol=1e-5)
        assert (cq != q64).mean() <= 0.02  # a code may flip only where fp32 vs fp64 straddles a rounding boundary
        tol = 2e-3 * np.abs(y64).max()
        assert np.abs(y - y64).max() <= tol
        yd, _, _ = oracle.mlp_row(*args, use_double=True)
        assert np.abs(yd - y64).max() <= tol
        # halves swapped <=> gate_first flag
        w13_sw = np.concatenate([inp["w13"][e][I:], inp["w13"][e][:I]])
        s_sw = np.concatenate([inp["w13_scale"][e][I // 128:], inp["w13_scale"][e][:I // 128]])
        y_sw, _, _ = oracle.mlp_row(args[0], args[1], w13_sw, s_sw, args[4], args[5], gate_first=False)
        assert np.array_equal(y_sw, y)


def _identity_problem(H, gate_val, x_vals):
    """H == I, all scales 1: up = identity, gate row n = gate_val * e_0, x[0] = 1."""
    I = H
    enc = lambda a: torch.tensor(a, dtype=torch.float32).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    x = np.array(x_vals, np.float32)
    x[0] = 1.0
    w13 = np.zeros((2 * I, H), np.float32)
    w13[:I, 0] = gate_val
    w13[I:, :] = np.eye(I, H)
    w2 = np.eye(H, I, dtype=np.float32)
    ones = lambda *s: np.ones(s, np.float32)
    return (enc(x), ones(H // 128), enc(w13), ones(2 * I // 128, H // 128), enc(w2), ones(H // 128, I // 128)), x


def test_mlp_identity_weight_closed_forms():
    rng = np.random.default_rng(4)
    H = 256
    xv = rng.integers(-8, 9, H).astype(np.float32)  # FP8-exact integers
    args, x = _identity_problem(H, 0.0, xv)
    y, cq, cs = oracle.mlp_row(*args)
    assert np.all(y == 0) and np.all(cq & 0x7F == 0) and np.all(cs == 1.0)  # gate 0 -> silu(0)*up = 0
    g0 = 1.5
    args, x = _identity_problem(H, g0, xv)
    y, cq, cs = oracle.mlp_row(*args)
    want = (g0 / (1 + math.exp(-g0))) * x.astype(np.float64)
    for blk in range(H // 128):
        sl = slice(blk * 128, (blk + 1) * 128)
        amax = np.abs(want[sl]).max()
        assert np.isclose(cs[blk], amax / 448.0, rtol=1e-6)
        # e4m3 keeps 3 mantissa bits: relative error at most 2^-4 of each value (plus subnormal step)
        assert np.all(np.abs(y[sl] - want[sl]) <= 2.0 ** -4 * np.abs(want[sl]) + cs[blk] * 2.0 ** -10 + 1e-6)
        top = np.argmax(np.abs(want[sl]))
        assert np.isclose(y[sl][top], want[sl][top], rtol=1e-6)  # the block maximum maps to code 448 exactly


def _tiny_inputs(**kw):
    wl = syn.tiny_workload(**kw)
    return wl, syn.to_host(syn.make_inputs(wl))


def test_forward_single_expert_weight_is_scaling_factor():
    # E=2 experts in one group, K=1: the single selected weight is sig/sig*s = s exactly
    wl, inp = _tiny_inputs(tokens=4, hidden=256, intermediate=128, num_experts=2, num_local_experts=2,
                           n_group=1, topk_group=1, top_k=1, seed=7, scaling=2.5)
    r = oracle.forward(inp, 1, 1, 1)
    assert np.all(r["topk_w"] == np.float32(2.5))
    for t in range(4):
        e = int(r["topk_idx"][t, 0])
        y, _, _ = oracle.mlp_row(inp["hidden_fp8"][t], inp["hidden_scale"][t], inp["w13"][e], inp["w13_scale"][e],
                                 inp["w2"][e], inp["w2_scale"][e])
        want = torch.from_numpy(np.float32(2.5) * y).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
        assert np.array_equal(r["out"][t], want)


def test_forward_vs_dense_bruteforce_all_experts():
    wl, inp = _tiny_inputs(tokens=6, hidden=256, intermediate=128, num_experts=16, num_local_experts=8,
                           n_group=4, topk_group=2, top_k=3, seed=11, offset=4)
    d = wl.dims
    r = oracle.forward(inp, d.n_group, d.topk_group, d.top_k)
    dense = oracle.dense_bruteforce(inp, d.n_group, d.topk_group, d.top_k)
    out = oracle.bf16_decode(r["out"])
    assert np.abs(out - dense).max() <= 2e-3 * np.abs(dense).max() + 2.0 ** -8 * np.abs(dense).max()
    # tokens without any local expert are exactly zero
    local = (r["topk_idx"] >= 4) & (r["topk_idx"] < 12)
    for t in range(6):
        if not local[t].any():
            assert np.all(r["out"][t] == 0)
    assert local.any() and not local.all()


def test_forward_exact_invariants():
    wl, inp = _tiny_inputs(tokens=7, hidden=256, intermediate=256, num_experts=16, num_local_experts=16,
                           n_group=4, topk_group=2, top_k=4, seed=21)
    d = wl.dims
    base = oracle.forward(inp, d.n_group, d.topk_group, d.top_k)
    # doubling w2_scale, or the scaling factor, doubles the bf16 output bit for bit
    twice = oracle.bf16_encode(2.0 * oracle.bf16_decode(base["out"]))
    inp2 = dict(inp, w2_scale=inp["w2_scale"] * 2)
    assert np.array_equal(oracle.forward(inp2, d.n_group, d.topk_group, d.top_k)["out"], twice)
    inp3 = dict(inp, scaling_factor=5.0)
    assert np.array_equal(oracle.forward(inp3, d.n_group, d.topk_group, d.top_k)["out"], twice)
    # permuting tokens permutes output rows bit for bit
    perm = np.random.default_rng(0).permutation(7)
    inp4 = dict(inp, hidden_fp8=inp["hidden_fp8"][perm], hidden_scale=inp["hidden_scale"][perm],
                router_logits=inp["router_logits"][perm])
    assert np.array_equal(oracle.forward(inp4, d.n_group, d.topk_group, d.top_k)["out"], base["out"][perm])
    # token subset == rows of the full run; transposed scale layout == row-major
    sub = oracle.forward(inp, d.n_group, d.topk_group, d.top_k, tokens=[5, 0, 3])
    assert np.array_equal(sub["out"], base["out"][[5, 0, 3]])
    inp5 = dict(inp, hidden_scale=np.ascontiguousarray(inp["hidden_scale"].T))
    assert np.array_equal(oracle.forward(inp5, d.n_group, d.topk_group, d.top_k, scale_layout=1)["out"], base["out"])


def test_forward_expert_parallel_shards_sum_to_all_local():
    wl, inp = _tiny_inputs(tokens=6, hidden=128, intermediate=128, num_experts=16, num_local_experts=16,
                           n_group=4, topk_group=2, top_k=4, seed=31)
    d = wl.dims
    full = oracle.bf16_decode(oracle.forward(inp, d.n_group, d.topk_group, d.top_k)["out"]).astype(np.float64)
    acc = np.zeros_like(full)
    for off in range(0, 16, 4):
        shard = dict(inp, w13=inp["w13"][off:off + 4], w13_scale=inp["w13_scale"][off:off + 4],
                     w2=inp["w2"][off:off + 4], w2_scale=inp["w2_scale"][off:off + 4], local_expert_offset=off)
        acc += oracle.bf16_decode(oracle.forward(shard, d.n_group, d.topk_group, d.top_k)["out"])
    assert np.abs(acc - full).max() <= 4 * 2.0 ** -8 * np.abs(full).max()


# --------------------------------------------------------------------------
# router projection and input quantisation (the layer started from bf16 hidden states)
# --------------------------------------------------------------------------
def _bf16_bits(x):
    return torch.as_tensor(np.asarray(x, np.float32)).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)


def test_router_projection_hand_worked_cases():
    def vec(spec, ramp_ok=True):
        v = np.zeros(64, np.float32)
        spec = spec.strip()
        if spec == "ramp":
            return np.arange(1, 65, dtype=np.float32)
        if spec == "ones":
            return np.ones(64, np.float32)
        if spec == "alt":
            return np.where(np.arange(64) % 2 == 0, 1.0, -1.0).astype(np.float32)
        for item in spec.split():
            k, val = item.split(":")
            if k == "even":
                v[0::2] = float(val)
            else:
                v[int(k)] = float(val)
        return v

    n = 0
    for line in open(os.path.join(GOLDEN, "router_projection.txt")):
        if line.startswith("#") or not line.strip():
            continue
        _, xs, ws, want = [f.strip() for f in line.split("|")]
        x = vec(xs)[None, :]
        w = np.stack([vec(f) for f in ws.split(";")])
        got = oracle.router_logits(_bf16_bits(x), _bf16_bits(w))
        assert got.shape == (1, w.shape[0])
        assert got[0].tolist() == [float(v) for v in want.split()], line
        n += 1
    assert n == 2


@pytest.mark.parametrize("T,H,E,seed", [(5, 64, 7, 0), (9, 448, 16, 1), (3, 7168, 256, 2)])
def test_router_projection_vs_fp64_library_matmul(T, H, E, seed):
    rng = np.random.default_rng(seed)
    x = _bf16_bits(rng.standard_normal((T, H)))
    w = _bf16_bits(rng.standard_normal((E, H)) / np.sqrt(H))
    got = oracle.router_logits(x, w).astype(np.float64)
    xd = torch.from_numpy(oracle.bf16_decode(x).astype(np.float64))
    wd = torch.from_numpy(oracle.bf16_decode(w).astype(np.float64))
    ref = torch.matmul(xd, wd.t()).numpy()
    # fp32 summation: each of the (H/32 + 5) roundings on the path of a term is at most half an ulp of a
    # running value bounded by the sum of magnitudes
    bound = (H / 32 + 6) * 2.0 ** -24 * torch.matmul(xd.abs(), wd.abs().t()).numpy()
    assert (np.abs(got - ref) <= bound).all()
    # a transposed or mis-strided operand would fail by orders of magnitude; so would a dropped pair
    assert np.abs(got - ref).max() < 1e-4


def test_router_projection_rows_and_experts_are_independent():
    rng = np.random.default_rng(3)
    x = _bf16_bits(rng.standard_normal((6, 128)))
    w = _bf16_bits(rng.standard_normal((10, 128)))
    full = oracle.router_logits(x, w)
    assert np.array_equal(oracle.router_logits(x[2:5], w[3:9]), full[2:5, 3:9])
    # doubling a weight row doubles its logits bit for bit (powers of two commute with rounding)
    w2 = _bf16_bits(2.0 * oracle.bf16_decode(w))
    assert np.array_equal(oracle.router_logits(x, w2), 2.0 * full)


def test_input_quantisation_vs_torch_cast():
    rng = np.random.default_rng(4)
    x = rng.standard_normal((7, 512)).astype(np.float32) * rng.choice([1e-3, 0.3, 1.0, 40.0], (7, 1)).astype(np.float32)
    x[1, 128:256] = 0.0            # an all-zero block: scale 1, codes 0
    x[2, 5] = 448.0                # values at the format's edge
    xb = torch.from_numpy(x).to(torch.bfloat16)
    q, s = oracle.quantize_rows(xb.view(torch.int16).numpy().view(np.uint16))
    xf = xb.to(torch.float32).view(7, 4, 128)
    amax = xf.abs().amax(-1)
    ts = torch.where(amax == 0, torch.ones_like(amax), amax / 448.0)
    tq = (xf / ts.unsqueeze(-1)).to(torch.float8_e4m3fn).view(7, 512).view(torch.uint8).numpy()
    assert np.array_equal(s.view(np.uint32), ts.numpy().view(np.uint32))
    assert np.array_equal(q, tq)
    assert s[1, 1] == 1.0 and not q[1, 128:256].any()
    # the synthetic input recipe applies the same rule
    rq, rs = syn._quant_rows_128(xb.to(torch.float32))
    assert np.array_equal(q, rq.view(torch.uint8).numpy()) and np.array_equal(s, rs.numpy())


def test_forward_from_hidden_is_projection_then_quantisation_then_forward():
    wl = syn.tiny_workload(tokens=6, hidden=256, intermediate=128)
    inp = syn.to_host(syn.make_inputs(wl))
    r = syn.to_host(syn.make_router_inputs(wl))
    d = wl.dims
    res = oracle.forward_from_hidden({**inp, **r}, d.n_group, d.topk_group, d.top_k)
    logits = oracle.router_logits(r["hidden_bf16"], r["router_weight"])
    q, s = oracle.quantize_rows(r["hidden_bf16"])
    direct = oracle.forward(dict(inp, hidden_fp8=q, hidden_scale=s, router_logits=logits), d.n_group, d.topk_group,
                            d.top_k)
    assert np.array_equal(res["out"], direct["out"]) and np.array_equal(res["topk_idx"], direct["topk_idx"])
    # the recipe's own FP8 activations are the quantisation of the same bf16 hidden states
    assert np.array_equal(q, inp["hidden_fp8"]) and np.array_equal(s, inp["hidden_scale"])
