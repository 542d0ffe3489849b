"""Helpers shared by the GPU parity tests: run the CUDA path through the C ABI
binding, run the CPU oracle on the same seeded inputs, compare."""
from __future__ import annotations

import os
from concurrent.futures import ThreadPoolExecutor

import numpy as np
import torch

import oracle
from paper_2608_14560_b200 import MoeFp8
from paper_2608_14560_b200 import synthetic as syn

# Output tolerance of the workload definition: |gpu - ref| <= 1e-2 + 5e-2*|ref| on
# at least 99.5 % of the elements, and cosine similarity >= 0.999.
ABS_TOL, REL_TOL, MIN_FRACTION, MIN_COSINE = 1e-2, 5e-2, 0.995, 0.999


def bf16_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    return (bits.astype(np.uint32) << 16).view(np.float32)


def check_output(gpu_bits: np.ndarray, ref_bits: np.ndarray):
    g = bf16_bits_to_f32(gpu_bits).astype(np.float64)
    r = bf16_bits_to_f32(ref_bits).astype(np.float64)
    assert np.isfinite(g).all(), "non-finite values in the GPU output"
    ok = np.abs(g - r) <= ABS_TOL + REL_TOL * np.abs(r)
    frac = ok.mean() if ok.size else 1.0
    den = np.linalg.norm(g) * np.linalg.norm(r)
    cos = float((g * r).sum() / den) if den > 0 else 1.0
    if den == 0:
        assert np.array_equal(g, r)
    assert frac >= MIN_FRACTION, f"only {frac:.5f} of elements within tolerance"
    assert cos >= MIN_COSINE, f"cosine {cos:.6f}"
    return frac, cos


WORKERS = os.cpu_count() or 8


def oracle_forward_parallel(host: dict, dims: syn.LayerDims, tokens, workers: int = WORKERS, **kw) -> np.ndarray:
    """The unmodified single-thread oracle on disjoint token shards, one shard per
    thread (the C call releases the GIL).  -> bf16 bits [len(tokens), H]."""
    tokens = np.asarray(tokens, np.int32)
    if tokens.size == 0:
        return np.empty((0, dims.hidden), np.uint16)
    # several shards per worker: tokens differ in their number of local slots
    shards = [s for s in np.array_split(tokens, min(4 * workers, tokens.size)) if s.size]
    with ThreadPoolExecutor(workers) as ex:
        outs = list(ex.map(lambda s: oracle.forward(host, dims.n_group, dims.topk_group, dims.top_k,
                                                    tokens=s, **kw)["out"], shards))
    return np.concatenate(outs)


def segment_tile_rows(count: np.ndarray, offset: np.ndarray, tile: int = 128) -> np.ndarray:
    """Canonical rows of whole GEMM row tiles that span the shapes a persistent CTA meets: the first and the
    last (ragged) tile of the largest expert segment, every row of the smallest non-empty segment, and the
    first tile of a median-sized one."""
    nz = np.flatnonzero(count > 0)
    if nz.size == 0:
        return np.empty(0, np.int64)
    by_size = nz[np.argsort(count[nz], kind="stable")]
    big, small, med = int(by_size[-1]), int(by_size[0]), int(by_size[len(by_size) // 2])
    rows = []
    o, c = int(offset[big]), int(count[big])
    rows.append(np.arange(o, o + min(c, tile)))
    rows.append(np.arange(o + (c - 1) // tile * tile, o + c))
    rows.append(np.arange(int(offset[small]), int(offset[small]) + min(int(count[small]), tile)))
    rows.append(np.arange(int(offset[med]), int(offset[med]) + min(int(count[med]), tile)))
    return np.unique(np.concatenate(rows)).astype(np.int64)


def make_engine(wl: syn.Workload, device, max_tokens=None, poison=True, **kw) -> MoeFp8:
    d = wl.dims
    eng = MoeFp8(d.hidden, d.intermediate, d.num_experts, d.num_local_experts, d.n_group, d.topk_group, d.top_k,
                 max_tokens=max(wl.tokens, 1) if max_tokens is None else max_tokens, device=device,
                 poison_workspace=poison, **kw)  # unwritten scratch reads as NaN (fp8, fp32, bf16) or -1 (int32)
    return eng


def run_and_compare(wl: syn.Workload, device, inp=None, sample_tokens=None, check_rows=True, eng=None, **kw):
    """Forward on the GPU, oracle on the host, every comparison of one workload."""
    d = wl.dims
    if inp is None:
        inp = syn.make_inputs(wl, device)
    own = eng is None
    if own:
        eng = make_engine(wl, device, **kw)
    T = inp["router_logits"].shape[0]
    out = eng.forward(inp)
    dbg = eng.debug_export(T, rows=check_rows is not False)
    torch.cuda.synchronize()
    assert int(dbg["status"].item()) == 0, f"device status {int(dbg['status'].item())}"
    host = syn.to_host(inp)

    # routing: indices bit-exact, weights to fp32 rounding
    ridx, rw = oracle.route(host["router_logits"], host["routing_bias"], d.n_group, d.topk_group, d.top_k,
                            float(inp["scaling_factor"]))
    gidx = dbg["topk_idx"].cpu().numpy()
    assert np.array_equal(gidx, ridx), f"{(gidx != ridx).any(1).sum()} tokens with different expert lists"
    assert np.array_equal(dbg["topk_w"].cpu().numpy(), rw), "routing weights differ"

    # permutation: bit-exact
    perm = oracle.permute(ridx, int(inp["local_expert_offset"]), d.num_local_experts)
    S = perm["S"]
    assert np.array_equal(dbg["expert_count"].cpu().numpy(), perm["count"])
    assert np.array_equal(dbg["expert_offset"].cpu().numpy(), perm["offset"])
    assert np.array_equal(dbg["row_to_slot"].cpu().numpy()[:S], perm["row_to_slot"])

    # output
    tokens = np.arange(T, dtype=np.int32) if sample_tokens is None else np.asarray(sample_tokens, np.int32)
    scale_layout = eng.cfg.hidden_scale_layout
    ref = oracle_forward_parallel(host, d, tokens, scale_layout=scale_layout, gate_first=bool(eng.cfg.gate_first))
    gpu = out.view(torch.int16).cpu().numpy().view(np.uint16)[tokens]
    frac, cos = check_output(gpu, ref)
    local = (ridx >= inp["local_expert_offset"]) & (ridx < inp["local_expert_offset"] + d.num_local_experts)
    none_local = ~local.any(1)
    full = out.view(torch.int16).cpu().numpy()
    assert not full[none_local].any(), "tokens without a local expert must be exactly zero"

    stats = {"S": S, "frac": frac, "cos": cos, "active": int((perm["count"] > 0).sum())}
    if check_rows is not False and S > 0:
        # per slot: the re-quantised SwiGLU row and the down-projection row against the oracle's own
        # intermediates.  check_rows = True: every row of a small layer, else 24 spread rows;
        # "tiles": whole row tiles (see segment_tile_rows); an array: those canonical rows.
        if isinstance(check_rows, str) and check_rows == "tiles":
            rows = segment_tile_rows(perm["count"], perm["offset"])
        elif check_rows is True:
            n = S if (d.hidden * d.intermediate <= 1024 * 512 and S <= 8192) else min(S, 24)
            rows = np.unique(np.linspace(0, S - 1, n).astype(np.int64))
        else:
            rows = np.unique(np.asarray(check_rows, np.int64))
        sel = torch.as_tensor(rows, device=dbg["y_rows"].device)
        y_g = dbg["y_rows"][sel].float().cpu().numpy()
        a2 = dbg["a2_fp8"][sel].cpu().numpy()
        a2s = dbg["a2_scale"][sel].cpu().numpy()
        off = int(inp["local_expert_offset"])
        gate_first = bool(eng.cfg.gate_first)

        def one(i):
            slot = int(perm["row_to_slot"][rows[i]])
            t, j = divmod(slot, d.top_k)
            e = int(ridx[t, j]) - off
            xs = host["hidden_scale"][:, t] if scale_layout else host["hidden_scale"][t]
            yr, cq, cs = oracle.mlp_row(host["hidden_fp8"][t], xs, host["w13"][e], host["w13_scale"][e],
                                        host["w2"][e], host["w2_scale"][e], gate_first=gate_first)
            scales_ok = bool(np.allclose(a2s[i], cs, rtol=1e-5, atol=0))
            # the slot's down-projection row (bf16 in the kernel, fp32 in the oracle), before the weighted combine
            bad = int((np.abs(y_g[i] - yr) > 1e-2 + 5e-2 * np.abs(yr)).sum())
            return scales_ok, int((a2[i] != cq).sum()), cq.size, bad, yr.size

        with ThreadPoolExecutor(WORKERS) as ex:
            res = list(ex.map(one, range(len(rows))))
        assert all(r[0] for r in res), "re-quantisation scales differ"
        mism, tot = sum(r[1] for r in res), sum(r[2] for r in res)
        y_bad, y_tot = sum(r[3] for r in res), sum(r[4] for r in res)
        worst = max(r[1] / r[2] for r in res)
        stats["rows_checked"] = len(rows)
        stats["a2_mismatch"] = mism / tot
        assert mism / tot <= 2e-3, f"{mism}/{tot} re-quantised codes differ"
        assert worst <= 0.05, f"one row has {worst:.3f} of its re-quantised codes different"
        stats["y_rows_bad"] = y_bad / y_tot
        assert y_bad / y_tot <= 5e-3, f"{y_bad}/{y_tot} elements of the per-slot GEMM2 rows outside the tolerance"
    if own:
        eng.close()
    return stats
