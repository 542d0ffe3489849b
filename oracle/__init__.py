"""ctypes front end of the CPU oracle (TEST INFRASTRUCTURE).

Only tests, the smoke check and the benchmark's CPU-baseline leg import this
package.  It never touches CUDA and never imports the product package's
binding; arrays are numpy (fp8 as uint8 codes, bf16 as uint16 bits).
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "moe_oracle.c")
_LIB = os.path.join(_HERE, "libmoe_oracle.so")

CFLAGS = ["-O2", "-march=native", "-ffp-contract=off", "-fno-fast-math", "-std=c11", "-Wall", "-Wextra"]


def build(force: bool = False) -> str:
    """Compile moe_oracle.c with gcc into libmoe_oracle.so next to it."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(["gcc", *CFLAGS, "-shared", "-fPIC", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def lib() -> C.CDLL:
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.moe_ref_e4m3_decode.restype = C.c_float
        _lib.moe_ref_e4m3_decode.argtypes = [C.c_uint8]
        _lib.moe_ref_e4m3_encode.restype = C.c_uint8
        _lib.moe_ref_e4m3_encode.argtypes = [C.c_float]
        _lib.moe_ref_bf16_decode.restype = C.c_float
        _lib.moe_ref_bf16_decode.argtypes = [C.c_uint16]
        _lib.moe_ref_bf16_encode.restype = C.c_uint16
        _lib.moe_ref_bf16_encode.argtypes = [C.c_float]
        _lib.moe_ref_expdet.restype = C.c_float
        _lib.moe_ref_expdet.argtypes = [C.c_float]
        _lib.moe_ref_sigmoid.restype = C.c_float
        _lib.moe_ref_sigmoid.argtypes = [C.c_float]
    return _lib


def _p(a, ct):
    return None if a is None else a.ctypes.data_as(C.POINTER(ct))


def _c(a, dtype):
    a = np.ascontiguousarray(a, dtype=dtype)
    return a


def _check(rc: int, what: str):
    if rc < 0:
        raise RuntimeError(f"oracle {what} failed with code {rc}")


def e4m3_decode(codes) -> np.ndarray:
    codes = _c(codes, np.uint8)
    f = lib().moe_ref_e4m3_decode
    return np.array([f(int(c)) for c in codes.ravel()], dtype=np.float32).reshape(codes.shape)


def e4m3_encode(x) -> np.ndarray:
    x = _c(x, np.float32)
    f = lib().moe_ref_e4m3_encode
    return np.array([f(float(v)) for v in x.ravel()], dtype=np.uint8).reshape(x.shape)


def bf16_encode(x) -> np.ndarray:
    x = _c(x, np.float32)
    f = lib().moe_ref_bf16_encode
    return np.array([f(float(v)) for v in x.ravel()], dtype=np.uint16).reshape(x.shape)


def bf16_decode(bits) -> np.ndarray:
    bits = _c(bits, np.uint16)
    return (bits.astype(np.uint32) << 16).view(np.float32)


def expdet(x) -> np.ndarray:
    x = _c(x, np.float32)
    f = lib().moe_ref_expdet
    return np.array([f(float(v)) for v in x.ravel()], dtype=np.float32).reshape(x.shape)


def sigmoid(x) -> np.ndarray:
    x = _c(x, np.float32)
    f = lib().moe_ref_sigmoid
    return np.array([f(float(v)) for v in x.ravel()], dtype=np.float32).reshape(x.shape)


def router_logits(x_bf16, w_bf16) -> np.ndarray:
    """Router projection in the fixed fp32 summation order: x [T,H], w [E,H] bf16 bits -> logits [T,E] fp32."""
    x = _c(x_bf16, np.uint16)
    w = _c(w_bf16, np.uint16)
    T, H = x.shape
    E = w.shape[0]
    assert w.shape[1] == H
    out = np.empty((T, E), np.float32)
    _check(lib().moe_ref_router_logits(C.c_int(T), C.c_int(H), C.c_int(E), _p(x, C.c_uint16), _p(w, C.c_uint16),
                                       _p(out, C.c_float)), "router_logits")
    return out


def quantize_rows(x_bf16):
    """Input-side activation quantisation: x [T,H] bf16 bits -> (codes uint8 [T,H], scale fp32 [T,H/128])."""
    x = _c(x_bf16, np.uint16)
    T, H = x.shape
    q = np.empty((T, H), np.uint8)
    s = np.empty((T, H // 128), np.float32)
    _check(lib().moe_ref_quantize_rows(C.c_int(T), C.c_int(H), _p(x, C.c_uint16), _p(q, C.c_uint8), _p(s, C.c_float)),
           "quantize_rows")
    return q, s


def forward_from_hidden(inp: dict, n_group: int, topk_group: int, top_k: int, tokens=None, **kw):
    """The layer starting from bf16 hidden states: router projection, input quantisation, then forward().
    inp carries hidden_bf16 [T,H] and router_weight [E,H] (bf16 bits) instead of hidden_fp8 / hidden_scale /
    router_logits.  -> forward()'s dict plus the logits, codes and scales it was given."""
    logits = router_logits(inp["hidden_bf16"], inp["router_weight"])
    q, s = quantize_rows(inp["hidden_bf16"])
    full = dict(inp, hidden_fp8=q, hidden_scale=s, router_logits=logits)
    res = forward(full, n_group, topk_group, top_k, tokens=tokens, **kw)
    res.update(router_logits=logits, hidden_fp8=q, hidden_scale=s)
    return res


def route(logits, bias_bf16, n_group, topk_group, top_k, scaling, want_sig=False):
    """-> (topk_idx [T,K] int32, topk_w [T,K] fp32[, sig [T,E]])."""
    logits = _c(logits, np.float32)
    bias = _c(bias_bf16, np.uint16)
    T, E = logits.shape
    idx = np.empty((T, top_k), np.int32)
    w = np.empty((T, top_k), np.float32)
    sig = np.empty((T, E), np.float32) if want_sig else None
    rc = lib().moe_ref_route(C.c_int(T), C.c_int(E), C.c_int(n_group), C.c_int(topk_group), C.c_int(top_k),
                             _p(logits, C.c_float), _p(bias, C.c_uint16), C.c_float(scaling),
                             _p(idx, C.c_int32), _p(w, C.c_float), _p(sig, C.c_float))
    _check(rc, "route")
    return (idx, w, sig) if want_sig else (idx, w)


def permute(topk_idx, local_expert_offset, num_local_experts):
    """-> dict(count [E_loc], offset [E_loc+1], row_to_slot [S], slot_to_row [T*K], S)."""
    idx = _c(topk_idx, np.int32)
    T, K = idx.shape
    count = np.empty(num_local_experts, np.int32)
    offset = np.empty(num_local_experts + 1, np.int32)
    r2s = np.empty(max(T * K, 1), np.int32)
    s2r = np.empty(max(T * K, 1), np.int32)
    S = lib().moe_ref_permute(C.c_int(T), C.c_int(K), _p(idx, C.c_int32), C.c_int(local_expert_offset),
                              C.c_int(num_local_experts), _p(count, C.c_int32), _p(offset, C.c_int32),
                              _p(r2s, C.c_int32), _p(s2r, C.c_int32))
    _check(S, "permute")
    return {"count": count, "offset": offset, "row_to_slot": r2s[:S].copy(), "slot_to_row": s2r[: T * K].copy(), "S": S}


def mlp_row(x_q, x_s, w13, w13_s, w2, w2_s, gate_first=True, use_double=False):
    """One (token, expert) slot -> (y [H] fp32, c_q [I] uint8, c_s [I/128] fp32)."""
    x_q = _c(x_q, np.uint8)
    x_s = _c(x_s, np.float32)
    w13 = _c(w13, np.uint8)
    w13_s = _c(w13_s, np.float32)
    w2 = _c(w2, np.uint8)
    w2_s = _c(w2_s, np.float32)
    H = x_q.shape[0]
    I = w2.shape[1]
    assert w13.shape == (2 * I, H) and w2.shape == (H, I)
    y = np.empty(H, np.float32)
    c_q = np.empty(I, np.uint8)
    c_s = np.empty(I // 128, np.float32)
    rc = lib().moe_ref_mlp_row(C.c_int(H), C.c_int(I), _p(x_q, C.c_uint8), _p(x_s, C.c_float),
                               _p(w13, C.c_uint8), _p(w13_s, C.c_float), _p(w2, C.c_uint8), _p(w2_s, C.c_float),
                               C.c_int(int(gate_first)), C.c_int(int(use_double)), _p(y, C.c_float),
                               _p(c_q, C.c_uint8), _p(c_s, C.c_float))
    _check(rc, "mlp_row")
    return y, c_q, c_s


def forward(inp: dict, n_group: int, topk_group: int, top_k: int, tokens=None, scale_layout=0,
            gate_first=True, use_double=False):
    """Whole layer on host arrays (see synthetic.to_host for the dict).

    tokens: None -> all T tokens, else a list of token ids.
    -> dict(out bf16 bits [n,H] uint16, topk_idx [T,K], topk_w [T,K])."""
    hq = _c(inp["hidden_fp8"], np.uint8)
    hs = _c(inp["hidden_scale"], np.float32)
    lg = _c(inp["router_logits"], np.float32)
    bias = _c(inp["routing_bias"], np.uint16)
    w13 = _c(inp["w13"], np.uint8)
    w13s = _c(inp["w13_scale"], np.float32)
    w2 = _c(inp["w2"], np.uint8)
    w2s = _c(inp["w2_scale"], np.float32)
    T, H = hq.shape
    E = lg.shape[1]
    E_loc, _, I = w2.shape
    tok = None if tokens is None else _c(tokens, np.int32)
    n = T if tok is None else tok.shape[0]
    out = np.empty((n, H), np.uint16)
    idx = np.empty((T, top_k), np.int32)
    w = np.empty((T, top_k), np.float32)
    rc = lib().moe_ref_forward(
        C.c_int(T), C.c_int(H), C.c_int(I), C.c_int(E), C.c_int(E_loc), C.c_int(n_group), C.c_int(topk_group),
        C.c_int(top_k), C.c_int(scale_layout), C.c_int(int(gate_first)), C.c_int(int(use_double)),
        _p(hq, C.c_uint8), _p(hs, C.c_float), _p(lg, C.c_float), _p(bias, C.c_uint16),
        _p(w13, C.c_uint8), _p(w13s, C.c_float), _p(w2, C.c_uint8), _p(w2s, C.c_float),
        C.c_int(int(inp["local_expert_offset"])), C.c_float(float(inp["scaling_factor"])),
        _p(tok, C.c_int32), C.c_int(n), _p(out, C.c_uint16), _p(idx, C.c_int32), _p(w, C.c_float))
    _check(rc, "forward")
    return {"out": out, "topk_idx": idx, "topk_w": w}


def dense_bruteforce(inp: dict, n_group: int, topk_group: int, top_k: int, gate_first=True) -> np.ndarray:
    """Every local expert for every token (tiny problems only) -> fp32 [T,H]."""
    hq = _c(inp["hidden_fp8"], np.uint8)
    hs = _c(inp["hidden_scale"], np.float32)
    lg = _c(inp["router_logits"], np.float32)
    bias = _c(inp["routing_bias"], np.uint16)
    w13 = _c(inp["w13"], np.uint8)
    w13s = _c(inp["w13_scale"], np.float32)
    w2 = _c(inp["w2"], np.uint8)
    w2s = _c(inp["w2_scale"], np.float32)
    T, H = hq.shape
    E = lg.shape[1]
    E_loc, _, I = w2.shape
    out = np.empty((T, H), np.float32)
    rc = lib().moe_ref_dense_bruteforce(
        C.c_int(T), C.c_int(H), C.c_int(I), C.c_int(E), C.c_int(E_loc), C.c_int(n_group), C.c_int(topk_group),
        C.c_int(top_k), C.c_int(int(gate_first)), _p(hq, C.c_uint8), _p(hs, C.c_float), _p(lg, C.c_float),
        _p(bias, C.c_uint16), _p(w13, C.c_uint8), _p(w13s, C.c_float), _p(w2, C.c_uint8), _p(w2s, C.c_float),
        C.c_int(int(inp["local_expert_offset"])), C.c_float(float(inp["scaling_factor"])), _p(out, C.c_float))
    _check(rc, "dense_bruteforce")
    return out
