"""ctypes binding of include/moe_fp8.h.  Argument marshalling only: every step
of the forward pass runs in the CUDA library.  PyTorch supplies device memory
and streams."""
from __future__ import annotations

import ctypes as C
import os

import torch

from .build import LIB_PATH

OK = 0
ERR_BAD_ARG, ERR_UNSUPPORTED_DIMS, ERR_NO_WORKSPACE, ERR_CUDA, ERR_ARCH = -1, -2, -3, -4, -5

EXPORTS = (
    "moe_fp8_create", "moe_fp8_destroy", "moe_fp8_workspace_bytes", "moe_fp8_set_workspace", "moe_fp8_forward",
    "moe_fp8_forward_host", "moe_fp8_debug_export", "moe_fp8_last_cuda_error", "moe_fp8_last_launch_count",
    "moe_fp8_strerror", "moe_fp8_set_stage_timing", "moe_fp8_num_stages", "moe_fp8_stage_name",
    "moe_fp8_get_stage_times", "moe_fp8_expert_histogram_static", "moe_fp8_debug_set_fault",
    "moe_fp8_debug_sigmoid", "moe_fp8_forward_from_hidden", "moe_fp8_debug_export_inputs",
    "moe_fp8_set_small_batch_fusion", "moe_fp8_forward_host_async", "moe_fp8_host_sync",
    "moe_fp8_debug_set_short_tiles", "moe_fp8_debug_set_k_split",
)


class Config(C.Structure):
    _fields_ = [(n, C.c_int) for n in (
        "hidden", "intermediate", "num_experts", "num_local_experts", "n_group", "topk_group", "top_k",
        "max_tokens", "hidden_scale_layout", "gate_first")]


class MoeFp8Error(RuntimeError):
    def __init__(self, rc: int, msg: str):
        super().__init__(f"moe_fp8 error {rc}: {msg}")
        self.rc = rc


_lib = None


def load_library() -> C.CDLL:
    """Loads the CUDA library; raises if it has not been built (no fallback)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise MoeFp8Error(ERR_CUDA, f"{LIB_PATH} is missing: run `python -m paper_2608_14560_b200.build` "
                                        "(there is no CPU or PyTorch fallback)")
        lib = C.CDLL(LIB_PATH)
        vp, ip, fp = C.c_void_p, C.c_void_p, C.c_void_p
        lib.moe_fp8_create.argtypes = [C.POINTER(Config), C.POINTER(C.c_void_p)]
        lib.moe_fp8_create.restype = C.c_int
        lib.moe_fp8_destroy.argtypes = [vp]
        lib.moe_fp8_destroy.restype = C.c_int
        lib.moe_fp8_workspace_bytes.argtypes = [vp]
        lib.moe_fp8_workspace_bytes.restype = C.c_size_t
        lib.moe_fp8_set_workspace.argtypes = [vp, vp, C.c_size_t]
        lib.moe_fp8_set_workspace.restype = C.c_int
        fwd = [vp, C.c_int, vp, fp, fp, vp, vp, fp, vp, fp, C.c_int, C.c_float, vp, vp]
        lib.moe_fp8_forward.argtypes = fwd
        lib.moe_fp8_forward.restype = C.c_int
        lib.moe_fp8_forward_host.argtypes = fwd
        lib.moe_fp8_forward_host.restype = C.c_int
        lib.moe_fp8_forward_host_async.argtypes = fwd
        lib.moe_fp8_forward_host_async.restype = C.c_int
        lib.moe_fp8_host_sync.argtypes = [vp]
        lib.moe_fp8_host_sync.restype = C.c_int
        lib.moe_fp8_forward_from_hidden.argtypes = [vp, C.c_int, vp, vp, vp, vp, fp, vp, fp, C.c_int, C.c_float, vp, vp]
        lib.moe_fp8_forward_from_hidden.restype = C.c_int
        lib.moe_fp8_debug_export_inputs.argtypes = [vp, C.c_int, fp, vp, fp, vp]
        lib.moe_fp8_debug_export_inputs.restype = C.c_int
        lib.moe_fp8_debug_export.argtypes = [vp, C.c_int, ip, fp, ip, ip, ip, vp, fp, vp, ip, vp]
        lib.moe_fp8_debug_export.restype = C.c_int
        lib.moe_fp8_last_cuda_error.argtypes = [vp]
        lib.moe_fp8_last_cuda_error.restype = C.c_int
        lib.moe_fp8_last_launch_count.argtypes = [vp]
        lib.moe_fp8_last_launch_count.restype = C.c_int
        lib.moe_fp8_set_stage_timing.argtypes = [vp, C.c_int]
        lib.moe_fp8_set_stage_timing.restype = C.c_int
        lib.moe_fp8_num_stages.argtypes = []
        lib.moe_fp8_num_stages.restype = C.c_int
        lib.moe_fp8_stage_name.argtypes = [C.c_int]
        lib.moe_fp8_stage_name.restype = C.c_char_p
        lib.moe_fp8_get_stage_times.argtypes = [vp, C.POINTER(C.c_float), C.c_int]
        lib.moe_fp8_get_stage_times.restype = C.c_int
        lib.moe_fp8_expert_histogram_static.argtypes = [C.c_int, ip, C.c_int, C.c_int, ip, ip, vp]
        lib.moe_fp8_expert_histogram_static.restype = C.c_int
        lib.moe_fp8_set_small_batch_fusion.argtypes = [vp, C.c_int]
        lib.moe_fp8_set_small_batch_fusion.restype = C.c_int
        lib.moe_fp8_debug_set_k_split.argtypes = [vp, C.c_int]
        lib.moe_fp8_debug_set_k_split.restype = C.c_int
        lib.moe_fp8_debug_set_short_tiles.argtypes = [vp, C.c_int]
        lib.moe_fp8_debug_set_short_tiles.restype = C.c_int
        lib.moe_fp8_debug_set_fault.argtypes = [vp, C.c_int, C.c_longlong]
        lib.moe_fp8_debug_set_fault.restype = C.c_int
        lib.moe_fp8_debug_sigmoid.argtypes = [C.c_int, fp, fp, vp]
        lib.moe_fp8_debug_sigmoid.restype = C.c_int
        lib.moe_fp8_strerror.argtypes = [C.c_int]
        lib.moe_fp8_strerror.restype = C.c_char_p
        _lib = lib
    return _lib


def _ptr(t):
    return None if t is None else C.c_void_p(t.data_ptr())


STATIC_HISTOGRAM_MAX_TOKENS = 16384
ERR_STATIC_LIMIT = -6


def expert_histogram_static(topk_idx: torch.Tensor, local_expert_offset: int, num_local_experts: int,
                            expert_count: torch.Tensor, expert_offset: torch.Tensor, stream=None) -> int:
    """moe_fp8_expert_histogram_static: per-expert counts and offsets from routing indices without any
    workspace or allocation (for callers that may not allocate: graph capture, serving loops, plug-ins
    without a memory pool).  The caller passes the preallocated int32 outputs; returns the C return code."""
    lib = load_library()
    for name, t, shape in (("topk_idx", topk_idx, None), ("expert_count", expert_count, (num_local_experts,)),
                           ("expert_offset", expert_offset, (num_local_experts + 1,))):
        if t.dtype != torch.int32 or not t.is_contiguous() or t.device != topk_idx.device or not t.is_cuda:
            raise TypeError(f"{name} must be a contiguous int32 CUDA tensor on the device of topk_idx")
        if shape is not None and tuple(t.shape) != shape:
            raise ValueError(f"{name} must have shape {shape}")
    if topk_idx.dim() != 2 or topk_idx.shape[1] != 8:
        raise ValueError("topk_idx must have shape [T, 8]")
    s = torch.cuda.current_stream(topk_idx.device) if stream is None else stream
    return int(lib.moe_fp8_expert_histogram_static(
        int(topk_idx.shape[0]), _ptr(topk_idx), int(local_expert_offset), int(num_local_experts),
        _ptr(expert_count), _ptr(expert_offset), C.c_void_p(s.cuda_stream)))


def debug_sigmoid(x: torch.Tensor, stream=None) -> torch.Tensor:
    """moe_fp8_debug_sigmoid: the routing stage's sigmoid on a contiguous fp32 CUDA tensor."""
    if x.dtype != torch.float32 or not x.is_contiguous() or not x.is_cuda:
        raise TypeError("x must be a contiguous fp32 CUDA tensor")
    y = torch.empty_like(x)
    s = torch.cuda.current_stream(x.device) if stream is None else stream
    rc = int(load_library().moe_fp8_debug_sigmoid(x.numel(), _ptr(x), _ptr(y), C.c_void_p(s.cuda_stream)))
    if rc != OK:
        raise MoeFp8Error(rc, load_library().moe_fp8_strerror(rc).decode())
    return y


class MoeFp8:
    """One layer shape + its workspace.  Same names as the C entry points."""

    def __init__(self, hidden=7168, intermediate=2048, num_experts=256, num_local_experts=32, n_group=8,
                 topk_group=4, top_k=8, max_tokens=1024, hidden_scale_layout=0, gate_first=True,
                 device="cuda:0", poison_workspace=False):
        self.lib = load_library()
        self.cfg = Config(hidden, intermediate, num_experts, num_local_experts, n_group, topk_group, top_k,
                          max_tokens, hidden_scale_layout, int(gate_first))
        self.device = torch.device(device)
        self.handle = C.c_void_p()
        if self.device.type == "cuda":
            torch.cuda.set_device(self.device)
        self._check(self.lib.moe_fp8_create(C.byref(self.cfg), C.byref(self.handle)))
        self.workspace_bytes = int(self.lib.moe_fp8_workspace_bytes(self.handle))
        self.workspace = torch.empty(self.workspace_bytes + 1024, dtype=torch.uint8, device=self.device)
        if poison_workspace:  # tests: scratch that is read before it is written shows up as NaN / -1
            self.workspace.fill_(0xFF)
            torch.cuda.synchronize(self.device)
        base = self.workspace.data_ptr()
        self._ws_ptr = (base + 1023) // 1024 * 1024
        self._check(self.lib.moe_fp8_set_workspace(self.handle, C.c_void_p(self._ws_ptr), self.workspace_bytes))

    def _check(self, rc: int):
        if rc != OK:
            msg = self.lib.moe_fp8_strerror(rc).decode()
            if rc == ERR_CUDA and self.handle:
                msg += f" (cudaError {self.lib.moe_fp8_last_cuda_error(self.handle)})"
            raise MoeFp8Error(rc, msg)

    def close(self):
        if self.handle:
            self.lib.moe_fp8_destroy(self.handle)
            self.handle = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def _stream(self, stream):
        s = torch.cuda.current_stream(self.device) if stream is None else stream
        return C.c_void_p(s.cuda_stream)

    def forward(self, inp: dict, out: torch.Tensor | None = None, stream=None) -> torch.Tensor:
        """moe_fp8_forward on device tensors (dict keys as synthetic.make_inputs)."""
        T = inp["router_logits"].shape[0]
        if out is None:
            out = torch.empty(T, self.cfg.hidden, dtype=torch.bfloat16, device=self.device)
        self._check(self.lib.moe_fp8_forward(
            self.handle, T, _ptr(inp["hidden_fp8"]), _ptr(inp["hidden_scale"]), _ptr(inp["router_logits"]),
            _ptr(inp["routing_bias"]), _ptr(inp["w13"]), _ptr(inp["w13_scale"]), _ptr(inp["w2"]),
            _ptr(inp["w2_scale"]), int(inp["local_expert_offset"]), float(inp["scaling_factor"]), _ptr(out),
            self._stream(stream)))
        return out

    def forward_from_hidden(self, inp: dict, out: torch.Tensor | None = None, stream=None) -> torch.Tensor:
        """moe_fp8_forward_from_hidden: inp carries hidden_bf16 [T,H] and router_weight [256,H] (bf16) besides
        the bias and the expert weights."""
        T = inp["hidden_bf16"].shape[0]
        if out is None:
            out = torch.empty(T, self.cfg.hidden, dtype=torch.bfloat16, device=self.device)
        self._check(self.lib.moe_fp8_forward_from_hidden(
            self.handle, T, _ptr(inp["hidden_bf16"]), _ptr(inp["router_weight"]), _ptr(inp["routing_bias"]),
            _ptr(inp["w13"]), _ptr(inp["w13_scale"]), _ptr(inp["w2"]), _ptr(inp["w2_scale"]),
            int(inp["local_expert_offset"]), float(inp["scaling_factor"]), _ptr(out), self._stream(stream)))
        return out

    def debug_export_inputs(self, T: int, stream=None) -> dict:
        """moe_fp8_debug_export_inputs -> router_logits, hidden_fp8 (uint8 codes), hidden_scale (device tensors)."""
        dev, H = self.device, self.cfg.hidden
        sshape = (H // 128, T) if self.cfg.hidden_scale_layout else (T, H // 128)
        r = {"router_logits": torch.empty(T, self.cfg.num_experts, dtype=torch.float32, device=dev),
             "hidden_fp8": torch.empty(T, H, dtype=torch.uint8, device=dev),
             "hidden_scale": torch.empty(sshape, dtype=torch.float32, device=dev)}
        self._check(self.lib.moe_fp8_debug_export_inputs(self.handle, T, _ptr(r["router_logits"]), _ptr(r["hidden_fp8"]),
                                                         _ptr(r["hidden_scale"]), self._stream(stream)))
        return r

    def forward_host(self, host_act: dict, weights: dict, host_out: torch.Tensor, stream=None) -> torch.Tensor:
        """moe_fp8_forward_host: hidden_fp8 / hidden_scale / router_logits / out in (pinned) host memory."""
        T = host_act["router_logits"].shape[0]
        self._check(self.lib.moe_fp8_forward_host(
            self.handle, T, _ptr(host_act["hidden_fp8"]), _ptr(host_act["hidden_scale"]),
            _ptr(host_act["router_logits"]), _ptr(weights["routing_bias"]), _ptr(weights["w13"]),
            _ptr(weights["w13_scale"]), _ptr(weights["w2"]), _ptr(weights["w2_scale"]),
            int(weights["local_expert_offset"]), float(weights["scaling_factor"]), _ptr(host_out),
            self._stream(stream)))
        return host_out

    def set_small_batch_fusion(self, enable):
        """moe_fp8_set_small_batch_fusion: False / 0 = separate kernels at every batch size; True / 1 = the fused
        kernel up to the default limit (80 tokens; a single launch per forward up to 16 tokens); 2..256 = the
        fused kernel up to that many tokens."""
        self._check(self.lib.moe_fp8_set_small_batch_fusion(self.handle, int(enable)))

    def debug_set_k_split(self, enable: bool):
        """moe_fp8_debug_set_k_split: batches of at most 4 tokens may cut a tile's K range over several CTAs
        (default on)."""
        self._check(self.lib.moe_fp8_debug_set_k_split(self.handle, int(enable)))

    def debug_set_short_tiles(self, min_tokens: int):
        """moe_fp8_debug_set_short_tiles: batch size from which row tiles of at most 32 rows run with the weights
        on the M side of the MMAs inside the large-tile GEMM kernels (0: never)."""
        self._check(self.lib.moe_fp8_debug_set_short_tiles(self.handle, int(min_tokens)))

    def debug_set_fault(self, skip_iteration: int = -1, wait_clocks: int = 0):
        """moe_fp8_debug_set_fault (test hook of the bounded-wait failure path)."""
        self._check(self.lib.moe_fp8_debug_set_fault(self.handle, int(skip_iteration), int(wait_clocks)))

    def forward_host_async(self, host_act: dict, weights: dict, host_out: torch.Tensor, stream=None) -> torch.Tensor:
        """moe_fp8_forward_host_async: as forward_host, but returns once the step is enqueued; call host_sync()
        before reading host_out."""
        T = host_act["router_logits"].shape[0]
        self._check(self.lib.moe_fp8_forward_host_async(
            self.handle, T, _ptr(host_act["hidden_fp8"]), _ptr(host_act["hidden_scale"]),
            _ptr(host_act["router_logits"]), _ptr(weights["routing_bias"]), _ptr(weights["w13"]),
            _ptr(weights["w13_scale"]), _ptr(weights["w2"]), _ptr(weights["w2_scale"]),
            int(weights["local_expert_offset"]), float(weights["scaling_factor"]), _ptr(host_out),
            self._stream(stream)))
        return host_out

    def host_sync(self):
        self._check(self.lib.moe_fp8_host_sync(self.handle))

    def set_stage_timing(self, enable: bool):
        self._check(self.lib.moe_fp8_set_stage_timing(self.handle, int(enable)))

    def stage_names(self):
        return [self.lib.moe_fp8_stage_name(i).decode() for i in range(self.lib.moe_fp8_num_stages())]

    def get_stage_times(self) -> dict:
        """Device milliseconds per kernel of the last forward (stage timing must be on)."""
        n = self.lib.moe_fp8_num_stages()
        buf = (C.c_float * n)()
        k = self.lib.moe_fp8_get_stage_times(self.handle, buf, n)
        if k < 0:
            self._check(k)
        return dict(zip(self.stage_names(), list(buf)[:k]))

    def last_launch_count(self) -> int:
        return int(self.lib.moe_fp8_last_launch_count(self.handle))

    def debug_export(self, T: int, rows: bool = True, stream=None) -> dict:
        """moe_fp8_debug_export -> dict of device tensors (see the header for shapes)."""
        dev, EL = self.device, self.cfg.num_local_experts
        I, H = self.cfg.intermediate, self.cfg.hidden
        r = {
            "topk_idx": torch.empty(T, 8, dtype=torch.int32, device=dev),
            "topk_w": torch.empty(T, 8, dtype=torch.float32, device=dev),
            "expert_count": torch.empty(EL, dtype=torch.int32, device=dev),
            "expert_offset": torch.empty(EL + 1, dtype=torch.int32, device=dev),
            "row_to_slot": torch.full((T * 8,), -1, dtype=torch.int32, device=dev),
            "status": torch.zeros(1, dtype=torch.int32, device=dev),
        }
        if rows:
            r["a2_fp8"] = torch.zeros(T * 8, I, dtype=torch.uint8, device=dev)
            r["a2_scale"] = torch.zeros(T * 8, I // 128, dtype=torch.float32, device=dev)
            r["y_rows"] = torch.zeros(T * 8, H, dtype=torch.bfloat16, device=dev)
        self._check(self.lib.moe_fp8_debug_export(
            self.handle, T, _ptr(r["topk_idx"]), _ptr(r["topk_w"]), _ptr(r["expert_count"]),
            _ptr(r["expert_offset"]), _ptr(r["row_to_slot"]), _ptr(r.get("a2_fp8")), _ptr(r.get("a2_scale")),
            _ptr(r.get("y_rows")), _ptr(r["status"]), self._stream(stream)))
        return r

    def status(self) -> int:
        s = torch.zeros(1, dtype=torch.int32, device=self.device)
        self._check(self.lib.moe_fp8_debug_export(self.handle, 0, None, None, None, None, None, None, None, None,
                                                  _ptr(s), self._stream(None)))
        return int(s.item())
