"""Thin Python binding over the C ABI of libd2moe.so (see include/d2moe.h).

Argument marshalling only: torch is used for device memory and streams; every step of the layer
runs in the library's CUDA kernels.  There is no fallback: if the library is missing or a call
fails, an exception is raised.
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass, field
from typing import List, Optional, Sequence, Tuple

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.environ.get("D2MOE_LIB_PATH") or os.path.join(_HERE, "libd2moe.so")

PATH_AUTO, PATH_CUDA_CORE, PATH_TENSOR = 0, 1, 2

DEV_NONFINITE, DEV_TIMEOUT, DEV_BAD_INDEX = 1, 2, 4


class D2MoEError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: d2moe status {code} ({status_string(code)})")


class _Config(ctypes.Structure):
    _fields_ = [("d_model", ctypes.c_int32), ("d_ffn", ctypes.c_int32), ("n_experts", ctypes.c_int32),
                ("top_k", ctypes.c_int32), ("n_shared", ctypes.c_int32), ("group_size", ctypes.c_int32),
                ("n_bits", ctypes.c_int32), ("bits", ctypes.c_int32 * 8),
                ("renormalize", ctypes.c_int32), ("scale_mode", ctypes.c_int32),
                ("kernel_path", ctypes.c_int32), ("reserved", ctypes.c_int32 * 3)]


class _PlanItem(ctypes.Structure):
    _fields_ = [("expert", ctypes.c_int32), ("segment", ctypes.c_int32)]


class _Segment(ctypes.Structure):
    _fields_ = [("layer", ctypes.c_int32), ("expert", ctypes.c_int32), ("segment", ctypes.c_int32),
                ("reserved", ctypes.c_int32), ("bytes", ctypes.c_int64)]


class _RouteIn(ctypes.Structure):
    _fields_ = [("gate_w_bf16", ctypes.c_void_p), ("logits", ctypes.c_void_p),
                ("bit_w_bf16", ctypes.c_void_p), ("forced_bit_idx", ctypes.c_void_p)]


class _RouteOut(ctypes.Structure):
    _fields_ = [("topk_idx", ctypes.c_void_p), ("topk_w", ctypes.c_void_p), ("bit_idx", ctypes.c_void_p),
                ("perm", ctypes.c_void_p), ("inv_perm", ctypes.c_void_p), ("group_off", ctypes.c_void_p)]


_lib = None

EXPORTS = ["d2moe_status_string", "d2moe_check_config", "d2moe_packed_bytes", "d2moe_pack_mwq",
           "d2moe_unpack_codes", "d2moe_workspace_bytes", "d2moe_route", "d2moe_moe_forward",
           "d2moe_stack_layer", "d2moe_moe_forward_events", "d2moe_forward_launch_count",
           "d2moe_route_static_scratch", "d2moe_selftest_wait_expiry", "d2moe_unpack_scales", "d2moe_plan_load_order", "d2moe_plan_simulate", "d2moe_plan_budget_step", "d2moe_pack_mwq_calibrated"]


def lib() -> ctypes.CDLL:
    """Loads libd2moe.so (built by ``python -m paper_2504_15299_b200.build``)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise FileNotFoundError(f"{LIB_PATH} is missing: run `python -m paper_2504_15299_b200.build`")
    L = ctypes.CDLL(LIB_PATH)
    vp, i64, sz = ctypes.c_void_p, ctypes.c_int64, ctypes.c_size_t
    cfgp = ctypes.POINTER(_Config)
    L.d2moe_status_string.restype = ctypes.c_char_p
    L.d2moe_status_string.argtypes = [ctypes.c_int]
    L.d2moe_check_config.argtypes = [cfgp]
    L.d2moe_packed_bytes.argtypes = [cfgp, i64, i64, ctypes.POINTER(sz), ctypes.POINTER(sz), ctypes.POINTER(sz)]
    L.d2moe_pack_mwq.argtypes = [cfgp, vp, i64, i64, vp, sz, vp]
    L.d2moe_unpack_codes.argtypes = [cfgp, vp, i64, i64, ctypes.c_int, vp, vp, vp, vp]
    L.d2moe_pack_mwq_calibrated.argtypes = [cfgp, vp, i64, i64, vp, vp, vp, sz, vp]
    L.d2moe_unpack_scales.argtypes = [cfgp, vp, i64, i64, vp, vp]
    i32p, dp = ctypes.POINTER(ctypes.c_int32), ctypes.POINTER(ctypes.c_double)
    L.d2moe_plan_load_order.argtypes = [ctypes.c_int32, ctypes.c_int32, i32p, ctypes.c_int32, ctypes.POINTER(_PlanItem),
                                        ctypes.c_int32, i32p]
    L.d2moe_plan_simulate.argtypes = [ctypes.c_int32, ctypes.c_int32, i32p, ctypes.POINTER(_PlanItem), ctypes.c_int32, dp, dp,
                                      dp, dp]
    segp = ctypes.POINTER(_Segment)
    L.d2moe_plan_budget_step.argtypes = [segp, ctypes.c_int32, segp, ctypes.c_int32, ctypes.c_int64, segp, i32p, segp, i32p,
                                         segp, i32p, ctypes.c_int32]
    L.d2moe_workspace_bytes.restype = sz
    L.d2moe_workspace_bytes.argtypes = [cfgp, i64]
    L.d2moe_route.argtypes = [cfgp, i64, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, sz, vp]
    L.d2moe_route_static_scratch.argtypes = [cfgp, i64, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp]
    L.d2moe_moe_forward.argtypes = [cfgp, i64, vp, ctypes.POINTER(vp), ctypes.POINTER(_RouteIn),
                                    ctypes.POINTER(_RouteOut), vp, vp, vp, sz, vp]
    L.d2moe_moe_forward_events.argtypes = [cfgp, i64, vp, ctypes.POINTER(vp), ctypes.POINTER(_RouteIn),
                                           ctypes.POINTER(_RouteOut), vp, vp, vp, sz, vp, ctypes.POINTER(vp)]
    L.d2moe_forward_launch_count.argtypes = [cfgp, i64, ctypes.c_int]
    L.d2moe_selftest_wait_expiry.argtypes = [ctypes.c_int, vp, vp]
    L.d2moe_stack_layer.argtypes = [cfgp, i64, vp, vp, ctypes.c_float, ctypes.POINTER(vp),
                                    ctypes.POINTER(_RouteIn), vp, vp, sz, vp]
    for name in EXPORTS:
        getattr(L, name)
    _lib = L
    return L


def status_string(code: int) -> str:
    return lib().d2moe_status_string(int(code)).decode()


@dataclass
class Config:
    d_model: int
    d_ffn: int
    n_experts: int
    top_k: int
    group_size: int
    bits: Tuple[int, ...]
    n_shared: int = 0
    renormalize: int = 1
    scale_mode: int = 0
    kernel_path: int = PATH_AUTO

    def c(self) -> _Config:
        c = _Config()
        c.d_model, c.d_ffn, c.n_experts, c.top_k = self.d_model, self.d_ffn, self.n_experts, self.top_k
        c.n_shared, c.group_size, c.n_bits = self.n_shared, self.group_size, len(self.bits)
        for i in range(8):
            c.bits[i] = self.bits[i] if i < len(self.bits) else 0
        c.renormalize, c.scale_mode, c.kernel_path = self.renormalize, self.scale_mode, self.kernel_path
        return c

    @staticmethod
    def from_workload(wl, kernel_path: int = PATH_AUTO, scale_mode: int = 0) -> "Config":
        return Config(wl.d_model, wl.d_ffn, wl.n_experts, wl.top_k, wl.group_size, tuple(wl.bits),
                      n_shared=wl.n_shared, renormalize=wl.renormalize, kernel_path=kernel_path, scale_mode=scale_mode)


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    if t is None:
        return None
    assert t.is_contiguous()
    return t.data_ptr()


def _stream(stream: Optional[torch.cuda.Stream]) -> Optional[int]:
    if stream is None:
        stream = torch.cuda.current_stream()
    return stream.cuda_stream or None


def _check(code: int, where: str) -> None:
    if code != 0:
        raise D2MoEError(code, where)


def check_config(cfg: Config) -> int:
    return lib().d2moe_check_config(ctypes.byref(cfg.c()))


def packed_bytes(cfg: Config, rows: int, cols: int) -> Tuple[int, int, int]:
    tot, code, meta = ctypes.c_size_t(), ctypes.c_size_t(), ctypes.c_size_t()
    _check(lib().d2moe_packed_bytes(ctypes.byref(cfg.c()), rows, cols, ctypes.byref(tot), ctypes.byref(code),
                                    ctypes.byref(meta)), "d2moe_packed_bytes")
    return tot.value, code.value, meta.value


def workspace_bytes(cfg: Config, max_tokens: int) -> int:
    n = lib().d2moe_workspace_bytes(ctypes.byref(cfg.c()), max_tokens)
    if n == 0:
        raise D2MoEError(2, "d2moe_workspace_bytes")
    return n


def pack_mwq(cfg: Config, W: torch.Tensor, out: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    """MWQ-quantize and pack a device fp32 [rows, cols] matrix; returns the packed uint8 blob."""
    assert W.is_cuda and W.dtype == torch.float32 and W.dim() == 2
    rows, cols = W.shape
    total, _, _ = packed_bytes(cfg, rows, cols)
    if out is None:
        out = torch.empty(total, dtype=torch.uint8, device=W.device)
    _check(lib().d2moe_pack_mwq(ctypes.byref(cfg.c()), _ptr(W.contiguous()), rows, cols, _ptr(out),
                                out.numel(), _stream(stream)), "d2moe_pack_mwq")
    return out


def pack_mwq_calibrated(cfg: Config, W: torch.Tensor, hc: Optional[torch.Tensor] = None,
                        col_energy: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    """Calibration-aware MWQ of a device fp32 matrix (a copy of W is made: the library overwrites its input)."""
    assert W.is_cuda and W.dtype == torch.float32 and W.dim() == 2
    rows, cols = W.shape
    total, _, _ = packed_bytes(cfg, rows, cols)
    out = torch.empty(total, dtype=torch.uint8, device=W.device)
    work = W.contiguous().clone()
    _check(lib().d2moe_pack_mwq_calibrated(ctypes.byref(cfg.c()), _ptr(work), rows, cols, _ptr(hc), _ptr(col_energy),
                                           _ptr(out), out.numel(), _stream(stream)), "d2moe_pack_mwq_calibrated")
    return out


def unpack_codes(cfg: Config, packed: torch.Tensor, rows: int, cols: int, bits: int, stream=None):
    """Canonical codes at width ``bits`` plus the stored (s1, lo): uint8 [rows, cols], fp32 x2."""
    codes = torch.empty((rows, cols), dtype=torch.uint8, device=packed.device)
    ng = cols // cfg.group_size
    scale = torch.empty((rows, ng), dtype=torch.float32, device=packed.device)
    offset = torch.empty((rows, ng), dtype=torch.float32, device=packed.device)
    _check(lib().d2moe_unpack_codes(ctypes.byref(cfg.c()), _ptr(packed), rows, cols, bits, _ptr(codes),
                                    _ptr(scale), _ptr(offset), _stream(stream)), "d2moe_unpack_codes")
    return codes, scale, offset


def unpack_scales(cfg: Config, packed: torch.Tensor, rows: int, cols: int, stream=None) -> torch.Tensor:
    """scale_mode 1: the free scale of every residual step, fp32 [rows, cols / g, top - b1]."""
    n_steps = cfg.bits[-1] - cfg.bits[0]
    out = torch.empty((rows, cols // cfg.group_size, n_steps), dtype=torch.float32, device=packed.device)
    _check(lib().d2moe_unpack_scales(ctypes.byref(cfg.c()), _ptr(packed), rows, cols, _ptr(out), _stream(stream)),
           "d2moe_unpack_scales")
    return out


@dataclass
class RouteResult:
    topk_idx: torch.Tensor
    topk_w: torch.Tensor
    bit_idx: torch.Tensor
    perm: torch.Tensor
    inv_perm: torch.Tensor
    group_off: torch.Tensor
    device_status: torch.Tensor

    def c(self) -> _RouteOut:
        return _RouteOut(_ptr(self.topk_idx), _ptr(self.topk_w), _ptr(self.bit_idx), _ptr(self.perm),
                         _ptr(self.inv_perm), _ptr(self.group_off))


def route(cfg: Config, x: torch.Tensor, *, gate_w=None, logits=None, bit_w=None, forced_bit_idx=None,
          workspace: Optional[torch.Tensor] = None, stream=None) -> RouteResult:
    T = x.shape[0]
    dev = x.device
    A = T * cfg.top_k
    r = RouteResult(torch.empty((T, cfg.top_k), dtype=torch.int32, device=dev),
                    torch.empty((T, cfg.top_k), dtype=torch.float32, device=dev),
                    torch.empty((T, cfg.top_k), dtype=torch.int8, device=dev),
                    torch.empty(A, dtype=torch.int32, device=dev),
                    torch.empty(A, dtype=torch.int32, device=dev),
                    torch.empty(cfg.n_experts * len(cfg.bits) + 1, dtype=torch.int32, device=dev),
                    torch.zeros(1, dtype=torch.int32, device=dev))
    if workspace is None:
        workspace = torch.empty(workspace_bytes(cfg, max(T, 1)), dtype=torch.uint8, device=dev)
    _check(lib().d2moe_route(ctypes.byref(cfg.c()), T, _ptr(x), _ptr(gate_w), _ptr(logits), _ptr(bit_w),
                             _ptr(forced_bit_idx), _ptr(r.topk_idx), _ptr(r.topk_w), _ptr(r.bit_idx),
                             _ptr(r.perm), _ptr(r.inv_perm), _ptr(r.group_off), _ptr(r.device_status),
                             _ptr(workspace), workspace.numel(), _stream(stream)), "d2moe_route")
    return r


STATIC_MAX_ASSIGNMENTS, STATIC_MAX_KEYS = 16384, 2048


def route_static_scratch(cfg: Config, x: torch.Tensor, *, gate_w=None, logits=None, bit_w=None,
                         forced_bit_idx=None, out: Optional[RouteResult] = None, stream=None) -> RouteResult:
    """d2moe_route for callers that cannot provide a workspace: the library's built-in scratch array is
    used instead (see the limits in include/d2moe.h).  Pass ``out`` (a RouteResult whose tensors were
    allocated earlier) to make the call itself allocation-free on the Python side too."""
    T = x.shape[0]
    dev = x.device
    A = T * cfg.top_k
    r = out
    if r is None:
        r = RouteResult(torch.empty((T, cfg.top_k), dtype=torch.int32, device=dev),
                        torch.empty((T, cfg.top_k), dtype=torch.float32, device=dev),
                        torch.empty((T, cfg.top_k), dtype=torch.int8, device=dev),
                        torch.empty(A, dtype=torch.int32, device=dev),
                        torch.empty(A, dtype=torch.int32, device=dev),
                        torch.empty(cfg.n_experts * len(cfg.bits) + 1, dtype=torch.int32, device=dev),
                        torch.zeros(1, dtype=torch.int32, device=dev))
    _check(lib().d2moe_route_static_scratch(ctypes.byref(cfg.c()), T, _ptr(x), _ptr(gate_w), _ptr(logits),
                                            _ptr(bit_w), _ptr(forced_bit_idx), _ptr(r.topk_idx), _ptr(r.topk_w),
                                            _ptr(r.bit_idx), _ptr(r.perm), _ptr(r.inv_perm), _ptr(r.group_off),
                                            _ptr(r.device_status), _stream(stream)), "d2moe_route_static_scratch")
    return r


def selftest_wait_expiry(which: int, device_status: torch.Tensor, stream=None) -> None:
    """Launches the block whose bounded wait nothing satisfies (see include/d2moe.h); asynchronous."""
    _check(lib().d2moe_selftest_wait_expiry(which, _ptr(device_status), _stream(stream)), "d2moe_selftest_wait_expiry")


def _expert_ptr_array(expert_w: Sequence[torch.Tensor]):
    arr = (ctypes.c_void_p * len(expert_w))()
    for i, t in enumerate(expert_w):
        arr[i] = t.data_ptr()
    return arr


N_STAGES = 4
STAGE_NAMES = ("route", "gate_up", "down", "combine")


def forward_launch_count(cfg: Config, T: int, routing_precomputed: bool = False) -> int:
    return lib().d2moe_forward_launch_count(ctypes.byref(cfg.c()), T, int(routing_precomputed))


def moe_forward(cfg: Config, x: torch.Tensor, expert_w: Sequence[torch.Tensor], *, gate_w=None, logits=None,
                bit_w=None, forced_bit_idx=None, pre: Optional[RouteResult] = None,
                y: Optional[torch.Tensor] = None, workspace: Optional[torch.Tensor] = None,
                device_status: Optional[torch.Tensor] = None, stream=None,
                stage_events: Optional[Sequence[torch.cuda.Event]] = None) -> torch.Tensor:
    """One dual-routed MWQ MoE layer.  expert_w: packed blobs, order [expert][gate, up, down].
    stage_events: optional N_STAGES+1 torch.cuda.Event(enable_timing=True), each recorded once before
    (so that its handle exists); the library records them around its stages."""
    assert x.is_cuda and x.dtype == torch.bfloat16
    T = x.shape[0]
    if y is None:
        y = torch.empty_like(x)
    if workspace is None:
        workspace = torch.empty(workspace_bytes(cfg, max(T, 1)), dtype=torch.uint8, device=x.device)
    rin = _RouteIn(_ptr(gate_w), _ptr(logits), _ptr(bit_w), _ptr(forced_bit_idx))
    rout = pre.c() if pre is not None else None
    if stage_events is not None:
        assert len(stage_events) == N_STAGES + 1
        evs = (ctypes.c_void_p * (N_STAGES + 1))(*[e.cuda_event for e in stage_events])
        _check(lib().d2moe_moe_forward_events(ctypes.byref(cfg.c()), T, _ptr(x), _expert_ptr_array(expert_w),
                                              ctypes.byref(rin), ctypes.byref(rout) if rout is not None else None,
                                              _ptr(y), _ptr(device_status), _ptr(workspace), workspace.numel(),
                                              _stream(stream), evs), "d2moe_moe_forward_events")
        return y
    _check(lib().d2moe_moe_forward(ctypes.byref(cfg.c()), T, _ptr(x), _expert_ptr_array(expert_w),
                                   ctypes.byref(rin), ctypes.byref(rout) if rout is not None else None,
                                   _ptr(y), _ptr(device_status), _ptr(workspace), workspace.numel(),
                                   _stream(stream)), "d2moe_moe_forward")
    return y


def stack_layer(cfg: Config, x: torch.Tensor, xn: torch.Tensor, expert_w: Sequence[torch.Tensor], *,
                gate_w=None, logits=None, bit_w=None, forced_bit_idx=None, eps: float = 1e-5,
                workspace: Optional[torch.Tensor] = None, device_status=None, stream=None) -> torch.Tensor:
    """x <- bf16(x + MoE(bf16(RMSNorm(x)))) in place."""
    T = x.shape[0]
    if workspace is None:
        workspace = torch.empty(workspace_bytes(cfg, max(T, 1)), dtype=torch.uint8, device=x.device)
    rin = _RouteIn(_ptr(gate_w), _ptr(logits), _ptr(bit_w), _ptr(forced_bit_idx))
    _check(lib().d2moe_stack_layer(ctypes.byref(cfg.c()), T, _ptr(x), _ptr(xn), ctypes.c_float(eps),
                                   _expert_ptr_array(expert_w), ctypes.byref(rin), _ptr(device_status),
                                   _ptr(workspace), workspace.numel(), _stream(stream)), "d2moe_stack_layer")
    return x


# ---- host-side pipeline planning (Section 3.4): marshalling of plain Python lists ----
PLAN_HEBF, PLAN_BY_ID = 0, 1


def _flat_B(B):
    E, K = len(B), len(B[0])
    arr = (ctypes.c_int32 * (E * K))(*[int(v) for row in B for v in row])
    return E, K, arr


def plan_load_order(B, policy: int = PLAN_HEBF) -> List[Tuple[int, int]]:
    E, K, arr = _flat_B(B)
    q = (_PlanItem * (E * K))()
    n = ctypes.c_int32()
    _check(lib().d2moe_plan_load_order(E, K, arr, policy, q, E * K, ctypes.byref(n)), "d2moe_plan_load_order")
    return [(q[i].expert, q[i].segment) for i in range(n.value)]


def plan_simulate(B, order: Sequence[Tuple[int, int]], t_io: Sequence[float], t_comp: Sequence[float]) -> Tuple[float, float]:
    E, K, arr = _flat_B(B)
    q = (_PlanItem * max(len(order), 1))(*[_PlanItem(j, k) for j, k in order])
    io, comp = (ctypes.c_double * K)(*t_io), (ctypes.c_double * K)(*t_comp)
    span, wait = ctypes.c_double(), ctypes.c_double()
    _check(lib().d2moe_plan_simulate(E, K, arr, q, len(order), io, comp, ctypes.byref(span), ctypes.byref(wait)),
           "d2moe_plan_simulate")
    return span.value, wait.value


def plan_budget_step(resident, need, budget: int):
    """resident / need: lists of (layer, expert, segment, bytes); returns (new resident, loads, evictions)."""
    cap = len(resident) + len(need) + 1
    mk = lambda v: (_Segment * max(len(v), 1))(*[_Segment(l, e, k, 0, b) for l, e, k, b in v])
    out = [(_Segment * cap)() for _ in range(3)]
    ns = [ctypes.c_int32() for _ in range(3)]
    _check(lib().d2moe_plan_budget_step(mk(resident), len(resident), mk(need), len(need), budget, out[0], ctypes.byref(ns[0]),
                                        out[1], ctypes.byref(ns[1]), out[2], ctypes.byref(ns[2]), cap), "d2moe_plan_budget_step")
    conv = lambda a, n: [(a[i].layer, a[i].expert, a[i].segment, a[i].bytes) for i in range(n.value)]
    return conv(out[0], ns[0]), conv(out[1], ns[1]), conv(out[2], ns[2])
