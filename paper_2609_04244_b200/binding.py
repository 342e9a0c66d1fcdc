"""Thin ctypes binding of the C ABI in include/moe_b200.h.

Argument marshalling only: every step of the operator runs inside the CUDA library.
Functions carry the names of the C entry points; `MoEPlan` is a small convenience
wrapper that owns a plan and a torch-allocated workspace.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

import torch

SCORE_SOFTMAX = 0
SCORE_SIGMOID_BIAS = 1

EXPORTS = ["moe_plan", "moe_plan_ex", "moe_plan_destroy", "moe_workspace_bytes", "moe_workspace_init", "moe_forward",
           "moe_forward_noalloc", "moe_forward_host", "moe_forward_debug", "moe_sync_status", "moe_debug_stamps", "moe_plan_info", "moe_plan_variant", "moe_tokens_per_launch", "moe_plan_set_knob", "moe_plan_get_knob", "moe_plan_set_timeout_ms", "moe_last_error"]

_lib = None


class MoEError(RuntimeError):
    def __init__(self, code: int, msg: str):
        super().__init__(f"moe_b200 error {code}: {msg}")
        self.code = code


def lib_path() -> str:
    return os.path.join(os.path.dirname(os.path.abspath(__file__)), "csrc", "libmoe_b200.so")


def load_library():
    """dlopen the in-tree CUDA library; fails loudly if it has not been built."""
    global _lib
    if _lib is not None:
        return _lib
    path = lib_path()
    if not os.path.exists(path):
        raise MoEError(-8, f"{path} is missing: run `python -m paper_2609_04244_b200.build` (needs nvcc); "
                           "there is no CPU fallback")
    lib = ctypes.CDLL(path)
    vp, i, f, sz = ctypes.c_void_p, ctypes.c_int, ctypes.c_float, ctypes.c_size_t
    lib.moe_plan.restype = i
    lib.moe_plan.argtypes = [i, i, i, i, i, i, ctypes.POINTER(vp)]
    lib.moe_plan_ex.restype = i
    lib.moe_plan_ex.argtypes = [i, i, i, i, i, i, f, ctypes.POINTER(vp)]
    lib.moe_plan_destroy.restype = None
    lib.moe_plan_destroy.argtypes = [vp]
    lib.moe_workspace_bytes.restype = sz
    lib.moe_workspace_bytes.argtypes = [vp, i]
    lib.moe_workspace_init.restype = i
    lib.moe_workspace_init.argtypes = [vp, vp, sz, vp]
    lib.moe_forward.restype = i
    lib.moe_forward.argtypes = [vp, i] + [vp] * 9 + [sz, vp]
    lib.moe_forward_noalloc.restype = i
    lib.moe_forward_noalloc.argtypes = [vp, i] + [vp] * 8 + [vp]
    lib.moe_forward_host.restype = i
    lib.moe_forward_host.argtypes = [vp, i] + [vp] * 9 + [sz, vp]
    lib.moe_forward_debug.restype = i
    lib.moe_forward_debug.argtypes = [vp, i] + [vp] * 9 + [sz, vp] + [vp] * 5
    lib.moe_sync_status.restype = i
    lib.moe_sync_status.argtypes = [vp, vp, vp]
    lib.moe_debug_stamps.restype = i
    lib.moe_debug_stamps.argtypes = [vp, vp, vp, vp]
    lib.moe_plan_info.restype = i
    lib.moe_plan_info.argtypes = [vp, i] + [ctypes.POINTER(i)] * 4
    lib.moe_plan_variant.restype = i
    lib.moe_plan_variant.argtypes = [vp, i] + [ctypes.POINTER(i)] * 2
    lib.moe_plan_set_knob.restype = i
    lib.moe_plan_set_knob.argtypes = [vp, i, i, i]
    lib.moe_plan_get_knob.restype = i
    lib.moe_plan_get_knob.argtypes = [vp, i, i, ctypes.POINTER(i)]
    lib.moe_tokens_per_launch.restype = i
    lib.moe_tokens_per_launch.argtypes = [vp]
    lib.moe_plan_set_timeout_ms.restype = i
    lib.moe_plan_set_timeout_ms.argtypes = [vp, i]
    lib.moe_last_error.restype = ctypes.c_char_p
    lib.moe_last_error.argtypes = []
    _lib = lib
    return lib


def _check(rc: int):
    if rc != 0:
        raise MoEError(rc, load_library().moe_last_error().decode())


def _p(t: Optional[torch.Tensor]):
    if t is None:
        return None
    if not t.is_cuda or not t.is_contiguous():
        raise MoEError(-1, "tensors must be contiguous CUDA tensors")
    return ctypes.c_void_p(t.data_ptr())


def _stream(stream) -> ctypes.c_void_p:
    s = torch.cuda.current_stream() if stream is None else stream
    return ctypes.c_void_p(s.cuda_stream)


def moe_plan(H: int, E: int, I: int, top_k: int, scoring: int, renorm: int, routed_scale: float = 1.0):
    h = ctypes.c_void_p()
    lib = load_library()
    _check(lib.moe_plan_ex(H, E, I, top_k, scoring, renorm, ctypes.c_float(routed_scale), ctypes.byref(h)))
    return h


def moe_plan_destroy(plan) -> None:
    load_library().moe_plan_destroy(plan)


def moe_workspace_bytes(plan, T_max: int) -> int:
    return int(load_library().moe_workspace_bytes(plan, T_max))


def moe_workspace_init(plan, workspace: torch.Tensor, stream=None) -> None:
    _check(load_library().moe_workspace_init(plan, _p(workspace), workspace.numel() * workspace.element_size(),
                                             _stream(stream)))


def moe_forward(plan, T, hidden, Wr, sel_bias, W13q, W13s, W2q, W2s, out, workspace, stream=None) -> None:
    _check(load_library().moe_forward(plan, T, _p(hidden), _p(Wr), _p(sel_bias), _p(W13q), _p(W13s), _p(W2q), _p(W2s),
                                      _p(out), _p(workspace), workspace.numel() * workspace.element_size(),
                                      _stream(stream)))


def moe_forward_host(plan, T, hidden_host, Wr, sel_bias, W13q, W13s, W2q, W2s, out_host, workspace, stream=None) -> None:
    """One decode step with the activations in (pinned) host tensors; weights and workspace stay on the device."""
    if hidden_host.is_cuda or out_host.is_cuda or not hidden_host.is_contiguous() or not out_host.is_contiguous():
        raise MoEError(-1, "hidden_host and out_host must be contiguous host tensors")
    _check(load_library().moe_forward_host(plan, T, ctypes.c_void_p(hidden_host.data_ptr()), _p(Wr), _p(sel_bias),
                                           _p(W13q), _p(W13s), _p(W2q), _p(W2s), ctypes.c_void_p(out_host.data_ptr()),
                                           _p(workspace), workspace.numel() * workspace.element_size(), _stream(stream)))


def moe_forward_noalloc(plan, T, hidden, Wr, sel_bias, W13q, W13s, W2q, W2s, out, stream=None) -> None:
    """One decode step using the library's built-in scratch array instead of a caller workspace.

    For callers that cannot allocate device memory where they run the step; see include/moe_b200.h for the size
    limit, the first-call set-up and the rule that calls sharing a device must not overlap.
    """
    _check(load_library().moe_forward_noalloc(plan, T, _p(hidden), _p(Wr), _p(sel_bias), _p(W13q), _p(W13s), _p(W2q),
                                              _p(W2s), _p(out), _stream(stream)))


def moe_forward_debug(plan, T, hidden, Wr, sel_bias, W13q, W13s, W2q, W2s, out, workspace, stream=None,
                      topk_ids=None, topk_w=None, xq=None, xs=None, logits=None) -> None:
    _check(load_library().moe_forward_debug(plan, T, _p(hidden), _p(Wr), _p(sel_bias), _p(W13q), _p(W13s), _p(W2q),
                                            _p(W2s), _p(out), _p(workspace),
                                            workspace.numel() * workspace.element_size(), _stream(stream),
                                            _p(topk_ids), _p(topk_w), _p(xq), _p(xs), _p(logits)))


def moe_sync_status(plan, workspace, stream=None) -> None:
    _check(load_library().moe_sync_status(plan, _p(workspace), _stream(stream)))


def moe_debug_stamps(plan, workspace, grid: int, stream=None):
    """Phase time stamps and wait-time accumulators [grid, 32] (ns) of the last launch on this workspace; see include/moe_b200.h."""
    import numpy as np
    sms = torch.cuda.get_device_properties(workspace.device).multi_processor_count   # the call fills one row per SM
    buf = np.zeros((max(sms, grid), 32), dtype=np.uint64)
    _check(load_library().moe_debug_stamps(plan, _p(workspace), _stream(stream), ctypes.c_void_p(buf.ctypes.data)))
    return buf[:grid]


KNOBS = {"stages": 0, "split_slack_kib": 1, "route_all_tokens": 2, "compact_min": 3, "pdl": 4, "split_weight": 5,
         "fused": 6, "cluster": 7, "stamps": 8, "debug_skip": 9, "split_units": 10, "host_direct": 11}


def moe_plan_set_knob(plan, T: int, knob, value: int) -> None:
    """Set a schedule knob (name from KNOBS or its number) for token count T (0 = every token count)."""
    _check(load_library().moe_plan_set_knob(plan, int(T), KNOBS.get(knob, knob), int(value)))


def moe_plan_get_knob(plan, T: int, knob) -> int:
    v = ctypes.c_int()
    _check(load_library().moe_plan_get_knob(plan, int(T), KNOBS.get(knob, knob), ctypes.byref(v)))
    return v.value


def moe_tokens_per_launch(plan) -> int:
    return int(load_library().moe_tokens_per_launch(plan))


def moe_plan_info(plan, T: int) -> dict:
    g, s, n, b = ctypes.c_int(), ctypes.c_int(), ctypes.c_int(), ctypes.c_int()
    _check(load_library().moe_plan_info(plan, T, ctypes.byref(g), ctypes.byref(s), ctypes.byref(n), ctypes.byref(b)))
    f, c, dyn = moe_plan_variant(plan, T)
    return {"grid": g.value, "stages": s.value, "n_hw": n.value, "smem_bytes": b.value, "fused": f, "cluster": c,
            "pairs_at_runtime": dyn}


def moe_plan_variant(plan, T: int):
    """(fused, cluster, pairs_at_runtime): whether T tokens get the fused-unit kernel variant, the CTAs per cluster of the
    launch, and whether the kernel decides after routing if the CTAs of a pair share units or work alone."""
    f, c = ctypes.c_int(), ctypes.c_int()
    _check(load_library().moe_plan_variant(plan, T, ctypes.byref(f), ctypes.byref(c)))
    return bool(f.value), c.value, f.value == 2


class MoEPlan:
    """Owns a plan handle and a workspace sized for `T_max` tokens on the current CUDA device."""

    def __init__(self, H, E, I, top_k, scoring=SCORE_SOFTMAX, renorm=1, routed_scale=1.0, T_max=64, schedule=None):
        self.H, self.E, self.I, self.top_k = H, E, I, top_k
        self.T_max = T_max
        self.handle = moe_plan(H, E, I, top_k, scoring, renorm, routed_scale)
        self.workspace = None
        if schedule:
            self.apply_schedule(schedule)
        self._size_workspace()

    def _size_workspace(self):
        need = moe_workspace_bytes(self.handle, self.T_max)
        if self.workspace is None or self.workspace.numel() < need:
            self.workspace = torch.empty(need, dtype=torch.uint8, device="cuda")
            moe_workspace_init(self.handle, self.workspace)

    def set_knob(self, T, knob, value):
        """Schedule knob for token count T (0 = all); the scratch is re-sized if the knob changes its layout."""
        torch.cuda.synchronize()
        moe_plan_set_knob(self.handle, T, knob, value)
        if self.workspace is not None:
            self._size_workspace()

    def get_knob(self, T, knob):
        return moe_plan_get_knob(self.handle, T, knob)

    def apply_schedule(self, schedule):
        """Apply a schedule table as written by paper_2609_04244_b200.tune: {"plan": {knob: value}, "per_tokens":
        {"T": {knob: value}}}; unknown token counts keep the defaults."""
        for knob, value in schedule.get("plan", {}).items():
            self.set_knob(0, knob, value)
        for T, knobs in schedule.get("per_tokens", {}).items():
            for knob, value in knobs.items():
                self.set_knob(int(T), knob, value)

    def forward(self, hidden, Wr, sel_bias, W13q, W13s, W2q, W2s, out=None, stream=None):
        T = hidden.shape[0]
        if out is None:
            out = torch.empty((T, self.H), dtype=torch.bfloat16, device=hidden.device)
        moe_forward(self.handle, T, hidden, Wr, sel_bias, W13q, W13s, W2q, W2s, out, self.workspace, stream)
        return out

    def forward_host(self, hidden_host, Wr, sel_bias, W13q, W13s, W2q, W2s, out_host, stream=None):
        moe_forward_host(self.handle, hidden_host.shape[0], hidden_host, Wr, sel_bias, W13q, W13s, W2q, W2s, out_host,
                         self.workspace, stream)
        return out_host

    def bind_forward_host(self, hidden_host, Wr, sel_bias, W13q, W13s, W2q, W2s, out_host, stream=None):
        """moe_forward_host with its arguments marshalled once: returns a zero-argument callable that enqueues the step on
        `stream`.  For callers that repeat a step on the same buffers (a decode loop re-filling `hidden_host` in place):
        only the C call remains per step."""
        if hidden_host.is_cuda or out_host.is_cuda or not hidden_host.is_contiguous() or not out_host.is_contiguous():
            raise MoEError(-1, "hidden_host and out_host must be contiguous host tensors")
        fn = load_library().moe_forward_host
        args = (self.handle, hidden_host.shape[0], ctypes.c_void_p(hidden_host.data_ptr()), _p(Wr), _p(sel_bias), _p(W13q),
                _p(W13s), _p(W2q), _p(W2s), ctypes.c_void_p(out_host.data_ptr()), _p(self.workspace),
                self.workspace.numel() * self.workspace.element_size(), _stream(stream))
        keep = (hidden_host, Wr, sel_bias, W13q, W13s, W2q, W2s, out_host)      # the tensors must outlive the callable

        def step(_keep=keep):
            rc = fn(*args)
            if rc != 0:
                _check(rc)
        return step

    def forward_debug(self, hidden, Wr, sel_bias, W13q, W13s, W2q, W2s, stream=None):
        T, dev = hidden.shape[0], hidden.device
        out = torch.empty((T, self.H), dtype=torch.bfloat16, device=dev)
        dbg = {"ids": torch.empty((T, self.top_k), dtype=torch.int32, device=dev),
               "w": torch.empty((T, self.top_k), dtype=torch.float32, device=dev),
               "xq": torch.empty((T, self.H), dtype=torch.uint8, device=dev),
               "xs": torch.empty((T, self.H // 128), dtype=torch.float32, device=dev),
               "logits": torch.empty((T, self.E), dtype=torch.float32, device=dev)}
        moe_forward_debug(self.handle, T, hidden, Wr, sel_bias, W13q, W13s, W2q, W2s, out, self.workspace, stream,
                          dbg["ids"], dbg["w"], dbg["xq"], dbg["xs"], dbg["logits"])
        dbg["out"] = out
        return dbg

    def sync_status(self, stream=None):
        moe_sync_status(self.handle, self.workspace, stream)

    def stamps(self, T=1, stream=None):
        """Phase time stamps of the last launch (of T tokens); needs the "stamps" knob set before that launch."""
        return moe_debug_stamps(self.handle, self.workspace, self.info(T)["grid"], stream)

    def info(self, T):
        return moe_plan_info(self.handle, T)

    def tokens_per_launch(self):
        return moe_tokens_per_launch(self.handle)

    def close(self):
        if self.handle is not None:
            moe_plan_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
