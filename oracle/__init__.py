"""ctypes front-end of the CPU oracle (`moe_oracle.c`).

TEST INFRASTRUCTURE ONLY.  Nothing in the product package imports this; only
the tests, the smoke check and the benchmark's cpu-baseline / reference legs do.
The shared object is compiled on first use with gcc (plain C, -O2, OpenMP over
(token, slot) pairs, no fast-math, no FMA contraction).
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "moe_oracle.c")
_LIB = os.path.join(_HERE, "libmoe_oracle.so")
_lib = None

SCORE_SOFTMAX = 0
SCORE_SIGMOID_BIAS = 1


def build(force: bool = False) -> str:
    """Compile the oracle's C source into a shared object next to it; returns the path."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-std=c99", "-fPIC", "-shared", "-fopenmp", "-ffp-contract=off",
               "-fno-fast-math", "-o", _LIB, _SRC, "-lm"]
        subprocess.run(cmd, check=True, cwd=_HERE)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        lib.oracle_bf16_to_double.restype = ctypes.c_double
        lib.oracle_bf16_to_double.argtypes = [ctypes.c_uint16]
        lib.oracle_double_to_bf16.restype = ctypes.c_uint16
        lib.oracle_double_to_bf16.argtypes = [ctypes.c_double]
        lib.oracle_e4m3_to_double.restype = ctypes.c_double
        lib.oracle_e4m3_to_double.argtypes = [ctypes.c_uint8]
        lib.oracle_e4m3_from_float.restype = ctypes.c_uint8
        lib.oracle_e4m3_from_float.argtypes = [ctypes.c_float]
        lib.oracle_quantize_groups.restype = None
        lib.oracle_quantize_groups.argtypes = [ctypes.c_void_p, ctypes.c_int, ctypes.c_int,
                                               ctypes.c_void_p, ctypes.c_void_p]
        lib.moe_oracle.restype = ctypes.c_int
        lib.moe_oracle.argtypes = [ctypes.c_int] * 7 + [ctypes.c_float, ctypes.c_int] + [ctypes.c_void_p] * 22
        lib.moe_oracle_threads.restype = ctypes.c_int
        lib.moe_oracle_set_threads.argtypes = [ctypes.c_int]
        _lib = lib
    return _lib


def threads() -> int:
    return int(_load().moe_oracle_threads())


def set_threads(n: int) -> None:
    _load().moe_oracle_set_threads(int(n))


def bf16_to_double(bits: int) -> float:
    return float(_load().oracle_bf16_to_double(int(bits)))


def double_to_bf16(x: float) -> int:
    return int(_load().oracle_double_to_bf16(float(x)))


def e4m3_to_double(code: int) -> float:
    return float(_load().oracle_e4m3_to_double(int(code)))


def e4m3_from_float(v: float) -> int:
    return int(_load().oracle_e4m3_from_float(np.float32(v)))


def quantize_groups(x: np.ndarray, group: int = 128):
    """fp32 vector (length a multiple of group) -> (E4M3 bytes, fp32 scales)."""
    x = np.ascontiguousarray(x, dtype=np.float32).ravel()
    q = np.empty(x.size, dtype=np.uint8)
    s = np.empty(x.size // group, dtype=np.float32)
    _load().oracle_quantize_groups(x.ctypes.data, x.size, group, q.ctypes.data, s.ctypes.data)
    return q, s


def _ptr(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data


def moe_forward(hidden_bf16: np.ndarray, Wr_bf16: np.ndarray, bias: Optional[np.ndarray],
                W13q: np.ndarray, W13s: np.ndarray, W2q: np.ndarray, W2s: np.ndarray,
                top_k: int, scoring: int = SCORE_SOFTMAX, renorm: int = 1, routed_scale: float = 1.0,
                group: int = 128, expert_map: Optional[np.ndarray] = None,
                ids_in: Optional[np.ndarray] = None, w_in: Optional[np.ndarray] = None,
                want_slots: bool = False):
    """Run the oracle on host arrays.

    hidden_bf16 uint16 [T,H] (bf16 bit patterns), Wr_bf16 uint16 [E,H], bias fp32 [E] or None,
    W13q uint8 [E',2I,H], W13s fp32 [E',2I/g,H/g], W2q uint8 [E',H,I], W2s fp32 [E',H/g,I/g]
    (E' = E, or the number of compacted experts when expert_map int32 [E] is given).
    Returns a dict of numpy arrays: out (uint16 bf16 bits [T,H]), out_f64, ids, w, margin,
    logits, xq, xs, act (fp32 SwiGLU output [T*K,I]), hq, hs and optionally y_slots.
    """
    lib = _load()
    hidden_bf16 = np.ascontiguousarray(hidden_bf16, dtype=np.uint16)
    Wr_bf16 = np.ascontiguousarray(Wr_bf16, dtype=np.uint16)
    T, H = hidden_bf16.shape
    E = Wr_bf16.shape[0]
    assert Wr_bf16.shape[1] == H
    W13q = np.ascontiguousarray(W13q, dtype=np.uint8)
    W2q = np.ascontiguousarray(W2q, dtype=np.uint8)
    W13s = np.ascontiguousarray(W13s, dtype=np.float32)
    W2s = np.ascontiguousarray(W2s, dtype=np.float32)
    I = W2q.shape[2]
    assert W13q.shape[1:] == (2 * I, H) and W2q.shape[1] == H
    assert W13s.shape[1:] == (2 * I // group, H // group) and W2s.shape[1:] == (H // group, I // group)
    n_w = W13q.shape[0]
    if expert_map is not None:
        expert_map = np.ascontiguousarray(expert_map, dtype=np.int32)
        assert expert_map.shape == (E,) and int(expert_map.max()) < n_w
    else:
        assert n_w == E
    if bias is not None:
        bias = np.ascontiguousarray(bias, dtype=np.float32)
        assert bias.shape == (E,)
    K = int(top_k)
    if ids_in is not None:
        ids_in = np.ascontiguousarray(ids_in, dtype=np.int32).reshape(T, K)
        w_in = np.ascontiguousarray(w_in, dtype=np.float32).reshape(T, K)
    r = {
        "out": np.zeros((T, H), np.uint16), "ids": np.zeros((T, K), np.int32), "w": np.zeros((T, K), np.float32),
        "margin": np.zeros((T,), np.float64), "logits": np.zeros((T, E), np.float32),
        "xq": np.zeros((T, H), np.uint8), "xs": np.zeros((T, H // group), np.float32),
        "act": np.zeros((T * K, I), np.float32), "hq": np.zeros((T * K, I), np.uint8),
        "hs": np.zeros((T * K, I // group), np.float32), "out_f64": np.zeros((T, H), np.float64),
    }
    y_slots = np.zeros((T, K, H), np.float64) if want_slots else None
    rc = lib.moe_oracle(T, H, E, I, K, int(scoring), int(renorm), ctypes.c_float(routed_scale), int(group),
                        _ptr(hidden_bf16), _ptr(Wr_bf16), _ptr(bias), _ptr(expert_map),
                        _ptr(W13q), _ptr(W13s), _ptr(W2q), _ptr(W2s), _ptr(ids_in), _ptr(w_in),
                        _ptr(r["out"]), _ptr(r["ids"]), _ptr(r["w"]), _ptr(r["margin"]), _ptr(r["logits"]),
                        _ptr(r["xq"]), _ptr(r["xs"]), _ptr(r["act"]), _ptr(r["hq"]), _ptr(r["hs"]),
                        _ptr(y_slots), _ptr(r["out_f64"]))
    if rc != 0:
        raise RuntimeError(f"moe_oracle failed with status {rc}")
    if want_slots:
        r["y_slots"] = y_slots
    return r


def bf16_bits_to_f64(bits: np.ndarray) -> np.ndarray:
    """Decode bf16 bit patterns (uint16) to float64 (exact)."""
    b = np.ascontiguousarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)
    return b.view(np.float32).astype(np.float64)


def route_and_quantize(hidden_bf16: np.ndarray, Wr_bf16: np.ndarray, bias: Optional[np.ndarray], top_k: int,
                       scoring: int = SCORE_SOFTMAX, renorm: int = 1, routed_scale: float = 1.0, group: int = 128):
    """Steps 1-5 only (logits, scores, top-k, weights, input quantisation).

    Implemented by running the full oracle against one all-zero stand-in expert, so no step is duplicated here.
    """
    E, H = Wr_bf16.shape
    z13 = np.zeros((1, 2 * group, H), np.uint8)
    z2 = np.zeros((1, H, group), np.uint8)
    s13 = np.ones((1, 2, H // group), np.float32)
    s2 = np.ones((1, H // group, 1), np.float32)
    r = moe_forward(hidden_bf16, Wr_bf16, bias, z13, s13, z2, s2, top_k=top_k, scoring=scoring, renorm=renorm,
                    routed_scale=routed_scale, group=group, expert_map=np.zeros(E, np.int32))
    return {k: r[k] for k in ("ids", "w", "margin", "logits", "xq", "xs")}
