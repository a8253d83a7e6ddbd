"""ctypes access to the CPU oracle (oracle/hola_verify_ref.cpp).

Test infrastructure only: imported by tests/, by the smoke check and by the benchmark's CPU-baseline leg.
Nothing on the product path may import this module, and this module imports nothing from the CUDA package.

Arrays are numpy.  bf16 data travels as uint16 bit patterns (numpy has no bf16); the helpers below convert.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "hola_verify_ref.cpp")
_LIB = os.path.join(_HERE, "libhola_verify_ref.so")

BF16, F32, F64 = 0, 1, 2
FLAG_BAD_TOKEN, FLAG_BAD_UNIFORM, FLAG_R_ZERO = 1, 2, 8


def build(force: bool = False) -> str:
    """Compile the oracle with g++ (no fast-math: summation order is part of its definition)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["g++", "-O2", "-fopenmp", "-shared", "-fPIC", "-std=c++17", "-o", _LIB, _SRC]
        subprocess.run(cmd, check=True)
    return _LIB


_lib = None


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.hola_ref_max_threads.restype = ctypes.c_int
    return _lib


def max_threads() -> int:
    return int(lib().hola_ref_max_threads())


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round-to-nearest-even fp32 -> bf16 bit patterns (uint16).  Input synthesis helper, not method maths."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32).astype(np.uint64)
    rounded = (u + 0x7FFF + ((u >> 16) & 1)) >> 16
    return rounded.astype(np.uint16)


def bf16_bits_to_f64(b: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def _dtype_code(a: np.ndarray) -> int:
    if a.dtype == np.uint16:
        return BF16
    if a.dtype == np.float32:
        return F32
    if a.dtype == np.float64:
        return F64
    raise TypeError(f"unsupported dtype {a.dtype}: use uint16 (bf16 bits), float32 or float64")


def _ptr(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


@dataclass
class RefResult:
    accept_len: np.ndarray      # int32 [B]
    next_tok: np.ndarray        # int32 [B]
    entropy: np.ndarray         # float64 [B, k+1]
    logZ: np.ndarray            # float64 [B, k+1]
    margin_accept: np.ndarray   # float64 [B, k]; +inf where the ratio test was not evaluated
    margin_gate: np.ndarray     # float64 [B, k]; +inf where the gate was not evaluated
    margin_cdf: np.ndarray      # float64 [B]
    flags: np.ndarray           # uint32 [B]
    logits: np.ndarray | None   # float64 [B, k+1, V]
    draft_entropy: np.ndarray | None = None    # float64 [B, k]: entropy of each draft row
    margin_argmax: np.ndarray | None = None    # float64 [B, k+1]: top-1 minus top-2 logit (greedy verifier only)
    gate_source: int = 0        # 0: entropy of the target distribution gates; 1: entropy of the draft distribution
    fallback: int = 0           # 0: speculative-sampling test and residual draw; 1: greedy verifier


def logits(hidden: np.ndarray, W: np.ndarray, nthreads: int = 0) -> np.ndarray:
    """Step 1: logits[r, v] = sum_h hidden[r, h] * W[v, h] in fp64.  hidden [M, H], W [V, H], same dtype."""
    hidden = np.ascontiguousarray(hidden)
    W = np.ascontiguousarray(W)
    code = _dtype_code(hidden)
    assert _dtype_code(W) == code and hidden.ndim == 2 and W.ndim == 2 and hidden.shape[1] == W.shape[1]
    M, H = hidden.shape
    V = W.shape[0]
    out = np.empty((M, V), dtype=np.float64)
    rc = lib().hola_ref_logits(M, H, V, _ptr(hidden), _ptr(W), code, _ptr(out), nthreads)
    if rc:
        raise ValueError("hola_ref_logits rejected its arguments")
    return out


def softmax_entropy(logits64: np.ndarray):
    """Steps 2-3: (logZ, H) per row of fp64 logits [M, V]."""
    logits64 = np.ascontiguousarray(logits64, dtype=np.float64)
    M, V = logits64.shape
    logZ = np.empty(M)
    H = np.empty(M)
    rc = lib().hola_ref_softmax_entropy(M, V, _ptr(logits64), _ptr(logZ), _ptr(H))
    if rc:
        raise ValueError("hola_ref_softmax_entropy rejected its arguments")
    return logZ, H


GATE_TARGET, GATE_DRAFT = 0, 1
FALLBACK_SAMPLE, FALLBACK_GREEDY = 0, 1


def _outputs(B, k):
    return dict(
        accept_len=np.empty(B, dtype=np.int32), next_tok=np.empty(B, dtype=np.int32),
        entropy=np.empty((B, k + 1)), logZ=np.empty((B, k + 1)),
        margin_accept=np.empty((B, k)), margin_gate=np.empty((B, k)), margin_cdf=np.empty(B),
        flags=np.zeros(B, dtype=np.uint32), draft_entropy=np.zeros((B, k)), margin_argmax=np.full((B, k + 1), np.inf))


def verify_from_logits(logits64, draft_tok, draft_q, uniforms, tau, gate_source: int = 0,
                       fallback: int = 0) -> RefResult:
    """Steps 2-6 from fp64 logits [B, k+1, V]; draft_q [B, k, V] (uint16 bf16 bits, float32 or float64)."""
    logits64 = np.ascontiguousarray(logits64, dtype=np.float64)
    B, k1, V = logits64.shape
    k = k1 - 1
    draft_tok = np.ascontiguousarray(draft_tok, dtype=np.int32).reshape(B, k)
    draft_q = np.ascontiguousarray(draft_q).reshape(B, k, V)
    uniforms = np.ascontiguousarray(uniforms, dtype=np.float32).reshape(B, k + 1)
    o = _outputs(B, k)
    rc = lib().hola_verify_from_logits_ref_ex(
        B, k, V, _ptr(logits64), _ptr(draft_tok), _ptr(draft_q), _dtype_code(draft_q), _ptr(uniforms),
        ctypes.c_double(float(tau)), int(gate_source), int(fallback), _ptr(o["accept_len"]), _ptr(o["next_tok"]),
        _ptr(o["entropy"]), _ptr(o["logZ"]), _ptr(o["margin_accept"]), _ptr(o["margin_gate"]), _ptr(o["margin_cdf"]),
        _ptr(o["draft_entropy"]), _ptr(o["margin_argmax"]), _ptr(o["flags"]))
    if rc:
        raise ValueError("hola_verify_from_logits_ref_ex rejected its arguments")
    return RefResult(logits=logits64, gate_source=int(gate_source), fallback=int(fallback), **o)


def verify(hidden, W, draft_tok, draft_q, uniforms, tau, keep_logits: bool = False, nthreads: int = 0,
           gate_source: int = 0, fallback: int = 0) -> RefResult:
    """The whole verify step.  hidden [B, k+1, H] and W [V, H] share a dtype (uint16 bf16 bits / f32 / f64)."""
    hidden = np.ascontiguousarray(hidden)
    W = np.ascontiguousarray(W)
    B, k1, H = hidden.shape
    k = k1 - 1
    V = W.shape[0]
    code = _dtype_code(hidden)
    assert _dtype_code(W) == code and W.shape[1] == H
    draft_tok = np.ascontiguousarray(draft_tok, dtype=np.int32).reshape(B, k)
    draft_q = np.ascontiguousarray(draft_q).reshape(B, k, V)
    uniforms = np.ascontiguousarray(uniforms, dtype=np.float32).reshape(B, k + 1)
    o = _outputs(B, k)
    lg = np.empty((B, k + 1, V)) if keep_logits else None
    rc = lib().hola_verify_ref_ex(
        B, k, H, V, _ptr(hidden), _ptr(W), code, _ptr(draft_tok), _ptr(draft_q), _dtype_code(draft_q),
        _ptr(uniforms), ctypes.c_double(float(tau)), int(gate_source), int(fallback), _ptr(o["accept_len"]),
        _ptr(o["next_tok"]), _ptr(o["entropy"]), _ptr(o["logZ"]), _ptr(o["margin_accept"]), _ptr(o["margin_gate"]),
        _ptr(o["margin_cdf"]), _ptr(o["draft_entropy"]), _ptr(o["margin_argmax"]), _ptr(lg), _ptr(o["flags"]),
        nthreads)
    if rc:
        raise ValueError("hola_verify_ref_ex rejected its arguments")
    return RefResult(logits=lg, gate_source=int(gate_source), fallback=int(fallback), **o)
