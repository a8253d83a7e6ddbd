"""ctypes binding of libhola_verify.so: argument marshalling only, every step runs in the CUDA kernels.

Function names mirror the C ABI (include/hola_verify.h).  Tensors are torch CUDA tensors; torch is used for
device memory and streams, nothing else.
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass

import torch

from . import build as _build

HOLA_OK = 0
HOLA_Q_BF16, HOLA_Q_F32 = 0, 1
HOLA_GATE_TARGET_ENTROPY, HOLA_GATE_DRAFT_ENTROPY = 0, 1
HOLA_FALLBACK_SAMPLE, HOLA_FALLBACK_GREEDY = 0, 1
HOLA_W_BF16, HOLA_W_INT8, HOLA_W8A8, HOLA_W8A16, HOLA_W_MIXED = 0, 1, 2, 3, 4
GROUP_ROWS, SUB_BLOCK = 256, 128
FLAG_BAD_TOKEN, FLAG_BAD_UNIFORM, FLAG_TIMEOUT, FLAG_R_ZERO = 1, 2, 4, 8
HOLA_OPT_RING_SLOTS, HOLA_OPT_ROTATING_UNITS, HOLA_OPT_HOST_OVERLAP, HOLA_OPT_HOST_ROWS_ON_DEMAND, HOLA_OPT_PASSES, HOLA_OPT_PAIR_MMA, HOLA_OPT_HOST_IN_PLACE, HOLA_OPT_CONVERTER_GROUP, HOLA_OPT_FUSED_PASSES = 1, 2, 3, 4, 5, 6, 7, 8, 9

EXPORTS = ["hola_create", "hola_destroy", "hola_workspace_bytes", "hola_verify", "hola_verify_host",
           "hola_lm_head_entropy", "hola_accept_sample", "hola_host_traffic", "hola_shard_record_bytes", "hola_shard_lm_head",
           "hola_shard_accept", "hola_shard_sample", "hola_lm_head_entropy_static", "hola_quantize_w8", "hola_quantize_w4", "hola_plan", "hola_plan_ex", "hola_plan_for_shape", "hola_set_option", "hola_selftest_bounded_wait", "hola_profile_begin", "hola_profile_end", "hola_strerror", "hola_last_cuda_error",
           "hola_version"]


class HolaError(RuntimeError):
    pass


class hola_verify_args(ctypes.Structure):
    _fields_ = [("B", ctypes.c_int32), ("k", ctypes.c_int32), ("H", ctypes.c_int32), ("V", ctypes.c_int32),
                ("hidden", ctypes.c_void_p), ("W_lm", ctypes.c_void_p), ("draft_tok", ctypes.c_void_p),
                ("draft_q", ctypes.c_void_p), ("q_dtype", ctypes.c_int32), ("uniforms", ctypes.c_void_p),
                ("tau", ctypes.c_float), ("accept_len", ctypes.c_void_p), ("next_tok", ctypes.c_void_p),
                ("entropy", ctypes.c_void_p), ("logZ", ctypes.c_void_p), ("logits_out", ctypes.c_void_p),
                ("status_word", ctypes.c_void_p), ("gate_source", ctypes.c_int32), ("fallback", ctypes.c_int32),
                ("draft_entropy", ctypes.c_void_p), ("w_dtype", ctypes.c_int32), ("reserved_", ctypes.c_int32),
                ("w_scale", ctypes.c_void_p), ("wmix", ctypes.c_void_p)]


class hola_wmix(ctypes.Structure):
    _fields_ = [("W16", ctypes.c_void_p), ("W8", ctypes.c_void_p), ("W4", ctypes.c_void_p), ("shift4", ctypes.c_void_p),
                ("group_width", ctypes.c_void_p), ("group_row", ctypes.c_void_p), ("rows16", ctypes.c_int32),
                ("rows8", ctypes.c_int32), ("rows4", ctypes.c_int32), ("reserved_", ctypes.c_int32)]


class hola_shard_args(ctypes.Structure):
    _fields_ = [("world", ctypes.c_int32), ("rank", ctypes.c_int32), ("v_offset", ctypes.c_int32),
                ("V_global", ctypes.c_int32), ("q_tok", ctypes.c_void_p), ("record_out", ctypes.c_void_p),
                ("records", ctypes.c_void_p), ("mass_out", ctypes.c_void_p), ("masses", ctypes.c_void_p)]


class hola_plan_info(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in ("tile_v", "grid", "stages", "rows_per_pass", "passes", "kernels_per_call")]


_lib = None


def load_library(path: str | None = None) -> ctypes.CDLL:
    """Loads the C-ABI library (building it first if the source is newer).  Raises if it cannot be had."""
    global _lib
    if _lib is not None and path is None:
        return _lib
    p = path or (_build.LIB if os.path.exists(_build.LIB) and not _build.needs_build() else _build.build())
    lib = ctypes.CDLL(p)
    lib.hola_create.restype = ctypes.c_int
    lib.hola_create.argtypes = [ctypes.POINTER(ctypes.c_void_p), ctypes.c_int, ctypes.c_int, ctypes.c_int,
                                ctypes.c_int, ctypes.c_int]
    lib.hola_destroy.restype = ctypes.c_int
    lib.hola_destroy.argtypes = [ctypes.c_void_p]
    lib.hola_workspace_bytes.restype = ctypes.c_size_t
    lib.hola_workspace_bytes.argtypes = [ctypes.c_int] * 4
    for name in ("hola_verify", "hola_verify_host", "hola_lm_head_entropy", "hola_accept_sample"):
        fn = getattr(lib, name)
        fn.restype = ctypes.c_int
        fn.argtypes = [ctypes.c_void_p, ctypes.POINTER(hola_verify_args), ctypes.c_void_p]
    lib.hola_lm_head_entropy_static.restype = ctypes.c_int
    lib.hola_lm_head_entropy_static.argtypes = [ctypes.POINTER(hola_verify_args), ctypes.c_void_p]
    lib.hola_quantize_w8.restype = ctypes.c_int
    lib.hola_quantize_w8.argtypes = [ctypes.c_void_p, ctypes.c_int, ctypes.c_int, ctypes.c_void_p, ctypes.c_void_p,
                                     ctypes.c_void_p]
    lib.hola_quantize_w4.restype = ctypes.c_int
    lib.hola_quantize_w4.argtypes = [ctypes.c_void_p, ctypes.c_int, ctypes.c_int, ctypes.c_void_p, ctypes.c_void_p,
                                     ctypes.c_int, ctypes.c_void_p, ctypes.c_void_p]
    lib.hola_plan.restype = ctypes.c_int
    lib.hola_plan.argtypes = [ctypes.c_void_p, ctypes.c_int, ctypes.c_int, ctypes.POINTER(hola_plan_info)]
    lib.hola_plan_for_shape.restype = ctypes.c_int
    lib.hola_plan_for_shape.argtypes = [ctypes.c_int] * 5 + [ctypes.POINTER(hola_plan_info)]
    lib.hola_plan_ex.restype = ctypes.c_int
    lib.hola_plan_ex.argtypes = [ctypes.c_void_p, ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.POINTER(hola_plan_info)]
    lib.hola_profile_begin.restype = ctypes.c_int
    lib.hola_profile_begin.argtypes = [ctypes.c_void_p, ctypes.c_int]
    lib.hola_set_option.restype = ctypes.c_int
    lib.hola_set_option.argtypes = [ctypes.c_void_p, ctypes.c_int, ctypes.c_int]
    lib.hola_selftest_bounded_wait.restype = ctypes.c_int
    lib.hola_selftest_bounded_wait.argtypes = [ctypes.c_void_p, ctypes.c_longlong, ctypes.c_void_p, ctypes.c_void_p,
                                               ctypes.c_void_p]
    lib.hola_shard_record_bytes.restype = ctypes.c_size_t
    lib.hola_shard_record_bytes.argtypes = [ctypes.c_int, ctypes.c_int]
    for name in ("hola_shard_lm_head", "hola_shard_accept", "hola_shard_sample"):
        fn = getattr(lib, name)
        fn.restype = ctypes.c_int
        fn.argtypes = [ctypes.c_void_p, ctypes.POINTER(hola_verify_args), ctypes.POINTER(hola_shard_args),
                       ctypes.c_void_p]
    lib.hola_host_traffic.restype = ctypes.c_int
    lib.hola_host_traffic.argtypes = [ctypes.c_void_p, ctypes.POINTER(ctypes.c_ulonglong),
                                      ctypes.POINTER(ctypes.c_ulonglong)]
    lib.hola_profile_end.restype = ctypes.c_int
    lib.hola_profile_end.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.POINTER(ctypes.c_double),
                                     ctypes.POINTER(ctypes.c_double), ctypes.POINTER(ctypes.c_int)]
    lib.hola_strerror.restype = ctypes.c_char_p
    lib.hola_strerror.argtypes = [ctypes.c_int]
    lib.hola_last_cuda_error.restype = ctypes.c_char_p
    lib.hola_last_cuda_error.argtypes = [ctypes.c_void_p]
    lib.hola_version.restype = ctypes.c_char_p
    if path is None:
        _lib = lib
    return lib


def _check(lib, ctx, status: int, what: str):
    if status != HOLA_OK:
        msg = lib.hola_strerror(status).decode()
        detail = lib.hola_last_cuda_error(ctx).decode() if ctx else ""
        raise HolaError(f"{what}: {msg}" + (f" [{detail}]" if detail else ""))


def _dptr(t: torch.Tensor | None):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _stream_ptr(stream) -> ctypes.c_void_p:
    s = torch.cuda.current_stream() if stream is None else stream
    return ctypes.c_void_p(s.cuda_stream)


def hola_quantize_w8(W_lm: torch.Tensor, stream=None):
    """8-bit form of a bf16 W_lm [V, H] on the device: returns (q int8 [V, H], scale fp32 [V]).  The integers and the
    scales are computed by the library's kernel; torch only provides the two output buffers."""
    if W_lm.dtype != torch.bfloat16 or not W_lm.is_cuda or not W_lm.is_contiguous():
        raise HolaError("hola_quantize_w8 takes a contiguous bfloat16 device tensor")
    lib = load_library()
    V, H = W_lm.shape
    q = torch.empty((V, H), dtype=torch.int8, device=W_lm.device)
    scale = torch.empty((V,), dtype=torch.float32, device=W_lm.device)
    with torch.cuda.device(W_lm.device):
        _check(lib, None, lib.hola_quantize_w8(_dptr(W_lm), V, H, _dptr(q), _dptr(scale), _stream_ptr(stream)),
               "hola_quantize_w8")
    return q, scale


@dataclass
class MixedHead:
    """An LM head stored as groups of 256 vocabulary rows at 4, 8 or 16 bits (HOLA_W_MIXED): the device buffers and the
    hola_wmix struct that points at them.  Keep the object alive while calls that use it are in flight."""
    V: int
    H: int
    widths: list
    W16: torch.Tensor | None
    W8: torch.Tensor | None
    W4: torch.Tensor | None
    shift4: torch.Tensor | None
    w_scale: torch.Tensor
    group_width: torch.Tensor
    group_row: torch.Tensor
    struct: "hola_wmix" = None

    def weight_bytes(self) -> int:
        """Bytes of weights, scales and exponents one pass over the head streams."""
        n = self.w_scale.numel() * 4
        for t in (self.W16, self.W8, self.W4, self.shift4):
            n += 0 if t is None else t.numel() * t.element_size()
        return n


def hola_quantize_mixed(W_lm: torch.Tensor, widths, stream=None) -> MixedHead:
    """bf16 W_lm [V, H] -> the mixed-width form: widths[g] in {4, 8, 16} for group g of 256 vocabulary rows.  The codes,
    scales and exponents are made by the library's quantiser kernels, each run of groups of one width in one launch that
    writes straight into that width's compact buffer; 16-bit rows are copied as they are.  torch provides the buffers."""
    if W_lm.dtype != torch.bfloat16 or not W_lm.is_cuda or not W_lm.is_contiguous():
        raise HolaError("hola_quantize_mixed takes a contiguous bfloat16 device tensor")
    lib = load_library()
    V, H = W_lm.shape
    ng = -(-V // GROUP_ROWS)
    widths = [int(x) for x in widths]
    if len(widths) != ng or any(x not in (4, 8, 16) for x in widths) or H % SUB_BLOCK:
        raise HolaError(f"need {ng} widths out of 4, 8, 16 and H a multiple of {SUB_BLOCK}")
    dev = W_lm.device
    rows = {4: 0, 8: 0, 16: 0}
    group_row = []
    for g, wd in enumerate(widths):
        group_row.append(rows[wd])
        rows[wd] += min(V, (g + 1) * GROUP_ROWS) - g * GROUP_ROWS
    W16 = torch.empty((rows[16], H), dtype=torch.bfloat16, device=dev) if rows[16] else None
    W8 = torch.empty((rows[8], H), dtype=torch.int8, device=dev) if rows[8] else None
    W4 = torch.empty((rows[4], H // 2), dtype=torch.uint8, device=dev) if rows[4] else None
    shift4 = torch.zeros((H // SUB_BLOCK, rows[4]), dtype=torch.uint8, device=dev) if rows[4] else None
    w_scale = torch.ones((V,), dtype=torch.float32, device=dev)
    sp = _stream_ptr(stream)
    with torch.cuda.device(dev):
        g = 0
        while g < ng:                                            # runs of consecutive groups of one width
            g1 = g
            while g1 < ng and widths[g1] == widths[g]:
                g1 += 1
            v0, v1 = g * GROUP_ROWS, min(V, g1 * GROUP_ROWS)
            n, r0, wd = v1 - v0, group_row[g], widths[g]
            src = ctypes.c_void_p(W_lm.data_ptr() + v0 * H * 2)
            scale = ctypes.c_void_p(w_scale.data_ptr() + v0 * 4)
            if wd == 16:
                W16[r0:r0 + n].copy_(W_lm[v0:v1])
            elif wd == 8:
                _check(lib, None, lib.hola_quantize_w8(src, n, H, ctypes.c_void_p(W8.data_ptr() + r0 * H), scale, sp),
                       "hola_quantize_w8")
            else:
                _check(lib, None, lib.hola_quantize_w4(src, n, H, ctypes.c_void_p(W4.data_ptr() + r0 * (H // 2)),
                                                       ctypes.c_void_p(shift4.data_ptr() + r0), rows[4], scale, sp),
                       "hola_quantize_w4")
            g = g1
    head = MixedHead(V, H, widths, W16, W8, W4, shift4, w_scale,
                     torch.tensor(widths, dtype=torch.uint8, device=dev),
                     torch.tensor(group_row, dtype=torch.int32, device=dev))
    st = hola_wmix()
    st.W16, st.W8, st.W4, st.shift4 = (t.data_ptr() if t is not None else None for t in (W16, W8, W4, shift4))
    st.group_width, st.group_row = head.group_width.data_ptr(), head.group_row.data_ptr()
    st.rows16, st.rows8, st.rows4 = rows[16], rows[8], rows[4]
    head.struct = st
    return head


def hola_lm_head_entropy_static(hidden, W_lm, logits, entropy, logZ, stream=None, status=None) -> None:
    """Steps 1-2 through the entry point that allocates no device memory (no context needed).

    For callers that cannot call cudaMalloc (all of HBM already handed to their own pool, a fixed memory budget,
    an allocator that is locked at this point): the library's only scratch for this call is a 1.25 MiB array
    built into it.  Every tensor is the caller's and lives on the current device: hidden bf16 [B, k+1, H],
    W_lm bf16 [V, H], and the outputs logits fp32 [B, k+1, V], entropy and logZ fp32 [B, k+1].
    At most 512 verify rows (B * (k+1)); larger calls raise HolaError and launch nothing.  Calls share the
    built-in array, so do not let two of them overlap on one GPU.  `status` (int32 [1] on the device, optional) gets
    HOLA_FLAG_TIMEOUT OR-ed in should an on-chip wait run out: it is the only way to learn of that here.
    """
    lib = load_library()
    B, k1, H = hidden.shape
    a = hola_verify_args()
    a.B, a.k, a.H, a.V = B, k1 - 1, H, W_lm.shape[0]
    a.hidden, a.W_lm = _dptr(hidden), _dptr(W_lm)
    a.logits_out, a.entropy, a.logZ = _dptr(logits), _dptr(entropy), _dptr(logZ)
    a.status_word = _dptr(status)
    _check(lib, None, lib.hola_lm_head_entropy_static(ctypes.byref(a), _stream_ptr(stream)),
           "hola_lm_head_entropy_static")


@dataclass
class VerifyOutputs:
    accept_len: torch.Tensor   # int32 [B]
    next_tok: torch.Tensor     # int32 [B]
    entropy: torch.Tensor      # fp32 [B, k+1]
    logZ: torch.Tensor         # fp32 [B, k+1]
    logits: torch.Tensor | None
    status: torch.Tensor       # uint32 as int32 [1]
    draft_entropy: torch.Tensor | None = None   # fp32 [B, k], filled when the gate looks at the draft rows


class HolaVerify:
    """Owns one hola_ctx.  Methods are named after the C entry points they call."""

    def __init__(self, maxB: int, maxK: int, H: int, V: int, device: int | None = None):
        if not torch.cuda.is_available():
            raise HolaError("hola_create: no CUDA device; this library has no CPU path")
        self.lib = load_library()
        self.device = torch.cuda.current_device() if device is None else int(device)
        self.maxB, self.maxK, self.H, self.V = maxB, maxK, H, V
        self._ctx = ctypes.c_void_p()
        st = self.lib.hola_create(ctypes.byref(self._ctx), self.device, maxB, maxK, H, V)
        _check(self.lib, None, st, "hola_create")

    def close(self):
        if getattr(self, "_ctx", None) and self._ctx.value:
            self.lib.hola_destroy(self._ctx)
            self._ctx = ctypes.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def __enter__(self):
        return self

    def __exit__(self, *exc):
        self.close()

    # -------------------------------------------------------------------------------------------------
    def hola_plan(self, B: int, k: int, w_dtype: int = HOLA_W_BF16) -> dict:
        info = hola_plan_info()
        _check(self.lib, self._ctx, self.lib.hola_plan_ex(self._ctx, B, k, w_dtype, ctypes.byref(info)), "hola_plan_ex")
        return {n: getattr(info, n) for n, _ in info._fields_}

    def hola_set_option(self, option: int, value: int):
        _check(self.lib, self._ctx, self.lib.hola_set_option(self._ctx, int(option), int(value)), "hola_set_option")

    def hola_selftest_bounded_wait(self, limit_cycles: int = 100000, stream=None) -> tuple[int, int, int]:
        """Runs the bounded-wait self-test; returns (status word, threads that reached the end, waits that gave up)
        after synchronising the stream."""
        dev = torch.device("cuda", self.device)
        status = torch.zeros(1, dtype=torch.int32, device=dev)
        counters = torch.zeros(2, dtype=torch.int32, device=dev)
        st = self.lib.hola_selftest_bounded_wait(self._ctx, int(limit_cycles), _dptr(status), _dptr(counters),
                                                 _stream_ptr(stream))
        _check(self.lib, self._ctx, st, "hola_selftest_bounded_wait")
        (torch.cuda.current_stream() if stream is None else stream).synchronize()
        return int(status.item()), int(counters[0].item()), int(counters[1].item())

    def hola_profile_begin(self, max_calls: int):
        _check(self.lib, self._ctx, self.lib.hola_profile_begin(self._ctx, max_calls), "hola_profile_begin")

    def hola_shard_call(self, which: str, args, shard, stream=None):
        """hola_shard_lm_head / hola_shard_accept / hola_shard_sample on prepared argument structs."""
        if which not in ("hola_shard_lm_head", "hola_shard_accept", "hola_shard_sample"):
            raise HolaError(f"unknown entry point {which}")
        st = getattr(self.lib, which)(self._ctx, ctypes.byref(args), ctypes.byref(shard), _stream_ptr(stream))
        _check(self.lib, self._ctx, st, which)

    def hola_host_traffic(self) -> tuple[int, int]:
        """(host-to-device, device-to-host) bytes of the last hola_verify_host call."""
        up, down = ctypes.c_ulonglong(0), ctypes.c_ulonglong(0)
        _check(self.lib, self._ctx, self.lib.hola_host_traffic(self._ctx, ctypes.byref(up), ctypes.byref(down)),
               "hola_host_traffic")
        return int(up.value), int(down.value)

    def hola_profile_end(self, stream=None) -> dict:
        a, b, n = ctypes.c_double(), ctypes.c_double(), ctypes.c_int()
        st = self.lib.hola_profile_end(self._ctx, _stream_ptr(stream), ctypes.byref(a), ctypes.byref(b), ctypes.byref(n))
        _check(self.lib, self._ctx, st, "hola_profile_end")
        return {"lm_head_ms": a.value, "accept_sample_ms": b.value, "calls": n.value}

    def _args(self, hidden, W_lm, draft_tok, draft_q, uniforms, tau, out: VerifyOutputs, B, k,
              gate_source: int = HOLA_GATE_TARGET_ENTROPY, fallback: int = HOLA_FALLBACK_SAMPLE, w_scale=None,
              a8: bool = False):
        mixed = W_lm if isinstance(W_lm, MixedHead) else None
        if mixed is not None:
            if mixed.V != self.V or mixed.H != self.H or w_scale is not None or a8:
                raise HolaError("a MixedHead carries its own scales and takes bf16 activations; its shape must be the context's")
            W_lm, w_scale = (mixed.W8 if mixed.W8 is not None else (mixed.W4 if mixed.W4 is not None else mixed.W16)), mixed.w_scale
        if hidden.dtype != torch.bfloat16 or (mixed is None and W_lm.dtype not in (torch.bfloat16, torch.int8)):
            raise HolaError("hidden must be bfloat16, W_lm bfloat16 or int8")
        if mixed is None and (W_lm.dtype == torch.int8) != (w_scale is not None):
            raise HolaError("an int8 W_lm goes with w_scale (fp32 per vocabulary row), a bfloat16 one without")
        if draft_q is not None and draft_q.dtype not in (torch.bfloat16, torch.float32):
            raise HolaError("draft_q must be bfloat16 or float32")
        for t in (hidden, W_lm, draft_tok, draft_q, uniforms):
            if t is not None and not t.is_contiguous():
                raise HolaError("all inputs must be contiguous")
        a = hola_verify_args()
        a.B, a.k, a.H, a.V = B, k, self.H, self.V
        a.hidden, a.W_lm = _dptr(hidden), _dptr(W_lm)
        a.draft_tok = _dptr(draft_tok) if k > 0 else None
        a.draft_q = _dptr(draft_q) if k > 0 else None
        a.q_dtype = HOLA_Q_F32 if (draft_q is not None and draft_q.dtype == torch.float32) else HOLA_Q_BF16
        a.uniforms = _dptr(uniforms)
        a.tau = float(tau)
        a.accept_len, a.next_tok = _dptr(out.accept_len), _dptr(out.next_tok)
        a.entropy, a.logZ = _dptr(out.entropy), _dptr(out.logZ)
        a.logits_out = _dptr(out.logits)
        a.status_word = _dptr(out.status)
        a.gate_source, a.fallback = int(gate_source), int(fallback)
        a.draft_entropy = _dptr(out.draft_entropy)
        # a8: True = one 8-bit plane per hidden row (W8A8); "a16" = two planes (16-bit-class activations, W8A16)
        if a8 and w_scale is None:
            raise HolaError("8-bit activation planes (a8) go with an int8 W_lm and its scales")
        act = HOLA_W8A16 if a8 == "a16" else (HOLA_W8A8 if a8 else HOLA_W_INT8)
        a.w_dtype = act if w_scale is not None else HOLA_W_BF16
        a.w_scale = _dptr(w_scale)
        if mixed is not None:
            a.w_dtype, a.W_lm = HOLA_W_MIXED, None
            a.wmix = ctypes.addressof(mixed.struct)
        return a

    def alloc_outputs(self, B: int, k: int, want_logits: bool = False, device=None) -> VerifyOutputs:
        dev = torch.device("cuda", self.device) if device is None else device
        return VerifyOutputs(
            accept_len=torch.empty(B, dtype=torch.int32, device=dev),
            next_tok=torch.empty(B, dtype=torch.int32, device=dev),
            entropy=torch.empty((B, k + 1), dtype=torch.float32, device=dev),
            logZ=torch.empty((B, k + 1), dtype=torch.float32, device=dev),
            logits=torch.empty((B, k + 1, self.V), dtype=torch.float32, device=dev) if want_logits else None,
            status=torch.zeros(1, dtype=torch.int32, device=dev),
            draft_entropy=torch.zeros((B, k), dtype=torch.float32, device=dev))

    def hola_verify(self, hidden, W_lm, draft_tok, draft_q, uniforms, tau, out: VerifyOutputs | None = None,
                    want_logits: bool = False, stream=None, gate_source: int = HOLA_GATE_TARGET_ENTROPY,
                    fallback: int = HOLA_FALLBACK_SAMPLE, w_scale=None, a8: bool = False) -> VerifyOutputs:
        """The whole verify step on device tensors, asynchronous on the stream.  With w_scale, W_lm is the int8 form
        made by hola_quantize_w8; with a8 as well, the hidden rows are quantised on the fly and the products run on
        the 8-bit tensor-core kind."""
        B, k = hidden.shape[0], hidden.shape[1] - 1
        out = out or self.alloc_outputs(B, k, want_logits)
        a = self._args(hidden, W_lm, draft_tok, draft_q, uniforms, tau, out, B, k, gate_source, fallback, w_scale, a8)
        _check(self.lib, self._ctx, self.lib.hola_verify(self._ctx, ctypes.byref(a), _stream_ptr(stream)), "hola_verify")
        return out

    def hola_lm_head_entropy(self, hidden, W_lm, out: VerifyOutputs | None = None, want_logits: bool = True,
                             stream=None, w_scale=None, a8: bool = False) -> VerifyOutputs:
        B, k = hidden.shape[0], hidden.shape[1] - 1
        out = out or self.alloc_outputs(B, k, want_logits)
        a = self._args(hidden, W_lm, None, None, None, 0.0, out, B, k, w_scale=w_scale, a8=a8)
        _check(self.lib, self._ctx, self.lib.hola_lm_head_entropy(self._ctx, ctypes.byref(a), _stream_ptr(stream)),
               "hola_lm_head_entropy")
        return out

    def hola_accept_sample(self, logits, entropy, logZ, draft_tok, draft_q, uniforms, tau, stream=None) -> VerifyOutputs:
        """Steps 3-5 from given fp32 logits [B, k+1, V] and their entropy / logZ."""
        B, k = logits.shape[0], logits.shape[1] - 1
        out = self.alloc_outputs(B, k, False)
        out.logits = logits
        out.entropy.copy_(entropy)
        out.logZ.copy_(logZ)
        a = hola_verify_args()
        a.B, a.k, a.H, a.V = B, k, self.H, self.V
        a.draft_tok = _dptr(draft_tok) if k > 0 else None
        a.draft_q = _dptr(draft_q) if k > 0 else None
        a.q_dtype = HOLA_Q_F32 if (draft_q is not None and draft_q.dtype == torch.float32) else HOLA_Q_BF16
        a.uniforms, a.tau = _dptr(uniforms), float(tau)
        a.accept_len, a.next_tok = _dptr(out.accept_len), _dptr(out.next_tok)
        a.entropy, a.logZ, a.logits_out, a.status_word = _dptr(out.entropy), _dptr(out.logZ), _dptr(logits), _dptr(out.status)
        _check(self.lib, self._ctx, self.lib.hola_accept_sample(self._ctx, ctypes.byref(a), _stream_ptr(stream)),
               "hola_accept_sample")
        return out

    def hola_verify_host(self, hidden, W_lm, draft_tok, draft_q, uniforms, tau, out: VerifyOutputs | None = None,
                         stream=None, gate_source: int = HOLA_GATE_TARGET_ENTROPY,
                         fallback: int = HOLA_FALLBACK_SAMPLE, w_scale=None, a8: bool = False) -> VerifyOutputs:
        """End-to-end form: per-step inputs and all outputs are HOST tensors (pinned for async copies);
        W_lm is the resident device weight.  Returns after the stream has been synchronised."""
        B, k = hidden.shape[0], hidden.shape[1] - 1
        if not isinstance(W_lm, MixedHead) and W_lm.device.type != "cuda":
            raise HolaError("W_lm must be resident on the device")
        for t in (hidden, draft_tok, draft_q, uniforms):
            if t is not None and t.device.type != "cpu":
                raise HolaError("hola_verify_host takes host tensors for the per-step inputs")
        out = out or self.alloc_outputs(B, k, False, device=torch.device("cpu"))
        a = self._args(hidden, W_lm, draft_tok, draft_q, uniforms, tau, out, B, k, gate_source, fallback, w_scale, a8)
        a.logits_out = None
        _check(self.lib, self._ctx, self.lib.hola_verify_host(self._ctx, ctypes.byref(a), _stream_ptr(stream)),
               "hola_verify_host")
        return out


def hola_plan_for_shape(num_sms: int, H: int, V: int, rows: int, w_dtype: int = 0) -> dict:
    """Launch geometry for a shape alone (host arithmetic; needs the library, not a device)."""
    lib = load_library()
    info = hola_plan_info()
    st = lib.hola_plan_for_shape(int(num_sms), int(H), int(V), int(rows), int(w_dtype), ctypes.byref(info))
    if st != 0:
        raise HolaError(f"hola_plan_for_shape: status {st}")
    return {n: getattr(info, n) for n, _ in hola_plan_info._fields_}
