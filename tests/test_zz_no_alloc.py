"""hola_lm_head_entropy_static: the entry point for callers that may not allocate device memory.

Some users of the library cannot call cudaMalloc when they need a verify step (an engine that gave all of HBM to
its own pool, a plugin under a fixed budget), so they cannot create a context.  The static entry point keeps its only
scratch, the per-CTA softmax statistics, in an array built into the library.  Here it is called twice in a row
through the C ABI, on different inputs of different sizes, and each result is compared with what the ordinary
context-based entry point gives for the same inputs, and with the CPU oracle.  The second call finds the first call's leftovers in the
shared array and must not be disturbed by them.

This file is collected last on purpose: a run that stops at the first failure has then already run everything else.
It passes on its own in a fresh process (the first call does the per-device set-up) and after the other tests.
"""
import ctypes

import numpy as np
import pytest
import torch

from oracle import compare
from oracle import ref as oracle_ref
from paper_2506_18952_b200 import workloads

pytestmark = pytest.mark.gpu

DEV = "cuda"


def _both_ways(binding, w):
    B, k, V = w.B, w.k, w.V
    with binding.HolaVerify(B, k, w.H, V) as ctx:
        want = ctx.hola_lm_head_entropy(w.hidden, w.W_lm, want_logits=True)
        torch.cuda.synchronize()
    logits = torch.full((B, k + 1, V), float("nan"), dtype=torch.float32, device=DEV)
    entropy = torch.full((B, k + 1), float("nan"), dtype=torch.float32, device=DEV)
    logZ = torch.full((B, k + 1), float("nan"), dtype=torch.float32, device=DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    binding.hola_lm_head_entropy_static(w.hidden, w.W_lm, logits, entropy, logZ, status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0                     # no wait ran out (the only place such a thing would show)
    return want, logits, entropy, logZ


def _check(want, logits, entropy, logZ):
    n = compare.torch_to_numpy
    assert np.isfinite(n(entropy)).all() and np.isfinite(n(logZ)).all() and np.isfinite(n(logits)).all()
    assert np.max(np.abs(n(entropy) - n(want.entropy))) <= compare.ENTROPY_ATOL
    assert np.max(np.abs(n(logZ) - n(want.logZ))) <= compare.ENTROPY_ATOL
    ref = n(want.logits).astype(np.float64)
    assert np.max(np.abs(n(logits) - ref) / np.maximum(np.abs(ref), 1.0)) <= compare.LOGIT_RTOL


def _check_oracle(w, logits, entropy, logZ):
    """The static entry against the CPU oracle's steps 1-3 directly."""
    n = compare.torch_to_numpy
    lg = oracle_ref.logits(n(w.hidden).reshape(w.M, w.H), n(w.W_lm))
    lz, H = oracle_ref.softmax_entropy(lg)
    assert np.max(np.abs(n(logits).reshape(w.M, w.V) - lg) / np.maximum(np.abs(lg), 1.0)) <= compare.LOGIT_RTOL
    assert np.max(np.abs(n(entropy).reshape(-1) - H)) <= compare.ENTROPY_ATOL
    assert np.max(np.abs(n(logZ).reshape(-1) - lz)) <= compare.ENTROPY_ATOL


def test_static_entry_matches_context_entry_on_two_calls_in_a_row():
    from paper_2506_18952_b200 import binding
    # first call: 60 sequences x 6 positions = 360 rows, several vocab tiles with a ragged tail
    w1 = workloads.gaussian_head("static-1", 60, 5, 256, 5000, seed=21, device=DEV, w_std=0.3)
    r1 = _both_ways(binding, w1)
    _check(*r1)
    _check_oracle(w1, *r1[1:])
    # second call, right after: fewer rows, other sizes, peaked rows - the array still holds the first call's data
    w2 = workloads.make_config("wide", DEV, B=7, k=3, H=128, V=3001)
    r2 = _both_ways(binding, w2)
    _check(*r2)
    _check_oracle(w2, *r2[1:])


def test_static_entry_rejects_what_does_not_fit():
    from paper_2506_18952_b200 import binding
    lib = binding.load_library()
    B, k, H, V = 103, 4, 64, 100                      # 515 rows > 512
    hidden = torch.zeros((B, k + 1, H), dtype=torch.bfloat16, device=DEV)
    W = torch.zeros((V, H), dtype=torch.bfloat16, device=DEV)
    out = torch.full((B, k + 1, V), -7.0, dtype=torch.float32, device=DEV)
    e = torch.zeros((B, k + 1), dtype=torch.float32, device=DEV)
    with pytest.raises(binding.HolaError, match="512 verify rows"):
        binding.hola_lm_head_entropy_static(hidden, W, out, e, e.clone())
    torch.cuda.synchronize()
    assert torch.all(out == -7.0)                     # nothing was launched
    a = binding.hola_verify_args()
    assert lib.hola_lm_head_entropy_static(ctypes.byref(a), None) == 1      # all-null arguments
    assert lib.hola_lm_head_entropy_static(None, None) == 1


def test_static_entry_refuses_the_8_bit_weight_modes():
    """They need a context's workspace for the quantised hidden rows (and their scales), which this entry does not have."""
    from paper_2506_18952_b200 import binding
    lib = binding.load_library()
    B, k, H, V = 2, 1, 64, 96
    hidden = torch.zeros((B, k + 1, H), dtype=torch.bfloat16, device=DEV)
    Wq = torch.zeros((V, H), dtype=torch.int8, device=DEV)
    scale = torch.ones(V, dtype=torch.float32, device=DEV)
    out = torch.full((B, k + 1, V), -7.0, dtype=torch.float32, device=DEV)
    e = torch.zeros((B, k + 1), dtype=torch.float32, device=DEV)
    z = e.clone()
    for mode in (binding.HOLA_W_INT8, binding.HOLA_W8A8, binding.HOLA_W8A16):
        a = binding.hola_verify_args()
        a.B, a.k, a.H, a.V = B, k, H, V
        a.hidden, a.W_lm, a.w_scale = hidden.data_ptr(), Wq.data_ptr(), scale.data_ptr()
        a.logits_out, a.entropy, a.logZ = out.data_ptr(), e.data_ptr(), z.data_ptr()
        a.w_dtype = mode
        assert lib.hola_lm_head_entropy_static(ctypes.byref(a), None) == 1
    torch.cuda.synchronize()
    assert torch.all(out == -7.0)
