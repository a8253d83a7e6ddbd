"""GPU parity: the CUDA path, called through the C ABI, against the CPU oracle on identical seeded inputs."""
import math

import numpy as np
import pytest
import torch

from oracle import compare, ref
from paper_2506_18952_b200 import workloads

pytestmark = pytest.mark.gpu

DEV = "cuda"


@pytest.fixture(scope="module")
def binding():
    from paper_2506_18952_b200 import binding as b
    b.load_library()
    return b


def _np(t):
    return compare.torch_to_numpy(t)


def run_gpu(binding, w, want_logits=False, tau=None, ctx=None, gate_source=0, fallback=0):
    own = ctx is None
    ctx = ctx or binding.HolaVerify(max(w.B, 1), w.k, w.H, w.V)
    try:
        out = ctx.hola_verify(w.hidden, w.W_lm, w.draft_tok, w.draft_q, w.uniforms, w.tau if tau is None else tau,
                              want_logits=want_logits, gate_source=gate_source, fallback=fallback)
        torch.cuda.synchronize()
    finally:
        if own:
            ctx.close()
    return out


def check_against_oracle(binding, w, seqs=None, want_logits=True, tau=None, out=None, gate_source=0, fallback=0):
    """Runs the GPU path on the whole workload and the oracle on `seqs` (all sequences when None)."""
    tau = w.tau if tau is None else tau
    out = out or run_gpu(binding, w, want_logits=want_logits, tau=tau, gate_source=gate_source, fallback=fallback)
    status = int(out.status.item())
    assert status & binding.FLAG_TIMEOUT == 0, "a device-side wait timed out"
    sub = w if seqs is None else w.slice(seqs)
    idx = np.arange(w.B) if seqs is None else np.asarray(list(seqs))
    sub.tau = tau
    orc = compare.run_oracle(sub, keep_logits=True, gate_source=gate_source, fallback=fallback)
    if gate_source == 1 and w.k > 0:
        assert np.max(np.abs(_np(out.draft_entropy)[idx] - orc.draft_entropy)) <= compare.ENTROPY_ATOL
    pick = torch.as_tensor(idx, device=out.accept_len.device)
    rep = compare.compare(orc, _np(sub.draft_q), _np(sub.uniforms), _np(out.accept_len[pick]), _np(out.next_tok[pick]),
                          _np(out.entropy[pick]), _np(out.logZ[pick]),
                          _np(out.logits[pick]) if out.logits is not None else None)
    print(w.name, "tau", tau, rep.summary())
    assert rep.ok, rep.summary() + f" accept_fail={rep.accept_failures[:5]} token_fail={rep.token_failures[:5]}"
    # margin cases are reported, and must stay rare
    assert rep.accept_margin_cases <= max(1, rep.n_seq // 20)
    assert rep.token_margin_cases <= max(1, rep.n_seq // 10)
    return out, orc, rep


def check_ranges(w, out):
    a, t = _np(out.accept_len), _np(out.next_tok)
    assert a.min() >= 0 and a.max() <= w.k
    assert t.min() >= 0 and t.max() < w.V
    H = _np(out.entropy)
    assert np.isfinite(H).all() and H.min() >= 0 and H.max() <= math.log(w.V) + 1e-3
    assert np.isfinite(_np(out.logZ)).all()


# ------------------------------------------------------------------------------------------ the projection
def _int_workload(B, k, H, V, seed, identity=False):
    g = torch.Generator().manual_seed(seed)
    hidden = torch.randint(-4, 5, (B, k + 1, H), generator=g).float()
    W = torch.eye(V, H) if identity else torch.randint(-4, 5, (V, H), generator=g).float()
    q = torch.full((B, k, V), 1.0 / V)
    tok = torch.randint(0, V, (B, k), generator=g, dtype=torch.int32)
    u = torch.rand((B, k + 1), generator=g)
    return workloads.VerifyInputs("ints", B, k, H, V, 0.0, hidden.bfloat16().to(DEV), W.bfloat16().to(DEV),
                                  tok.to(DEV), q.to(DEV), u.to(DEV))


@pytest.mark.parametrize("B,k,H,V", [(7, 0, 128, 37), (2, 3, 64, 300), (40, 3, 192, 520), (150, 3, 64, 96)])
def test_small_integer_logits_are_bit_exact(binding, B, k, H, V):
    # |values| <= 4: every product and partial sum is an integer far below 2^24, so bf16 inputs, fp32 tensor-core
    # accumulation and the fp64 oracle must agree exactly, tile tails and row-block tails included.
    w = _int_workload(B, k, H, V, seed=B * 1000 + V)
    with binding.HolaVerify(B, k, H, V) as ctx:
        out = ctx.hola_lm_head_entropy(w.hidden, w.W_lm, want_logits=True)
        torch.cuda.synchronize()
    want = ref.logits(_np(w.hidden).reshape(-1, H), _np(w.W_lm)).reshape(B, k + 1, V)
    assert np.array_equal(_np(out.logits).astype(np.float64), want)
    logZ, Hn = ref.softmax_entropy(want.reshape(-1, V))
    assert np.max(np.abs(_np(out.logZ).reshape(-1) - logZ)) < 2e-3
    assert np.max(np.abs(_np(out.entropy).reshape(-1) - Hn)) < 2e-3


def test_identity_weight_returns_hidden(binding):
    w = _int_workload(5, 1, 64, 64, seed=5, identity=True)
    with binding.HolaVerify(5, 1, 64, 64) as ctx:
        out = ctx.hola_lm_head_entropy(w.hidden, w.W_lm, want_logits=True)
        torch.cuda.synchronize()
    assert torch.equal(out.logits, w.hidden.float())


@pytest.mark.parametrize("V", [8, 16, 1000, 32000])
def test_zero_weight_gives_uniform_entropy(binding, V):
    B, k, H = 3, 2, 64
    hidden = torch.randn((B, k + 1, H), device=DEV).bfloat16()
    W = torch.zeros((V, H), device=DEV, dtype=torch.bfloat16)
    with binding.HolaVerify(B, k, H, V) as ctx:
        out = ctx.hola_lm_head_entropy(hidden, W, want_logits=False)
        torch.cuda.synchronize()
    assert torch.allclose(out.logZ, torch.full_like(out.logZ, math.log(V)), atol=1e-4)
    assert torch.allclose(out.entropy, torch.full_like(out.entropy, math.log(V)), atol=1e-4)


def test_peaked_rows_keep_entropy_accuracy(binding):
    # one logit 15 above the rest at V = 32000: H = 0.1551462, logZ - l_max = ln(1 + (V-1) e^-15)
    V, H = 32000, 64
    W = torch.zeros((V, H)); W[12345, 0] = 1.0
    hidden = torch.zeros((1, 1, H)); hidden[0, 0, 0] = 15.0
    with binding.HolaVerify(1, 0, H, V) as ctx:
        out = ctx.hola_lm_head_entropy(hidden.bfloat16().to(DEV), W.bfloat16().to(DEV), want_logits=False)
        torch.cuda.synchronize()
    tail = (V - 1) * math.exp(-15.0)
    p = 1 / (1 + tail)
    H_want = -p * math.log(p) - (1 - p) * math.log((1 - p) / (V - 1))
    assert abs(out.entropy.item() - H_want) < 1e-4
    assert abs(out.logZ.item() - (15.0 + math.log1p(tail))) < 1e-4


# ------------------------------------------------------------------------------------------ whole path, small
@pytest.mark.parametrize("tau", [None, 0.0, 1.5, float("inf"), float("nan")])
def test_tiny_config(binding, tau):
    w = workloads.make_config("tiny", DEV)
    check_against_oracle(binding, w, tau=w.tau if tau is None else tau)


@pytest.mark.parametrize("B,k,H,V,qd", [
    (3, 4, 200, 1000, torch.float32),      # K tail (H not a multiple of 64), vocab tail
    (37, 6, 256, 5000, torch.bfloat16),    # 259 rows: three row blocks, the last one ragged
    (5, 2, 64, 1001, torch.bfloat16),      # odd V: scalar load/store paths
    (130, 0, 64, 777, torch.bfloat16),     # k = 0: plain draw from p
    (90, 7, 128, 640, torch.float32),      # 720 rows: more row blocks than one pass holds
    (50, 5, 128, 80000, torch.bfloat16),   # 300 rows on rotating accumulator units (N = 112: the last 32-column
                                           # chunk half empty); five tiles per CTA pair = a full rotation period
    (46, 5, 64, 60000, torch.bfloat16),    # 276 rows: N = 96, one epilogue warp group without a chunk; four tiles
])
def test_ragged_shapes(binding, B, k, H, V, qd):
    w = workloads.gaussian_head("ragged", B, k, H, V, seed=B + V, device=DEV, w_std=0.3, sigma=1.0, q_dtype=qd,
                                tau=1.5 + 0.1 * k, sigma_far=0.2)
    out, _, _ = check_against_oracle(binding, w)
    check_ranges(w, out)


@pytest.mark.parametrize("V", [8, 16])
def test_brute_force_grid_matches_oracle_and_p(binding, V):
    # every draft token x, a grid of accept uniforms and of sampling uniforms, laid out as one batch; k = 1.
    # The emitted-token histogram, weighted by q(x), reproduces p to the grid resolution (gate off).
    rng = np.random.default_rng(V)
    H, G = 8, 24
    pw = rng.integers(1, 30, size=(2, V)).astype(np.float64); p = pw / pw.sum(-1, keepdims=True)
    qw = rng.integers(1, 30, size=V).astype(np.float64); q = qw / qw.sum()
    Wt = np.zeros((V, H), np.float32); Wt[:, 0] = np.log(p[0]); Wt[:, 1] = np.log(p[1])
    xs, ua, us = np.meshgrid(np.arange(V), (np.arange(G) + 0.5) / G, (np.arange(G) + 0.5) / G, indexing="ij")
    B = xs.size
    hidden = np.zeros((B, 2, H), np.float32); hidden[:, 0, 0] = 1.0; hidden[:, 1, 1] = 1.0
    w = workloads.VerifyInputs(
        "grid", B, 1, H, V, 0.0, torch.from_numpy(hidden).bfloat16().to(DEV), torch.from_numpy(Wt).bfloat16().to(DEV),
        torch.from_numpy(xs.reshape(B, 1).astype(np.int32)).to(DEV),
        torch.from_numpy(np.tile(q.astype(np.float32), (B, 1, 1))).to(DEV),
        torch.from_numpy(np.stack([ua.ravel(), us.ravel()], 1).astype(np.float32)).to(DEV))
    out, orc, _ = check_against_oracle(binding, w)
    # marginal of the emitted token at position 0, from the GPU outputs; p as the GPU sees it (bf16-rounded logs)
    lw = ref.bf16_bits_to_f64(ref.f32_to_bf16_bits(Wt[:, 0])); p0 = np.exp(lw) / np.exp(lw).sum()
    acc, nxt = _np(out.accept_len), _np(out.next_tok)
    emitted = np.where(acc >= 1, xs.ravel(), nxt)
    marg = np.bincount(emitted, weights=q[xs.ravel()] / (G * G), minlength=V)
    np.testing.assert_allclose(marg, p0, atol=2.0 / G)


def test_accept_sample_entry_from_oracle_logits(binding):
    # steps 3-5 alone, fed with logits, entropy and logZ made by the oracle (rounded to fp32)
    w = workloads.gaussian_head("k3", 48, 4, 64, 3000, seed=77, device="cpu", w_std=0.4, sigma=0.8, tau=0.0)
    orc0 = compare.run_oracle(w, keep_logits=True)
    l32 = orc0.logits.astype(np.float32)
    lz, Hn = ref.softmax_entropy(l32.astype(np.float64).reshape(-1, w.V))
    orc = ref.verify_from_logits(l32.astype(np.float64), _np(w.draft_tok), _np(w.draft_q), _np(w.uniforms), w.tau)
    with binding.HolaVerify(w.B, w.k, w.H, w.V) as ctx:
        out = ctx.hola_accept_sample(torch.from_numpy(l32).to(DEV), torch.from_numpy(Hn.astype(np.float32)).reshape(w.B, -1).to(DEV),
                                     torch.from_numpy(lz.astype(np.float32)).reshape(w.B, -1).to(DEV), w.draft_tok.to(DEV),
                                     w.draft_q.to(DEV), w.uniforms.to(DEV), w.tau)
        torch.cuda.synchronize()
    rep = compare.compare(orc, _np(w.draft_q), _np(w.uniforms), _np(out.accept_len), _np(out.next_tok),
                          Hn.reshape(w.B, -1), lz.reshape(w.B, -1))
    assert rep.ok and rep.accept_exact >= w.B - 1, rep.summary()
    assert 0 < _np(out.accept_len).mean() < w.k       # both branches taken


def test_maximum_sizes(binding):
    # the largest k the library takes (k + 1 = 64 positions per sequence) and the largest vocabulary (524288):
    # 2115 vocabulary tiles per launch, 4096 chunks in the accept/sample pass
    w = workloads.gaussian_head("max-k", 3, 63, 64, 300, seed=63, device=DEV, w_std=0.4, sigma=0.3, tau=3.0)
    out, _, _ = check_against_oracle(binding, w)
    check_ranges(w, out)
    assert _np(out.accept_len).max() > 5
    w = workloads.gaussian_head("max-v", 2, 1, 64, 524288, seed=64, device=DEV, w_std=0.3, sigma=1.0, tau=1.5)
    out, _, _ = check_against_oracle(binding, w)
    check_ranges(w, out)
    lib = binding.load_library()
    import ctypes
    ctx = ctypes.c_void_p()
    assert lib.hola_create(ctypes.byref(ctx), 0, 1, 1, 64, 524289) == 2      # one past the largest vocabulary


# ------------------------------------------------------------------------------------------ gate / verifier variants
@pytest.mark.parametrize("gate_source,fallback", [(1, 0), (0, 1), (1, 1)])
@pytest.mark.parametrize("B,k,H,V,qd", [(41, 5, 128, 3001, torch.bfloat16), (9, 3, 64, 1000, torch.float32)])
def test_draft_entropy_gate_and_greedy_verifier(binding, gate_source, fallback, B, k, H, V, qd):
    # w_std large enough that target rows are peaked sometimes (greedy accepts happen), draft noise small in the
    # first half; tau in the middle of the draft entropies so that both gate branches are taken.
    w = workloads.gaussian_head("variants", B, k, H, V, seed=31 * B + V, device=DEV, w_std=0.6, sigma=0.3, q_dtype=qd,
                                tau=0.0, sigma_far=1.5)
    probe = compare.run_oracle(w, keep_logits=False, gate_source=1)
    w.tau = float(np.median(probe.draft_entropy if gate_source == 1 else probe.entropy[:, :k]))
    if fallback == 1:                                    # let half of the draft tokens be the verifier's own choice
        am = torch.from_numpy(compare.run_oracle(w, keep_logits=True).logits.argmax(-1)[:, :k].astype(np.int32)).to(DEV)
        take = torch.rand((B, k), device=DEV, generator=torch.Generator(device=DEV).manual_seed(5)) < 0.6
        w.draft_tok = torch.where(take, am, w.draft_tok).contiguous()
    out, orc, rep = check_against_oracle(binding, w, gate_source=gate_source, fallback=fallback)
    check_ranges(w, out)
    acc = _np(out.accept_len)
    assert 0 < acc.mean() < k                            # some runs break, some survive
    gated = (orc.margin_gate < np.inf) & ((orc.draft_entropy if gate_source == 1 else orc.entropy[:, :k]) < w.tau)
    assert gated.any() and (~gated).any()                # both branches of the gate were evaluated
    if fallback == 1:                                    # the emitted token is always the verifier's arg-max
        lg = _np(out.logits)
        nxt = _np(out.next_tok)
        assert np.array_equal(nxt, lg[np.arange(B), acc].argmax(-1))


def test_greedy_verifier_on_the_large_vocabulary_shape(binding):
    w = workloads.make_config("large_vocab", DEV)
    out, _, _ = check_against_oracle(binding, w, seqs=[3, 30, 59], gate_source=1, fallback=1, want_logits=False)
    check_ranges(w, out)


def test_variant_arguments_are_validated(binding):
    w = workloads.gaussian_head("v", 2, 2, 64, 100, seed=1, device=DEV)
    with binding.HolaVerify(2, 2, 64, 100) as ctx:
        with pytest.raises(binding.HolaError, match="invalid argument"):
            ctx.hola_verify(w.hidden, w.W_lm, w.draft_tok, w.draft_q, w.uniforms, 1.5, gate_source=2)
        with pytest.raises(binding.HolaError, match="invalid argument"):
            ctx.hola_verify(w.hidden, w.W_lm, w.draft_tok, w.draft_q, w.uniforms, 1.5, fallback=-1)
        # a bad token still ends the run under the greedy verifier, and is flagged
        w.draft_tok[1, 0] = 100
        out = ctx.hola_verify(w.hidden, w.W_lm, w.draft_tok, w.draft_q, w.uniforms, 0.0, fallback=1)
        torch.cuda.synchronize()
        assert int(out.accept_len[1]) == 0 and int(out.status.item()) & binding.FLAG_BAD_TOKEN


# ------------------------------------------------------------------------------------------ degenerate inputs
def test_degenerate_inputs_are_flagged_not_fatal(binding):
    B, k, H, V = 4, 2, 64, 500
    w = workloads.gaussian_head("edge", B, k, H, V, seed=3, device=DEV, w_std=0.3, q_dtype=torch.float32, tau=0.0)
    w.draft_tok[0, 0] = V              # bad token -> rejection at position 0
    w.draft_tok[1, 1] = -3
    w.uniforms[2, k] = 1.0             # clamped
    w.draft_q[3] = 2.0 * torch.softmax(workloads._target_logits(w.hidden, w.W_lm)[3, :k], -1)   # q = 2p: R = 0
    w.uniforms[3, 0] = 0.75
    out, orc, _ = check_against_oracle(binding, w)
    st = int(out.status.item())
    assert st & binding.FLAG_BAD_TOKEN and st & binding.FLAG_BAD_UNIFORM and st & binding.FLAG_R_ZERO
    assert _np(out.accept_len)[0] == 0 and _np(out.accept_len)[1] <= 1 and _np(out.accept_len)[3] == 0
    assert orc.flags[3] & ref.FLAG_R_ZERO


def test_empty_batch_and_argument_errors(binding):
    import ctypes
    lib = binding.load_library()
    bad = ctypes.c_void_p()
    assert lib.hola_create(ctypes.byref(bad), 0, 1, 1, 60, 100) == 2          # H % 8 != 0
    assert lib.hola_create(ctypes.byref(bad), 0, 0, 1, 64, 100) == 1
    assert lib.hola_create(ctypes.byref(bad), 0, 1, 80, 64, 100) == 2         # k + 1 > 64
    with binding.HolaVerify(4, 2, 64, 100) as ctx:
        w = workloads.gaussian_head("e", 4, 2, 64, 100, seed=1, device=DEV)
        empty = w.slice([])
        out = ctx.hola_verify(empty.hidden, w.W_lm, empty.draft_tok, empty.draft_q, empty.uniforms, 1.5)
        assert out.accept_len.numel() == 0
        big = workloads.gaussian_head("e", 5, 2, 64, 100, seed=1, device=DEV)
        with pytest.raises(binding.HolaError, match="unsupported shape"):
            ctx.hola_verify(big.hidden, big.W_lm, big.draft_tok, big.draft_q, big.uniforms, 1.5)
        # misaligned hidden pointer
        raw = torch.zeros(4 * 3 * 64 + 8, dtype=torch.bfloat16, device=DEV)
        mis = raw[1:1 + 4 * 3 * 64].view(4, 3, 64)
        with pytest.raises(binding.HolaError, match="invalid argument"):
            ctx.hola_verify(mis, w.W_lm, w.draft_tok, w.draft_q, w.uniforms, 1.5)
        a = binding.hola_verify_args()
        assert lib.hola_verify(ctx._ctx, ctypes.byref(a), None) != 0          # all-null arguments
        assert lib.hola_verify(None, ctypes.byref(a), None) == 1


# ------------------------------------------------------------------------------------------ properties
def test_deterministic_and_batch_order_equivariant(binding):
    w = workloads.gaussian_head("perm", 33, 3, 128, 2048, seed=9, device=DEV, w_std=0.3, sigma=1.0, tau=4.0)
    a = run_gpu(binding, w, want_logits=True)
    b = run_gpu(binding, w, want_logits=True)
    for x, y in [(a.accept_len, b.accept_len), (a.next_tok, b.next_tok), (a.entropy, b.entropy), (a.logZ, b.logZ),
                 (a.logits, b.logits)]:
        assert torch.equal(x, y)
    perm = torch.randperm(w.B, generator=torch.Generator().manual_seed(1)).tolist()
    c = run_gpu(binding, w.slice(perm))
    idx = torch.tensor(perm, device=DEV)
    assert torch.equal(c.accept_len, a.accept_len[idx]) and torch.equal(c.next_tok, a.next_tok[idx])
    assert torch.allclose(c.entropy, a.entropy[idx], atol=1e-5)


@pytest.mark.parametrize("gate", [0, 1])
def test_call_can_be_captured_in_a_cuda_graph(binding, gate):
    """hola_verify neither allocates nor synchronises: a stream capture records it, and a replay on new contents of
    the same buffers gives what a direct call gives."""
    w = workloads.gaussian_head("graph", 12, 4, 128, 6000, seed=5, device=DEV, w_std=0.3, sigma=1.0, tau=4.0)
    w2 = workloads.gaussian_head("graph2", 12, 4, 128, 6000, seed=6, device=DEV, w_std=0.3, sigma=1.0, tau=4.0)
    with binding.HolaVerify(w.B, w.k, w.H, w.V) as ctx:
        bufs = [t.clone() for t in (w.hidden, w.W_lm, w.draft_tok, w.draft_q, w.uniforms)]
        out = ctx.alloc_outputs(w.B, w.k, False)
        ctx.hola_verify(*bufs, w.tau, out=out, gate_source=gate)   # warm-up outside the capture
        torch.cuda.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            ctx.hola_verify(*bufs, w.tau, out=out, gate_source=gate)
        for src in (w2, w):
            for dst, t in zip(bufs, (src.hidden, src.W_lm, src.draft_tok, src.draft_q, src.uniforms)):
                dst.copy_(t)
            out.accept_len.fill_(-1); out.next_tok.fill_(-1)
            graph.replay()
            torch.cuda.synchronize()
            ref_out = ctx.hola_verify(src.hidden, src.W_lm, src.draft_tok, src.draft_q, src.uniforms, src.tau,
                                      gate_source=gate)
            torch.cuda.synchronize()
            assert torch.equal(out.accept_len, ref_out.accept_len) and torch.equal(out.next_tok, ref_out.next_tok)
            assert torch.equal(out.entropy, ref_out.entropy) and torch.equal(out.logZ, ref_out.logZ)


@pytest.mark.parametrize("quant", [False, True])
def test_back_to_back_calls_do_not_disturb_each_other(binding, quant):
    """Calls queue on one stream without synchronisation, and each call's kernels may be scheduled while the call
    before still runs (programmatic dependent launch): 60 calls alternating between two problems must each give
    exactly what the problem gives alone."""
    ws = [workloads.gaussian_head(f"b2b{i}", 6, 4, 256, 20000, seed=40 + i, device=DEV, w_std=0.3, sigma=1.0, tau=4.0)
          for i in range(2)]
    with binding.HolaVerify(6, 4, 256, 20000) as ctx:
        Ws, scales = [], []
        for w in ws:
            if quant:
                q8, sc = binding.hola_quantize_w8(w.W_lm)
                Ws.append(q8); scales.append(sc)
            else:
                Ws.append(w.W_lm); scales.append(None)
        kw = [dict(w_scale=sc, a8=True) if quant else {} for sc in scales]
        alone = []
        for w, W, k in zip(ws, Ws, kw):
            alone.append(ctx.hola_verify(w.hidden, W, w.draft_tok, w.draft_q, w.uniforms, w.tau, **k))
            torch.cuda.synchronize()
        outs = [ctx.alloc_outputs(6, 4, False) for _ in range(60)]
        for i, o in enumerate(outs):
            w, W, k = ws[i & 1], Ws[i & 1], kw[i & 1]
            ctx.hola_verify(w.hidden, W, w.draft_tok, w.draft_q, w.uniforms, w.tau, out=o, **k)
        torch.cuda.synchronize()
    for i, o in enumerate(outs):
        r = alone[i & 1]
        assert torch.equal(o.accept_len, r.accept_len) and torch.equal(o.next_tok, r.next_tok), i
        assert torch.equal(o.entropy, r.entropy) and torch.equal(o.logZ, r.logZ), i


def test_outputs_stay_inside_their_buffers(binding):
    # canary words before and after every output
    B, k, H, V = 6, 3, 64, 333
    w = workloads.gaussian_head("canary", B, k, H, V, seed=4, device=DEV, w_std=0.3)
    pad = 64

    def padded(n, dtype, fill):
        buf = torch.full((n + 2 * pad,), fill, dtype=dtype, device=DEV)
        return buf, buf[pad:pad + n]

    bufs = {}
    with binding.HolaVerify(B, k, H, V) as ctx:
        out = ctx.alloc_outputs(B, k, True)
        bufs["a"], a = padded(B, torch.int32, -7); out.accept_len = a
        bufs["n"], n = padded(B, torch.int32, -7); out.next_tok = n
        bufs["e"], e = padded(B * (k + 1), torch.float32, -7.0); out.entropy = e.view(B, k + 1)
        bufs["z"], z = padded(B * (k + 1), torch.float32, -7.0); out.logZ = z.view(B, k + 1)
        bufs["l"], l = padded(B * (k + 1) * V, torch.float32, -7.0); out.logits = l.view(B, k + 1, V)
        ctx.hola_verify(w.hidden, w.W_lm, w.draft_tok, w.draft_q, w.uniforms, 1.5, out=out)
        torch.cuda.synchronize()
    for name, buf in bufs.items():
        assert torch.all(buf[:pad] == -7) and torch.all(buf[-pad:] == -7), name
    assert torch.all(out.accept_len >= 0) and torch.all(out.logits != -7.0)


def test_host_entry_equals_device_entry(binding):
    w = workloads.gaussian_head("host", 9, 3, 128, 4000, seed=12, device=DEV, w_std=0.3, tau=5.0)
    with binding.HolaVerify(w.B, w.k, w.H, w.V) as ctx:
        d = ctx.hola_verify(w.hidden, w.W_lm, w.draft_tok, w.draft_q, w.uniforms, w.tau)
        torch.cuda.synchronize()
        h = ctx.hola_verify_host(w.hidden.cpu().pin_memory(), w.W_lm, w.draft_tok.cpu().pin_memory(),
                                 w.draft_q.cpu().pin_memory(), w.uniforms.cpu().pin_memory(), w.tau)
    assert torch.equal(h.accept_len, d.accept_len.cpu()) and torch.equal(h.next_tok, d.next_tok.cpu())
    assert torch.equal(h.entropy, d.entropy.cpu()) and torch.equal(h.logZ, d.logZ.cpu())


@pytest.mark.parametrize("pinned", [True, False])
def test_host_entry_reads_missing_rows_in_place_or_copies_them(binding, pinned):
    """With the draft tensor in pinned host memory the rows not sent ahead are read in place by the accept/sample kernel;
    with pageable memory, or with the option off, they are copied after a read-back of accept_len.  Same results, same
    byte count, either way."""
    w = workloads.gaussian_head("in-place", 21, 4, 128, 5000, seed=78, device=DEV, w_std=0.3, tau=0.0)
    mem = (lambda t: t.cpu().pin_memory()) if pinned else (lambda t: t.cpu().clone())
    host = [mem(t) for t in (w.hidden, w.draft_tok, w.draft_q, w.uniforms)]
    outs, traffic = [], []
    with binding.HolaVerify(w.B, w.k, w.H, w.V) as ctx:
        ctx.hola_set_option(binding.HOLA_OPT_HOST_ROWS_ON_DEMAND, 1)
        d = ctx.hola_verify(w.hidden, w.W_lm, w.draft_tok, w.draft_q, w.uniforms, w.tau)
        torch.cuda.synchronize()
        for in_place in (1, 0):
            ctx.hola_set_option(binding.HOLA_OPT_HOST_IN_PLACE, in_place)
            outs.append(ctx.hola_verify_host(host[0], w.W_lm, host[1], host[2], host[3], w.tau))
            traffic.append(ctx.hola_host_traffic()[0])
    for h in outs:
        assert torch.equal(h.accept_len, d.accept_len.cpu()) and torch.equal(h.next_tok, d.next_tok.cpu())
        assert torch.equal(h.entropy, d.entropy.cpu()) and torch.equal(h.logZ, d.logZ.cpu())
    assert traffic[0] == traffic[1]
    assert len(set(d.accept_len.tolist())) >= 3              # rows beyond the ones sent ahead are needed


@pytest.mark.parametrize("q_dtype", [torch.bfloat16, torch.float32])
@pytest.mark.parametrize("gate,fallback", [(0, 0), (0, 1), (1, 0)])
@pytest.mark.parametrize("tau", [0.0, None, 100.0])
def test_host_entry_sends_only_the_rows_it_reads(binding, q_dtype, gate, fallback, tau):
    """hola_verify_host against hola_verify on the same data, over accept lengths from 0 to k (tau = 0: gate off;
    None: the median entropy; 100: every draft kept), with poisoned staging so that a row that was needed but not copied would show."""
    w = workloads.gaussian_head("host_rows", 21, 4, 128, 5000, seed=77, device=DEV, w_std=0.3, tau=tau,
                                q_dtype=q_dtype)
    pin = lambda t: t.cpu().pin_memory()
    with binding.HolaVerify(w.B, w.k, w.H, w.V) as ctx:
        ctx.hola_set_option(binding.HOLA_OPT_HOST_ROWS_ON_DEMAND, 1)     # this small tensor would otherwise be copied whole
        # a first host call with a wrong draft tensor leaves stale rows in the staging area
        ctx.hola_verify_host(pin(w.hidden), w.W_lm, pin(w.draft_tok), pin(torch.flip(w.draft_q, dims=[2])),
                             pin(w.uniforms), w.tau, gate_source=gate, fallback=fallback)
        d = ctx.hola_verify(w.hidden, w.W_lm, w.draft_tok, w.draft_q, w.uniforms, w.tau, gate_source=gate,
                            fallback=fallback)
        torch.cuda.synchronize()
        h = ctx.hola_verify_host(pin(w.hidden), w.W_lm, pin(w.draft_tok), pin(w.draft_q), pin(w.uniforms), w.tau,
                                 gate_source=gate, fallback=fallback)
        up, down = ctx.hola_host_traffic()
    assert torch.equal(h.accept_len, d.accept_len.cpu()) and torch.equal(h.next_tok, d.next_tok.cpu())
    assert torch.equal(h.entropy, d.entropy.cpu()) and torch.equal(h.logZ, d.logZ.cpu())
    assert int(h.status.item()) == int(d.status.item())
    if tau == 0.0 and fallback == 0:
        assert len(set(h.accept_len.tolist())) >= 3      # the case does spread over several accept lengths
    q_bytes = w.draft_q.numel() * w.draft_q.element_size()
    row = w.V * w.draft_q.element_size()
    # hidden rows, then tokens + uniforms (+ gathered probabilities) as one copy of a workspace span whose pieces
    # start on 256-byte boundaries: up to 255 bytes of padding after each piece but the last
    small = w.hidden.numel() * 2 + w.draft_tok.numel() * 4 + w.uniforms.numel() * 4
    if gate == 1:
        assert 0 <= up - (small + q_bytes) < 256          # the draft entropy reads every row
    elif fallback == 1:
        assert 0 <= up - (small + w.B * w.k * 4) < 512    # greedy: no row at all
    else:
        n = h.accept_len                                  # rows 0 .. ahead-1 go first, then the rows still missing
        pad = [up - (small + w.B * w.k * 4 + (w.B * ahead + int(((n >= ahead) & (n < w.k)).sum())) * row)
               for ahead in range(1, w.k + 1)]
        assert any(0 <= x < 512 for x in pad)
        assert up < small + q_bytes                       # and that is less than the whole tensor


# ------------------------------------------------------------------------------------------ 8-bit LM head
def _w8_oracle(w, q8, scale, a8=False, **kw):
    """The oracle on the dequantised head: hidden widened to fp64 (or, with a8, quantised row by row with the same
    rule and dequantised), W8 = scale * q in fp64."""
    from oracle import lobi
    hid = ref.bf16_bits_to_f64(_np(w.hidden))
    if a8:
        B, k1, H = hid.shape
        hq, hs = lobi.quantize_rows_int8(hid.reshape(B * k1, H).astype(np.float32))
        hid = lobi.dequantize_rows(hq, hs).reshape(B, k1, H)
    W8 = lobi.dequantize_rows(_np(q8), _np(scale))
    return ref.verify(hid, W8, _np(w.draft_tok), _np(w.draft_q), _np(w.uniforms), w.tau, keep_logits=True, **kw)


@pytest.mark.parametrize("V,H", [(1000, 64), (4099, 208), (32000, 128)])
def test_quantiser_is_bit_exact(binding, V, H):
    from oracle import lobi
    g = torch.Generator(device=DEV).manual_seed(V)
    W = (torch.randn((V, H), generator=g, device=DEV) * 0.02).bfloat16()
    W[3] = 0
    W[5, :4] = torch.tensor([1.0, 0.00390625, -0.01171875, 0.01953125], device=DEV).bfloat16()    # exact ties at 127 steps
    W[5, 4:] = 0
    q8, scale = binding.hola_quantize_w8(W)
    torch.cuda.synchronize()
    want_q, want_s = lobi.quantize_rows_int8(W.float().cpu().numpy())
    assert np.array_equal(_np(scale), want_s)
    assert np.array_equal(_np(q8), want_q)


@pytest.mark.parametrize("B,k,H,V,qd", [
    (1, 4, 64, 1000, torch.float32),       # the tiny shape
    (37, 6, 256, 5000, torch.bfloat16),    # 259 rows: two passes of the 8-bit kernel, ragged vocabulary tail
    (5, 2, 80, 1001, torch.bfloat16),      # K tail (H = 80), odd V
    (70, 3, 128, 640, torch.float32),      # 280 rows
])
def test_int8_head_matches_oracle_on_dequantised_weights(binding, B, k, H, V, qd):
    w = workloads.gaussian_head("w8", B, k, H, V, seed=B + V, device=DEV, w_std=0.3, sigma=1.0, q_dtype=qd,
                                tau=1.5 + 0.1 * k, sigma_far=0.2)
    q8, scale = binding.hola_quantize_w8(w.W_lm)
    with binding.HolaVerify(B, k, H, V) as ctx:
        out = ctx.hola_verify(w.hidden, q8, w.draft_tok, w.draft_q, w.uniforms, w.tau, want_logits=True, w_scale=scale)
        torch.cuda.synchronize()
    assert int(out.status.item()) & binding.FLAG_TIMEOUT == 0
    orc = _w8_oracle(w, q8, scale)
    rep = compare.compare(orc, _np(w.draft_q), _np(w.uniforms), _np(out.accept_len), _np(out.next_tok),
                          _np(out.entropy), _np(out.logZ), _np(out.logits))
    print(rep.summary())
    assert rep.ok, rep.summary()
    assert rep.accept_margin_cases <= max(1, B // 20) and rep.token_margin_cases <= max(1, B // 10)
    check_ranges(w, out)
    # and the quantised head stays close to the bf16 head it came from
    full = compare.run_oracle(w, keep_logits=False)
    assert np.max(np.abs(orc.entropy - full.entropy)) < 0.25


@pytest.mark.parametrize("B,k,H,V,qd", [
    (1, 4, 64, 1000, torch.float32),       # 5 rows: N = 32
    (37, 6, 256, 5000, torch.bfloat16),    # 259 rows: three MMAs of N = 96 per K step, ragged vocabulary tail
    (5, 2, 80, 1001, torch.bfloat16),      # K tail (H = 80 < one 128-wide block), odd V
    (90, 7, 384, 640, torch.float32),      # 720 rows: two passes
    (50, 5, 128, 80000, torch.bfloat16),   # 300 rows, N = 128 on rotating units, five tiles per CTA pair
    (75, 5, 128, 3000, torch.bfloat16),    # 450 rows: two MMAs of N = 256 fill the tensor memory
])
def test_w8a8_head_matches_oracle_on_dequantised_operands(binding, B, k, H, V, qd):
    w = workloads.gaussian_head("w8a8", B, k, H, V, seed=B + V, device=DEV, w_std=0.3, sigma=1.0, q_dtype=qd,
                                tau=1.5 + 0.1 * k, sigma_far=0.2)
    q8, scale = binding.hola_quantize_w8(w.W_lm)
    with binding.HolaVerify(B, k, H, V) as ctx:
        out = ctx.hola_verify(w.hidden, q8, w.draft_tok, w.draft_q, w.uniforms, w.tau, want_logits=True, w_scale=scale,
                              a8=True)
        torch.cuda.synchronize()
    assert int(out.status.item()) & binding.FLAG_TIMEOUT == 0
    orc = _w8_oracle(w, q8, scale, a8=True)
    rep = compare.compare(orc, _np(w.draft_q), _np(w.uniforms), _np(out.accept_len), _np(out.next_tok),
                          _np(out.entropy), _np(out.logZ), _np(out.logits))
    print(rep.summary())
    assert rep.ok, rep.summary()
    assert rep.accept_margin_cases <= max(1, B // 20) and rep.token_margin_cases <= max(1, B // 10)
    check_ranges(w, out)


def test_w8a8_integer_operands_are_bit_exact(binding):
    # integer weights and hidden rows with row maximum 127: both scales are 1, every product and sum is exact
    g = torch.Generator().manual_seed(10)
    B, k, H, V = 40, 3, 192, 520
    hf = torch.randint(-6, 7, (B, k + 1, H), generator=g).float()
    hf[..., 0] = 127.0
    Wf = torch.randint(-5, 6, (V, H), generator=g).float()
    Wf[:, 1] = -127.0
    hidden, W = hf.bfloat16().to(DEV), Wf.bfloat16().to(DEV)
    q8, scale = binding.hola_quantize_w8(W)
    with binding.HolaVerify(B, k, H, V) as ctx:
        out = ctx.hola_lm_head_entropy(hidden, q8, want_logits=True, w_scale=scale, a8=True)
        torch.cuda.synchronize()
    want = ref.logits(_np(hidden).reshape(-1, H), _np(W)).reshape(B, k + 1, V)
    assert np.array_equal(_np(out.logits).astype(np.float64), want)


def test_w8a8_on_the_large_vocabulary_shape(binding):
    w = workloads.make_config("large_vocab", DEV)
    q8, scale = binding.hola_quantize_w8(w.W_lm)
    with binding.HolaVerify(w.B, w.k, w.H, w.V) as ctx:
        out = ctx.hola_verify(w.hidden, q8, w.draft_tok, w.draft_q, w.uniforms, w.tau, want_logits=True, w_scale=scale,
                              a8=True)
        torch.cuda.synchronize()
    seqs = [1, 22, 63]
    sub = w.slice(seqs)
    orc = _w8_oracle(sub, q8, scale, a8=True)
    idx = np.asarray(seqs)
    rep = compare.compare(orc, _np(sub.draft_q), _np(sub.uniforms), _np(out.accept_len)[idx], _np(out.next_tok)[idx],
                          _np(out.entropy)[idx], _np(out.logZ)[idx], _np(out.logits)[idx])
    assert rep.ok, rep.summary()
    check_ranges(w, out)


# ---- 8-bit weights, 16-bit-class activations (two 8-bit planes)
def _w8a16_oracle(w, q8, scale, **kw):
    """The oracle on both operands as the kernel sees them: hidden rows = s1 q1 + s2 q2 (fp64), W8 = scale * q."""
    from oracle import lobi
    hid = ref.bf16_bits_to_f64(_np(w.hidden))
    B, k1, H = hid.shape
    h16 = lobi.dequantize_two_plane(*lobi.quantize_rows_two_plane(hid.reshape(B * k1, H).astype(np.float32)))
    W8 = lobi.dequantize_rows(_np(q8), _np(scale))
    return ref.verify(h16.reshape(B, k1, H), W8, _np(w.draft_tok), _np(w.draft_q), _np(w.uniforms), w.tau,
                      keep_logits=True, **kw)


@pytest.mark.parametrize("B,k,H,V,qd", [
    (1, 4, 64, 1000, torch.float32),       # 5 rows: one block of 32, N = 64
    (37, 6, 256, 5000, torch.bfloat16),    # 259 rows: two passes (at most 256 verify rows each)
    (5, 2, 80, 1001, torch.bfloat16),      # K tail, odd V
    (33, 3, 128, 40000, torch.bfloat16),   # 132 rows: 320 operand rows, two MMAs of N = 192, last block of 32 ragged
    (75, 2, 128, 3000, torch.bfloat16),    # 225 rows: 512 operand rows, two MMAs of N = 256
    (21, 5, 128, 3000, torch.float32),     # 126 rows: N = 256, double-buffered accumulators
])
def test_w8a16_head_matches_oracle_on_two_plane_rows(binding, B, k, H, V, qd):
    w = workloads.gaussian_head("w8a16", B, k, H, V, seed=B + V, device=DEV, w_std=0.3, sigma=1.0, q_dtype=qd,
                                tau=1.5 + 0.1 * k, sigma_far=0.2)
    q8, scale = binding.hola_quantize_w8(w.W_lm)
    with binding.HolaVerify(B, k, H, V) as ctx:
        out = ctx.hola_verify(w.hidden, q8, w.draft_tok, w.draft_q, w.uniforms, w.tau, want_logits=True, w_scale=scale,
                              a8="a16")
        torch.cuda.synchronize()
    assert int(out.status.item()) & binding.FLAG_TIMEOUT == 0
    orc = _w8a16_oracle(w, q8, scale)
    rep = compare.compare(orc, _np(w.draft_q), _np(w.uniforms), _np(out.accept_len), _np(out.next_tok),
                          _np(out.entropy), _np(out.logZ), _np(out.logits))
    print(rep.summary())
    assert rep.ok, rep.summary()
    assert rep.accept_margin_cases <= max(1, B // 20) and rep.token_margin_cases <= max(1, B // 10)
    check_ranges(w, out)
    # and the two planes keep the logits within 1e-3 of the 8-bit head on the unquantised bf16 rows
    exact = _w8_oracle(w, q8, scale)
    assert np.max(np.abs(_np(out.logits) - exact.logits)) < 2e-3


def test_w8a16_integer_operands_are_bit_exact(binding):
    # integer rows with maximum 127: s1 = 1, the first plane is the row, the second plane is zero
    g = torch.Generator().manual_seed(11)
    B, k, H, V = 40, 3, 192, 520
    hf = torch.randint(-6, 7, (B, k + 1, H), generator=g).float()
    hf[..., 0] = 127.0
    Wf = torch.randint(-5, 6, (V, H), generator=g).float()
    Wf[:, 1] = -127.0
    hidden, W = hf.bfloat16().to(DEV), Wf.bfloat16().to(DEV)
    q8, scale = binding.hola_quantize_w8(W)
    with binding.HolaVerify(B, k, H, V) as ctx:
        out = ctx.hola_lm_head_entropy(hidden, q8, want_logits=True, w_scale=scale, a8="a16")
        torch.cuda.synchronize()
    want = ref.logits(_np(hidden).reshape(-1, H), _np(W)).reshape(B, k + 1, V)
    assert np.array_equal(_np(out.logits).astype(np.float64), want)


@pytest.mark.parametrize("name", ["edge", "large_vocab_b32"])
def test_w8a16_on_the_bandwidth_bound_shapes(binding, name):
    w = workloads.make_config(name, DEV)
    q8, scale = binding.hola_quantize_w8(w.W_lm)
    with binding.HolaVerify(w.B, w.k, w.H, w.V) as ctx:
        out = ctx.hola_verify(w.hidden, q8, w.draft_tok, w.draft_q, w.uniforms, w.tau, want_logits=True, w_scale=scale,
                              a8="a16")
        torch.cuda.synchronize()
    seqs = [0] if w.B == 1 else [0, 13, w.B - 1]
    sub = w.slice(seqs)
    orc = _w8a16_oracle(sub, q8, scale)
    idx = np.asarray(seqs)
    rep = compare.compare(orc, _np(sub.draft_q), _np(sub.uniforms), _np(out.accept_len)[idx], _np(out.next_tok)[idx],
                          _np(out.entropy)[idx], _np(out.logZ)[idx], _np(out.logits)[idx])
    assert rep.ok, rep.summary()
    check_ranges(w, out)


def test_int8_head_small_integer_weights_are_bit_exact(binding):
    # integer weights with row maximum 127: scale = 1, q = W, every product and sum exact
    g = torch.Generator().manual_seed(9)
    B, k, H, V = 40, 3, 192, 520
    hidden = torch.randint(-4, 5, (B, k + 1, H), generator=g).float().bfloat16().to(DEV)
    Wf = torch.randint(-5, 6, (V, H), generator=g).float()
    Wf[:, 0] = 127.0
    W = Wf.bfloat16().to(DEV)
    q8, scale = binding.hola_quantize_w8(W)
    assert torch.all(scale == 1.0) and torch.equal(q8.float(), W.float())
    with binding.HolaVerify(B, k, H, V) as ctx:
        out = ctx.hola_lm_head_entropy(hidden, q8, want_logits=True, w_scale=scale)
        torch.cuda.synchronize()
    want = ref.logits(_np(hidden).reshape(-1, H), _np(W)).reshape(B, k + 1, V)
    assert np.array_equal(_np(out.logits).astype(np.float64), want)


def test_int8_head_on_the_edge_shape(binding):
    w = workloads.make_config("edge", DEV)
    q8, scale = binding.hola_quantize_w8(w.W_lm)
    with binding.HolaVerify(w.B, w.k, w.H, w.V) as ctx:
        out = ctx.hola_verify(w.hidden, q8, w.draft_tok, w.draft_q, w.uniforms, w.tau, want_logits=True, w_scale=scale)
        torch.cuda.synchronize()
        with pytest.raises(binding.HolaError):
            ctx.hola_verify(w.hidden, q8, w.draft_tok, w.draft_q, w.uniforms, w.tau)          # int8 without scales
    orc = _w8_oracle(w, q8, scale)
    rep = compare.compare(orc, _np(w.draft_q), _np(w.uniforms), _np(out.accept_len), _np(out.next_tok),
                          _np(out.entropy), _np(out.logZ), _np(out.logits))
    assert rep.ok and rep.max_logit_rel_err < 1e-3, rep.summary()


# ------------------------------------------------------------------------------------------ multi-round decode loop
@pytest.mark.parametrize("gate_source,fallback", [(0, 0), (1, 1)])
def test_multi_round_decode_loop(binding, gate_source, fallback):
    # Algorithm 1 as a loop: every round's verify call agrees with the oracle on that round's arrays, and the
    # context grows by exactly the accepted drafts plus the verifier's token.
    from paper_2506_18952_b200 import driver
    B, k, H, V, rounds = 6, 3, 128, 2000, 5
    models = driver.SyntheticPair(V, H, seed=77, device=torch.device(DEV))
    prompt = torch.randint(0, V, (B, 2), device=DEV, generator=torch.Generator(device=DEV).manual_seed(3))
    with binding.HolaVerify(B, k, H, V) as ctx:
        res = driver.hsd_decode(ctx, models, prompt, k, 1.5, rounds, seed=11, gate_source=gate_source,
                                fallback=fallback, keep_records=True)
    want = [list(map(int, prompt[b])) for b in range(B)]
    gated = 0
    for rec in res.records:
        w = workloads.VerifyInputs("round", B, k, H, V, 1.5, rec.hidden, models.W_lm, rec.draft_tok, rec.draft_q,
                                   rec.uniforms)
        check_against_oracle(binding, w, out=rec.out, gate_source=gate_source, fallback=fallback)
        gated += int((rec.out.entropy[:, :k] < 1.5).sum())
        for b in range(B):
            n = int(rec.out.accept_len[b])
            want[b] += list(map(int, rec.draft_tok[b, :n])) + [int(rec.out.next_tok[b])]
    for b in range(B):
        assert int(res.lengths[b]) == len(want[b]) and list(map(int, res.tokens[b, :len(want[b])])) == want[b]
    emitted = int((res.lengths - 2).sum())
    assert B * rounds <= emitted <= B * rounds * (k + 1) and emitted > B * rounds     # more than one token per call
    assert res.verify_ms > 0 and res.total_ms >= res.verify_ms


# ------------------------------------------------------------------------------------------ failure path, options
def test_a_wait_that_runs_out_is_reported_and_leaves_the_device_usable(binding):
    """The bounded waits, exercised for real but in miniature: a barrier that nothing signals, a limit of 1e5 cycles.
    The wait must give up, raise the time-out flag, make the whole CTA pair leave through the common tail (tensor
    memory released), and an ordinary verify call right behind it must be unaffected."""
    w = workloads.gaussian_head("after-timeout", 6, 3, 128, 3000, seed=5, device=DEV, w_std=0.3)
    with binding.HolaVerify(w.B, w.k, w.H, w.V) as ctx:
        want = ctx.hola_verify(w.hidden, w.W_lm, w.draft_tok, w.draft_q, w.uniforms, w.tau)
        torch.cuda.synchronize()
        for limit in (20000, 100000):
            status, reached, gave_up = ctx.hola_selftest_bounded_wait(limit)
            assert status & binding.FLAG_TIMEOUT and status & ~binding.FLAG_TIMEOUT == 0
            assert reached == 128 and gave_up == 4
        got = ctx.hola_verify(w.hidden, w.W_lm, w.draft_tok, w.draft_q, w.uniforms, w.tau)
        torch.cuda.synchronize()
        assert int(got.status.item()) == 0
        for f in ("accept_len", "next_tok", "entropy", "logZ"):
            assert torch.equal(getattr(got, f), getattr(want, f))
        with pytest.raises(binding.HolaError):
            ctx.hola_selftest_bounded_wait(10)                       # below the accepted range: nothing launched
        with pytest.raises(binding.HolaError):
            ctx.hola_selftest_bounded_wait(10 ** 12)
    check_against_oracle(binding, w, out=got, want_logits=False)


def test_inputs_written_by_the_kernel_just_before_the_call_are_seen(binding):
    """Tokens, uniforms and draft probabilities produced on the same stream right before the call (no synchronisation in
    between) must be the ones the step uses: the accept/sample kernel may be scheduled early, but reads its inputs only
    once the work in front of it is known to be complete."""
    w = workloads.gaussian_head("fresh-inputs", 40, 5, 128, 6000, seed=31, device=DEV, w_std=0.3, sigma=1.0)
    orc = compare.run_oracle(w, keep_logits=True)
    lg = torch.from_numpy(orc.logits).float().to(DEV)
    ent = torch.from_numpy(orc.entropy).float().to(DEV)
    lz = torch.from_numpy(orc.logZ).float().to(DEV)
    with binding.HolaVerify(w.B, w.k, w.H, w.V) as ctx:
        for _ in range(5):
            tok = torch.full_like(w.draft_tok, -1)                   # stale values a too-early read would pick up
            u = torch.full_like(w.uniforms, 2.0)
            q = torch.zeros_like(w.draft_q)
            big = torch.empty(64 << 20, dtype=torch.uint8, device=DEV)
            torch.cuda.synchronize()
            big.zero_()                                              # keeps the stream busy while the copies queue up
            tok.copy_(w.draft_tok); u.copy_(w.uniforms); q.copy_(w.draft_q)
            a = ctx.hola_accept_sample(lg, ent, lz, tok, q, u, w.tau)
            b = ctx.hola_verify(w.hidden, w.W_lm, tok, q, u, w.tau)
            torch.cuda.synchronize()
            for out in (a, b):
                assert int(out.status.item()) == 0
                rep = compare.compare(orc, _np(w.draft_q), _np(w.uniforms), _np(out.accept_len), _np(out.next_tok),
                                      _np(out.entropy), _np(out.logZ))
                assert rep.ok and rep.accept_margin_cases + rep.token_margin_cases <= 2, rep.summary()


def test_options_change_speed_knobs_not_results(binding):
    w = workloads.gaussian_head("options", 50, 5, 256, 9000, seed=17, device=DEV, w_std=0.3)     # 300 rows: rotating units
    with binding.HolaVerify(w.B, w.k, w.H, w.V) as ctx:
        base = ctx.hola_verify(w.hidden, w.W_lm, w.draft_tok, w.draft_q, w.uniforms, w.tau)
        plan0 = ctx.hola_plan(w.B, w.k)
        torch.cuda.synchronize()
        for opt, val in ((binding.HOLA_OPT_RING_SLOTS, 3), (binding.HOLA_OPT_ROTATING_UNITS, 0)):
            ctx.hola_set_option(opt, val)
            out = ctx.hola_verify(w.hidden, w.W_lm, w.draft_tok, w.draft_q, w.uniforms, w.tau)
            torch.cuda.synchronize()
            assert torch.equal(out.accept_len, base.accept_len) and torch.equal(out.next_tok, base.next_tok)
            assert torch.allclose(out.entropy, base.entropy, atol=1e-5) and torch.allclose(out.logZ, base.logZ, atol=1e-5)
        assert ctx.hola_plan(w.B, w.k)["stages"] == 3 and plan0["stages"] > 3
        with pytest.raises(binding.HolaError):
            ctx.hola_set_option(99, 1)
        with pytest.raises(binding.HolaError):
            ctx.hola_set_option(binding.HOLA_OPT_RING_SLOTS, 1)


@pytest.mark.parametrize("a8", [False, True])
def test_pair_mma_on_rotating_units_matches_oracle_and_the_three_mma_form(binding, a8):
    """378 rows: three row blocks of 128 (the last one ragged) on rotating units, two of them under one MMA of N = 256;
    20 000 vocabulary rows give every CTA pair a tile, the first pairs two, so both placements of the pair occur."""
    w = workloads.gaussian_head("pair-mma", 63, 5, 256, 20000, seed=23, device=DEV, w_std=0.3, sigma=1.0, sigma_far=0.2)
    W, sc = (binding.hola_quantize_w8(w.W_lm) if a8 else (w.W_lm, None))
    with binding.HolaVerify(w.B, w.k, w.H, w.V) as ctx:
        out = ctx.hola_verify(w.hidden, W, w.draft_tok, w.draft_q, w.uniforms, w.tau, want_logits=True, w_scale=sc, a8=a8)
        torch.cuda.synchronize()
        ctx.hola_set_option(binding.HOLA_OPT_PAIR_MMA, 0)
        three = ctx.hola_verify(w.hidden, W, w.draft_tok, w.draft_q, w.uniforms, w.tau, want_logits=True, w_scale=sc, a8=a8)
        torch.cuda.synchronize()
    assert int(out.status.item()) == 0
    assert torch.equal(out.accept_len, three.accept_len) and torch.equal(out.next_tok, three.next_tok)
    assert torch.allclose(out.logits, three.logits, rtol=1e-5, atol=1e-5)
    if a8:
        orc = _w8_oracle(w, W, sc, a8=True)
        rep = compare.compare(orc, _np(w.draft_q), _np(w.uniforms), _np(out.accept_len), _np(out.next_tok),
                              _np(out.entropy), _np(out.logZ), _np(out.logits))
        assert rep.ok, rep.summary()
    else:
        check_against_oracle(binding, w, out=out)


def test_repeated_calls_reuse_the_set_up_and_new_pointers_do_not(binding):
    """Same pointers and sizes: the second call takes its tensor maps from the context.  Other tensors of the same shape,
    or another batch size, must not be served from what the first call left."""
    w1 = workloads.gaussian_head("cache-1", 12, 3, 128, 4000, seed=1, device=DEV, w_std=0.3)
    w2 = workloads.gaussian_head("cache-2", 12, 3, 128, 4000, seed=2, device=DEV, w_std=0.3)
    w3 = workloads.gaussian_head("cache-3", 7, 3, 128, 4000, seed=3, device=DEV, w_std=0.3)
    with binding.HolaVerify(12, 3, 128, 4000) as ctx:
        for w in (w1, w1, w2, w3, w1, w2):
            out = ctx.hola_verify(w.hidden, w.W_lm, w.draft_tok, w.draft_q, w.uniforms, w.tau, want_logits=True)
            torch.cuda.synchronize()
            check_against_oracle(binding, w, out=out)


# ------------------------------------------------------------------------------------------ the named workloads
def test_edge_decode_config_full(binding):
    w = workloads.make_config("edge", DEV)
    out, _, rep = check_against_oracle(binding, w)
    check_ranges(w, out)
    assert rep.max_logit_rel_err < 1e-3


def test_batched_serving_config(binding):
    w = workloads.make_config("batched", DEV)
    out, orc, rep = check_against_oracle(binding, w)       # all 64 sequences, logits included
    assert rep.n_seq == w.B
    check_ranges(w, out)
    acc = _np(out.accept_len)
    assert acc[:32].mean() > acc[32:].mean() + 1.0      # near-p half keeps more drafts than the far half


def test_large_vocab_config(binding):
    """All 64 sequences, all three thresholds of the sweep.  The fp64 logits do not depend on tau, so the oracle makes
    them once and repeats only its steps 2-6 for each threshold."""
    w = workloads.make_config("large_vocab", DEV)
    lg = ref.logits(_np(w.hidden).reshape(w.M, w.H), _np(w.W_lm)).reshape(w.B, w.k + 1, w.V)
    with binding.HolaVerify(w.B, w.k, w.H, w.V) as ctx:
        for tau in (1.0, 2.0, 4.0):
            out = run_gpu(binding, w, want_logits=True, tau=tau, ctx=ctx)
            assert int(out.status.item()) & binding.FLAG_TIMEOUT == 0
            orc = ref.verify_from_logits(lg, _np(w.draft_tok), _np(w.draft_q), _np(w.uniforms), tau)
            rep = compare.compare(orc, _np(w.draft_q), _np(w.uniforms), _np(out.accept_len), _np(out.next_tok),
                                  _np(out.entropy), _np(out.logZ), _np(out.logits))
            print("large_vocab tau", tau, rep.summary())
            assert rep.ok and rep.n_seq == w.B, rep.summary() + f" {rep.accept_failures[:5]} {rep.token_failures[:5]}"
            assert rep.accept_margin_cases <= 3 and rep.token_margin_cases <= 6
            check_ranges(w, out)
            gated = (_np(out.entropy)[:, :w.k] < tau).sum()
            assert 0 < gated < w.B * w.k                    # the sweep exercises both branches of the gate
    H = _np(out.entropy)
    assert H.min() < 1.0 and H.max() > 6.0              # the entropy spread the workload asks for


def wide_sample(B=256, k1=9, rows_per_pass=384, n=32):
    """Sequences of the `wide` workload, evenly spread, such that every pass over W_lm and every 128-row accumulator
    unit inside a pass holds rows of at least one of them, peaked and flat rows alike."""
    seqs = sorted({round(i * (B - 1) / (n - 1)) for i in range(n)})
    hit = {((b * k1 + j) // rows_per_pass, ((b * k1 + j) % rows_per_pass) // 128) for b in seqs for j in range(k1)}
    passes = (B * k1 + rows_per_pass - 1) // rows_per_pass
    assert hit == {(p, u) for p in range(passes) for u in range(3)}
    return seqs


def test_wide_head_config(binding):
    w = workloads.make_config("wide", DEV)
    with binding.HolaVerify(w.B, w.k, w.H, w.V) as ctx:
        plan = ctx.hola_plan(w.B, w.k)
    seqs = wide_sample(w.B, w.k + 1, plan["rows_per_pass"])
    assert len(seqs) >= 32
    out, _, rep = check_against_oracle(binding, w, seqs=seqs, want_logits=True)
    assert rep.n_seq == len(seqs)
    check_ranges(w, out)
    H = _np(out.entropy).reshape(-1)
    assert (H[0::2] < 1.5).mean() > 0.9 and (H[1::2] > 10).mean() > 0.9     # peaked and flat rows


@pytest.mark.parametrize("B,k,H,V,weights", [
    (150, 5, 256, 9000, "bf16"),       # 900 rows: several passes, the last one ragged; more tiles than groups of pairs
    (150, 5, 256, 700, "bf16"),        # three tiles only: fewer tiles than groups of pairs
    (100, 7, 128, 5000, "w8a8"),       # 800 rows on the 8-bit kind
    (130, 3, 256, 4000, "mixed"),      # 520 rows, at most 256 per pass in the on-chip expansion
])
def test_all_passes_in_one_launch_match_the_oracle_and_the_launch_per_pass(binding, B, k, H, V, weights):
    """More verify rows than one pass over W_lm holds: by default every pass runs in the same launch (groups of CTA
    pairs share the vocabulary tiles, one pass each); the option brings back one launch per pass.  Same results, and
    both agree with the oracle."""
    w = workloads.gaussian_head("fused-passes", B, k, H, V, seed=B + V, device=DEV, w_std=0.3, sigma=1.0, sigma_far=0.2,
                                tau=1.6)
    kw, head, orc = {}, w.W_lm, None
    if weights == "w8a8":
        head, sc = binding.hola_quantize_w8(w.W_lm)
        kw = dict(w_scale=sc, a8=True)
    elif weights == "mixed":
        widths = [[4, 8, 16][g % 3] for g in range(-(-V // 256))]
        head = binding.hola_quantize_mixed(w.W_lm, widths)
    with binding.HolaVerify(B, k, H, V) as ctx:
        wd = {"bf16": binding.HOLA_W_BF16, "w8a8": binding.HOLA_W8A8, "mixed": binding.HOLA_W_MIXED}[weights]
        plan = ctx.hola_plan(B, k, wd)
        assert plan["passes"] >= 2 and plan["kernels_per_call"] == 2
        one = ctx.hola_verify(w.hidden, head, w.draft_tok, w.draft_q, w.uniforms, w.tau, want_logits=True, **kw)
        torch.cuda.synchronize()
        ctx.hola_set_option(binding.HOLA_OPT_FUSED_PASSES, 0)
        assert ctx.hola_plan(B, k, wd)["kernels_per_call"] == plan["passes"] + 1
        per = ctx.hola_verify(w.hidden, head, w.draft_tok, w.draft_q, w.uniforms, w.tau, want_logits=True, **kw)
        torch.cuda.synchronize()
    assert int(one.status.item()) == 0 and int(per.status.item()) == 0
    with binding.HolaVerify(B, k, H, V) as ctx:            # all passes in one launch, the groups of pairs free-running
        ctx.hola_set_option(binding.HOLA_OPT_FUSED_PASSES, 2)
        free = ctx.hola_verify(w.hidden, head, w.draft_tok, w.draft_q, w.uniforms, w.tau, want_logits=True, **kw)
        torch.cuda.synchronize()
        with pytest.raises(binding.HolaError):
            ctx.hola_set_option(binding.HOLA_OPT_FUSED_PASSES, 3)
    assert int(free.status.item()) == 0 and torch.equal(free.logits, one.logits)
    assert torch.equal(free.accept_len, one.accept_len) and torch.equal(free.next_tok, one.next_tok)
    assert torch.equal(one.logits, per.logits)
    assert torch.equal(one.accept_len, per.accept_len) and torch.equal(one.next_tok, per.next_tok)
    assert torch.allclose(one.entropy, per.entropy, atol=2e-5) and torch.allclose(one.logZ, per.logZ, atol=2e-5)
    if weights == "bf16":
        check_against_oracle(binding, w, out=one, seqs=range(0, B, 7))
    elif weights == "w8a8":
        orc = _w8_oracle(w.slice(range(0, B, 9)), head, sc, a8=True)
        pick = torch.arange(0, B, 9, device=DEV)
        sub = w.slice(range(0, B, 9))
        rep = compare.compare(orc, _np(sub.draft_q), _np(sub.uniforms), _np(one.accept_len[pick]), _np(one.next_tok[pick]),
                              _np(one.entropy[pick]), _np(one.logZ[pick]), _np(one.logits[pick]))
        assert rep.ok, rep.summary()


def test_split_entry_points_on_a_shape_with_several_passes(binding):
    """hola_lm_head_entropy (steps 1-2, statistics finished by the small finalising kernel) and hola_accept_sample
    (steps 3-5 from given logits) on 600 verify rows, which take several passes in one launch: the same logits, entropy,
    logZ and decisions as hola_verify, whose results the oracle checks."""
    w = workloads.gaussian_head("split-passes", 100, 5, 256, 6000, seed=41, device=DEV, w_std=0.3, sigma=1.0, sigma_far=0.2,
                                tau=1.6)
    with binding.HolaVerify(w.B, w.k, w.H, w.V) as ctx:
        assert ctx.hola_plan(w.B, w.k)["passes"] >= 2 and ctx.hola_plan(w.B, w.k)["kernels_per_call"] == 2
        whole = ctx.hola_verify(w.hidden, w.W_lm, w.draft_tok, w.draft_q, w.uniforms, w.tau, want_logits=True)
        torch.cuda.synchronize()
        first = ctx.hola_lm_head_entropy(w.hidden, w.W_lm, want_logits=True)
        torch.cuda.synchronize()
        assert torch.equal(first.logits, whole.logits)
        assert torch.allclose(first.entropy, whole.entropy, atol=2e-5) and torch.allclose(first.logZ, whole.logZ, atol=2e-5)
        second = ctx.hola_accept_sample(first.logits, first.entropy, first.logZ, w.draft_tok, w.draft_q, w.uniforms, w.tau)
        torch.cuda.synchronize()
    # (the statistics went through fp32 outputs on the way: a decision within 2e-5 of a tie may differ)
    same = (second.accept_len == whole.accept_len)
    assert int((~same).sum().item()) <= 1
    assert torch.equal(second.next_tok[same], whole.next_tok[same])
    check_against_oracle(binding, w, out=whole, seqs=range(0, w.B, 9))
