"""GPU parity of the mixed-width LM head (groups of 256 vocabulary rows at 4, 8 or 16 bits, HOLA_W_MIXED) and of the
4-bit quantiser kernel, against oracle/lobi.py and the fp64 verify oracle on the dequantised matrix."""
import numpy as np
import pytest
import torch

from oracle import compare, lobi, ref
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


def _widths(V, pattern):
    ng = -(-V // 256)
    return [pattern[g % len(pattern)] for g in range(ng)]


@pytest.mark.parametrize("V,H", [(300, 128), (1000, 512), (4099, 256)])
def test_w4_quantiser_is_bit_exact(binding, V, H):
    g = torch.Generator(device=DEV).manual_seed(V + H)
    W = (torch.randn((V, H), generator=g, device=DEV) * 0.02).bfloat16()
    W[:, 128:256] *= 0.05 if H >= 256 else 1.0          # a quiet sub-block: smaller exponents
    W[3] = 0                                            # an all-zero row
    W[5] = 0
    W[5, 0] = 0.4375                                    # 112 * 2^-8: scale 2^-8, ties at half steps below
    W[5, 1:4] = torch.tensor([0.03125 * 0.5, 0.03125 * 1.5, -0.03125 * 2.5], device=DEV).bfloat16()
    lib = binding.load_library()
    packed = torch.empty((V, H // 2), dtype=torch.uint8, device=DEV)
    shifts = torch.full((H // 128, V), 255, dtype=torch.uint8, device=DEV)
    scale = torch.empty((V,), dtype=torch.float32, device=DEV)
    import ctypes
    st = lib.hola_quantize_w4(ctypes.c_void_p(W.data_ptr()), V, H, ctypes.c_void_p(packed.data_ptr()),
                              ctypes.c_void_p(shifts.data_ptr()), V, ctypes.c_void_p(scale.data_ptr()), None)
    assert st == 0
    torch.cuda.synchronize()
    c, e, s = lobi.quantize_rows_w4(W.float().cpu().numpy())
    assert np.array_equal(_np(scale), s)
    assert np.array_equal(_np(shifts).T, e)
    assert np.array_equal(_np(packed), lobi.pack_nibbles(c))
    assert lib.hola_quantize_w4(ctypes.c_void_p(W.data_ptr()), V, 100, ctypes.c_void_p(packed.data_ptr()),
                                ctypes.c_void_p(shifts.data_ptr()), V, ctypes.c_void_p(scale.data_ptr()), None) == 2


def _mixed_oracle(w, widths, **kw):
    hid = ref.bf16_bits_to_f64(_np(w.hidden))
    Wd = lobi.dequantize_mixed(ref.bf16_bits_to_f64(_np(w.W_lm)).astype(np.float32), widths)
    return ref.verify(hid, Wd, _np(w.draft_tok), _np(w.draft_q), _np(w.uniforms), w.tau, keep_logits=True, **kw)


@pytest.mark.parametrize("B,k,H,V,pattern", [
    (1, 4, 128, 1000, [16, 4, 8, 4]),          # the tiny batch: four groups, every width, ragged last group
    (9, 3, 256, 700, [4, 8, 16]),              # three groups, two sub-blocks per row
    (37, 6, 256, 5000, [8, 8, 4, 16, 8]),      # 259 rows: two passes over the head
    (20, 3, 384, 2048, [4]),                   # every group at 4 bits, whole groups only
    (6, 2, 128, 3001, [16, 8]),                # no 4-bit group at all
])
def test_mixed_width_head_matches_oracle_on_the_dequantised_matrix(binding, B, k, H, V, pattern):
    w = workloads.gaussian_head("mixed", B, k, H, V, seed=B + V, device=DEV, w_std=0.3, sigma=1.0, tau=1.5 + 0.1 * k,
                                sigma_far=0.2)
    widths = _widths(V, pattern)
    head = binding.hola_quantize_mixed(w.W_lm, widths)
    with binding.HolaVerify(B, k, H, V) as ctx:
        out = ctx.hola_verify(w.hidden, head, w.draft_tok, w.draft_q, w.uniforms, w.tau, want_logits=True)
        torch.cuda.synchronize()
    assert int(out.status.item()) & binding.FLAG_TIMEOUT == 0
    orc = _mixed_oracle(w, widths)
    rep = compare.compare(orc, _np(w.draft_q), _np(w.uniforms), _np(out.accept_len), _np(out.next_tok),
                          _np(out.entropy), _np(out.logZ), _np(out.logits))
    print(rep.summary())
    assert rep.ok, rep.summary()
    assert rep.accept_margin_cases <= max(1, B // 20) and rep.token_margin_cases <= max(1, B // 10)


def test_mixed_width_integer_weights_are_bit_exact(binding):
    """Weights that are of the stored forms already (4-bit: c << e with a 112 per row; 8-bit: integers with a 127 per
    row; 16-bit: small integers) and small-integer hidden rows: every product and sum is exact, so the logits must
    equal the integer matrix product."""
    g = torch.Generator().manual_seed(4)
    V, H, B, k = 768, 256, 4, 2
    W = torch.zeros((V, H))
    c = torch.randint(-7, 8, (256, 2, 128), generator=g)
    e = torch.randint(0, 5, (256, 2), generator=g)
    c[:, :, 0] = 7
    e[:, 0] = 4
    W[0:256] = (c * (2 ** e)[:, :, None]).reshape(256, H).float()          # group 0: 4 bits
    W[256:512] = torch.randint(-127, 128, (256, H), generator=g).float()   # group 1: 8 bits
    W[256:512, 0] = 127
    W[512:768] = torch.randint(-8, 9, (256, H), generator=g).float()       # group 2: 16 bits
    hidden = torch.randint(-2, 3, (B, k + 1, H), generator=g).float()
    want = (hidden.reshape(-1, H).double() @ W.double().T).reshape(B, k + 1, V)
    q = torch.full((B, k, V), 1.0 / V)
    tok = torch.randint(0, V, (B, k), generator=g, dtype=torch.int32)
    u = torch.rand((B, k + 1), generator=g)
    head = binding.hola_quantize_mixed(W.bfloat16().to(DEV), [4, 8, 16])
    assert torch.all(head.w_scale == 1.0)
    with binding.HolaVerify(B, k, H, V) as ctx:
        out = ctx.hola_verify(hidden.bfloat16().to(DEV), head, tok.to(DEV), q.to(DEV), u.to(DEV), 0.0, want_logits=True)
        torch.cuda.synchronize()
    assert torch.equal(out.logits.cpu().double(), want)


def test_mixed_width_arguments_are_validated(binding):
    w = workloads.gaussian_head("mixed-args", 2, 2, 128, 600, seed=3, device=DEV, w_std=0.3)
    with pytest.raises(binding.HolaError):
        binding.hola_quantize_mixed(w.W_lm, [4, 8])                 # three groups, two widths
    with pytest.raises(binding.HolaError):
        binding.hola_quantize_mixed(w.W_lm, [4, 8, 5])
    head = binding.hola_quantize_mixed(w.W_lm, [4, 8, 16])
    assert head.weight_bytes() < w.W_lm.numel() * 2
    with binding.HolaVerify(2, 2, 128, 600) as ctx:
        with pytest.raises(binding.HolaError):
            ctx.hola_verify(w.hidden, head, w.draft_tok, w.draft_q, w.uniforms, w.tau, a8=True)
    with binding.HolaVerify(2, 2, 128, 856) as ctx:                 # a head of another vocabulary size
        with pytest.raises(binding.HolaError):
            ctx.hola_verify(w.hidden, head, w.draft_tok, w.draft_q, w.uniforms, w.tau)


@pytest.mark.parametrize("name", ["edge", "large_vocab_b32"])
def test_mixed_width_on_the_bandwidth_bound_shapes(binding, name):
    """Full size, widths in the proportions the paper reports (most groups at 8 bits, some at 4, a few kept at 16);
    sampled sequences against the oracle on the dequantised matrix."""
    w = workloads.make_config(name, DEV)
    ng = -(-w.V // 256)
    rng = np.random.default_rng(11)
    widths = rng.choice([4, 8, 16], size=ng, p=[0.2, 0.7, 0.1]).tolist()
    head = binding.hola_quantize_mixed(w.W_lm, widths)
    with binding.HolaVerify(w.B, w.k, w.H, w.V) as ctx:
        out = ctx.hola_verify(w.hidden, head, w.draft_tok, w.draft_q, w.uniforms, w.tau, want_logits=True)
        torch.cuda.synchronize()
    assert int(out.status.item()) & binding.FLAG_TIMEOUT == 0
    seqs = list(range(w.B)) if w.B <= 4 else [0, 9, 20, 31]
    sub = w.slice(seqs)
    orc = _mixed_oracle(sub, widths)
    pick = torch.as_tensor(seqs, device=DEV)
    rep = compare.compare(orc, _np(sub.draft_q), _np(sub.uniforms), _np(out.accept_len[pick]), _np(out.next_tok[pick]),
                          _np(out.entropy[pick]), _np(out.logZ[pick]), _np(out.logits[pick]))
    print(name, rep.summary())
    assert rep.ok, rep.summary()


def test_converter_group_size_changes_speed_not_results(binding):
    """The number of converter warps that share a K block is a speed knob: the expansion is exact whoever does it, so
    every setting gives the same logits bit for bit (few K blocks, many K blocks, more groups than ring slots in use)."""
    for B, k, H, V in ((3, 2, 128, 1300), (40, 4, 1024, 2600)):
        w = workloads.gaussian_head("conv-group", B, k, H, V, seed=V, device=DEV, w_std=0.3, sigma=1.0, tau=1.7)
        head = binding.hola_quantize_mixed(w.W_lm, _widths(V, [4, 8, 16, 8, 4]))
        with binding.HolaVerify(B, k, H, V) as ctx:
            base = ctx.hola_verify(w.hidden, head, w.draft_tok, w.draft_q, w.uniforms, w.tau, want_logits=True)
            torch.cuda.synchronize()
            assert int(base.status.item()) == 0
            for G in (1, 2, 3, 4, 8, 0):
                ctx.hola_set_option(binding.HOLA_OPT_CONVERTER_GROUP, G)
                out = ctx.hola_verify(w.hidden, head, w.draft_tok, w.draft_q, w.uniforms, w.tau, want_logits=True)
                torch.cuda.synchronize()
                assert int(out.status.item()) == 0, G
                assert torch.equal(out.logits, base.logits), G
                assert torch.equal(out.accept_len, base.accept_len) and torch.equal(out.next_tok, base.next_tok)
            for bad in (-1, 9):
                with pytest.raises(binding.HolaError):
                    ctx.hola_set_option(binding.HOLA_OPT_CONVERTER_GROUP, bad)
            # fewer ring slots than groups of converter warps: only as many groups as slots take part
            for slots, G in ((2, 1), (3, 2), (2, 4)):
                ctx.hola_set_option(binding.HOLA_OPT_RING_SLOTS, slots)
                ctx.hola_set_option(binding.HOLA_OPT_CONVERTER_GROUP, G)
                assert ctx.hola_plan(B, k, binding.HOLA_W_MIXED)["stages"] == slots
                out = ctx.hola_verify(w.hidden, head, w.draft_tok, w.draft_q, w.uniforms, w.tau, want_logits=True)
                torch.cuda.synchronize()
                assert int(out.status.item()) == 0, (slots, G)
                assert torch.equal(out.logits, base.logits), (slots, G)
    orc = _mixed_oracle(w, _widths(V, [4, 8, 16, 8, 4]))
    rep = compare.compare(orc, _np(w.draft_q), _np(w.uniforms), _np(base.accept_len), _np(base.next_tok),
                          _np(base.entropy), _np(base.logZ), _np(base.logits))
    assert rep.ok, rep.summary()
