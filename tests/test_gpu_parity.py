"""GPU parity: every CUDA entry point, called through the C-ABI binding, against the fp64 CPU
oracle on the same seeded inputs.

Tolerances:
  * packed bits: bit-exact, except in groups the oracle flags as near-ties (decision margin
    below 2^-20 of mean|w|), where rounding order may legitimately flip a bit;
  * quantizer alpha: |a - a_ref| <= 1e-5 * max(|a_ref|, mean|w_group|);
  * fp32 outputs of fwd / dX / dalpha: max|out - ref| / max|ref| <= 2e-3 (the bound the task
    states for bf16 inputs with fp32 accumulation; the kernels round the scaled weight once to
    fp16 and land near 3e-4; dalpha multiplies exact bf16 values and lands near 3e-7);
  * bf16 outputs: the same bound plus one bf16 rounding (2^-8 relative).
"""
import numpy as np
import pytest

import oracle
import paper_2210_03858_b200 as bcq
from paper_2210_03858_b200 import build as bcq_build
from paper_2210_03858_b200 import synth

pytestmark = pytest.mark.gpu
torch = pytest.importorskip("torch")

TOL = 2e-3


@pytest.fixture(scope="module", autouse=True)
def _built():
    bcq_build.build_library()
    assert torch.cuda.is_available()
    yield
    bcq.check_device()  # raises if a kernel reported an expired wait
    assert bcq.device_timeout_flag() == 0, "a kernel reported an expired wait"


def dev_bf16(a_u16):
    return torch.from_numpy(a_u16.view(np.int16)).cuda().view(torch.bfloat16)


def dev_bits(bits_u32):
    return torch.from_numpy(bits_u32.view(np.int32)).cuda()


def host_bits(t):
    return t.cpu().numpy().view(np.uint32)


def rel_err(out, ref):
    return float(np.abs(out.astype(np.float64) - ref).max() / np.abs(ref).max())


def make_case(seed, n, d_in, d_out, q, g, alt=0, outliers=0.0):
    key = (100, seed, 0)
    W = synth.weights(d_out, d_in, key, outlier_frac=outliers)
    X = synth.activations(n, d_in, key, synth.ROLE_X)
    dY = synth.activations(n, d_out, key, synth.ROLE_DY)
    bits, alpha, sq_err, margin = oracle.quantize(W, q, g, alt_iters=alt)
    return W, X, dY, bits, alpha, sq_err, margin


# --------------------------------------------------------------------------- quantizer

QUANT_CASES = [
    # d_out, d_in, q, g, alt, outliers
    (64, 128, 3, 128, 0, 0.0),
    (37, 1000, 3, 1000, 0, 0.0),      # row-wise, d_in not a multiple of 32
    (50, 1600, 4, 128, 0, 0.0),       # ragged last group (64)
    (24, 1024, 1, 32, 0, 0.0),
    (9, 4096, 2, 4096, 0, 0.0),       # CTA-wide teams
    (3, 20480, 2, 20480, 0, 0.0),
    (5, 8192, 8, 2048, 0, 0.0),
    (40, 512, 2, 128, 5, 1e-3),
    (40, 512, 3, 128, 5, 1e-3),
    (40, 640, 4, 128, 5, 1e-3),
    (16, 1024, 3, 1024, 3, 0.0),
    (6, 2304, 4, 2304, 2, 0.0),
    (12, 200, 5, 200, 1, 0.0),
    (32, 768, 3, 128, 15, 1e-3),      # the 15 alternating rounds of the paper's appendix
    (32, 768, 4, 128, 15, 1e-3),
]


@pytest.mark.parametrize("d_out,d_in,q,g,alt,outl", QUANT_CASES)
def test_quantize_matches_oracle(d_out, d_in, q, g, alt, outl):
    W, _, _, bits_ref, alpha_ref, sq_ref, margin = make_case(d_in + q, 1, d_in, d_out, q, g, alt, outl)
    bits, alpha, sq_err = bcq.quantize(torch.from_numpy(W).cuda(), q, g, alt, want_sq_err=True)
    torch.cuda.synchronize()
    bits, alpha, sq_err = host_bits(bits), alpha.cpu().numpy(), sq_err.cpu().numpy()
    G = oracle.num_groups(d_in, g)
    # padding bits are zero
    total = bits.shape[2] * 32
    kk = np.arange(d_in, total)
    if kk.size:
        assert not ((bits[:, :, kk >> 5] >> (kk & 31).astype(np.uint32)) & 1).any()
    flagged = margin < 2.0 ** -20
    diff_words = bits != bits_ref
    if diff_words.any():
        # every differing bit must sit in a flagged group
        k = np.arange(d_in)
        dbit = ((bits ^ bits_ref)[:, :, k >> 5] >> (k & 31).astype(np.uint32)) & 1
        for c in range(G):
            bad = dbit[:, :, c * g:(c + 1) * g].any(axis=(0, 2))
            assert not (bad & ~flagged[:, c]).any(), "bits differ in a group that is not a near-tie"
    same = ~np.stack([(bits != bits_ref)[:, :, (c * g) >> 5:((min((c + 1) * g, d_in) + 31) >> 5)].any(axis=(0, 2))
                      for c in range(G)], axis=1)
    assert same.mean() > 0.999
    mean_abs = np.stack([np.abs(W[:, c * g:(c + 1) * g]).mean(axis=1) for c in range(G)], axis=1)
    tol = 1e-5 * np.maximum(np.abs(alpha_ref), mean_abs[None])
    ok = np.abs(alpha - alpha_ref) <= tol
    assert ok[:, same].all()
    np.testing.assert_allclose(sq_err[same], sq_ref[same], rtol=1e-6, atol=1e-18)


def test_quantize_strided_input_and_determinism():
    W = synth.weights(48, 384, (101, 0, 0))
    Wp = np.zeros((48, 400), dtype=np.float32)
    Wp[:, :384] = W
    ref_bits, ref_alpha, _, _ = oracle.quantize(W, 3, 128)
    Wd = torch.from_numpy(Wp).cuda()[:, :384]
    b1, a1, _ = bcq.quantize(Wd, 3, 128)
    b2, a2, _ = bcq.quantize(Wd, 3, 128)
    torch.cuda.synchronize()
    assert torch.equal(b1, b2) and torch.equal(a1, a2)
    np.testing.assert_array_equal(host_bits(b1), ref_bits)
    np.testing.assert_array_equal(a1.cpu().numpy(), ref_alpha)


def test_dequantize_matches_oracle():
    for (d_out, d_in, q, g) in ((33, 1000, 3, 1000), (20, 1600, 4, 128), (7, 96, 2, 32)):
        _, _, _, bits, alpha, _, _ = make_case(7, 1, d_in, d_out, q, g)
        out = bcq.dequantize(dev_bits(bits), torch.from_numpy(alpha).cuda(), d_in, g).cpu().numpy()
        ref = oracle.dequantize(bits, alpha, d_in, g)
        np.testing.assert_allclose(out, ref, rtol=1e-6, atol=1e-9)


# --------------------------------------------------------------------------- linear layer

LINEAR_CASES = [
    # n, d_in, d_out, q, g
    (512, 1024, 1024, 3, 1024),    # the single-layer workload: several tiles, row-wise
    (300, 1000, 200, 4, 1000),     # ragged everywhere, row-wise with d_in % 32 != 0
    (257, 1600, 336, 4, 128),      # ragged last group, partial tiles in every dimension
    (64, 256, 128, 1, 32),         # smallest group size
    (130, 320, 384, 2, 96),        # groups not aligned to the tile widths
    (1100, 512, 640, 3, 256),      # more token tiles than one wave of a small grid
    (96, 2048, 256, 8, 512),       # q = 8
]


def _upload(X, dY, bits, alpha):
    return dev_bf16(X), dev_bf16(dY), dev_bits(bits), torch.from_numpy(alpha).cuda()


@pytest.mark.parametrize("n,d_in,d_out,q,g", LINEAR_CASES)
def test_fwd_matches_oracle(n, d_in, d_out, q, g):
    _, X, dY, bits, alpha, _, _ = make_case(n, n, d_in, d_out, q, g)
    Xd, _, bd, ad = _upload(X, dY, bits, alpha)
    ref = oracle.fwd(X, bits, alpha, d_in, g)
    Y = bcq.linear_fwd(Xd, bd, ad, d_in, g)
    Y2 = bcq.linear_fwd(Xd, bd, ad, d_in, g)
    torch.cuda.synchronize()
    assert torch.equal(Y, Y2), "two runs differ"
    assert rel_err(Y.cpu().numpy(), ref) <= TOL
    # bias and bf16 output
    bias = synth.bias(d_out, (100, n, 0))
    Yb = bcq.linear_fwd(Xd, bd, ad, d_in, g, bias=torch.from_numpy(bias).cuda(),
                        out_dtype=torch.bfloat16)
    Yb2 = bcq.linear_fwd(Xd, bd, ad, d_in, g, bias=torch.from_numpy(bias).cuda(),
                         out_dtype=torch.bfloat16)
    refb = ref + bias.astype(np.float64)
    assert torch.equal(Yb, Yb2), "two bf16 runs differ"
    assert rel_err(Yb.float().cpu().numpy(), refb) <= TOL + 2.0 ** -8


@pytest.mark.parametrize("n,d_in,d_out,q,g", LINEAR_CASES)
def test_bwd_x_matches_oracle(n, d_in, d_out, q, g):
    _, X, dY, bits, alpha, _, _ = make_case(n, n, d_in, d_out, q, g)
    _, dYd, bd, ad = _upload(X, dY, bits, alpha)
    ref = oracle.bwd_x(dY, bits, alpha, d_in, g)
    dX = bcq.linear_bwd_x(dYd, bd, ad, d_in, g)
    dX2 = bcq.linear_bwd_x(dYd, bd, ad, d_in, g)
    torch.cuda.synchronize()
    assert torch.equal(dX, dX2)
    assert rel_err(dX.cpu().numpy(), ref) <= TOL
    dXb = bcq.linear_bwd_x(dYd, bd, ad, d_in, g, out_dtype=torch.bfloat16)
    dXb2 = bcq.linear_bwd_x(dYd, bd, ad, d_in, g, out_dtype=torch.bfloat16)
    assert torch.equal(dXb, dXb2), "two bf16 runs differ"
    assert rel_err(dXb.float().cpu().numpy(), ref) <= TOL + 2.0 ** -8


@pytest.mark.parametrize("n,d_in,d_out,q,g", LINEAR_CASES)
def test_bwd_alpha_matches_oracle(n, d_in, d_out, q, g):
    _, X, dY, bits, alpha, _, _ = make_case(n, n, d_in, d_out, q, g)
    Xd, dYd, bd, _ = _upload(X, dY, bits, alpha)
    ref = oracle.bwd_alpha(dY, X, bits, d_in, g)
    dA = bcq.linear_bwd_alpha(dYd, Xd, bd, d_in, g)
    dA2 = bcq.linear_bwd_alpha(dYd, Xd, bd, d_in, g)
    torch.cuda.synchronize()
    assert torch.equal(dA, dA2)
    assert rel_err(dA.cpu().numpy(), ref) <= TOL
    # alpha_1 only, the paper's 1/g scale, accumulate on top of existing values
    out = torch.full_like(dA, 3.0)
    bcq.linear_bwd_alpha(dYd, Xd, bd, d_in, g, plane_mask=1, scale=1.0 / g, accumulate=True, out=out)
    o = out.cpu().numpy()
    assert (o[1:] == 3.0).all()
    assert np.abs(o[0] - 3.0 - ref[0] / g).max() <= TOL * np.abs(ref[0] / g).max() + 1e-6


@pytest.mark.parametrize("n", [1, 4, 16, 5])
@pytest.mark.parametrize("d_in,d_out,q,g", [(4096, 1536, 3, 128), (1024, 520, 4, 128), (2048, 256, 3, 2048)])
def test_decode_matches_oracle(n, d_in, d_out, q, g):
    _, X, dY, bits, alpha, _, _ = make_case(n + d_out, n, d_in, d_out, q, g)
    Xd, _, bd, ad = _upload(X, dY, bits, alpha)
    ref = oracle.fwd(X, bits, alpha, d_in, g)
    Y = bcq.linear_decode(Xd, bd, ad, d_in, g)
    Y2 = bcq.linear_decode(Xd, bd, ad, d_in, g)
    torch.cuda.synchronize()
    assert torch.equal(Y, Y2)
    assert rel_err(Y.cpu().numpy(), ref) <= TOL


@pytest.mark.parametrize("n,d_in,d_out,q,g", [c for c in LINEAR_CASES if c[3] <= 4] + [(200, 640, 304, 2, 128),
                                                                                       (300, 1600, 4800, 4, 128)])
def test_prepared_planes_give_the_same_results(n, d_in, d_out, q, g):
    # B is frozen: the planes regrouped once must give, bit for bit, what the per-call regrouping gives
    _, X, dY, bits, alpha, _, _ = make_case(n, n, d_in, d_out, q, g)
    Xd, dYd, bd, ad = _upload(X, dY, bits, alpha)
    pf = bcq.prepare_planes(bcq.OP_FWD, bd, d_in, g)
    px = bcq.prepare_planes(bcq.OP_BWD_X, bd, d_in, g)
    for dt in (torch.float32, torch.bfloat16):
        assert torch.equal(bcq.linear_fwd(Xd, pf, ad, d_in, g, out_dtype=dt), bcq.linear_fwd(Xd, bd, ad, d_in, g, out_dtype=dt))
        assert torch.equal(bcq.linear_bwd_x(dYd, px, ad, d_in, g, out_dtype=dt),
                           bcq.linear_bwd_x(dYd, bd, ad, d_in, g, out_dtype=dt))
    assert rel_err(bcq.linear_fwd(Xd, pf, ad, d_in, g).cpu().numpy(), oracle.fwd(X, bits, alpha, d_in, g)) <= TOL
    assert rel_err(bcq.linear_bwd_x(dYd, px, ad, d_in, g).cpu().numpy(), oracle.bwd_x(dY, bits, alpha, d_in, g)) <= TOL
    # alpha may change between calls (it is what AlphaTuning trains); the prepared planes stay valid
    ad2 = ad * 1.25
    ref2 = oracle.fwd(X, bits, (alpha * np.float32(1.25)).astype(np.float32), d_in, g)
    assert rel_err(bcq.linear_fwd(Xd, pf, ad2, d_in, g).cpu().numpy(), ref2) <= TOL


def test_prepared_planes_need_at_most_four_planes():
    assert bcq.lib().bcq_prepared_bytes(bcq.OP_FWD, 64, 256, 5, 64) == 0
    assert bcq.lib().bcq_prepared_bytes(bcq.OP_BWD_X, 64, 256, 4, 64) > 0
    assert bcq.lib().bcq_prepared_bytes(bcq.OP_DECODE, 64, 256, 4, 64) == 0


# --------------------------------------------------------------------------- tile-schedule corners

@pytest.mark.parametrize("n", [129, 145, 257, 300, 530, 1000])
def test_fwd_and_bwd_x_with_token_counts_between_tile_widths(n):
    # above 128 tokens the token-tile width is any multiple of 16 up to 256, chosen per call: these
    # counts give widths that are not powers of two, ragged last tiles and single tiles wider than n
    d_in, d_out, q, g = 640, 2560, 4, 128
    _, X, dY, bits, alpha, _, _ = make_case(900 + n, n, d_in, d_out, q, g)
    Xd, dYd, bd, ad = _upload(X, dY, bits, alpha)
    ref_y = oracle.fwd(X, bits, alpha, d_in, g)
    ref_dx = oracle.bwd_x(dY, bits, alpha, d_in, g)
    for dt, tol in ((torch.float32, TOL), (torch.bfloat16, TOL + 2.0 ** -8)):
        assert rel_err(bcq.linear_fwd(Xd, bd, ad, d_in, g, out_dtype=dt).float().cpu().numpy(), ref_y) <= tol
        assert rel_err(bcq.linear_bwd_x(dYd, bd, ad, d_in, g, out_dtype=dt).float().cpu().numpy(), ref_dx) <= tol


@pytest.mark.parametrize("n", [1, 17, 31, 32])
def test_fwd_and_bwd_x_with_few_tokens(n):
    # the prefill entry points accept any n >= 1; n <= 32 takes the narrowest token tile
    d_in, d_out, q, g = 640, 384, 3, 128
    _, X, dY, bits, alpha, _, _ = make_case(700 + n, n, d_in, d_out, q, g)
    Xd, dYd, bd, ad = _upload(X, dY, bits, alpha)
    ref_y = oracle.fwd(X, bits, alpha, d_in, g)
    ref_dx = oracle.bwd_x(dY, bits, alpha, d_in, g)
    for dt, tol in ((torch.float32, TOL), (torch.bfloat16, TOL + 2.0 ** -8)):
        assert rel_err(bcq.linear_fwd(Xd, bd, ad, d_in, g, out_dtype=dt).float().cpu().numpy(), ref_y) <= tol
        assert rel_err(bcq.linear_bwd_x(dYd, bd, ad, d_in, g, out_dtype=dt).float().cpu().numpy(), ref_dx) <= tol


@pytest.mark.parametrize("d_in", [64, 128, 192])
def test_many_tiles_per_cta_with_short_k(d_in):
    # 320 output tiles of 128 x 256 on 148 SMs: every persistent CTA walks three tiles, so both
    # accumulators are reused (second phase of their barriers) and, with K this short, the worker
    # warps are far ahead of the tensor core when they reach the last tile's epilogue
    n, d_out, q, g = 4096, 2560, 3, 64
    _, X, dY, bits, alpha, _, _ = make_case(800 + d_in, n, d_in, d_out, q, g)
    Xd, _, bd, ad = _upload(X, dY, bits, alpha)
    ref = oracle.fwd(X, bits, alpha, d_in, g)
    Yb = bcq.linear_fwd(Xd, bd, ad, d_in, g, out_dtype=torch.bfloat16)
    Yb2 = bcq.linear_fwd(Xd, bd, ad, d_in, g, out_dtype=torch.bfloat16)
    assert torch.equal(Yb, Yb2)
    assert rel_err(Yb.float().cpu().numpy(), ref) <= TOL + 2.0 ** -8
    assert rel_err(bcq.linear_fwd(Xd, bd, ad, d_in, g).cpu().numpy(), ref) <= TOL


def test_bwd_x_many_tiles_per_cta_with_short_k():
    n, d_in, d_out, q, g = 4096, 2560, 64, 4, 128
    _, X, dY, bits, alpha, _, _ = make_case(811, n, d_in, d_out, q, g)
    _, dYd, bd, ad = _upload(X, dY, bits, alpha)
    ref = oracle.bwd_x(dY, bits, alpha, d_in, g)
    assert rel_err(bcq.linear_bwd_x(dYd, bd, ad, d_in, g, out_dtype=torch.bfloat16).float().cpu().numpy(),
                   ref) <= TOL + 2.0 ** -8
    assert rel_err(bcq.linear_bwd_x(dYd, bd, ad, d_in, g).cpu().numpy(), ref) <= TOL


# --------------------------------------------------------------------------- dynamic range

def _bf16(x):
    return synth.f32_to_bf16_bits(np.asarray(x, dtype=np.float32))


def test_token_with_one_huge_channel():
    # one channel of one token is 1e4 among N(0,1): the per-token power-of-two scale has to keep
    # both the outlier and the ordinary channels inside the fp16 operands' range
    n, d_in, d_out, q, g = 96, 512, 256, 3, 128
    _, X, dY, bits, alpha, _, _ = make_case(900, n, d_in, d_out, q, g)
    Xf = synth.bf16_bits_to_f32(X)
    Xf[5, 77] = 1.0e4
    Xf[40, 300] = -3.0e4
    X = _bf16(Xf)
    Xd, _, bd, ad = _upload(X, dY, bits, alpha)
    ref = oracle.fwd(X, bits, alpha, d_in, g)
    Y = bcq.linear_fwd(Xd, bd, ad, d_in, g).cpu().numpy()
    assert np.isfinite(Y).all()
    # per token, since the two outlier tokens dwarf the others
    for t in (0, 5, 40, 95):
        assert np.abs(Y[t] - ref[t]).max() <= TOL * np.abs(ref[t]).max()
    pack = bcq.decode_pack(bd, ad, d_in, g)
    for nn in (1, 16):
        refd = ref[:nn * 6:6]
        Xs = Xd[:nn * 6:6].contiguous()
        for Yd in (bcq.linear_decode(Xs, bd, ad, d_in, g).cpu().numpy(),
                   bcq.linear_decode_packed(Xs, pack, d_out, d_in, q, g).cpu().numpy()):
            for t in range(nn):
                assert np.abs(Yd[t] - refd[t]).max() <= TOL * np.abs(refd[t]).max()


def test_tiny_output_gradients():
    # dY ~ 1e-6: far below the smallest normal fp16 number unless each token row is rescaled
    n, d_in, d_out, q, g = 200, 384, 256, 4, 128
    _, X, dY, bits, alpha, _, _ = make_case(901, n, d_in, d_out, q, g)
    dY = _bf16(synth.bf16_bits_to_f32(dY) * np.float32(1e-6))
    Xd, dYd, bd, ad = _upload(X, dY, bits, alpha)
    ref = oracle.bwd_x(dY, bits, alpha, d_in, g)
    assert rel_err(bcq.linear_bwd_x(dYd, bd, ad, d_in, g).cpu().numpy(), ref) <= TOL
    ref = oracle.bwd_alpha(dY, X, bits, d_in, g)
    assert rel_err(bcq.linear_bwd_alpha(dYd, Xd, bd, d_in, g).cpu().numpy(), ref) <= TOL


def test_scales_spread_over_4096x_between_rows_and_groups():
    # alpha differs by 2^12 between rows and, inside a row, between groups (also: the first groups
    # of a row are ~1e-6 of the later ones, and the other way round)
    n, d_in, d_out, q, g = 80, 1024, 256, 3, 128
    W = synth.weights(d_out, d_in, (100, 902, 0))
    row_mul = np.float32(2.0) ** -(np.arange(d_out) % 13).astype(np.float32)
    W = W * row_mul[:, None]
    W[64:128, :512] *= np.float32(1e-6)     # tiny first four groups
    W[128:192, 512:] *= np.float32(1e-6)    # tiny last four groups
    W[192:, 256:384] *= np.float32(4096.0)  # one large group in the middle
    X = synth.activations(n, d_in, (100, 902, 0), synth.ROLE_X)
    dY = synth.activations(n, d_out, (100, 902, 0), synth.ROLE_DY)
    bits, alpha, _, _ = oracle.quantize(W.astype(np.float32), q, g)
    Xd, dYd, bd, ad = _upload(X, dY, bits, alpha)
    ref = oracle.fwd(X, bits, alpha, d_in, g)
    # decode, column by column: every weight row has its own magnitude and its own scale
    pack = bcq.decode_pack(bd, ad, d_in, g)
    for nn in (1, 4, 16):
        Xs = Xd[:nn].contiguous()
        for Yd in (bcq.linear_decode(Xs, bd, ad, d_in, g).cpu().numpy(),
                   bcq.linear_decode_packed(Xs, pack, d_out, d_in, q, g).cpu().numpy()):
            assert np.isfinite(Yd).all()
            e = np.abs(Yd - ref[:nn]).max(axis=0) / np.abs(ref).max(axis=0)
            assert e.max() <= TOL
    # the prefill kernels scale all weights by one power of two: rows 2^12 below the largest keep
    # the absolute accuracy of the largest, which the per-tensor metric is about
    assert rel_err(bcq.linear_fwd(Xd, bd, ad, d_in, g).cpu().numpy(), ref) <= TOL
    assert rel_err(bcq.linear_bwd_x(dYd, bd, ad, d_in, g).cpu().numpy(),
                   oracle.bwd_x(dY, bits, alpha, d_in, g)) <= TOL


@pytest.mark.parametrize("n", [1, 2, 4, 7, 16])
@pytest.mark.parametrize("d_in,d_out,q,g", [
    (4096, 1536, 3, 128), (1024, 520, 4, 128), (2048, 256, 3, 2048), (1000, 200, 4, 1000),
    (1600, 336, 4, 128), (320, 384, 2, 96), (256, 128, 1, 32), (2304, 4100, 2, 64),
])
def test_decode_packed_matches_oracle(n, d_in, d_out, q, g):
    _, X, dY, bits, alpha, _, _ = make_case(n + d_out + q, n, d_in, d_out, q, g)
    Xd, _, bd, ad = _upload(X, dY, bits, alpha)
    ref = oracle.fwd(X, bits, alpha, d_in, g)
    pack = bcq.decode_pack(bd, ad, d_in, g)
    Y = bcq.linear_decode_packed(Xd, pack, d_out, d_in, q, g)
    Y2 = bcq.linear_decode_packed(Xd, pack, d_out, d_in, q, g)   # the pack's counters are back at zero
    torch.cuda.synchronize()
    assert torch.equal(Y, Y2)
    assert rel_err(Y.cpu().numpy(), ref) <= TOL
    bias = synth.bias(d_out, (100, n, 1))
    Yb = bcq.linear_decode_packed(Xd, pack, d_out, d_in, q, g, bias=torch.from_numpy(bias).cuda(),
                                  out_dtype=torch.bfloat16)
    assert rel_err(Yb.float().cpu().numpy(), ref + bias.astype(np.float64)) <= TOL + 2.0 ** -8


def test_decode_pack_rejects_more_than_four_planes():
    assert bcq.lib().bcq_decode_pack_bytes(64, 256, 5, 64) == 0
    assert bcq.lib().bcq_decode_pack_bytes(64, 256, 4, 64) > 0


def test_strided_activations_and_outputs():
    n, d_in, d_out, q, g = 70, 256, 192, 3, 128
    _, X, dY, bits, alpha, _, _ = make_case(3, n, d_in, d_out, q, g)
    Xd, dYd, bd, ad = _upload(X, dY, bits, alpha)
    Xp = torch.zeros((n, d_in + 8), dtype=torch.bfloat16, device="cuda")
    Xp[:, :d_in] = Xd
    Yp = torch.full((n, d_out + 5), -7.0, dtype=torch.float32, device="cuda")
    bcq.linear_fwd(Xp[:, :d_in], bd, ad, d_in, g, out=Yp[:, :d_out])
    ref = oracle.fwd(X, bits, alpha, d_in, g)
    assert rel_err(Yp[:, :d_out].cpu().numpy(), ref) <= TOL
    assert (Yp[:, d_out:] == -7.0).all()       # nothing written past the row


def test_quantize_then_layer_end_to_end():
    # the whole path on device: W -> (bits, alpha) -> fwd, dX, dalpha, all against the oracle
    n, d_in, d_out, q, g = 256, 512, 384, 3, 128
    W, X, dY, bits_ref, alpha_ref, _, _ = make_case(11, n, d_in, d_out, q, g)
    bits, alpha, _ = bcq.quantize(torch.from_numpy(W).cuda(), q, g)
    np.testing.assert_array_equal(host_bits(bits), bits_ref)
    Xd, dYd = dev_bf16(X), dev_bf16(dY)
    assert rel_err(bcq.linear_fwd(Xd, bits, alpha, d_in, g).cpu().numpy(),
                   oracle.fwd(X, bits_ref, alpha_ref, d_in, g)) <= TOL
    assert rel_err(bcq.linear_bwd_x(dYd, bits, alpha, d_in, g).cpu().numpy(),
                   oracle.bwd_x(dY, bits_ref, alpha_ref, d_in, g)) <= TOL
    assert rel_err(bcq.linear_bwd_alpha(dYd, Xd, bits, d_in, g).cpu().numpy(),
                   oracle.bwd_alpha(dY, X, bits_ref, d_in, g)) <= TOL
