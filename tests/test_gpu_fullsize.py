"""Parity at the full sizes of the benchmark workloads, in the launch configuration the benchmark
times (bf16 outputs leave through the TMA-store epilogue; fp32 outputs are checked as well).

  * GPT-2-medium block (2048 tokens, q = 3, row-wise): the WHOLE Y, dX and dalpha of all four
    linears against the oracle.
  * GPT-2-XL linears (4096 tokens, q = 4, g = 128, ragged last group), all four shapes: the oracle
    computes outputs one by one, so the comparison is on a stratified sample -- two positions in
    every 128 x 256 output tile of every tensor, plus whole rows and whole columns through the
    ragged last tile and the short last group.
  * OPT-13B linears (2048 tokens, q in {2, 3, 4}, g = 128) quantized on the device with greedy +
    5 alternating rounds from weights with 0.1 % outliers x 20: quantizer on sampled rows, then
    the prefill forward on a stratified sample.
  * OPT-6.7B decode shapes: the whole GEMV.
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
BF16 = 2.0 ** -8   # one more rounding for bf16 outputs


@pytest.fixture(scope="module", autouse=True)
def _built():
    bcq_build.build_library()
    yield
    assert bcq.device_timeout_flag() == 0


def dev_bf16(a):
    return torch.from_numpy(a.view(np.int16)).cuda().view(torch.bfloat16)


def _layer(n, d_in, d_out, q, g, key, alt=0, outliers=0.0, check_rows=24):
    """Seeded layer; quantized on the device, the quantizer itself checked on sampled rows."""
    W = synth.weights(d_out, d_in, key, outlier_frac=outliers)
    X = synth.activations(n, d_in, key, synth.ROLE_X)
    dY = synth.activations(n, d_out, key, synth.ROLE_DY)
    bits, alpha, _ = bcq.quantize(torch.from_numpy(W).cuda(), q, g, alt)
    rows = synth.sample_indices(check_rows, [d_out], key)[0]
    rb, ra, _, margin = oracle.quantize(W[rows], q, g, alt_iters=alt)
    hb = bits.cpu().numpy().view(np.uint32)
    ha = alpha.cpu().numpy()
    if alt == 0:
        np.testing.assert_array_equal(hb[:, rows], rb)
        np.testing.assert_array_equal(ha[:, rows], ra)
    else:
        G = oracle.num_groups(d_in, g)
        same = np.stack([(hb[:, rows] == rb)[:, :, (c * g) >> 5:((min((c + 1) * g, d_in) + 31) >> 5)].all(axis=(0, 2))
                         for c in range(G)], axis=1)
        assert (same | (margin < 2.0 ** -20)).all(), "bits differ in a group that is not a near-tie"
        assert same.mean() > 0.999
    return X, dY, bits, alpha, hb, ha


# ------------------------------------------------------------------------------------------
# GPT-2 medium block: whole tensors
# ------------------------------------------------------------------------------------------

@pytest.mark.parametrize("d_in,d_out", [(1024, 3072), (1024, 1024), (1024, 4096), (4096, 1024)])
def test_gpt2_medium_layer_whole_tensors(d_in, d_out):
    n, q, g = 2048, 3, d_in
    key = (1, 0, d_out % 7)
    X, dY, bits, alpha, hb, ha = _layer(n, d_in, d_out, q, g, key)
    Xd, dYd = dev_bf16(X), dev_bf16(dY)
    ref_y = oracle.fwd(X, hb, ha, d_in, g)
    ref_dx = oracle.bwd_x(dY, hb, ha, d_in, g)
    ref_da = oracle.bwd_alpha(dY, X, hb, d_in, g)

    def err(out, ref):
        return float(np.abs(out.double().cpu().numpy() - ref).max() / np.abs(ref).max())

    assert err(bcq.linear_fwd(Xd, bits, alpha, d_in, g, out_dtype=torch.bfloat16), ref_y) <= TOL + BF16
    assert err(bcq.linear_bwd_x(dYd, bits, alpha, d_in, g, out_dtype=torch.bfloat16), ref_dx) <= TOL + BF16
    assert err(bcq.linear_fwd(Xd, bits, alpha, d_in, g), ref_y) <= TOL
    assert err(bcq.linear_bwd_x(dYd, bits, alpha, d_in, g), ref_dx) <= TOL
    assert err(bcq.linear_bwd_alpha(dYd, Xd, bits, d_in, g), ref_da) <= TOL


# ------------------------------------------------------------------------------------------
# GPT-2 XL linears: stratified samples
# ------------------------------------------------------------------------------------------

def _sample_positions(rows, cols, tile_rows, tile_cols, key, row_lines, col_lines):
    r1, c1 = synth.stratified_indices(rows, cols, tile_rows, tile_cols, 2, key)
    r2, c2 = synth.line_indices(rows, cols, row_lines, col_lines)
    return np.concatenate([r1, r2]), np.concatenate([c1, c2])


@pytest.mark.parametrize("d_in,d_out", [(1600, 4800), (1600, 1600), (1600, 6400), (6400, 1600)])
def test_gpt2_xl_layer_stratified(d_in, d_out):
    n, q, g = 4096, 4, 128
    key = (2, 0, d_out % 7)
    X, dY, bits, alpha, hb, ha = _layer(n, d_in, d_out, q, g, key)
    G = oracle.num_groups(d_in, g)
    Xd, dYd = dev_bf16(X), dev_bf16(dY)
    # Y[t][j]: tiles of 256 tokens x 128 rows; a whole token row, the last token, and columns in
    # the ragged last row tile (d_out = 1600, 4800, 6400 are 12.5, 37.5, 50 tiles of 128)
    t, j = _sample_positions(n, d_out, 256, 128, key, [0, n - 1], [d_out - 1, d_out - 33])
    ref = oracle.fwd_at(X, hb, ha, d_in, g, t, j)
    scale = np.abs(ref).max()
    Y = bcq.linear_fwd(Xd, bits, alpha, d_in, g).cpu().numpy()
    Yb = bcq.linear_fwd(Xd, bits, alpha, d_in, g, out_dtype=torch.bfloat16).float().cpu().numpy()
    assert np.abs(Y[t, j] - ref).max() <= TOL * scale
    assert np.abs(Yb[t, j] - ref).max() <= (TOL + BF16) * scale
    # dX[t][k]: tiles of 256 tokens x 128 columns k; lines through the short last group
    t, k = _sample_positions(n, d_in, 256, 128, (key[0], 1, key[2]), [1, n - 2], [d_in - 1, d_in - 40])
    ref = oracle.bwd_x_at(dY, hb, ha, d_in, g, t, k)
    scale = np.abs(ref).max()
    dX = bcq.linear_bwd_x(dYd, bits, alpha, d_in, g).cpu().numpy()
    dXb = bcq.linear_bwd_x(dYd, bits, alpha, d_in, g, out_dtype=torch.bfloat16).float().cpu().numpy()
    assert np.abs(dX[t, k] - ref).max() <= TOL * scale
    assert np.abs(dXb[t, k] - ref).max() <= (TOL + BF16) * scale
    # dalpha[i][j][c]: the product tile is 128 rows x 256 columns = two groups; every (row tile,
    # group) gets two samples per plane, plus the whole last row and the whole last group
    jj, cc = _sample_positions(d_out, G, 128, 1, (key[0], 2, key[2]), [d_out - 1], [G - 1])
    ii = synth.sample_indices(len(jj), [q], (key[0], 3, key[2]))[0]
    ref = oracle.bwd_alpha_at(dY, X, hb, d_in, g, ii, jj, cc)
    dA = bcq.linear_bwd_alpha(dYd, Xd, bits, d_in, g).cpu().numpy()
    assert np.abs(dA[ii, jj, cc] - ref).max() <= TOL * np.abs(ref).max()


# ------------------------------------------------------------------------------------------
# OPT-13B: alternating quantizer with outliers, then the 2048-token prefill forward
# ------------------------------------------------------------------------------------------

@pytest.mark.parametrize("q", [2, 3, 4])
@pytest.mark.parametrize("d_in,d_out", [(5120, 15360), (5120, 5120), (5120, 20480), (20480, 5120)])
def test_opt13b_quantize_then_prefill(d_in, d_out, q):
    n, g = 2048, 128
    key = (4, q, d_out % 7)
    X, _, bits, alpha, hb, ha = _layer(n, d_in, d_out, q, g, key, alt=5, outliers=1e-3, check_rows=8)
    t, j = _sample_positions(n, d_out, 256, 128, key, [n - 1], [d_out - 1])
    ref = oracle.fwd_at(X, hb, ha, d_in, g, t, j)
    scale = np.abs(ref).max()
    Xd = dev_bf16(X)
    Yb = bcq.linear_fwd(Xd, bits, alpha, d_in, g, out_dtype=torch.bfloat16).float().cpu().numpy()
    assert np.abs(Yb[t, j] - ref).max() <= (TOL + BF16) * scale
    del Yb
    Y = bcq.linear_fwd(Xd, bits, alpha, d_in, g).cpu().numpy()
    assert np.abs(Y[t, j] - ref).max() <= TOL * scale


@pytest.mark.parametrize("q", [2, 3, 4])
def test_quantizer_opt13b_shape_with_alternating_refits(q):
    # one 5120 -> 5120 layer, g = 128, greedy + 5 alternating rounds, 0.1 % outliers x20
    d_in = d_out = 5120
    key = (4, q, 0)
    W = synth.weights(d_out, d_in, key, outlier_frac=1e-3, outlier_mult=20.0)
    bits, alpha, _ = bcq.quantize(torch.from_numpy(W).cuda(), q, 128, alt_iters=5)
    rows = synth.sample_indices(48, [d_out], key)[0]
    rb, ra, _, margin = oracle.quantize(W[rows], q, 128, alt_iters=5)
    hb = bits.cpu().numpy().view(np.uint32)[:, rows]
    a = alpha.cpu().numpy()[:, rows]
    same = np.stack([(hb == rb)[:, :, 4 * c:4 * c + 4].all(axis=(0, 2)) for c in range(40)], axis=1)
    assert (same | (margin < 2.0 ** -20)).all(), "bits differ in a group that is not a near-tie"
    assert same.mean() > 0.999
    mean_abs = np.abs(W[rows]).reshape(len(rows), 40, 128).mean(axis=2)
    ok = np.abs(a - ra) <= 1e-5 * np.maximum(np.abs(ra), mean_abs[None])
    assert ok[:, same].all()


# ------------------------------------------------------------------------------------------
# OPT-6.7B decode: the whole GEMV
# ------------------------------------------------------------------------------------------

@pytest.mark.parametrize("d_in,d_out", [(4096, 12288), (4096, 16384), (16384, 4096), (4096, 4096)])
@pytest.mark.parametrize("q", [3, 4])
def test_decode_layer(d_in, d_out, q):
    g = 128
    key = (3, q, d_out % 5)
    X, _, bits, alpha, hb, ha = _layer(16, d_in, d_out, q, g, key)
    pack = bcq.decode_pack(bits, alpha, d_in, g)
    for n in (1, 4, 16):
        ref = oracle.fwd(X[:n], hb, ha, d_in, g)
        Y = bcq.linear_decode(dev_bf16(X[:n]), bits, alpha, d_in, g).cpu().numpy()
        assert np.abs(Y - ref).max() <= TOL * np.abs(ref).max()
        Yb = bcq.linear_decode(dev_bf16(X[:n]), bits, alpha, d_in, g, out_dtype=torch.bfloat16)
        assert np.abs(Yb.float().cpu().numpy() - ref).max() <= (TOL + BF16) * np.abs(ref).max()
        # the packed path (what the benchmark's decode table times)
        Yp = bcq.linear_decode_packed(dev_bf16(X[:n]), pack, d_out, d_in, q, g).cpu().numpy()
        assert np.abs(Yp - ref).max() <= TOL * np.abs(ref).max()
