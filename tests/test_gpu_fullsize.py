"""Parity at the full sizes of the benchmark workloads, in the launch configuration the benchmark
times, on sampled outputs that the oracle computes one by one.

Covers the GPT-2-medium block (2048 tokens, q = 3, row-wise), the GPT-2-XL linears (4096 tokens,
q = 4, g = 128, ragged last group), the OPT-6.7B decode shapes and one OPT-13B-shaped layer of the
quantizer with alternating refits and outliers (rows sampled)."""
import numpy as np
import pytest

import oracle
import paper_2210_03858_b200 as bcq
from paper_2210_03858_b200 import build as bcq_build
from paper_2210_03858_b200 import synth

pytestmark = pytest.mark.gpu
torch = pytest.importorskip("torch")
TOL = 2e-3
NS = 400  # sampled outputs per tensor


@pytest.fixture(scope="module", autouse=True)
def _built():
    bcq_build.build_library()
    yield
    assert bcq.device_timeout_flag() == 0


def dev_bf16(a):
    return torch.from_numpy(a.view(np.int16)).cuda().view(torch.bfloat16)


def _check_sampled(out, ref_vals, idx, scale):
    got = out[idx].astype(np.float64)
    assert np.abs(got - ref_vals).max() <= TOL * scale


def _layer(workload, n, d_in, d_out, q, g, key):
    W = synth.weights(d_out, d_in, key)
    X = synth.activations(n, d_in, key, synth.ROLE_X)
    dY = synth.activations(n, d_out, key, synth.ROLE_DY)
    Wd = torch.from_numpy(W).cuda()
    bits, alpha, _ = bcq.quantize(Wd, q, g)
    # the device quantizer is itself checked on sampled rows against the oracle
    rows = synth.sample_indices(24, [d_out], key)[0]
    rb, ra, _, _ = oracle.quantize(W[rows], q, g)
    hb = bits.cpu().numpy().view(np.uint32)
    np.testing.assert_array_equal(hb[:, rows], rb)
    np.testing.assert_array_equal(alpha.cpu().numpy()[:, rows], ra)
    return X, dY, bits, alpha, hb, alpha.cpu().numpy()


PREFILL = [
    # workload, n, d_in, d_out, q, g
    (1, 2048, 1024, 3072, 3, 1024), (1, 2048, 1024, 1024, 3, 1024),
    (1, 2048, 1024, 4096, 3, 1024), (1, 2048, 4096, 1024, 3, 4096),
    (2, 4096, 1600, 4800, 4, 128), (2, 4096, 6400, 1600, 4, 128),
]


@pytest.mark.parametrize("workload,n,d_in,d_out,q,g", PREFILL)
def test_prefill_layer_sampled(workload, n, d_in, d_out, q, g):
    key = (workload, 0, d_out % 7)
    X, dY, bits, alpha, hb, ha = _layer(workload, n, d_in, d_out, q, g, key)
    G = oracle.num_groups(d_in, g)
    Xd, dYd = dev_bf16(X), dev_bf16(dY)
    Y = bcq.linear_fwd(Xd, bits, alpha, d_in, g).cpu().numpy()
    dX = bcq.linear_bwd_x(dYd, bits, alpha, d_in, g).cpu().numpy()
    dA = bcq.linear_bwd_alpha(dYd, Xd, bits, d_in, g).cpu().numpy()
    t, j, k = synth.sample_indices(NS, [n, d_out, d_in], key)
    i, c = synth.sample_indices(NS // 8, [q, G], (workload, 1, 0))
    # typical magnitudes: rms(Y) ~ rms(W_hat) sqrt(d_in); the tolerance is relative to max |ref|, for
    # which max over the samples is a (smaller, hence stricter) stand-in
    ref = oracle.fwd_at(X, hb, ha, d_in, g, t, j)
    _check_sampled(Y, ref, (t, j), np.abs(ref).max())
    ref_dx = oracle.bwd_x_at(dY, hb, ha, d_in, g, t, k)
    _check_sampled(dX, ref_dx, (t, k), np.abs(ref_dx).max())
    # bf16 outputs, as bench.py launches the layer (another epilogue: one more rounding, 2^-8)
    Yb = bcq.linear_fwd(Xd, bits, alpha, d_in, g, out_dtype=torch.bfloat16).float().cpu().numpy()
    dXb = bcq.linear_bwd_x(dYd, bits, alpha, d_in, g, out_dtype=torch.bfloat16).float().cpu().numpy()
    assert np.abs(Yb[(t, j)] - ref).max() <= (TOL + 2.0 ** -8) * np.abs(ref).max()
    assert np.abs(dXb[(t, k)] - ref_dx).max() <= (TOL + 2.0 ** -8) * np.abs(ref_dx).max()
    # and the whole bf16 output against the fp32 one: a misplaced tile would show here
    assert np.abs(Yb - Y).max() <= 2.0 ** -7 * np.abs(Y).max()
    assert np.abs(dXb - dX).max() <= 2.0 ** -7 * np.abs(dX).max()
    jj = j[: NS // 8]
    ref = oracle.bwd_alpha_at(dY, X, hb, d_in, g, i, jj, c)
    _check_sampled(dA, ref, (i, jj, c), np.abs(ref).max())


@pytest.mark.parametrize("d_in,d_out", [(4096, 12288), (4096, 16384), (16384, 4096)])
@pytest.mark.parametrize("q", [3, 4])
def test_decode_layer(d_in, d_out, q):
    # the oracle computes the whole GEMV for n = 1, 4, 16 in a few seconds
    g = 128
    key = (3, q, d_out % 5)
    X, _, bits, alpha, hb, ha = _layer(3, 16, d_in, d_out, q, g, key)
    for n in (1, 4, 16):
        Y = bcq.linear_decode(dev_bf16(X[:n]), bits, alpha, d_in, g).cpu().numpy()
        ref = oracle.fwd(X[:n], hb, ha, d_in, g)
        assert np.abs(Y - ref).max() <= TOL * np.abs(ref).max()


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
