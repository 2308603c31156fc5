"""Pins for the oracle's forward (Eq. 2) and backward (Eq. 3, Eq. 4).

The forward is compared with a dense fp64 matmul (numpy) against the reconstructed matrix of
Eq. 1, the backward with central finite differences of the forward and with the adjoint and
Euler identities; none of these go through the code under test.
"""
import numpy as np

import oracle
from paper_2210_03858_b200 import synth


def _unpack_py(bits, d_in):
    k = np.arange(d_in)
    b = (bits[:, :, k >> 5] >> (k & 31).astype(np.uint32)) & 1
    return b.astype(np.float64) * 2 - 1


def _dense_w(bits, alpha, d_in, g):
    b = _unpack_py(bits, d_in)
    return (alpha.astype(np.float64)[:, :, np.arange(d_in) // g] * b).sum(axis=0)


def _case(seed, n, d_in, d_out, q, g, alt=0):
    rng = np.random.default_rng(seed)
    W = (rng.standard_normal((d_out, d_in)) * 0.02).astype(np.float32)
    bits, alpha, _, _ = oracle.quantize(W, q, g, alt_iters=alt)
    X = synth.f32_to_bf16_bits(rng.standard_normal((n, d_in)).astype(np.float32))
    dY = synth.f32_to_bf16_bits(rng.standard_normal((n, d_out)).astype(np.float32))
    return bits, alpha, X, dY


CASES = [(20, 5, 70, 9, 3, 32), (21, 3, 128, 4, 1, 128), (22, 4, 100, 6, 4, 100),
         (23, 2, 33, 3, 2, 7), (24, 6, 64, 5, 3, 16)]


def test_bf16_conversion_round_trip_and_rne():
    x = np.array([1.0, -2.5, 1.00390625, 1.01171875, 3.14159, 1e-3], dtype=np.float32)
    b = synth.f32_to_bf16_bits(x)
    f = synth.bf16_bits_to_f32(b)
    assert f[0] == 1.0 and f[1] == -2.5
    assert f[2] == 1.0            # 1 + 2^-8 is a tie: rounds to even (1.0)
    assert f[3] == 1.015625       # 1 + 3*2^-8 is a tie: rounds to even (1 + 2^-6)
    assert np.all(np.abs(f - x) <= np.abs(x) * 2.0 ** -8)
    np.testing.assert_array_equal(synth.f32_to_bf16_bits(f), b)


def test_fwd_equals_dense_matmul_with_reconstructed_w():
    for seed, n, d_in, d_out, q, g in CASES:
        bits, alpha, X, _ = _case(seed, n, d_in, d_out, q, g)
        Wd = _dense_w(bits, alpha, d_in, g)
        Xd = synth.bf16_bits_to_f32(X).astype(np.float64)
        Y = oracle.fwd(X, bits, alpha, d_in, g)
        np.testing.assert_allclose(Y, Xd @ Wd.T, rtol=1e-12, atol=1e-13)
        bias = np.linspace(-1, 1, d_out).astype(np.float32)
        Yb = oracle.fwd(X, bits, alpha, d_in, g, bias=bias)
        np.testing.assert_allclose(Yb, Xd @ Wd.T + bias.astype(np.float64), rtol=1e-12, atol=1e-13)


def test_fwd_q1_rowwise_special_case():
    # Y = (X sign(W)^T) diag(alpha) for q = 1 and g = d_in
    rng = np.random.default_rng(30)
    W = (rng.standard_normal((6, 40)) * 0.02).astype(np.float32)
    bits, alpha, _, _ = oracle.quantize(W, 1, 40)
    X = synth.f32_to_bf16_bits(rng.standard_normal((3, 40)).astype(np.float32))
    Xd = synth.bf16_bits_to_f32(X).astype(np.float64)
    ref = (Xd @ np.where(W >= 0, 1.0, -1.0).T) * np.abs(W.astype(np.float64)).mean(axis=1).astype(np.float32)
    np.testing.assert_allclose(oracle.fwd(X, bits, alpha, 40, 40), ref, rtol=1e-12, atol=1e-14)


def test_sampled_entry_points_match_full():
    seed, n, d_in, d_out, q, g = CASES[0]
    bits, alpha, X, dY = _case(seed, n, d_in, d_out, q, g)
    G = oracle.num_groups(d_in, g)
    Y = oracle.fwd(X, bits, alpha, d_in, g)
    dX = oracle.bwd_x(dY, bits, alpha, d_in, g)
    dA = oracle.bwd_alpha(dY, X, bits, d_in, g)
    rng = np.random.default_rng(0)
    t = rng.integers(0, n, 50); j = rng.integers(0, d_out, 50); k = rng.integers(0, d_in, 50)
    i = rng.integers(0, q, 50); c = rng.integers(0, G, 50)
    np.testing.assert_allclose(oracle.fwd_at(X, bits, alpha, d_in, g, t, j), Y[t, j], rtol=1e-13)
    np.testing.assert_allclose(oracle.bwd_x_at(dY, bits, alpha, d_in, g, t, k), dX[t, k], rtol=1e-12, atol=1e-14)
    np.testing.assert_allclose(oracle.bwd_alpha_at(dY, X, bits, d_in, g, i, j, c), dA[i, j, c], rtol=1e-12, atol=1e-13)


def test_bwd_x_dense_and_finite_difference():
    for seed, n, d_in, d_out, q, g in CASES:
        bits, alpha, X, dY = _case(seed, n, d_in, d_out, q, g)
        Wd = _dense_w(bits, alpha, d_in, g)
        dYd = synth.bf16_bits_to_f32(dY).astype(np.float64)
        dX = oracle.bwd_x(dY, bits, alpha, d_in, g)
        np.testing.assert_allclose(dX, dYd @ Wd, rtol=1e-12, atol=1e-13)
        # L(X) = <dY, fwd(X)> is linear in X: a central difference with a bf16-exact step is
        # exact up to rounding.  Perturb single entries through the oracle's own forward.
        Xf = synth.bf16_bits_to_f32(X)
        rng = np.random.default_rng(seed)
        for _ in range(6):
            t, k = int(rng.integers(n)), int(rng.integers(d_in))
            h = 0.5
            Xp, Xm = Xf.copy(), Xf.copy()
            Xp[t, k] = np.float32(np.round(Xf[t, k] * 4) / 4 + h)
            Xm[t, k] = np.float32(np.round(Xf[t, k] * 4) / 4 - h)
            Lp = (dYd * oracle.fwd(synth.f32_to_bf16_bits(Xp), bits, alpha, d_in, g)).sum()
            Lm = (dYd * oracle.fwd(synth.f32_to_bf16_bits(Xm), bits, alpha, d_in, g)).sum()
            assert abs((Lp - Lm) / (2 * h) - dX[t, k]) <= 1e-9 * max(1.0, abs(dX[t, k]))


def test_bwd_alpha_dense_finite_difference_and_scale():
    for seed, n, d_in, d_out, q, g in CASES:
        bits, alpha, X, dY = _case(seed, n, d_in, d_out, q, g)
        G = oracle.num_groups(d_in, g)
        b = _unpack_py(bits, d_in)
        Xd = synth.bf16_bits_to_f32(X).astype(np.float64)
        dYd = synth.bf16_bits_to_f32(dY).astype(np.float64)
        P = dYd.T @ Xd                                   # (d_out, d_in) = dY^T X
        ref = np.zeros((q, d_out, G))
        for c in range(G):
            sl = slice(c * g, min((c + 1) * g, d_in))
            ref[:, :, c] = (b[:, :, sl] * P[None, :, sl]).sum(axis=2)
        dA = oracle.bwd_alpha(dY, X, bits, d_in, g)
        np.testing.assert_allclose(dA, ref, rtol=1e-11, atol=1e-11)
        # Eq. 4's empirical 1/g_L factor is just a scale on the gradient
        np.testing.assert_allclose(oracle.bwd_alpha(dY, X, bits, d_in, g, scale=1.0 / g), ref / g,
                                   rtol=1e-11, atol=1e-12)
        # finite differences through the forward: L(alpha) is linear in alpha
        rng = np.random.default_rng(seed + 100)
        for _ in range(6):
            i, j, c = int(rng.integers(q)), int(rng.integers(d_out)), int(rng.integers(G))
            ap, am = alpha.copy(), alpha.copy()
            base = np.float32(np.round(alpha[i, j, c] * 64) / 64)
            ap[i, j, c] = base + np.float32(0.25)
            am[i, j, c] = base - np.float32(0.25)
            Lp = (dYd * oracle.fwd(X, bits, ap, d_in, g)).sum()
            Lm = (dYd * oracle.fwd(X, bits, am, d_in, g)).sum()
            assert abs((Lp - Lm) / 0.5 - dA[i, j, c]) <= 1e-9 * max(1.0, abs(dA[i, j, c]))


def test_plane_mask_leaves_other_planes_untouched():
    seed, n, d_in, d_out, q, g = CASES[0]
    bits, alpha, X, dY = _case(seed, n, d_in, d_out, q, g)
    full = oracle.bwd_alpha(dY, X, bits, d_in, g)
    out = np.full_like(full, 123.0)
    oracle.bwd_alpha(dY, X, bits, d_in, g, plane_mask=0b001, out=out)   # alpha_1 only
    np.testing.assert_array_equal(out[0], full[0])
    assert (out[1:] == 123.0).all()


def test_adjoint_and_euler_identities():
    for seed, n, d_in, d_out, q, g in CASES:
        bits, alpha, X, dY = _case(seed, n, d_in, d_out, q, g, alt=2)
        Xd = synth.bf16_bits_to_f32(X).astype(np.float64)
        dYd = synth.bf16_bits_to_f32(dY).astype(np.float64)
        Y = oracle.fwd(X, bits, alpha, d_in, g)
        dX = oracle.bwd_x(dY, bits, alpha, d_in, g)
        dA = oracle.bwd_alpha(dY, X, bits, d_in, g)
        lhs = (dYd * Y).sum()
        assert abs(lhs - (dX * Xd).sum()) <= 1e-10 * max(1.0, abs(lhs))           # <dY, Y> = <dX, X>
        # Y is homogeneous of degree one in alpha:  sum alpha * dalpha = <dY, Y>, row by row
        per_row = (alpha.astype(np.float64) * dA).sum(axis=(0, 2))
        np.testing.assert_allclose(per_row, (dYd * Y).sum(axis=0), rtol=1e-9, atol=1e-9)
