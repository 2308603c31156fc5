"""Pins for the oracle's quantizer and container format.

Nothing here goes through the CUDA library.  Each test checks the oracle against something
the paper or the mathematics fixes independently of the oracle's own code: the q = 1 closed
form, exhaustive search over sign patterns, numpy's least squares, a hand-computed example,
the residual-energy identity of the greedy recurrence, and the sizes the paper prints.
"""
import itertools
import os

import numpy as np
import pytest

import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _rows(name):
    out = []
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            line = line.split("#")[0].strip()
            if line:
                out.append(line.split())
    return out


def _unpack_py(bits, d_in):
    """Independent unpack straight from the format definition (bit k&31 of word k>>5)."""
    q, d_out, _ = bits.shape
    k = np.arange(d_in)
    b = (bits[:, :, k >> 5] >> (k & 31).astype(np.uint32)) & 1
    return b.astype(np.int8) * 2 - 1


def _rng(seed):
    return np.random.default_rng(seed)


# ------------------------------------------------------------------ format


def test_pack_layout_and_padding():
    rng = _rng(1)
    for d_in in (1, 31, 32, 33, 127, 128, 129, 200):
        signs = rng.integers(0, 2, size=(3, 5, d_in)).astype(np.int8) * 2 - 1
        bits = oracle.pack(signs)
        assert bits.shape == (3, 5, 4 * ((d_in + 127) // 128))
        np.testing.assert_array_equal(_unpack_py(bits, d_in), signs)
        np.testing.assert_array_equal(oracle.unpack(bits, d_in), signs)
        # padding bits are zero
        total = bits.shape[2] * 32
        kk = np.arange(d_in, total)
        if kk.size:
            pad = (bits[:, :, kk >> 5] >> (kk & 31).astype(np.uint32)) & 1
            assert not pad.any()


def test_single_bit_position():
    signs = -np.ones((1, 1, 70), dtype=np.int8)
    signs[0, 0, 37] = 1
    bits = oracle.pack(signs)
    assert bits[0, 0, 1] == (1 << 5) and bits[0, 0, 0] == 0 and bits[0, 0, 2] == 0


def test_table1_sizes():
    for layer, d_out, d_in, g, *cells in _rows("table1_sizes.txt"):
        for q, cell in zip((1, 2, 3), cells):
            if cell == "-":
                continue
            mb = oracle.payload_bytes(int(d_out), int(d_in), q, int(g)) / 1e6
            assert abs(mb - float(cell)) <= 0.0051, (layer, g, q, mb, cell)


def _alpha_count(hidden, ffn, layers, planes, g):
    total = 0
    for d_in, d_out in ((hidden, 3 * hidden), (hidden, hidden), (hidden, ffn), (ffn, hidden)):
        gg = d_in if g == "row" else int(g)
        total += planes * d_out * oracle.num_groups(d_in, gg)
    return total * layers


def test_trainable_parameter_counts():
    for name, hidden, ffn, layers, planes, g, printed in _rows("param_counts.txt"):
        cnt = _alpha_count(int(hidden), int(ffn), int(layers), int(planes), g)
        assert abs(cnt / 1e6 - float(printed)) <= 0.0055, (name, cnt, printed)
    assert _alpha_count(1024, 4096, 24, 1, "row") == 221184
    assert _alpha_count(1024, 4096, 24, 3, "row") == 663552


def test_model_sizes():
    quantized = 24 * 12 * 1024 * 1024
    rest_bytes = (354.9e6 - quantized) * 4
    for q, printed in _rows("model_sizes.txt"):
        q = int(q)
        qbytes = 0.0
        for d_in, d_out in ((1024, 3072), (1024, 1024), (1024, 4096), (4096, 1024)):
            qbytes += 24 * oracle.payload_bytes(d_out, d_in, q, d_in)
        assert abs((qbytes + rest_bytes) / 1e6 - float(printed)) <= 1.0


# ------------------------------------------------------------------ q = 1 and greedy


def test_q1_closed_form():
    rng = _rng(2)
    W = (rng.standard_normal((7, 96)) * 0.02).astype(np.float32)
    W[0, 3] = 0.0
    W[1, 5] = -0.0
    for g in (96, 32, 40):
        bits, alpha, sq_err, _ = oracle.quantize(W, 1, g)
        b = _unpack_py(bits, 96)[0]
        np.testing.assert_array_equal(b, np.where(W >= 0, 1, -1))  # sign(0) = sign(-0) = +1
        G = oracle.num_groups(96, g)
        for c in range(G):
            seg = W[:, c * g:min((c + 1) * g, 96)].astype(np.float64)
            np.testing.assert_array_equal(alpha[0, :, c], np.abs(seg).mean(axis=1).astype(np.float32))
            a = alpha[0, :, c].astype(np.float64)[:, None]
            e = ((seg - a * np.where(seg >= 0, 1, -1)) ** 2).sum(axis=1)
            np.testing.assert_allclose(sq_err[:, c], e, rtol=1e-12)


def test_q1_is_the_global_optimum_by_brute_force():
    rng = _rng(3)
    for m in (1, 2, 5, 8):
        W = rng.standard_normal((6, m)).astype(np.float32)
        _, _, sq_err, _ = oracle.quantize(W, 1, m)
        for j in range(6):
            w = W[j].astype(np.float64)
            best = np.inf
            for s in itertools.product((-1.0, 1.0), repeat=m):
                b = np.array(s)
                a = w @ b / m
                best = min(best, ((w - a * b) ** 2).sum())
            assert abs(sq_err[j, 0] - best) <= 1e-6 * max(best, 1e-12) + 1e-12


def test_greedy_hand_example():
    rows = {r[0]: [float(v) for v in r[1:]] for r in _rows("greedy_dyadic.txt")}
    w = np.array([rows["w"]], dtype=np.float32)
    for q in (1, 2, 3):
        bits, alpha, sq_err, _ = oracle.quantize(w, q, 4)
        b = _unpack_py(bits, 4)
        np.testing.assert_array_equal(alpha[:, 0, 0], np.array(rows["alpha"][:q], dtype=np.float32))
        for i in range(q):
            np.testing.assert_array_equal(b[i, 0], np.array(rows["b%d" % (i + 1)], dtype=np.int8))
        assert sq_err[0, 0] == rows["sqerr"][q - 1]


def test_greedy_energy_identity_and_monotone_error():
    # From r_{i-1}^T b_i = m alpha_i:  |r_i|^2 = |r_{i-1}|^2 - m alpha_i^2.
    rng = _rng(4)
    W = (rng.standard_normal((5, 256)) * 0.02).astype(np.float32)
    prev = None
    for q in range(1, 7):
        bits, alpha, sq_err, _ = oracle.quantize(W, q, 64)
        assert (alpha >= 0).all()
        Wd = W.astype(np.float64).reshape(5, 4, 64)
        e = (Wd ** 2).sum(axis=2) - 64 * (alpha.astype(np.float64) ** 2).sum(axis=0)
        # alpha is stored rounded to fp32, so the identity holds to ~1e-7 of the row energy
        assert (np.abs(sq_err - e) <= 1e-6 * (Wd ** 2).sum(axis=2)).all()
        if prev is not None:
            assert (sq_err <= prev + 1e-15).all()
            np.testing.assert_array_equal(alpha[:q - 1], prev_alpha)  # planes are nested
            np.testing.assert_array_equal(bits[:q - 1], prev_bits)
        prev, prev_alpha, prev_bits = sq_err, alpha, bits


def test_greedy_matches_stepwise_numpy():
    rng = _rng(5)
    W = (rng.standard_normal((4, 100)) * 0.02).astype(np.float32)
    g, q = 48, 4  # groups of 48, 48 and a ragged 4
    bits, alpha, _, _ = oracle.quantize(W, q, g)
    b = _unpack_py(bits, 100)
    for c, (k0, k1) in enumerate(((0, 48), (48, 96), (96, 100))):
        r = W[:, k0:k1].astype(np.float64)
        for i in range(q):
            s = np.where(r >= 0, 1.0, -1.0)
            a = np.abs(r).mean(axis=1).astype(np.float32)
            np.testing.assert_array_equal(b[i, :, k0:k1], s.astype(np.int8))
            np.testing.assert_array_equal(alpha[i, :, c], a)
            r = r - a.astype(np.float64)[:, None] * s


def test_dequantize_definition():
    rng = _rng(6)
    W = (rng.standard_normal((9, 70)) * 0.02).astype(np.float32)
    bits, alpha, sq_err, _ = oracle.quantize(W, 3, 32)
    b = _unpack_py(bits, 70).astype(np.float64)
    grp = np.arange(70) // 32
    W_hat = (alpha.astype(np.float64)[:, :, grp] * b).sum(axis=0)
    np.testing.assert_allclose(oracle.dequantize(bits, alpha, 70, 32), W_hat, rtol=0, atol=1e-15)
    e = np.zeros((9, 3))
    for c in range(3):
        sel = grp == c
        e[:, c] = ((W.astype(np.float64)[:, sel] - W_hat[:, sel]) ** 2).sum(axis=1)
    np.testing.assert_allclose(sq_err, e, rtol=1e-10, atol=1e-18)


# ------------------------------------------------------------------ alternating


def _sq_err_of(w, b, a):
    return ((w - (a[:, None] * b).sum(axis=0)) ** 2).sum()


def test_alternating_alpha_is_least_squares_for_its_bits():
    rng = _rng(7)
    W = (rng.standard_normal((6, 192)) * 0.02).astype(np.float32)
    for q in (1, 2, 3, 4):
        for T in (1, 3):
            bits, alpha, sq_err, _ = oracle.quantize(W, q, 64, alt_iters=T)
            b = _unpack_py(bits, 192).astype(np.float64)
            for j in range(6):
                for c in range(3):
                    B = b[:, j, c * 64:(c + 1) * 64].T  # (m, q)
                    w = W[j, c * 64:(c + 1) * 64].astype(np.float64)
                    ref, *_ = np.linalg.lstsq(B, w, rcond=None)
                    a = alpha[:, j, c]
                    np.testing.assert_allclose(a, ref, rtol=3e-7, atol=1e-9)
                    # normal equations B^T (w - B a) ~ 0 up to the fp32 rounding of a
                    resid = B.T @ (w - B @ a.astype(np.float64))
                    assert np.abs(resid).max() <= 64 * q * 1e-7 * np.abs(ref).max() + 1e-12
                    # no small change of any scale lowers the error
                    e0 = _sq_err_of(w, B.T, a.astype(np.float64))
                    assert abs(e0 - sq_err[j, c]) <= 1e-9 * e0 + 1e-18
                    for i in range(q):
                        for d in (-1e-3, 1e-3):
                            a2 = a.astype(np.float64).copy()
                            a2[i] += d * max(abs(a2[i]), 1e-3)
                            assert _sq_err_of(w, B.T, a2) >= e0 * (1 - 1e-9)


def test_alternating_error_chain():
    # greedy >= alternating(T) and the error does not grow with more iterations
    rng = _rng(8)
    W = (rng.standard_normal((8, 128)) * 0.02).astype(np.float32)
    W[rng.random((8, 128)) < 0.01] *= 20
    for q in (2, 3, 4):
        _, _, e_prev, _ = oracle.quantize(W, q, 128, alt_iters=0)
        for T in (1, 2, 5, 15):
            _, _, e, _ = oracle.quantize(W, q, 128, alt_iters=T)
            assert (e <= e_prev * (1 + 1e-6) + 1e-15).all(), (q, T)
            e_prev = e


def test_alternating_nearest_level_assignment():
    # after the last refit every element sits on the level nearest to it for the alphas that
    # were current when the bits were chosen; check with one iteration, where those alphas are
    # the least-squares fit to the greedy bits.
    rng = _rng(9)
    W = (rng.standard_normal((3, 64)) * 0.02).astype(np.float32)
    q = 3
    gbits, _, _, _ = oracle.quantize(W, q, 64, alt_iters=0)
    bg = _unpack_py(gbits, 64).astype(np.float64)
    bits, _, _, _ = oracle.quantize(W, q, 64, alt_iters=1)
    b = _unpack_py(bits, 64)
    codes = np.array(list(itertools.product((-1.0, 1.0), repeat=q)))  # (8, q)
    for j in range(3):
        w = W[j].astype(np.float64)
        a, *_ = np.linalg.lstsq(bg[:, j, :].T, w, rcond=None)
        a = a.astype(np.float32).astype(np.float64)
        levels = codes @ a
        nearest = np.abs(w[:, None] - levels[None, :]).min(axis=1)
        chosen = (a[:, None] * b[:, j, :]).sum(axis=0)
        np.testing.assert_allclose(np.abs(w - chosen), nearest, rtol=1e-12, atol=1e-18)


def test_alternating_tie_prefers_largest_code():
    # w = 0 is equidistant from +a and -a for q = 1; the larger code (+1) must win, as for sign(0)
    W = np.array([[0.5, -0.5, 0.0, 0.0]], dtype=np.float32)
    bits, alpha, _, margin = oracle.quantize(W, 1, 4, alt_iters=2)
    np.testing.assert_array_equal(_unpack_py(bits, 4)[0, 0], [1, -1, 1, 1])
    assert margin[0, 0] == 0.0


def test_alternating_not_below_global_optimum():
    rng = _rng(10)
    for m, q in ((5, 2), (6, 2), (4, 3)):
        W = rng.standard_normal((4, m)).astype(np.float32)
        _, _, e_alt, _ = oracle.quantize(W, q, m, alt_iters=15)
        _, _, e_gr, _ = oracle.quantize(W, q, m, alt_iters=0)
        for j in range(4):
            w = W[j].astype(np.float64)
            best = np.inf
            for s in itertools.product((-1.0, 1.0), repeat=m * q):
                B = np.array(s).reshape(q, m).T
                a, *_ = np.linalg.lstsq(B, w, rcond=None)
                best = min(best, ((w - B @ a) ** 2).sum())
            assert e_alt[j, 0] >= best - 1e-9
            assert e_alt[j, 0] <= e_gr[j, 0] * (1 + 1e-6) + 1e-15


def test_singular_planes_keep_previous_alpha():
    # integer-valued row whose residual vanishes after one plane: plane 2 becomes all +1 with
    # alpha 0 while plane 1 is all +1 too, so B^T B is singular and the refit is skipped.
    W = np.full((1, 8), 0.25, dtype=np.float32)
    bits, alpha, sq_err, _ = oracle.quantize(W, 2, 8, alt_iters=3)
    assert np.isfinite(alpha).all()
    np.testing.assert_array_equal(alpha[:, 0, 0], np.array([0.25, 0.0], dtype=np.float32))
    assert sq_err[0, 0] == 0.0


def test_margin_flags_near_ties_only():
    rng = _rng(11)
    W = (rng.standard_normal((16, 128)) * 0.02).astype(np.float32)
    _, _, _, margin = oracle.quantize(W, 3, 128)
    assert (margin > 0).all()
    W[3, 7] = 0.0  # exact tie in the first plane
    _, _, _, margin = oracle.quantize(W, 3, 128)
    assert margin[3, 0] == 0.0 and (np.delete(margin[:, 0], 3) > 0).all()


def test_invalid_arguments():
    W = np.zeros((2, 8), dtype=np.float32)
    for q, g in ((0, 8), (9, 8), (2, 0), (2, 9)):
        with pytest.raises(ValueError):
            oracle.quantize(W, q, g)
