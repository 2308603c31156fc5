"""Pins of the oracle's optimiser step (AdamW on the scales, linear-decay learning rate), none of
which goes through the oracle's own arithmetic: a hand-computed two-step example, torch's AdamW in
fp64 as an independent library implementation, closed-form special cases, and a small end-to-end
check that training alpha_1 alone lowers a regression loss through the BCQ layer."""
import os

import numpy as np
import pytest
import torch

import oracle
from paper_2210_03858_b200 import synth

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def test_adamw_hand_computed_two_steps():
    p = np.array([1.0, -2.0], dtype=np.float32)
    m = np.zeros(2, dtype=np.float32)
    v = np.zeros(2, dtype=np.float32)
    with open(os.path.join(GOLDEN, "adamw_two_steps.txt")) as f:
        rows = [l.split() for l in f if l.strip() and not l.startswith("#")]
    for step, g0, g1, p0, p1 in rows:
        oracle.adamw(p, np.array([float(g0), float(g1)], dtype=np.float32), m, v, int(step), lr=0.1, beta1=0.9,
                     beta2=0.999, eps=0.0, wd=0.1)
        np.testing.assert_allclose(p, [float(p0), float(p1)], rtol=2e-6)


def test_adamw_matches_torch_adamw():
    rng = np.random.default_rng(5)
    p0 = rng.standard_normal(257).astype(np.float32)
    tp = torch.nn.Parameter(torch.from_numpy(p0.astype(np.float64)))
    opt = torch.optim.AdamW([tp], lr=3e-3, betas=(0.85, 0.98), eps=1e-7, weight_decay=0.05)
    p, m, v = p0.copy(), np.zeros_like(p0), np.zeros_like(p0)
    for step in range(1, 8):
        g = rng.standard_normal(257).astype(np.float32)
        tp.grad = torch.from_numpy(g.astype(np.float64) * 0.25)
        opt.step()
        oracle.adamw(p, g, m, v, step, lr=3e-3, beta1=0.85, beta2=0.98, eps=1e-7, wd=0.05, grad_scale=0.25)
        # the oracle rounds its state to fp32 after every step, torch keeps fp64
        np.testing.assert_allclose(p, tp.detach().numpy(), rtol=0, atol=step * 4e-7)


def test_adamw_special_cases():
    p = np.array([2.0, -3.0], dtype=np.float32)
    m, v = np.zeros(2, np.float32), np.zeros(2, np.float32)
    # zero gradient: only the decoupled weight decay acts
    oracle.adamw(p, np.zeros(2, np.float32), m, v, 1, lr=0.5, eps=1e-8, wd=0.2)
    np.testing.assert_allclose(p, [2.0 * 0.9, -3.0 * 0.9], rtol=1e-6)
    assert not m.any() and not v.any()
    # first step without decay and eps: the step is lr * sign(g), whatever |g| and the gradient scale
    p = np.zeros(3, np.float32)
    m, v = np.zeros(3, np.float32), np.zeros(3, np.float32)
    oracle.adamw(p, np.array([1e-3, -7.0, 40.0], np.float32), m, v, 1, lr=0.01, eps=0.0, wd=0.0, grad_scale=1.0 / 1024)
    np.testing.assert_allclose(p, [-0.01, 0.01, -0.01], rtol=1e-6)


def test_linear_decay_schedule():
    assert oracle.lr_linear(1e-4, 0, 0, 100) == pytest.approx(1e-4)
    assert oracle.lr_linear(1e-4, 50, 0, 100) == pytest.approx(0.5e-4)
    assert oracle.lr_linear(1e-4, 100, 0, 100) == 0.0
    assert oracle.lr_linear(1e-4, 250, 500, 1000) == pytest.approx(0.5e-4)     # warm-up (ablation table)
    assert oracle.lr_linear(1e-4, 750, 500, 1000) == pytest.approx(0.5e-4)
    lrs = [oracle.lr_linear(1.0, s, 10, 60) for s in range(61)]
    assert np.argmax(lrs) == 10 and all(np.diff(lrs[10:]) < 0)


def test_training_alpha1_lowers_the_loss():
    # a tiny AlphaTuning loop on one layer: B frozen, only alpha_1 trained with Eq. 4's gradient
    # (scaled by 1/g_L) and AdamW under linear decay; the regression loss must go down
    n, d_in, d_out, q, g = 48, 64, 24, 3, 32
    key = (60, 0, 0)
    W = synth.weights(d_out, d_in, key)
    X = synth.activations(n, d_in, key, synth.ROLE_X)
    bits, alpha, _, _ = oracle.quantize(W, q, g)
    target = synth.bf16_bits_to_f32(X).astype(np.float64) @ (W.astype(np.float64).T * 1.3)
    a = alpha.copy()
    m, v = np.zeros_like(a[0]), np.zeros_like(a[0])
    losses = []
    for step in range(1, 21):
        Y = oracle.fwd(X, bits, a, d_in, g)
        losses.append(float(((Y - target) ** 2).sum()))
        dY = synth.f32_to_bf16_bits((2.0 * (Y - target)).astype(np.float32))
        grad = oracle.bwd_alpha(dY, X, bits, d_in, g, plane_mask=1)[0].astype(np.float32)
        lr = oracle.lr_linear(2e-3, step - 1, 0, 40)
        a1 = np.ascontiguousarray(a[0])
        oracle.adamw(a1, grad, m, v, step, lr=lr, wd=0.01, grad_scale=1.0 / g)
        a[0] = a1
    assert losses[-1] < 0.8 * losses[0]
    assert np.array_equal(a[1:], alpha[1:])      # the other planes' scales are untouched
