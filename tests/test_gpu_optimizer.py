"""GPU parity of the AlphaTuning update (bcq_alpha_adamw) and of the scale-only checkpoint
(bcq_alpha_pack / bcq_alpha_unpack) against the oracle, through the C ABI.

Tolerance: the kernel computes a step in fp32 (about ten rounded operations per element), the oracle
in fp64 with the state rounded to fp32 once per step, so after three steps the scales and moments
agree to a few fp32 ulps: 1e-6 relative to the largest magnitude of each array."""
import numpy as np
import pytest

import oracle
import paper_2210_03858_b200 as bcq
from paper_2210_03858_b200 import build as bcq_build
from paper_2210_03858_b200.dist import AlphaBucket

pytestmark = pytest.mark.gpu
torch = pytest.importorskip("torch")


@pytest.fixture(scope="module", autouse=True)
def _built():
    bcq_build.build_library()


def f32(x):
    """The value the C ABI receives: hyper-parameters cross it as fp32, so the oracle gets the same."""
    return float(np.float32(x))


def _close(dev_t, ref, rel=1e-6):
    got = dev_t.cpu().numpy().astype(np.float64)
    assert np.abs(got - ref).max() <= rel * max(1e-30, np.abs(ref).max())


def test_adamw_three_steps_alpha1_of_several_linears():
    shapes = [(3, 40, 2), (3, 24, 1), (4, 130, 13)]          # (q, d_out, G) of three linears
    groups = [64, 1024, 128]                                   # their group sizes g_L
    rng = np.random.default_rng(3)
    bucket_a, bucket_g = AlphaBucket(shapes, "cuda"), AlphaBucket(shapes, "cuda")
    a0 = (rng.standard_normal(bucket_a.flat.numel()) * 0.02).astype(np.float32)
    bucket_a.flat.copy_(torch.from_numpy(a0))
    m = torch.zeros_like(bucket_a.flat)
    v = torch.zeros_like(bucket_a.flat)
    runs = bucket_a.plane_segments(0b001)                      # alpha_1 only, as the paper trains
    seg = bcq.Segments(runs, "cuda", scales=[1.0 / g for g in groups])
    ra, rm, rv = a0.copy(), np.zeros_like(a0), np.zeros_like(a0)
    for step in (1, 2, 3):
        g = rng.standard_normal(a0.size).astype(np.float32)
        bucket_g.flat.copy_(torch.from_numpy(g))
        lr = bcq.lr_linear_decay(1e-3, step - 1, 0, 10)
        assert lr == pytest.approx(oracle.lr_linear(1e-3, step - 1, 0, 10), rel=1e-6)
        bcq.alpha_adamw(bucket_a.flat, bucket_g.flat, m, v, step, lr, 0.9, 0.999, 1e-8, 0.01, segments=seg)
        for (b, c), gl in zip(runs, groups):
            sa, sm, sv = ra[b:b + c].copy(), rm[b:b + c].copy(), rv[b:b + c].copy()
            oracle.adamw(sa, g[b:b + c], sm, sv, step, lr=lr, beta1=f32(0.9), beta2=f32(0.999), eps=f32(1e-8),
                         wd=f32(0.01), grad_scale=f32(1.0 / gl))
            ra[b:b + c], rm[b:b + c], rv[b:b + c] = sa, sm, sv
    _close(bucket_a.flat, ra.astype(np.float64))
    _close(m, rm.astype(np.float64))
    _close(v, rv.astype(np.float64))
    # everything outside alpha_1 is bit-for-bit what it was
    mask = np.ones(a0.size, bool)
    for b, c in runs:
        mask[b:b + c] = False
    assert np.array_equal(bucket_a.flat.cpu().numpy()[mask], a0[mask])
    assert not m.cpu().numpy()[mask].any()


def test_adamw_contiguous_and_warmup_schedule():
    rng = np.random.default_rng(4)
    a0 = rng.standard_normal(5000).astype(np.float32)
    a = torch.from_numpy(a0).cuda()
    m, v = torch.zeros_like(a), torch.zeros_like(a)
    ra, rm, rv = a0.copy(), np.zeros_like(a0), np.zeros_like(a0)
    for step in (1, 2, 3):
        g = rng.standard_normal(5000).astype(np.float32)
        lr = bcq.lr_linear_decay(5e-4, step, 2, 20)
        assert lr == pytest.approx(oracle.lr_linear(5e-4, step, 2, 20), rel=1e-6)
        bcq.alpha_adamw(a, torch.from_numpy(g).cuda(), m, v, step, lr, 0.8, 0.95, 1e-6, 0.1, grad_scale=0.5)
        oracle.adamw(ra, g, rm, rv, step, lr=lr, beta1=f32(0.8), beta2=f32(0.95), eps=f32(1e-6), wd=f32(0.1),
                     grad_scale=0.5)
    _close(a, ra.astype(np.float64))
    _close(m, rm.astype(np.float64))
    _close(v, rv.astype(np.float64))


def test_checkpoint_pack_unpack_round_trip():
    shapes = [(3, 17, 4), (2, 9, 1), (4, 33, 7)]
    bucket = AlphaBucket(shapes, "cuda")
    vals = torch.arange(bucket.flat.numel(), dtype=torch.float32, device="cuda")
    bucket.flat.copy_(vals)
    runs = bucket.plane_segments(0b001)
    seg = bcq.Segments(runs, "cuda")
    ckpt = bcq.alpha_pack(bucket.flat, seg)
    expect = np.concatenate([np.arange(b, b + c) for b, c in runs]).astype(np.float32)
    assert np.array_equal(ckpt.cpu().numpy(), expect)                # bit-exact gather, documented order
    bucket.flat.zero_()
    bcq.alpha_unpack(ckpt, bucket.flat, seg)
    back = bucket.flat.cpu().numpy()
    off = 0
    for i, (q, d_out, G) in enumerate(shapes):
        assert np.array_equal(bucket[i][0].cpu().numpy().ravel(), expect[off:off + d_out * G])
        off += d_out * G
    assert back.sum() == expect.sum()                                 # nothing else was written


def test_training_steps_end_to_end_on_device():
    # forward -> loss gradient -> dalpha (Eq. 4 with the 1/g_L scale) -> AdamW on alpha_1: the loss falls
    from paper_2210_03858_b200 import synth
    n, d_in, d_out, q, g = 128, 256, 192, 3, 64
    key = (61, 0, 0)
    W = synth.weights(d_out, d_in, key)
    X = synth.activations(n, d_in, key, synth.ROLE_X)
    bits, alpha, _ = bcq.quantize(torch.from_numpy(W).cuda(), q, g)
    G = bcq.num_groups(d_in, g)
    ba, bg = AlphaBucket([(q, d_out, G)], "cuda"), AlphaBucket([(q, d_out, G)], "cuda")
    ba[0].copy_(alpha)
    m, v = torch.zeros_like(ba.flat), torch.zeros_like(ba.flat)
    seg = bcq.Segments(ba.plane_segments(1), "cuda")
    Xd = torch.from_numpy(X.view(np.int16)).cuda().view(torch.bfloat16)
    target = (Xd.float() @ torch.from_numpy(W).cuda().t()) * 1.3
    losses = []
    for step in range(1, 13):
        Y = bcq.linear_fwd(Xd, bits, ba[0], d_in, g)
        losses.append(float(((Y - target) ** 2).sum()))
        dY = (2.0 * (Y - target)).bfloat16()
        bcq.linear_bwd_alpha(dY, Xd, bits, d_in, g, plane_mask=1, scale=1.0 / g, out=bg[0])
        bcq.alpha_adamw(ba.flat, bg.flat, m, v, step, bcq.lr_linear_decay(2e-3, step - 1, 0, 24), segments=seg,
                        weight_decay=0.01)
    assert losses[-1] < 0.8 * losses[0]
    assert torch.equal(ba[0][1:], alpha[1:])
