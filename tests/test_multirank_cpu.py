"""The data-parallel shape of the path, on CPU with two gloo ranks: tokens are split over ranks,
every rank computes the scale gradient (Eq. 4) of its own tokens for several linears into the
views of one flat bucket, and the library's helper (the one bench.py calls for N > 1) all-reduces
the bucket.  The result must be the oracle's gradient of the whole batch, in every linear's own
view.  Forward and dX need no exchange: each rank's rows are its own.  The per-rank arithmetic is
the oracle's; what is tested is the sharding, the bucket layout and the reduction."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import oracle
from paper_2210_03858_b200 import synth
from paper_2210_03858_b200.dist import AlphaBucket, allreduce_dalpha

N, Q = 24, 3
LINEARS = [(96, 40, 32), (64, 56, 64), (40, 24, 40)]   # d_in, d_out, g


def _inputs(li):
    d_in, d_out, g = LINEARS[li]
    key = (50, li, 0)
    W = synth.weights(d_out, d_in, key)
    X = synth.activations(N, d_in, key, synth.ROLE_X)
    dY = synth.activations(N, d_out, key, synth.ROLE_DY)
    bits, alpha, _, _ = oracle.quantize(W, Q, g)
    return X, dY, bits, alpha


def _shapes():
    return [(Q, d_out, oracle.num_groups(d_in, g)) for d_in, d_out, g in LINEARS]


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    bucket = AlphaBucket(_shapes(), "cpu")
    lo, hi = rank * N // world, (rank + 1) * N // world
    ys = []
    for li, (d_in, d_out, g) in enumerate(LINEARS):
        X, dY, bits, alpha = _inputs(li)
        bucket[li].copy_(torch.from_numpy(oracle.bwd_alpha(dY[lo:hi], X[lo:hi], bits, d_in, g)).float())
        ys.append(oracle.fwd(X[lo:hi], bits, alpha, d_in, g))
    allreduce_dalpha(bucket)
    gathered = [torch.zeros(hi - lo, LINEARS[0][1], dtype=torch.float64) for _ in range(world)]
    dist.all_gather(gathered, torch.from_numpy(ys[0]))
    if rank == 1:   # any rank holds the reduced gradients
        for li in range(len(LINEARS)):
            np.save(out + ".dalpha%d.npy" % li, bucket[li].numpy())
        np.save(out + ".y.npy", torch.cat(gathered).numpy())
    dist.destroy_process_group()


def test_token_sharding_and_bucket_allreduce(tmp_path):
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    out = str(tmp_path / "r")
    mp.spawn(_worker, args=(2, port, out), nprocs=2, join=True)
    for li, (d_in, d_out, g) in enumerate(LINEARS):
        X, dY, bits, alpha = _inputs(li)
        ref = oracle.bwd_alpha(dY, X, bits, d_in, g)
        got = np.load(out + ".dalpha%d.npy" % li)
        assert got.shape == ref.shape
        np.testing.assert_allclose(got, ref, rtol=2e-6, atol=2e-6 * np.abs(ref).max())
    X, dY, bits, alpha = _inputs(0)
    np.testing.assert_allclose(np.load(out + ".y.npy"), oracle.fwd(X, bits, alpha, LINEARS[0][0], LINEARS[0][2]),
                               rtol=1e-13)


def test_bucket_views_and_plane_segments():
    shapes = [(3, 4, 2), (2, 5, 1)]
    b = AlphaBucket(shapes, "cpu")
    assert b.flat.numel() == 24 + 10
    b[1].fill_(7.0)
    assert float(b.flat[:24].abs().sum()) == 0.0 and float(b.flat[24:].sum()) == 70.0
    # alpha_1 only: the first plane of every linear
    assert b.plane_segments(0b001) == [(0, 8), (24, 5)]
    assert b.plane_segments(0b110) == [(8, 8), (16, 8), (29, 5)]
