"""The data-parallel shape of the path, on CPU with two gloo ranks: tokens are split over ranks,
every rank computes the scale gradient (Eq. 4) of its own tokens, and one all-reduce (sum) gives
the gradient of the whole batch.  Forward and dX need no exchange: each rank's rows are its own.
Uses the oracle for the per-rank arithmetic; what is tested is the sharding and the reduction that
bench.py performs for N > 1."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import oracle
from paper_2210_03858_b200 import synth

N, D_IN, D_OUT, Q, G = 24, 96, 40, 3, 32


def _inputs():
    key = (50, 0, 0)
    W = synth.weights(D_OUT, D_IN, key)
    X = synth.activations(N, D_IN, key, synth.ROLE_X)
    dY = synth.activations(N, D_OUT, key, synth.ROLE_DY)
    bits, alpha, _, _ = oracle.quantize(W, Q, G)
    return X, dY, bits, alpha


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    X, dY, bits, alpha = _inputs()
    lo, hi = rank * N // world, (rank + 1) * N // world
    dA = torch.from_numpy(oracle.bwd_alpha(dY[lo:hi], X[lo:hi], bits, D_IN, G))
    dist.all_reduce(dA)
    Y = oracle.fwd(X[lo:hi], bits, alpha, D_IN, G)
    gathered = [torch.zeros(hi - lo, D_OUT, dtype=torch.float64) for _ in range(world)]
    dist.all_gather(gathered, torch.from_numpy(Y))
    if rank == 0:
        np.save(out + ".dalpha.npy", dA.numpy())
        np.save(out + ".y.npy", torch.cat(gathered).numpy())
    dist.destroy_process_group()


def test_token_sharding_and_dalpha_allreduce(tmp_path):
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    out = str(tmp_path / "r0")
    mp.spawn(_worker, args=(2, port, out), nprocs=2, join=True)
    X, dY, bits, alpha = _inputs()
    np.testing.assert_allclose(np.load(out + ".dalpha.npy"), oracle.bwd_alpha(dY, X, bits, D_IN, G),
                               rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(np.load(out + ".y.npy"), oracle.fwd(X, bits, alpha, D_IN, G), rtol=1e-13)
