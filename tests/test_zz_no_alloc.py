"""bcq_linear_decode_noalloc: the decode entry point for callers that cannot allocate.

A caller that may not call cudaMalloc (it runs where the allocator is off limits, or it was only
handed its inputs and outputs) cannot give bcq_linear_decode a workspace.  The no-alloc entry
point keeps the split-K partial sums in a fixed array inside the library instead.  This file
checks, through the C ABI, that it gives the same result as bcq_linear_decode -- twice in a row,
since the array is shared by all calls and keeps the previous call's contents -- and that a shape
whose partial sums do not fit is refused before anything is launched.

The file name sorts last on purpose: a run that stops at the first failure has then already run
every other test.
"""
import ctypes as C

import numpy as np
import pytest

import oracle
import paper_2210_03858_b200 as bcq
from paper_2210_03858_b200 import build as bcq_build
from paper_2210_03858_b200 import synth

TOL = 2e-3


@pytest.fixture(scope="module", autouse=True)
def _built():
    bcq_build.build_library()


@pytest.mark.gpu
def test_noalloc_decode_matches_decode_twice_in_a_row():
    import torch
    cases = [(4, 4096, 1536, 3, 128), (16, 2048, 520, 4, 128), (1, 1024, 256, 3, 1024)]
    for n, d_in, d_out, q, g in cases:
        key = (300, n, d_out)
        W = synth.weights(d_out, d_in, key)
        X = synth.activations(n, d_in, key, synth.ROLE_X)
        bits, alpha, _, _ = oracle.quantize(W, q, g)
        ref = oracle.fwd(X, bits, alpha, d_in, g)
        Xd = torch.from_numpy(X.view(np.int16)).cuda().view(torch.bfloat16)
        bd = torch.from_numpy(bits.view(np.int32)).cuda()
        ad = torch.from_numpy(alpha).cuda()
        assert bcq.workspace_bytes(bcq.OP_DECODE, d_out, d_in, q, g, n) <= bcq.NOALLOC_SCRATCH_BYTES
        expect = bcq.linear_decode(Xd, bd, ad, d_in, g)
        out1 = torch.full((n, d_out), float("nan"), device="cuda")
        out2 = torch.full((n, d_out), float("nan"), device="cuda")
        bcq.linear_decode_noalloc(Xd, bd, ad, d_in, g, out=out1)
        bcq.linear_decode_noalloc(Xd, bd, ad, d_in, g, out=out2)   # scratch still holds call 1's sums
        torch.cuda.synchronize()
        scale = float(expect.abs().max())
        for out in (out1, out2):
            assert float((out - expect).abs().max()) <= TOL * scale
            assert float(np.abs(out.cpu().numpy().astype(np.float64) - ref).max() / np.abs(ref).max()) <= TOL
    assert bcq.device_timeout_flag() == 0


def test_noalloc_decode_refuses_what_does_not_fit():
    # the arguments are checked on the host before the scratch symbol is resolved or anything is
    # launched, so the (16-byte aligned, never dereferenced) fake pointers are safe to pass
    lib = bcq.lib()
    p, null = C.c_void_p(256), C.c_void_p(0)
    d_out, d_in, q, g, n = 12288, 4096, 4, 128, 16       # 3 splits x 16 x 12288 floats > 2 MiB
    assert bcq.workspace_bytes(bcq.OP_DECODE, d_out, d_in, q, g, n) > bcq.NOALLOC_SCRATCH_BYTES
    assert lib.bcq_linear_decode_noalloc(d_out, d_in, q, g, n, p, d_in, p, p, null, p, d_out, 0, null) == -5
    assert lib.bcq_linear_decode_noalloc(64, 256, 2, 64, 17, p, 256, p, p, null, p, 64, 0, null) == -2
