"""Small single-kernel workloads for profiling (`python -m paper_2210_03858_b200.profile_cases CASE`).

Each case sets up one layer with synthetic data, calls one entry point a few times and exits, so
that a profiler can capture one or two launches of one kernel in a minute:

    fwd | dx | dalpha   one GPT-2-XL FFN linear (1600 -> 6400, q = 4, g = 128), 4096 tokens,
                        planes prepared once, bf16 outputs: three calls
    decode [q] [n]      OPT-6.7B att_qkv (4096 -> 12288, g = 128): eight random packs, three
                        rounds of bcq_linear_decode_packed over them (default q = 4, n = 1)
    quantize [alt]      greedy (alt = 0, five 6400 x 1600 matrices) or greedy + alt alternating
                        rounds (five 5120 x 5120 matrices), q = 4, g = 128
"""
import sys

import torch

import paper_2210_03858_b200 as bcq


def _linear(which):
    dev = torch.device("cuda", 0)
    n, q, g, d_in, d_out = 4096, 4, 128, 1600, 6400
    gen = torch.Generator(device=dev)
    gen.manual_seed(1)
    W = torch.randn((d_out, d_in), generator=gen, device=dev) * 0.02
    bits, alpha, _ = bcq.quantize(W, q, g)
    X = torch.randn((n, d_in), generator=gen, device=dev).bfloat16()
    dY = torch.randn((n, d_out), generator=gen, device=dev).bfloat16()
    pf = bcq.prepare_planes(bcq.OP_FWD, bits, d_in, g)
    px = bcq.prepare_planes(bcq.OP_BWD_X, bits, d_in, g)
    Y = torch.empty((n, d_out), device=dev, dtype=torch.bfloat16)
    dX = torch.empty((n, d_in), device=dev, dtype=torch.bfloat16)
    dA = torch.zeros_like(alpha)
    for _ in range(3):
        if which == "fwd":
            bcq.linear_fwd(X, pf, alpha, d_in, g, out=Y)
        elif which == "dx":
            bcq.linear_bwd_x(dY, px, alpha, d_in, g, out=dX)
        else:
            bcq.linear_bwd_alpha(dY, X, bits, d_in, g, out=dA)


def _decode(q, n):
    dev = torch.device("cuda", 0)
    g, d_out, d_in = 128, 12288, 4096
    gen = torch.Generator(device=dev)
    gen.manual_seed(1)
    packs = []
    for _ in range(8):
        bits = torch.randint(-2 ** 31, 2 ** 31 - 1, (q, d_out, bcq.pitch_words(d_in)), generator=gen,
                             dtype=torch.int32, device=dev)
        alpha = torch.rand((q, d_out, d_in // g), generator=gen, device=dev) * 0.02
        packs.append(bcq.decode_pack(bits, alpha, d_in, g))
    X = torch.randn((n, d_in), generator=gen, device=dev).bfloat16()
    Y = torch.empty((n, d_out), device=dev)
    ws = torch.empty(max(16, bcq.workspace_bytes(bcq.OP_DECODE_PACKED, d_out, d_in, q, g, n)), dtype=torch.uint8,
                     device=dev)
    for _ in range(3):
        for pack in packs:
            bcq.linear_decode_packed(X, pack, d_out, d_in, q, g, out=Y, ws=ws)


def _quantize(alt):
    dev = torch.device("cuda", 0)
    gen = torch.Generator(device=dev)
    gen.manual_seed(1)
    shape = (6400, 1600) if alt == 0 else (5120, 5120)
    Ws = [torch.randn(shape, generator=gen, device=dev) * 0.02 for _ in range(5)]
    for W in Ws:
        bcq.quantize(W, 4, 128, alt)


def main(argv):
    case = argv[1] if len(argv) > 1 else "fwd"
    if case in ("fwd", "dx", "dalpha"):
        _linear(case)
    elif case == "decode":
        _decode(int(argv[2]) if len(argv) > 2 else 4, int(argv[3]) if len(argv) > 3 else 1)
    elif case == "quantize":
        _quantize(int(argv[2]) if len(argv) > 2 else 0)
    else:
        raise SystemExit(__doc__)
    torch.cuda.synchronize()
    assert bcq.device_timeout_flag() == 0
    print("ok")


if __name__ == "__main__":
    main(sys.argv)
