"""Seeded synthetic inputs shaped like the paper's workloads.

This module only draws random numbers and converts number formats; it contains none of the
BCQ arithmetic.  Both the CUDA tests/benchmark and the CPU oracle are fed from here so that
they see the same bytes.

The paper fine-tunes GPT-2 medium/large and OPT-1.3B (Table 1 gives the four quantized
linears of a GPT-2 medium block for hidden size h = 1024: ATT_qkv (3h,h), ATT_output (h,h),
FFN_h_4h (4h,h), FFN_4h_h (h,4h)).  Its datasets and checkpoints are not used here; the
tensors below take those layer shapes and stand in for them:

  * weights  W ~ N(0, sigma = 0.02) fp32 (the GPT-2 initialiser scale), optionally with a
    fraction ``outlier_frac`` of entries multiplied by ``outlier_mult``;
  * activations X and output gradients dY ~ N(0, 1), rounded to bf16 (round to nearest even)
    and handed around as uint16 bit patterns.

Every tensor is drawn from ``numpy.random.Generator(PCG64(SeedSequence(key)))`` with
``key = (BASE_SEED, workload id, layer, linear, role)``.
"""
from __future__ import annotations

import numpy as np

BASE_SEED = 221003858
ROLE_W, ROLE_X, ROLE_DY, ROLE_BIAS, ROLE_IDX = 0, 1, 2, 3, 4


def rng_for(workload: int, layer: int, linear: int, role: int) -> np.random.Generator:
    ss = np.random.SeedSequence([BASE_SEED, int(workload), int(layer), int(linear), int(role)])
    return np.random.Generator(np.random.PCG64(ss))


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round fp32 to bf16 (nearest even); returns the uint16 bit patterns."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32).astype(np.uint64)
    rounded = (u + 0x7FFF + ((u >> 16) & 1)) >> 16
    return rounded.astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << 16).view(np.float32)


def weights(d_out: int, d_in: int, key, sigma: float = 0.02, outlier_frac: float = 0.0,
            outlier_mult: float = 20.0) -> np.ndarray:
    """W[d_out][d_in] fp32 ~ N(0, sigma); each entry independently an outlier."""
    rng = rng_for(*key, ROLE_W)
    W = rng.standard_normal((d_out, d_in), dtype=np.float32) * np.float32(sigma)
    if outlier_frac > 0.0:
        mask = rng.random((d_out, d_in), dtype=np.float32) < np.float32(outlier_frac)
        W = np.where(mask, W * np.float32(outlier_mult), W).astype(np.float32)
    return W


def activations(n: int, d: int, key, role: int = ROLE_X) -> np.ndarray:
    """[n][d] ~ N(0,1) rounded to bf16, as uint16 bit patterns."""
    rng = rng_for(*key, role)
    return f32_to_bf16_bits(rng.standard_normal((n, d), dtype=np.float32))


def bias(d_out: int, key) -> np.ndarray:
    rng = rng_for(*key, ROLE_BIAS)
    return (rng.standard_normal(d_out, dtype=np.float32) * np.float32(0.02)).astype(np.float32)


def sample_indices(count: int, bounds, key) -> list:
    """``count`` index tuples drawn uniformly from the box ``bounds`` (one array per axis)."""
    rng = rng_for(*key, ROLE_IDX)
    return [rng.integers(0, b, size=count, dtype=np.int64) for b in bounds]


def stratified_indices(rows: int, cols: int, tile_rows: int, tile_cols: int, per_tile: int, key) -> list:
    """``per_tile`` (row, column) positions drawn uniformly inside every tile_rows x tile_cols tile
    of a rows x cols matrix (edge tiles are clipped), so that no tile of an output is left
    without a sampled value.  Returns [row indices, column indices]."""
    rng = rng_for(*key, ROLE_IDX)
    rr, cc = [], []
    for r0 in range(0, rows, tile_rows):
        rh = min(tile_rows, rows - r0)
        for c0 in range(0, cols, tile_cols):
            cw = min(tile_cols, cols - c0)
            rr.append(r0 + rng.integers(0, rh, size=per_tile, dtype=np.int64))
            cc.append(c0 + rng.integers(0, cw, size=per_tile, dtype=np.int64))
    return [np.concatenate(rr), np.concatenate(cc)]


def line_indices(rows: int, cols: int, row_lines, col_lines) -> list:
    """Every position of the given whole rows and whole columns of a rows x cols matrix."""
    rr = [np.repeat(np.asarray(row_lines, dtype=np.int64), cols)]
    cc = [np.tile(np.arange(cols, dtype=np.int64), len(row_lines))]
    rr.append(np.tile(np.arange(rows, dtype=np.int64), len(col_lines)))
    cc.append(np.repeat(np.asarray(col_lines, dtype=np.int64), rows))
    return [np.concatenate(rr), np.concatenate(cc)]


# ----------------------------------------------------------------------------------------
# Workloads: (name, d_in, d_out) of the quantized linears of one Transformer block.
# ----------------------------------------------------------------------------------------

def block_linears(hidden: int, ffn: int):
    return [("att_qkv", hidden, 3 * hidden), ("att_out", hidden, hidden),
            ("ffn_h_4h", hidden, ffn), ("ffn_4h_h", ffn, hidden)]


WORKLOADS = {
    # id: dict(description of the synthetic stand-in)
    0: dict(name="single-1024", linears=[("lin", 1024, 1024)], layers=1, n=512, q=(3,), g="row",
            alt_iters=0),
    1: dict(name="gpt2-medium-block", linears=block_linears(1024, 4096), layers=24, n=2048,
            q=(3,), g="row", alt_iters=0),
    2: dict(name="gpt2-xl-block", linears=block_linears(1600, 6400), layers=48, n=4096, q=(4,),
            g=128, alt_iters=0),
    3: dict(name="opt-6.7b-decode", linears=[("att_qkv", 4096, 12288), ("ffn_h_4h", 4096, 16384),
                                             ("ffn_4h_h", 16384, 4096), ("att_out", 4096, 4096)],
            layers=32, n=(1, 4, 16), q=(3, 4), g=128, alt_iters=0),
    4: dict(name="opt-13b-ptq-prefill", linears=block_linears(5120, 20480), layers=40, n=2048,
            q=(2, 3, 4), g=128, alt_iters=5, outlier_frac=1e-3, outlier_mult=20.0),
}


def group_size(workload: dict, d_in: int) -> int:
    return d_in if workload["g"] == "row" else int(workload["g"])
