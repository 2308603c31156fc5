"""Host-side checks of the C-ABI library that need no GPU: it loads, exports every symbol the
header declares, its size helpers reproduce the paper's storage accounting, and argument
validation rejects bad calls before anything touches the device."""
import ctypes as C
import os
import re

import pytest

import paper_2210_03858_b200 as bcq
from paper_2210_03858_b200 import build as bcq_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


@pytest.fixture(scope="module", autouse=True)
def _built():
    bcq_build.build_library()


def test_exports_every_declared_symbol():
    header = open(os.path.join(ROOT, "include", "bcq.h")).read()
    declared = set(re.findall(r"\b(bcq_[a-z_0-9]+)\s*\(", header))
    assert declared == set(bcq.SYMBOLS)
    lib = bcq.lib()
    for name in declared:
        assert hasattr(lib, name), name


def test_size_helpers_and_table1():
    assert bcq.pitch_words(1) == 4 and bcq.pitch_words(128) == 4 and bcq.pitch_words(129) == 8
    assert bcq.pitch_words(1600) == 52
    assert bcq.num_groups(1600, 128) == 13 and bcq.num_groups(1024, 1024) == 1
    assert bcq.bits_bytes(1024, 1024, 3) == 393216
    assert bcq.alpha_count(1024, 1024, 3, 1024) == 3072
    with open(os.path.join(GOLDEN, "table1_sizes.txt")) as f:
        for line in f:
            line = line.split("#")[0].split()
            if not line:
                continue
            _, d_out, d_in, g, *cells = line
            for q, cell in zip((1, 2, 3), cells):
                if cell != "-":
                    mb = bcq.payload_bits(int(d_out), int(d_in), q, int(g)) / 8e6
                    assert abs(mb - float(cell)) <= 0.0051


def test_argument_validation_happens_before_any_launch():
    lib = bcq.lib()
    p = C.c_void_p(256)   # never dereferenced: every call below must fail validation first
    null = C.c_void_p(0)
    # shape / support
    assert lib.bcq_quantize(0, 8, 1, 8, p, 8, 0, p, p, null, null) == -2
    assert lib.bcq_quantize(4, 64, 9, 64, p, 64, 0, p, p, null, null) == -4
    assert lib.bcq_quantize(4, 64, 2, 48, p, 64, 0, p, p, null, null) == -4      # g not /32, not d_in
    assert lib.bcq_quantize(4, 64, 2, 128, p, 64, 0, p, p, null, null) == -2     # g > d_in
    assert lib.bcq_quantize(4, 64, 2, 64, null, 64, 0, p, p, null, null) == -1
    assert lib.bcq_quantize(4, 64, 2, 64, p, 32, 0, p, p, null, null) == -2      # ldw < d_in
    # forward: NULLs, pitch, alignment, decode token limit
    args = lambda X, ldx, n: (8, 64, 2, 64, n, X, ldx, p, p, null, p, 8, 0, null, 0, null)
    assert lib.bcq_linear_fwd(*args(null, 64, 4)) == -1
    assert lib.bcq_linear_fwd(*args(p, 60, 4)) == -2
    assert lib.bcq_linear_fwd(*args(p, 68, 4)) == -3
    assert lib.bcq_linear_fwd(*args(C.c_void_p(258), 64, 4)) == -3
    assert lib.bcq_linear_decode(*args(p, 64, 17)) == -2
    assert lib.bcq_linear_bwd_x(8, 64, 2, 64, 0, p, 8, p, p, p, 64, 0, null, 0, null) == -2
    assert lib.bcq_linear_bwd_alpha(8, 64, 2, 64, 4, p, 8, p, 64, p, 3, 1.0, 0, null, null, 0, null) == -1
    assert bcq.status_string(-4).startswith("shape not covered")
    assert bcq.workspace_bytes(bcq.OP_QUANTIZE, 8, 64, 2, 64, 0) == 0


def test_workspace_sizes_are_consistent():
    # decode splits K over CTAs and needs room for partial sums; prefill holds its fp16 activations
    assert bcq.workspace_bytes(bcq.OP_DECODE, 4096, 16384, 4, 128, 16) > 0
    assert bcq.workspace_bytes(bcq.OP_FWD, 3072, 1024, 3, 1024, 2048) >= 2048 * 1024 * 2
    assert bcq.workspace_bytes(bcq.OP_BWD_ALPHA, 1024, 1024, 3, 1024, 512) > 0
