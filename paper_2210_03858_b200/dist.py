"""Data-parallel plumbing of the scale gradients.

The path shards over tokens: every rank runs forward, dX and dalpha on its own tokens with the
same (B, alpha).  Only dalpha (Eq. 4) is a sum over tokens, so one all-reduce per step makes it
the gradient of the whole batch.  The gradients of all linears live in ONE flat fp32 buffer
(`AlphaBucket`): every linear's [q][d_out][G] tensor is a view into it, the kernels write through
the views, and the exchange is a single collective on the flat buffer -- no gather, no copy back.

Nothing here computes anything; torch.distributed does the exchange (NCCL on GPUs, gloo in the
CPU tests).
"""
from __future__ import annotations

from typing import Iterable, List, Sequence, Tuple


class AlphaBucket:
    """One flat fp32 buffer holding a [q][d_out][G] tensor per linear, in the given order."""

    def __init__(self, shapes: Sequence[Tuple[int, int, int]], device):
        import torch
        self.shapes = [tuple(int(x) for x in s) for s in shapes]
        self.offsets = [0]
        for q, d_out, G in self.shapes:
            self.offsets.append(self.offsets[-1] + q * d_out * G)
        self.flat = torch.zeros(self.offsets[-1], dtype=torch.float32, device=device)
        self.views: List = [self.flat[self.offsets[i]:self.offsets[i + 1]].view(*s)
                            for i, s in enumerate(self.shapes)]

    def __len__(self):
        return len(self.views)

    def __getitem__(self, i):
        return self.views[i]

    def plane_segments(self, plane_mask: int) -> List[Tuple[int, int]]:
        """(offset, count) of the elements of the planes in plane_mask, per linear: planes are the
        outermost index, so each selected plane of a linear is one contiguous run."""
        segs = []
        for i, (q, d_out, G) in enumerate(self.shapes):
            for pl in range(q):
                if (plane_mask >> pl) & 1:
                    segs.append((self.offsets[i] + pl * d_out * G, d_out * G))
        return segs


def allreduce_dalpha(bucket: AlphaBucket, group=None, average: bool = False):
    """Sums the scale gradients of all linears over the ranks of `group` (one collective on the flat
    buffer; the per-linear views see the result).  With average=True divides by the world size,
    the usual data-parallel mean over the global batch."""
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()):
        return bucket.flat
    dist.all_reduce(bucket.flat, op=dist.ReduceOp.SUM, group=group)
    if average:
        bucket.flat.div_(dist.get_world_size(group))
    return bucket.flat
