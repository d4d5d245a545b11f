"""One large picture over several GPUs: rows are sharded, every rank convolves its own strip.

The regression networks of the paper (VDSR, Table 4; the VRCNN in-loop filter on 2560 x 1600
frames, Table 6) are stride-1 stacks: an output row depends on input rows at most ``halo`` away,
``halo`` being the sum over the layers of the padding of the widest filter at that depth (6 rows
for the VRCNN shape, 20 for the 20-layer VDSR).  So a rank that owns output rows [o0, o1) takes
input rows [o0 - halo, o1 + halo) clipped to the picture, runs the whole network on that strip
(the rows near an artificial cut come out wrong, the rows near the picture's own border see the
same zero padding as the unsplit run) and keeps exactly its owned rows: they are bit-identical
to the unsplit result, the strips need no exchange between layers, and the only communication is
the final gather of the owned rows.

Host logic only; the layers run in the CUDA library through ``Network``.
"""
from dataclasses import dataclass
from typing import Callable, List

import numpy as np

from workloads.networks import Conv, Net


@dataclass
class Strip:
    rank: int
    own0: int        # first owned output row (of the whole picture)
    own1: int        # one past the last owned output row
    in0: int         # first input row of the strip
    in1: int         # one past the last input row of the strip

    @property
    def rows(self) -> int:
        return self.in1 - self.in0

    @property
    def keep(self) -> slice:
        """The owned rows, as a slice of the strip's own output."""
        return slice(self.own0 - self.in0, self.own1 - self.in0)


def halo_rows(net: Net) -> int:
    """Rows of context an output row needs on each side: every layer adds the padding of its
    widest branch (layers that write the same tensor are sibling branches of one depth).  Only
    stride-1, size-preserving stacks shard this way."""
    per_depth = {}
    for op in net.ops:
        if not isinstance(op, Conv) or op.stride != 1 or 2 * op.pad != op.k - 1:
            raise ValueError("row sharding needs a stack of stride-1, size-preserving convolutions (%s is not)" % getattr(op, "name", op))
        per_depth[op.dst] = max(per_depth.get(op.dst, 0), op.pad)
    return sum(per_depth.values())


def partition(h: int, parts: int, halo: int) -> List[Strip]:
    """Strips of a picture of h rows for `parts` ranks: owned rows split as evenly as possible,
    contiguous, in rank order; input rows = owned rows widened by the halo and clipped."""
    if h < 1 or parts < 1 or halo < 0:
        raise ValueError("partition: need h >= 1, parts >= 1, halo >= 0")
    base, extra = divmod(h, parts)
    strips, row = [], 0
    for r in range(parts):
        count = base + (1 if r < extra else 0)
        strips.append(Strip(r, row, row + count, max(0, row - halo), min(h, row + count + halo)))
        row += count
    return strips


def run_strip(picture: np.ndarray, strip: Strip, forward: Callable[[np.ndarray], np.ndarray]) -> np.ndarray:
    """The owned rows of one strip: `forward` maps an input strip [1][rows][w][c] to the network's
    output for it (same height).  A rank that owns no row returns an empty array."""
    if strip.own1 == strip.own0:
        return np.zeros((picture.shape[0], 0) + picture.shape[2:], dtype=np.uint8)
    out = forward(np.ascontiguousarray(picture[:, strip.in0:strip.in1]))
    assert out.shape[1] == strip.rows, "the network must preserve the picture's height"
    return np.ascontiguousarray(out[:, strip.keep])


def stitch(parts: List[np.ndarray]) -> np.ndarray:
    """The whole picture from the ranks' owned rows, in rank order."""
    return np.concatenate(parts, axis=1)


def gather_rows(owned: np.ndarray, strips: List[Strip], rank: int):
    """All ranks' owned rows at rank 0 (torch.distributed gather of uint8 tensors padded to the
    tallest strip); returns the stitched picture on rank 0, None elsewhere.  Without a process
    group (one rank) the owned rows are the picture."""
    import torch
    import torch.distributed as dist
    if not dist.is_initialized():
        return owned
    tallest = max(s.own1 - s.own0 for s in strips)
    n, _, w, c = owned.shape
    buf = torch.zeros((n, tallest, w, c), dtype=torch.uint8)
    buf[:, :owned.shape[1]] = torch.from_numpy(owned)
    if dist.get_backend() == "nccl":
        buf = buf.cuda()
    if rank == 0:
        got = [torch.empty_like(buf) for _ in strips]
        dist.gather(buf, got, dst=0)
        return stitch([g.cpu().numpy()[:, :s.own1 - s.own0] for g, s in zip(got, strips)])
    dist.gather(buf, None, dst=0)
    return None
