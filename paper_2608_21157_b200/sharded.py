"""One grid swept by several GPUs: slab decomposition along the slowest axis.

Each rank owns a contiguous slab of planes (rows for a 2D grid) plus R ghost
planes on either side.  Before every time step the ranks swap the R boundary
planes with their two neighbours (point-to-point ``torch.distributed`` sends:
NCCL between GPUs, gloo in the CPU tests), writing them into the receiver's own
ghost planes; the sweep itself is then the ordinary single-GPU ``stencil_apply``
on the local slab.  The outermost ghost planes of the first and last rank lie
outside the grid and are kept at zero (the zero boundary).  There is no
all-reduce or all-gather on the data path.

The paper runs every task on a single GPU and leaves multi-GPU execution open;
this module is the natural sharding of the sweep, kept outside the three-call C
ABI.  It has only been exercised with several ranks on CPU (gloo) and with one
rank on a GPU.

Zero boundary only: a periodic grid would also wrap the first rank's lower
ghost planes around to the last rank.
"""
from __future__ import annotations

from typing import Callable, Optional, Sequence, Tuple

import numpy as np

from . import binding

ZERO = binding.ZERO


def slab_range(n: int, world: int, rank: int) -> Tuple[int, int]:
    """Planes [z0, z1) of rank ``rank`` when ``n`` planes are dealt to ``world`` ranks
    as evenly as possible (the first ``n % world`` ranks get one more)."""
    if not (0 <= rank < world):
        raise ValueError("rank out of range")
    base, extra = divmod(int(n), int(world))
    z0 = rank * base + min(rank, extra)
    return z0, z0 + base + (1 if rank < extra else 0)


class ShardedSweep:
    """Iterated sweep of one grid across the ranks of a process group.

    ``local_apply(src, dst)`` performs ONE sweep of the local extended slab
    (``slab + 2R`` planes, zero boundary at its ends) from tensor ``src`` to tensor
    ``dst``; by default it is a ``binding.Plan`` on the current CUDA stream.  Tests
    pass their own callable to drive the exchange logic without a GPU.
    """

    def __init__(self, dims: Sequence[int], radius: int, shape: int, weights: np.ndarray,
                 boundary: int = ZERO, *, rank: int, world: int, dist=None, group=None,
                 local_apply: Optional[Callable] = None):
        if boundary != ZERO:
            raise ValueError("sharded sweeps support the zero boundary only")
        self.dims = tuple(int(d) for d in dims)
        self.R = int(radius)
        self.rank, self.world = int(rank), int(world)
        self.dist, self.group = dist, group
        self.z0, self.z1 = slab_range(self.dims[0], self.world, self.rank)
        self.nlocal = self.z1 - self.z0
        if self.world > 1 and self.nlocal < self.R:
            raise ValueError("every rank needs at least R planes of its own")
        if self.world > 1 and dist is None:
            raise ValueError("world > 1 needs torch.distributed")
        self.local_dims = (self.nlocal + 2 * self.R,) + self.dims[1:]
        self._plan = None
        if local_apply is None:
            self._plan = binding.Plan(self.local_dims, radius, shape, weights, boundary)
            import torch

            def local_apply(src, dst):
                self._plan.apply(src, dst, 1, torch.cuda.current_stream().cuda_stream)
        self._local_apply = local_apply

    # ---- layout helpers ---------------------------------------------------
    def scatter(self, global_field):
        """Local extended slab (a new tensor) cut from a global field tensor: own planes in
        the middle, ghost planes zero until the first exchange."""
        import torch
        R = self.R
        ext = torch.zeros(self.local_dims, dtype=global_field.dtype, device=global_field.device)
        ext[R:R + self.nlocal] = global_field[self.z0:self.z1]
        return ext

    def interior(self, ext):
        return ext[self.R:self.R + self.nlocal]

    # ---- halo exchange ----------------------------------------------------
    def exchange(self, ext) -> None:
        """Fill the ghost planes of ``ext`` from the neighbours' boundary planes (zeros where
        the neighbour would lie outside the grid)."""
        R, n = self.R, self.nlocal
        lo_ghost, hi_ghost = ext[:R], ext[R + n:]
        if self.rank == 0:
            lo_ghost.zero_()
        if self.rank == self.world - 1:
            hi_ghost.zero_()
        if self.world == 1:
            return
        d = self.dist
        ops = []
        send_lo = ext[R:2 * R].contiguous()              # my lowest planes -> lower neighbour's upper ghosts
        send_hi = ext[n:n + R].contiguous()              # my highest planes -> upper neighbour's lower ghosts
        recv_lo = lo_ghost.new_empty(lo_ghost.shape)
        recv_hi = hi_ghost.new_empty(hi_ghost.shape)
        if self.rank > 0:
            ops.append(d.P2POp(d.isend, send_lo, self.rank - 1, self.group))
            ops.append(d.P2POp(d.irecv, recv_lo, self.rank - 1, self.group))
        if self.rank < self.world - 1:
            ops.append(d.P2POp(d.isend, send_hi, self.rank + 1, self.group))
            ops.append(d.P2POp(d.irecv, recv_hi, self.rank + 1, self.group))
        for req in d.batch_isend_irecv(ops):
            req.wait()
        if self.rank > 0:
            lo_ghost.copy_(recv_lo)
        if self.rank < self.world - 1:
            hi_ghost.copy_(recv_hi)

    # ---- iteration ----------------------------------------------------------
    def apply(self, ext, steps: int = 1):
        """``steps`` sweeps of the distributed field; returns the extended slab holding the
        result in its interior (``ext`` is used as one of the two ping-pong buffers)."""
        if steps < 0:
            raise ValueError("steps must be >= 0")
        import torch
        cur, other = ext, torch.empty_like(ext)
        for _ in range(steps):
            self.exchange(cur)
            self._local_apply(cur, other)
            cur, other = other, cur
        return cur

    def close(self) -> None:
        if self._plan is not None:
            self._plan.destroy()
            self._plan = None
