"""One grid swept by several GPUs: slab decomposition along the slowest axis.

Each rank owns a contiguous slab of planes (rows for a 2D grid).  A rank with a
neighbour below (above) keeps ``G*R`` ghost planes on that side, where ``G`` is
the number of time steps between two halo exchanges (``halo_steps``).  A round
is: swap the ``G*R`` boundary planes with the neighbours (point-to-point
``torch.distributed`` sends: NCCL between GPUs, gloo in the CPU tests), then
advance the local extended slab by up to ``G`` steps with the ordinary
single-GPU ``stencil_apply``.  The ends of the extended slab see a zero
boundary that is wrong for them, and the error travels inwards by R planes per
step, so after ``G`` steps it has consumed the ghost planes and stopped at the
rank's own planes, which are exact.  ``G = 1`` exchanges before every step;
``G = 2`` sends half as many messages (the same bytes) and lets the local sweep
run its two-step fused passes.

With ``G = 1`` a round also overlaps the exchange with compute where the local
sweep can be restricted to a range of planes (``stencil_apply_planes``: tiled
kernels, zero boundary, 16-byte rows): the sends and receives are started, the planes that read no
ghost plane are swept meanwhile, and the R planes next to each neighbour follow
once the ghost planes have arrived.

Under the zero boundary the first rank has no ghost planes below and the last
none above: their slabs end at the grid's own boundary, which the local plan
imposes at every step.  Under the periodic boundary the ranks form a ring (the
first rank's lower neighbour is the last rank), every rank keeps ghost planes on
both sides, and the local plan is periodic: right along the two axes a rank holds
completely, and wrong only at the ends of the extended slab along the split
axis, where the ghost planes absorb it like the zero boundary's error.  There
is no all-reduce or all-gather on the data path.

The paper runs every task on a single GPU and leaves multi-GPU execution open;
this module is the natural sharding of the sweep, kept outside the three-call C
ABI.  It has been exercised with several ranks on CPU (gloo), with one rank on a
GPU, and with the slabs of several ranks swept one after the other on one GPU
(exchange by direct copies), never yet on several GPUs.
"""
from __future__ import annotations

from typing import Callable, Optional, Sequence, Tuple

import numpy as np

from . import binding

ZERO = binding.ZERO
PERIODIC = binding.PERIODIC


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

    ``local_apply(src, dst, steps)`` advances the local extended slab (own planes plus
    the ghost planes this rank has, zero boundary at its ends) by ``steps`` time steps
    from tensor ``src`` to tensor ``dst``; by default it is a ``binding.Plan`` on the
    current CUDA stream.  ``local_apply_planes(src, dst, z_begin, z_end)``, if given (or
    if the default plan supports it), does one sweep for the output planes
    [z_begin, z_end) of the extended slab only and enables the overlap of exchange and
    compute.  Tests pass their own callables to drive the exchange logic without a GPU.
    """

    def __init__(self, dims: Sequence[int], radius: int, shape: int, weights: np.ndarray,
                 boundary: int = ZERO, *, rank: int, world: int, dist=None, group=None,
                 halo_steps: int = 1, local_apply: Optional[Callable] = None,
                 local_apply_planes: Optional[Callable] = None, overlap: bool = True):
        if boundary not in (ZERO, PERIODIC):
            raise ValueError("boundary must be ZERO or PERIODIC")
        if halo_steps < 1:
            raise ValueError("halo_steps must be >= 1")
        self.dims = tuple(int(d) for d in dims)
        self.R = int(radius)
        self.G = int(halo_steps)
        self.rank, self.world = int(rank), int(world)
        self.dist, self.group = dist, group
        self.z0, self.z1 = slab_range(self.dims[0], self.world, self.rank)
        self.nlocal = self.z1 - self.z0
        self.depth = self.G * self.R                       # ghost planes per side that has a neighbour
        if self.world > 1 and self.nlocal < self.depth:
            raise ValueError("every rank needs at least halo_steps * R planes of its own")
        if self.world > 1 and dist is None:
            raise ValueError("world > 1 needs torch.distributed")
        # neighbours along the split axis: a chain under the zero boundary, a ring under the periodic one
        ring = boundary == PERIODIC and self.world > 1
        self.lower = (self.rank - 1) % self.world if (ring or self.rank > 0) else None
        self.upper = (self.rank + 1) % self.world if (ring or self.rank < self.world - 1) else None
        if self.world == 1:
            self.lower = self.upper = None
        self.lo = self.depth if self.lower is not None else 0       # ghost planes below / above the own planes
        self.hi = self.depth if self.upper is not None else 0
        self.local_dims = (self.lo + self.nlocal + self.hi,) + self.dims[1:]
        self._plan = None
        if local_apply is None:
            self._plan = binding.Plan(self.local_dims, radius, shape, weights, boundary)
            import torch

            def local_apply(src, dst, steps):
                self._plan.apply(src, dst, steps, torch.cuda.current_stream().cuda_stream)

            ranged = (self._plan.variant == "stream" and boundary == ZERO
                      and self.dims[-1] % (2 if self._plan.f64 else 4) == 0)
            if ranged and local_apply_planes is None:
                def local_apply_planes(src, dst, z_begin, z_end):
                    self._plan.apply_planes(src, dst, z_begin, z_end, torch.cuda.current_stream().cuda_stream)
        self._local_apply = local_apply
        self._local_apply_planes = local_apply_planes
        # overlap needs one step per exchange, a ranged sweep and own planes that read no ghost plane
        self.overlap = bool(overlap and self.G == 1 and self.world > 1 and local_apply_planes is not None
                            and self.nlocal > 2 * self.R)

    # ---- layout helpers ---------------------------------------------------
    def scatter(self, global_field):
        """Local extended slab (a new tensor) cut from a global field tensor: own planes in
        the middle, ghost planes zero until the first exchange."""
        import torch
        ext = torch.zeros(self.local_dims, dtype=global_field.dtype, device=global_field.device)
        ext[self.lo:self.lo + self.nlocal] = global_field[self.z0:self.z1]
        return ext

    def interior(self, ext):
        return ext[self.lo:self.lo + self.nlocal]

    # ---- halo exchange ----------------------------------------------------
    def start_exchange(self, ext):
        """Start the sends of the outermost own planes and the receives into the ghost planes
        of ``ext`` (slices along the slowest axis are contiguous, so both go straight from and
        to the slab).  Returns the pending requests."""
        if self.world == 1:
            return []
        d, D, n, lo = self.dist, self.depth, self.nlocal, self.lo
        # Messages travelling down the axis carry tag 1, those travelling up tag 0.  In a ring of two
        # ranks both neighbours are the same peer: the receives are listed in the order of that
        # peer's sends (its "down" arrives from above, its "up" from below) for backends that
        # match the messages of a pair by order instead of by tag.
        ops = []
        if self.lower is not None:                           # my lowest planes -> lower neighbour
            ops.append(d.P2POp(d.isend, ext[lo:lo + D], self.lower, self.group, 1))
        if self.upper is not None:                           # my highest planes -> upper neighbour
            ops.append(d.P2POp(d.isend, ext[lo + n - D:lo + n], self.upper, self.group, 0))
        if self.upper is not None:                           # upper ghost planes <- upper neighbour's lowest
            ops.append(d.P2POp(d.irecv, ext[lo + n:], self.upper, self.group, 1))
        if self.lower is not None:                           # lower ghost planes <- lower neighbour's highest
            ops.append(d.P2POp(d.irecv, ext[:lo], self.lower, self.group, 0))
        return d.batch_isend_irecv(ops)

    @staticmethod
    def finish_exchange(reqs) -> None:
        for req in reqs:
            req.wait()

    def exchange(self, ext) -> None:
        """Fill the ghost planes of ``ext`` with the neighbours' outermost own planes."""
        self.finish_exchange(self.start_exchange(ext))

    # ---- iteration ----------------------------------------------------------
    def apply(self, ext, steps: int = 1):
        """``steps`` sweeps of the distributed field; returns the extended slab holding the
        result in its interior (``ext`` is used as one of the two ping-pong buffers)."""
        if steps < 0:
            raise ValueError("steps must be >= 0")
        import torch
        cur, other = ext, torch.empty_like(ext)
        done = 0
        while done < steps:
            r = min(self.G, steps - done)
            if self.overlap:
                # own planes [lo + R, lo + n - R) read own planes only: sweep them while the ghost
                # planes travel, then the R planes next to each neighbour (an edge rank's outer
                # side has no ghosts: its planes belong to the first range)
                R, lo, n = self.R, self.lo, self.nlocal
                inner0 = lo + (R if self.lower is not None else 0)
                inner1 = lo + n - (R if self.upper is not None else 0)
                reqs = self.start_exchange(cur)
                self._local_apply_planes(cur, other, inner0, inner1)
                self.finish_exchange(reqs)
                if inner0 > lo:
                    self._local_apply_planes(cur, other, lo, inner0)
                if inner1 < lo + n:
                    self._local_apply_planes(cur, other, inner1, lo + n)
            else:
                self.exchange(cur)
                self._local_apply(cur, other, r)
            cur, other = other, cur
            done += r
        return cur

    def close(self) -> None:
        if self._plan is not None:
            self._plan.destroy()
            self._plan = None
