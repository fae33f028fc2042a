"""B200 (sm_100a) stencil sweep: out[p] = sum_o w[o] * in[p+o] on 2D/3D fp32 grids.

``binding`` wraps the C ABI of the CUDA library (no CPU fallback);
``workloads`` holds the seeded synthetic problems; ``build`` compiles the
library in-tree.  Importing the package does not load the library; the first
call into ``binding`` does, and fails loudly if it was not built.
"""
from . import workloads  # noqa: F401
from . import binding  # noqa: F401
from .binding import Plan, StencilError  # noqa: F401
