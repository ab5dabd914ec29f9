"""FiCoCo token reduction (filter, correlate, compress) as sm_100a CUDA kernels behind a C ABI.

``binding`` wraps ``libficoco.so`` (built in-tree by ``build``); ``synth`` generates seeded
synthetic workloads; ``packing`` lays them out for the ABI.  There is no CPU fallback: using
the binding without the built library raises.
"""
from . import synth  # noqa: F401
from .binding import (Context, FicocoError, ficoco_default_params, load_library, make_params,  # noqa: F401
                      to_numpy, to_torch)
from .packing import pack_l, pack_v  # noqa: F401
