"""Band-wise local-operator chains on NVIDIA B200: thin Python binding of the C-ABI library.

Everything numerical happens in ``liblop_b200.so`` (hand-written sm_100a kernels); this
package only marshals arguments.  There is no CPU path: importing :mod:`.binding` fails
loudly when the library cannot be loaded.
"""
from .binding import (  # noqa: F401
    LIB_PATH, LopError, LopLayer, LopRange, LopTiming, Plan, lib, run_chain_banded, run_chain_pipelined,
    LOP_F32, LOP_BF16, LOP_CONV2D, LOP_MAXPOOL2D, LOP_LINEAR, LOP_ACT_NONE, LOP_ACT_RELU, LOP_ACT_SILU,
    LOP_RES_NONE, LOP_RES_PRE_ACT, LOP_RES_POST_ACT, LOP_INPUT, LOP_NO_RESIDUAL,
    LOP_FLAG_REUSE_HALO, LOP_FLAG_TIME_LAYERS, LOP_FLAG_FORCE_SIMT, LOP_FLAG_PER_LAYER, LOP_FLAG_COPY_ENGINE, LOP_FLAG_DEBUG_BOUNDS, LOP_STATIC_SCRATCH_BYTES, EXPORTS,
)
