"""libtng: the data-parallel hot path of Trajectory Normalized Gradients
(arXiv 1901.08227) as hand-written sm_100a CUDA kernels behind a C ABI.

``tng`` is the ctypes binding (argument marshalling only; every step of the
path runs in the CUDA library).  ``workloads`` draws the seeded synthetic
inputs.  There is no CPU fallback: using the binding without the built shared
library, or a round without a CUDA device, raises.
"""
from . import tng  # noqa: F401
from .tng import (  # noqa: F401
    CODEC_QSGD4, CODEC_SIGN1, CODEC_TERN2, FUSE_AUTO, FUSE_HINDSIGHT, FUSE_LAST, FUSE_LSQ, FUSE_MEAN, NORM_DIFF,
    NORM_COMB, NORM_NONE, NORM_QUOT, SCALE_ABSMAX, SCALE_L2, Context, TngError)
