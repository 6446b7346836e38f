"""Layer-wise stochastic quantization + QODA update on one B200 (sm_100a), behind a C ABI.

`binding` marshals torch tensors into the C entry points of liblq.so (include/lq.h);
`workloads` draws the seeded synthetic gradient sets; `build` compiles the library in-tree.
"""
from .binding import (HIST_STRIDE, NUM_BINS, STATUS_NONFINITE, STATUS_ZERO_NORM, STEP_AUTO, LqError, Plan,
                      load_library, lq_code_build, lq_code_universal, lq_vector_norm_static)

__all__ = ["Plan", "LqError", "load_library", "lq_vector_norm_static", "lq_code_build", "lq_code_universal", "NUM_BINS", "HIST_STRIDE", "STATUS_ZERO_NORM",
           "STATUS_NONFINITE", "STEP_AUTO"]
