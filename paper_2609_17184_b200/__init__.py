"""B200-native LoopSpec decode path: a thin ctypes binding over the C-ABI library `libloopspec.so`.

Every step of the path (batched recurrence, readouts, drafting, gate, cascade verification, KV rollback,
scheduling) runs in the library's CUDA kernels; this package only marshals arguments.  PyTorch is used for
device memory and streams.  There is no CPU fallback: importing fails if the library cannot be loaded.
"""
from .binding import (LoopSpec, LoopSpecError, fit_envelope, lib, linear, linear_scratch_bytes, linear_static, linear_tc, time_linear_tc, max_branches,  # noqa: F401
                      pick_depths,
                      upload_weights, EXPORTS)
