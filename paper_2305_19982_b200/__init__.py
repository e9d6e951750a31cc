"""B200-native AdamA (arXiv 2305.19982): thin ctypes binding over libadama.so.

Every step of the method (Algorithm 2: fold, fused weight-gradient fold, update)
runs in the CUDA kernels behind the C ABI declared in include/adama.h; this
module only marshals arguments (device pointers of torch tensors, the current
stream).  There is no CPU fallback: importing works without a GPU, but creating
an ``AdamA`` context raises if the library or a sm_100 device is missing.
"""
from .binding import (AdamA, AdamAError, TensorList, Status, library_path, load_library, host_constants,
                      linear_wgrad_fold_noalloc, debug_setup_state, EXPORTED_SYMBOLS)

__all__ = ["AdamA", "AdamAError", "TensorList", "Status", "library_path", "load_library", "host_constants",
           "linear_wgrad_fold_noalloc", "debug_setup_state", "EXPORTED_SYMBOLS"]
