"""B200-native softmax / log-softmax / LayerNorm / RMSNorm over the last axis, and over a
non-last axis of x[outer, reduce, inner] (``rowop_axis``).

The operators live in ``libakg.so`` (hand-written sm_100a CUDA behind the C ABI of
``include/akg.h``); ``binding`` marshals torch tensors into it and ``workloads``
generates the seeded benchmark inputs.  There is no CPU implementation here.
"""
from . import workloads  # noqa: F401
from .binding import (AkgError, Mask, act_mul, add_norm, argmax, argmin, colnorm, cumprod, cumsum, device_status, last_error, last_kernel, layernorm,  # noqa: F401
                      lib, log_softmax, make_mask, rmsnorm, rowop_axis, set_tuning, set_variant, softmax, softmax_scaled,
                      status_string)
