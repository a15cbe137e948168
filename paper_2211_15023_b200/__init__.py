"""B200-native int8 Actor policy inference (AcceRL's data-collection hot path).

The work happens in ``libaccerl.so`` (hand-written CUDA for sm_100a behind the C
ABI of ``include/accerl.h``).  This package only marshals arguments: torch is
used for device memory and streams, nothing is computed in Python, and there
is no CPU fallback -- importing :class:`Policy` without the built library
raises.
"""
from .binding import (AccerlError, Policy, library, library_path, FLAG_FORCE_GENERIC,  # noqa: F401
                      FLAG_KEEP_ACTIVATIONS, FLAG_TAP_FUSED)
