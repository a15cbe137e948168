"""B200-native int8 Actor policy inference (AcceRL's data-collection hot path).

The work happens in ``libaccerl.so`` (hand-written CUDA for sm_100a behind the C
ABI of ``include/accerl.h``).  This package only marshals arguments: torch is
used for device memory and streams, nothing is computed in Python, and there
is no CPU fallback -- importing :class:`Policy` without the built library
raises.
"""
from .binding import (AccerlError, Policy, act_mixed, kl, library, library_path, tc_probe_i8,  # noqa: F401
                      vtrace, FLAG_FORCE_GENERIC, FLAG_KEEP_ACTIVATIONS, FLAG_TAP_FUSED,
                      FLAG_VALUE_HEAD, FLAG_TEST_NO_FASTDIV, FLAG_TEST_NO_AFFINE)
