"""CPU oracle of the int8 Actor policy-inference path (TEST INFRASTRUCTURE).

Only the tests, the smoke check and the benchmark's CPU-baseline leg may
import this package.  It shares no code with the CUDA library and never
imports it.  ``accerl_oracle.c`` holds the arithmetic (naive loops), this
package compiles it with gcc, loads it through ctypes and composes the
per-layer calls into a whole forward pass (``forward``), a post-training
quantiser and calibrator (``ptq``); ``corrector`` wraps the V-trace definition.
"""
from .clib import build, lib  # noqa: F401
from .corrector import vtrace  # noqa: F401
from .net import entropy, forward, forward_mixed, ingest, kl, layer_acc, layer_float  # noqa: F401
from .ptq import calibrate, prune_2_4, quantise_weights  # noqa: F401
