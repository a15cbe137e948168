"""Compile ``accerl_oracle.c`` with gcc and load it (TEST INFRASTRUCTURE)."""
from __future__ import annotations

import ctypes
import os
import subprocess

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "accerl_oracle.c")
_SO = os.path.join(_HERE, "liboracle.so")
_lib = None

CFLAGS = ["-O2", "-fopenmp", "-ffp-contract=off", "-fno-fast-math", "-shared", "-fPIC",
          "-std=c11", "-Wall"]


def build(force: bool = False) -> str:
    """Build liboracle.so next to the source if it is missing or stale."""
    if force or not os.path.exists(_SO) or os.path.getmtime(_SO) < os.path.getmtime(_SRC):
        tmp = _SO + ".%d.tmp" % os.getpid()
        subprocess.check_call(["gcc", *CFLAGS, "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _SO)
    return _SO


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        for name in ("oracle_ingest_u8", "oracle_ingest_f32", "oracle_conv_acc", "oracle_fc_acc",
                     "oracle_skip_add", "oracle_epilogue_float", "oracle_requant",
                     "oracle_maxpool", "oracle_sample", "oracle_entropy", "oracle_kl",
                     "oracle_vtrace"):
            getattr(_lib, name).restype = None
    return _lib
