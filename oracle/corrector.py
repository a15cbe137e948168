"""V-trace targets of the Corrector (TEST INFRASTRUCTURE): thin wrapper over the C definition."""
from __future__ import annotations

import ctypes as C

import numpy as np

from .clib import lib


def _p(a):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def vtrace(logp_smaller, logp_original, rewards, values, bootstrap, gamma: float,
           rho_hat: float = 1.0, c_hat: float = 1.0, discounts=None) -> dict:
    """All inputs time-major float32 [n, B] (bootstrap [B]); returns float64 ``vs`` and ``adv``."""
    arrs = [np.ascontiguousarray(a, np.float32) for a in (logp_smaller, logp_original, rewards, values)]
    n, b = arrs[0].shape
    assert all(a.shape == (n, b) for a in arrs)
    boot = np.ascontiguousarray(bootstrap, np.float32)
    assert boot.shape == (b,)
    disc = None if discounts is None else np.ascontiguousarray(discounts, np.float32)
    assert disc is None or disc.shape == (n, b)
    vs = np.empty((n, b), np.float64)
    adv = np.empty((n, b), np.float64)
    lib().oracle_vtrace(_p(arrs[0]), _p(arrs[1]), _p(arrs[2]), _p(arrs[3]), _p(boot), _p(disc),
                        n, b, C.c_float(gamma), C.c_float(rho_hat), C.c_float(c_hat), _p(vs), _p(adv))
    return dict(vs=vs, adv=adv)
