"""Shared helpers of the GPU parity tests: calibrated policies and the comparison itself."""
from __future__ import annotations

import functools

import numpy as np

import oracle
import workloads as W

# Tolerances of the parity bar: int8 activations and actions bit-exact (actions may differ only
# where the uniform lies within ACTION_MARGIN of a CDF edge; such cases are counted), float
# outputs within RTOL relative / ATOL absolute.
RTOL, ATOL, ACTION_MARGIN = 1e-5, 1e-6, 1e-5


@functools.lru_cache(maxsize=None)
def calibrated(name: str, rows: int = W.CALIBRATION_ROWS) -> dict:
    c = W.config(name)
    return oracle.calibrate(c["in_kind"], c["in_shape"], c["layers"], W.fp32_parameters(name),
                            W.calibration_batch(name, rows), c["prune24"])


def compare(ref: dict, logits, actions, logp, taps=None, n_taps=None) -> dict:
    """Assert parity of one batch; returns counters.  ``taps(layer, n)`` reads int8 activations."""
    logits, actions, logp = (np.asarray(a) for a in (logits, actions, logp))
    b = logits.shape[0]
    stats = dict(states=b, int8_compared=0, int8_mismatch=0, action_mismatch=0,
                 action_mismatch_near_edge=0)
    if taps is not None:
        n = b if n_taps is None else n_taps
        got = taps(-1, n)
        want = ref["input_q"][:n].reshape(got.shape)
        stats["int8_compared"] += want.size
        stats["int8_mismatch"] += int((got != want).sum())
        for i, a in enumerate(ref["activations"]):
            if a is None:
                continue
            got = taps(i, n)
            want = a[:n].reshape(got.shape)
            bad = int((got != want).sum())
            stats["int8_compared"] += want.size
            stats["int8_mismatch"] += bad
            assert bad == 0, "layer %d: %d of %d int8 activations differ" % (i, bad, want.size)
        assert stats["int8_mismatch"] == 0
    np.testing.assert_allclose(logits, ref["logits"], rtol=RTOL, atol=ATOL)
    diff = actions != ref["actions"]
    stats["action_mismatch"] = int(diff.sum())
    stats["action_mismatch_near_edge"] = int((diff & (ref["margin"] < ACTION_MARGIN)).sum())
    assert stats["action_mismatch"] == stats["action_mismatch_near_edge"], \
        "%d actions differ away from a CDF edge" % (stats["action_mismatch"] -
                                                    stats["action_mismatch_near_edge"])
    same = ~diff
    np.testing.assert_allclose(logp[same], ref["logp"][same], rtol=RTOL, atol=ATOL)
    # where the action legitimately differs, the log-prob must be the one of the action taken
    for i in np.nonzero(diff)[0]:
        np.testing.assert_allclose(logp[i], ref["logp_all"][i, actions[i]], rtol=RTOL, atol=ATOL)
    assert np.all((actions >= 0) & (actions < logits.shape[1]))
    assert np.all(np.isfinite(logp)) and np.all(logp <= 0)
    return stats
