"""The C-ABI library without a GPU: it builds, loads, exports what the header declares, and
rejects bad descriptions on the host before it ever touches a device."""
import ctypes as C
import os
import re
import subprocess

import numpy as np
import pytest

import workloads as W

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2211_15023_b200 import build, binding
    build.build()
    return binding.library()


def _declared():
    names = []
    for fn in sorted(os.listdir(os.path.join(ROOT, "include"))):
        text = open(os.path.join(ROOT, "include", fn)).read()
        text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
        names += re.findall(r"\b(accerl_[a-z_0-9]+)\s*\(", text)
    return sorted(set(names))


def test_library_exports_every_declared_symbol(lib):
    declared = _declared()
    assert {"accerl_policy_create", "accerl_policy_act", "accerl_policy_destroy"} <= set(declared)
    out = subprocess.check_output(["nm", "-D", "--defined-only", lib._name]).decode()
    exported = set(re.findall(r" T (accerl_\w+)", out))
    for name in declared:
        assert name in exported, name
        getattr(lib, name)
    assert lib.accerl_version().startswith(b"accerl-b200")
    assert lib.accerl_last_error() is not None


def _create(pol, max_batch=8, flags=0, mutate=None):
    from paper_2211_15023_b200 import binding
    import copy
    pol = copy.deepcopy(pol)
    if mutate:
        mutate(pol)
    try:
        binding.Policy(pol, max_batch, flags)
    except binding.AccerlError as e:
        return e.status, str(e)
    return 0, ""


def test_bad_descriptions_are_rejected_on_the_host(lib):
    pol = W.drawn_int8_policy("impala_resnet_b16384")
    INVALID, UNSUPPORTED = 1, 2

    def m_scale(p): p["layers"][2]["s_in"] = np.float32(0.5)
    def m_shape(p): p["layers"][2]["in_h"] = 40
    def m_logits(p): p["layers"][-1]["logits"] = False
    def m_w128(p): p["layers"][0]["w"][0, 0, 0, 0] = -128
    def m_skip_fwd(p): p["layers"][3]["skip_from"] = 7
    def m_skip_mul(p): p["layers"][3]["skip_mul"][0] = 40000
    def m_skip_shape(p): p["layers"][3]["skip_from"] = 0
    def m_neg_scale(p): p["s_input"] = np.float32(-1.0)
    def m_fc_k(p): p["layers"][-2]["in_c"] = 2591
    def m_pool_scale(p): p["layers"][1]["s_out"] = np.float32(0.7)
    def m_kind(p): p["in_kind"] = "f32"

    for mut in (m_scale, m_shape, m_logits, m_w128, m_skip_fwd, m_skip_mul, m_skip_shape,
                m_neg_scale, m_fc_k, m_pool_scale, m_kind):
        status, msg = _create(pol, mutate=mut)
        assert status == INVALID, (mut.__name__, status, msg)
        assert len(msg) > 10
    status, _ = _create(pol, max_batch=0)
    assert status == INVALID
    status, _ = _create(pol, flags=1 << 9)
    assert status == INVALID
    # a valid description passes validation and only then fails for want of a device
    import torch
    if not torch.cuda.is_available():
        status, msg = _create(pol)
        assert status == 5 and "device" in msg


def test_further_entry_points_reject_bad_arguments_on_the_host(lib):
    """Argument checks of the calls beside create / act happen before any device is touched."""
    import ctypes as C
    from paper_2211_15023_b200 import binding
    INVALID = 1
    buf = np.zeros(64, np.float32)
    p = buf.ctypes.data
    # V-trace: null array, non-positive sizes, bad clips, misaligned pointer
    assert lib.accerl_vtrace(None, p, p, p, p, None, 2, 4, 0.99, 1.0, 1.0, p, None, None) == INVALID
    assert lib.accerl_vtrace(p, p, p, p, p, None, 0, 4, 0.99, 1.0, 1.0, p, None, None) == INVALID
    assert lib.accerl_vtrace(p, p, p, p, p, None, 2, 4, 0.99, -1.0, 1.0, p, None, None) == INVALID
    assert lib.accerl_vtrace(p, p, p, p, p, None, 2, 4, 0.99, 1.0, 1.0, p + 2, None, None) == INVALID
    assert b"vtrace" in lib.accerl_last_error()
    # KL: null array, action count out of range
    assert lib.accerl_policy_kl(None, p, 4, 2, p, None, None) == INVALID
    assert lib.accerl_policy_kl(p, p, 4, 0, p, None, None) == INVALID
    assert lib.accerl_policy_kl(p, p, 4, 2000, p, None, None) == INVALID
    # handle-taking calls refuse a null handle
    assert lib.accerl_policy_act_ex(None, p, p, 1, p, p, p, None, None, None) == INVALID
    assert lib.accerl_policy_act_mixed(None, None, p, p, p, 0.5, 1, p, p, p, None, None, None, None) == INVALID
    assert lib.accerl_policy_selftest_wait(None, 100, None) == INVALID
    assert lib.accerl_policy_export(None, 0, None, 0, None, None, None, None) == INVALID
    # the probe checks its shape arguments first
    ms, cyc = C.c_float(), C.c_float()
    assert lib.accerl_tc_probe_i8(0, 24, 1, 64, 1, 128, 0, 0, C.byref(ms), C.byref(cyc)) == INVALID
    assert lib.accerl_tc_probe_i8(0, 256, 4, 64, 1, 128, 0, 0, C.byref(ms), C.byref(cyc)) == INVALID
    # quantisation on the device: shapes that do not chain are refused before the device is used
    layers = [dict(l) for l in W.config("cartpole_mlp")["layers"]]
    params = W.fp32_parameters("cartpole_mlp")
    calib = W.calibration_batch("cartpole_mlp", 8)
    layers[1]["in_c"] = 63
    with pytest.raises(binding.AccerlError) as e:
        binding.Policy.from_fp32("f32", (4, 1, 1), layers, params, calib, 8)
    assert e.value.status == INVALID and "layer 1" in str(e.value)
