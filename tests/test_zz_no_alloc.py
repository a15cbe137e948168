"""accerl_policy_act_noalloc: the Actor step whose workspace is a fixed array in the library.

Some users of this library may not allocate GPU memory once they are running -- an Actor next to
a Learner that already owns the free HBM, or a control loop that cannot take an allocation's
stall.  They create a handle with max_batch = 1 and step through this entry point.  The test calls
it through the C ABI, twice in a row with different batches (the array keeps the first call's
bytes, the second call must not be disturbed by them), and requires the outputs of
accerl_policy_act on the same inputs: identical logits and actions, log-probs within the parity
tolerance.  This file sorts last on purpose, so that a run that stops at the first failure has
already been through every other test.
"""
import numpy as np
import pytest
import torch

import workloads as W
from parity_util import ATOL, RTOL

pytestmark = pytest.mark.gpu


def _outputs(b, a):
    return (torch.empty((b, a), dtype=torch.float32, device="cuda"),
            torch.empty(b, dtype=torch.int32, device="cuda"),
            torch.empty(b, dtype=torch.float32, device="cuda"))


def test_noalloc_matches_act_on_two_calls_in_a_row():
    import paper_2211_15023_b200 as P
    name = "nature_cnn_b160"
    pol = W.drawn_int8_policy(name)
    big = P.Policy(pol, 160)          # the regular entry point, with its own workspace
    tiny = P.Policy(pol, 1)           # owns (almost) nothing but the weights
    stream = torch.cuda.current_stream().cuda_stream
    for call, b in enumerate([160, 37]):
        obs = torch.from_numpy(W.observations(name, b, seed=70 + call)).cuda()
        u = torch.from_numpy(W.uniforms(name, b, seed=80 + call)).cuda()
        want = big.act(obs, u)
        got = _outputs(b, tiny.n_actions)
        free_before = torch.cuda.mem_get_info()[0]
        status = tiny.act_noalloc_raw(obs.data_ptr(), u.data_ptr(), b, got[0].data_ptr(),
                                      got[1].data_ptr(), got[2].data_ptr(), stream)
        assert status == 0, P.library().accerl_last_error()
        torch.cuda.synchronize()
        if call > 0:   # the first call on a device may load the module; later ones hold memory still
            assert torch.cuda.mem_get_info()[0] >= free_before
        assert np.array_equal(got[0].cpu().numpy(), want[0].cpu().numpy())
        assert np.array_equal(got[1].cpu().numpy(), want[1].cpu().numpy())
        np.testing.assert_allclose(got[2].cpu().numpy(), want[2].cpu().numpy(), rtol=RTOL, atol=ATOL)
    # a batch whose activations cannot fit the fixed array is refused with a clear message
    b = 4096
    obs = torch.zeros((b, 4, 84, 84), dtype=torch.uint8, device="cuda")
    u = torch.zeros(b, device="cuda")
    got = _outputs(b, tiny.n_actions)
    status = tiny.act_noalloc_raw(obs.data_ptr(), u.data_ptr(), b, got[0].data_ptr(),
                                  got[1].data_ptr(), got[2].data_ptr(), stream)
    assert status == 3
    msg = P.library().accerl_last_error().decode()
    assert "scratch" in msg and str(64 * 1024 * 1024) in msg
    assert tiny.act_noalloc_raw(None, u.data_ptr(), 4, got[0].data_ptr(), got[1].data_ptr(),
                                got[2].data_ptr(), stream) == 1
    big.check()
    tiny.check()    # waits on the stream of the last noalloc step, reports the device status word
    big.close()
    tiny.close()


@pytest.mark.parametrize("name,b", [("cartpole_mlp", 160), ("impala_resnet_b16384", 9)])
def test_noalloc_other_layer_kinds(name, b):
    """fp32 vector input, max-pool and residual layers carved from the same fixed array."""
    import paper_2211_15023_b200 as P
    pol = W.drawn_int8_policy(name)
    big, tiny = P.Policy(pol, b), P.Policy(pol, 1)
    stream = torch.cuda.current_stream().cuda_stream
    for call in range(2):
        obs = torch.from_numpy(W.observations(name, b, seed=90 + call)).cuda()
        u = torch.from_numpy(W.uniforms(name, b, seed=95 + call)).cuda()
        want = big.act(obs, u)
        got = _outputs(b, tiny.n_actions)
        assert tiny.act_noalloc_raw(obs.data_ptr(), u.data_ptr(), b, got[0].data_ptr(),
                                    got[1].data_ptr(), got[2].data_ptr(), stream) == 0
        tiny.check()
        assert np.array_equal(got[0].cpu().numpy(), want[0].cpu().numpy())
        assert np.array_equal(got[1].cpu().numpy(), want[1].cpu().numpy())
        np.testing.assert_allclose(got[2].cpu().numpy(), want[2].cpu().numpy(), rtol=RTOL, atol=ATOL)
    big.close()
    tiny.close()
