"""GPU parity: the CUDA library, called through its C ABI, against the CPU oracle."""
import numpy as np
import pytest
import torch

import oracle
import workloads as W
from parity_util import calibrated, compare

pytestmark = pytest.mark.gpu

SMALL = {  # name -> batches that span several tiles plus ragged tails
    "cartpole_mlp": [1, 3, 127, 160],
    "lunarlander_mlp": [129, 4096],
    "nature_cnn_b160": [1, 3, 37],
    "student_cnn_b8192": [5, 33],
    "impala_resnet_b16384": [2, 9],
}


def _run(pol, obs, u, flags, max_batch=None):
    import paper_2211_15023_b200 as P
    g = P.Policy(pol, max_batch or obs.shape[0], flags=flags)
    out = g.act(torch.from_numpy(obs).cuda(), torch.from_numpy(u).cuda())
    torch.cuda.synchronize()
    g.check()
    return g, [t.cpu().numpy() for t in out]


# tensors the production plan never stores (no tap can exist): the quantised frames when the
# input stage runs inside the first conv; conv outputs that are pooled on their accumulators
# (first conv and the 16->32 conv of the ResNet) and the ReLU'd-only input of its first fc layer
FUSED_TAPS_MISSING = {"cartpole_mlp": 0, "lunarlander_mlp": 0, "nature_cnn_b160": 1,
                      "student_cnn_b8192": 1, "impala_resnet_b16384": 3}


@pytest.mark.parametrize("name", list(SMALL))
@pytest.mark.parametrize("flags", [1, 5, 3], ids=["unfused_plan", "production_plan", "generic_plan"])
def test_small_batches_every_activation(name, flags):
    """flags 1: every tensor exists (input stage, pools and MLP layers as launches of their own);
    flags 5: the kernels of the production plan (what flags = 0 runs), tapped wherever that plan
    stores a tensor; flags 3: the CUDA-core kernels."""
    pol = calibrated(name)
    for b in SMALL[name]:
        obs, u = W.observations(name, b), W.uniforms(name, b)
        ref = oracle.forward(pol, obs, u)
        g, (logits, actions, logp) = _run(pol, obs, u, flags)
        if flags == 5:
            g0 = __import__("paper_2211_15023_b200").Policy(pol, obs.shape[0], flags=0)
            assert g0.info()["plan"] == g.info()["plan"], "the tapped plan is not the production plan"
            g0.close()
        stats = compare(ref, logits, actions, logp, taps=g.read_activation, label=name)
        assert stats["int8_mismatch"] == 0
        assert stats["taps_missing"] == (FUSED_TAPS_MISSING[name] if flags == 5 else 0), stats
        # three runs must give identical bytes (races show up as nondeterminism)
        for _ in range(2):
            out2 = g.act(torch.from_numpy(obs).cuda(), torch.from_numpy(u).cuda())
            assert np.array_equal(out2[0].cpu().numpy(), logits)
            assert np.array_equal(out2[1].cpu().numpy(), actions)
        g.close()


FULL = ["cartpole_mlp", "lunarlander_mlp", "nature_cnn_b160", "nature_cnn_b8192",
        "student_cnn_b8192", "impala_resnet_b16384"]


@pytest.mark.parametrize("name", FULL)
def test_full_batch_every_state(name):
    """Full batch on the plan the benchmark times (flags = 0), EVERY state against the oracle:
    logits bit for bit, actions (mismatches next to a CDF edge counted), log-probs.  The oracle
    streams through the batch in chunks and keeps no activations."""
    import paper_2211_15023_b200 as P
    pol = calibrated(name)
    b = W.config(name)["batch"]
    obs, u = W.observations(name, b), W.uniforms(name, b)
    g = P.Policy(pol, b, flags=0)
    out = g.act(torch.from_numpy(obs).cuda(), torch.from_numpy(u).cuda())
    torch.cuda.synchronize()
    g.check()
    logits, actions, logp = [t.cpu().numpy() for t in out]
    near_edge = 0
    for lo in range(0, b, 512):
        hi = min(b, lo + 512)
        ref = oracle.forward(pol, obs[lo:hi], u[lo:hi], keep=False)
        st = compare(ref, logits[lo:hi], actions[lo:hi], logp[lo:hi], label=name + "/full_batch")
        near_edge += st["action_mismatch_near_edge"]
    assert near_edge <= max(2, b // 1000), near_edge   # a |u - cdf| < 1e-5 event is rare
    # the same states alone in a small batch give the same bytes (no cross-state coupling)
    idx = np.unique(np.concatenate([[0, b - 1], np.random.default_rng(99).choice(b, min(b, 5), replace=False)]))
    small = g.act(torch.from_numpy(obs[idx]).cuda(), torch.from_numpy(u[idx]).cuda())
    assert np.array_equal(small[0].cpu().numpy(), logits[idx])
    assert np.array_equal(small[1].cpu().numpy(), actions[idx])
    g.close()


@pytest.mark.parametrize("name", ["cartpole_mlp", "lunarlander_mlp"])
def test_single_launch_mlp_plan_odd_batches(name):
    """Vector-observation MLPs run as one fused launch; batches around the 8-row CTA granule."""
    import paper_2211_15023_b200 as P
    pol = calibrated(name)
    g = P.Policy(pol, 200, flags=0)
    info = g.info()
    assert info["launches_per_act"] == 1 and "mlp_fused_kernel" in info["plan"]
    for b in (1, 7, 8, 9, 160, 199):
        obs, u = W.observations(name, b, seed=b), W.uniforms(name, b, seed=100 + b)
        ref = oracle.forward(pol, obs, u, keep=False)
        out = [t.cpu().numpy() for t in g.act(torch.from_numpy(obs).cuda(), torch.from_numpy(u).cuda())]
        compare(ref, *out)
    g.close()


def test_act_host_matches_device_call():
    import paper_2211_15023_b200 as P
    name = "nature_cnn_b160"
    pol = calibrated(name)
    obs, u = W.observations(name, 20), W.uniforms(name, 20)
    g = P.Policy(pol, 32)
    dev = [t.cpu().numpy() for t in g.act(torch.from_numpy(obs).cuda(), torch.from_numpy(u).cuda())]
    host = (torch.empty((20, 18), dtype=torch.float32).pin_memory(),
            torch.empty(20, dtype=torch.int32).pin_memory(),
            torch.empty(20, dtype=torch.float32).pin_memory())
    g.act_host(torch.from_numpy(obs).pin_memory(), torch.from_numpy(u).pin_memory(), host)
    for a, b in zip(dev, host):
        assert np.array_equal(a, b.numpy())
    g.close()


def test_act_host_in_chunks_matches_device_call():
    """From 4096 states on the host-buffer call goes in eight chunks with the copies overlapped; a
    batch that does not divide evenly (4099 on the MLP, whose fp32 rows keep every chunk aligned)
    and two calls in a row must give what one device call gives."""
    import paper_2211_15023_b200 as P
    name, b = "lunarlander_mlp", 4099
    pol = calibrated(name)
    g = P.Policy(pol, b)
    for call in range(2):
        obs, u = W.observations(name, b, seed=call), W.uniforms(name, b, seed=10 + call)
        dev = [t.cpu().numpy() for t in g.act(torch.from_numpy(obs).cuda(), torch.from_numpy(u).cuda())]
        host = (torch.empty((b, 4), dtype=torch.float32).pin_memory(),
                torch.empty(b, dtype=torch.int32).pin_memory(),
                torch.empty(b, dtype=torch.float32).pin_memory())
        g.act_host(torch.from_numpy(obs).pin_memory(), torch.from_numpy(u).pin_memory(), host)
        for x, y in zip(dev, host):
            assert np.array_equal(x, y.numpy())
    g.check()
    g.close()


def test_saturating_inputs_and_extreme_uniforms():
    import paper_2211_15023_b200 as P
    name = "lunarlander_mlp"
    pol = calibrated(name)
    obs = (W.observations(name, 64) * 5).astype(np.float32)   # far outside the calibrated range
    u = np.concatenate([np.zeros(32), np.full(32, np.nextafter(np.float32(1), np.float32(0)))]
                       ).astype(np.float32)
    ref = oracle.forward(pol, obs, u)
    g = P.Policy(pol, 64, flags=1)
    out = [t.cpu().numpy() for t in g.act(torch.from_numpy(obs).cuda(), torch.from_numpy(u).cuda())]
    compare(ref, *out, taps=g.read_activation)
    g.close()


def test_many_actions_wide_sampler():
    # 40 actions exercise the sampler that strides a warp over the row
    import paper_2211_15023_b200 as P
    rng = np.random.default_rng(5)
    layers = W.mlp([6, 32, 40])
    params = [dict(w=rng.standard_normal((l["out_c"], l["in_c"], 1, 1)).astype(np.float32),
                   bias=rng.standard_normal(l["out_c"]).astype(np.float32) * 0.1) for l in layers]
    calib = rng.standard_normal((256, 6)).astype(np.float32)
    pol = oracle.calibrate("f32", (6, 1, 1), layers, params, calib)
    obs = rng.standard_normal((77, 6)).astype(np.float32)
    u = rng.random(77, dtype=np.float32)
    ref = oracle.forward(pol, obs, u)
    g = P.Policy(pol, 77, flags=1)
    out = [t.cpu().numpy() for t in g.act(torch.from_numpy(obs).cuda(), torch.from_numpy(u).cuda())]
    compare(ref, *out, taps=g.read_activation)
    g.close()


def test_odd_shapes_padding_stride_pool_residual():
    import paper_2211_15023_b200 as P
    rng = np.random.default_rng(11)
    layers = [W._conv(3, 11, 9, 5, 3, 2, 1, relu_out=False), W._pool(5, 6, 5, 3, 2),
              W._conv(5, 2, 2, 5, 3, 1, 1, relu_in=True),
              W._conv(5, 2, 2, 5, 3, 1, 1, relu_out=False, skip_from=1),
              W._fc(20, 7, relu_in=True), W._fc(7, 3, relu_out=False, logits=True)]
    params = [None if l["kind"] == "maxpool" else
              dict(w=rng.standard_normal((l["out_c"], l["in_c"], l["kh"], l["kw"])
                                         ).astype(np.float32) * 0.3,
                   bias=rng.standard_normal(l["out_c"]).astype(np.float32) * 0.1) for l in layers]
    calib = rng.integers(0, 256, (16, 3, 11, 9), dtype=np.uint8)
    pol = oracle.calibrate("u8", (3, 11, 9), layers, params, calib)
    obs = rng.integers(0, 256, (13, 3, 11, 9), dtype=np.uint8)
    u = rng.random(13, dtype=np.float32)
    ref = oracle.forward(pol, obs, u)
    g = P.Policy(pol, 13, flags=1)
    out = [t.cpu().numpy() for t in g.act(torch.from_numpy(obs).cuda(), torch.from_numpy(u).cuda())]
    compare(ref, *out, taps=g.read_activation)
    g.close()


@pytest.mark.parametrize("hw", [(44, 40), (37, 52)], ids=["19_wide_after_pool", "25_wide_after_pool"])
def test_multi_pixel_rows_ragged_widths(hw):
    """Residual 3x3 stacks on images whose width is no multiple of the pixels per GEMM row: the
    last group of a row is cut (19 = 2*8+3, 25 = 3*8+1; the 16->32 conv and the 32-channel block
    use 4 pixels per row), with and without taps, so that both the direct and the shared-memory
    staged epilogues, the residual read and the ReLU'd second copy are compared with the oracle."""
    import paper_2211_15023_b200 as P
    H, Wd = hw
    rng = np.random.default_rng(23)
    h1, w1 = (H - 3) // 2 + 1, (Wd - 3) // 2 + 1
    layers = [W._conv(4, H, Wd, 16, 3, 1, 1, relu_out=False), W._pool(16, H, Wd),
              W._conv(16, h1, w1, 16, 3, 1, 1, relu_in=True, relu_out=True),
              W._conv(16, h1, w1, 16, 3, 1, 1, relu_out=False, skip_from=1),
              W._conv(16, h1, w1, 32, 3, 1, 1, relu_out=False),
              W._conv(32, h1, w1, 32, 3, 1, 1, relu_in=True, relu_out=True),
              W._conv(32, h1, w1, 32, 3, 1, 1, relu_out=False, skip_from=4),
              W._pool(32, h1, w1)]
    h2, w2 = (h1 - 3) // 2 + 1, (w1 - 3) // 2 + 1
    layers += [W._fc(32 * h2 * w2, 64, relu_in=True), W._fc(64, 6, relu_out=False, logits=True)]
    params = [None if l["kind"] == "maxpool" else
              dict(w=(rng.standard_normal((l["out_c"], l["in_c"], l["kh"], l["kw"])) *
                      np.sqrt(2.0 / (l["in_c"] * l["kh"] * l["kw"]))).astype(np.float32),
                   bias=rng.standard_normal(l["out_c"]).astype(np.float32) * 0.05) for l in layers]
    calib = rng.integers(0, 256, (32, 4, H, Wd), dtype=np.uint8)
    pol = oracle.calibrate("u8", (4, H, Wd), layers, params, calib)
    b = 11
    obs = rng.integers(0, 256, (b, 4, H, Wd), dtype=np.uint8)
    u = rng.random(b, dtype=np.float32)
    ref = oracle.forward(pol, obs, u)
    for flags in (1, 5, 0):
        g = P.Policy(pol, b, flags=flags)
        assert "tc_gemm_kernel" in g.info()["plan"]
        out = [t.cpu().numpy() for t in g.act(torch.from_numpy(obs).cuda(), torch.from_numpy(u).cuda())]
        g.check()
        compare(ref, *out, taps=g.read_activation if flags else None)
        g.close()


@pytest.mark.parametrize("hw", [(44, 40), (37, 52), (52, 84)],
                         ids=["19_wide_after_pool", "25_wide_after_pool", "41_wide_after_pool"])
def test_conv_pooled_on_accumulators_ragged_widths(hw):
    """A 16->32 conv whose only reader is a 3x3 stride-2 max-pool pools along x on its int32
    accumulators (and so does the first conv): widths that are no multiple of the 4 pixels of a
    GEMM row, on the production plan with and without taps, against the oracle's pooled tensor
    and everything after it."""
    import paper_2211_15023_b200 as P
    H, Wd = hw
    rng = np.random.default_rng(29)
    h1, w1 = (H - 3) // 2 + 1, (Wd - 3) // 2 + 1
    h2, w2 = (h1 - 3) // 2 + 1, (w1 - 3) // 2 + 1
    layers = [W._conv(4, H, Wd, 16, 3, 1, 1, relu_out=False), W._pool(16, H, Wd),
              W._conv(16, h1, w1, 16, 3, 1, 1, relu_in=True, relu_out=True),
              W._conv(16, h1, w1, 16, 3, 1, 1, relu_out=False, skip_from=1),
              W._conv(16, h1, w1, 32, 3, 1, 1, relu_out=False), W._pool(32, h1, w1),
              W._conv(32, h2, w2, 32, 3, 1, 1, relu_in=True, relu_out=True),
              W._conv(32, h2, w2, 32, 3, 1, 1, relu_out=False, skip_from=5),
              W._fc(32 * h2 * w2, 64, relu_in=True), W._fc(64, 6, relu_out=False, logits=True)]
    params = [None if l["kind"] == "maxpool" else
              dict(w=(rng.standard_normal((l["out_c"], l["in_c"], l["kh"], l["kw"])) *
                      np.sqrt(2.0 / (l["in_c"] * l["kh"] * l["kw"]))).astype(np.float32),
                   bias=rng.standard_normal(l["out_c"]).astype(np.float32) * 0.05) for l in layers]
    calib = rng.integers(0, 256, (32, 4, H, Wd), dtype=np.uint8)
    pol = oracle.calibrate("u8", (4, H, Wd), layers, params, calib)
    b = 7
    obs = rng.integers(0, 256, (b, 4, H, Wd), dtype=np.uint8)
    u = rng.random(b, dtype=np.float32)
    ref = oracle.forward(pol, obs, u)
    plans = {}
    for flags in (1, 5, 0):
        g = P.Policy(pol, b, flags=flags)
        plans[flags] = g.info()["plan"]
        out = [t.cpu().numpy() for t in g.act(torch.from_numpy(obs).cuda(), torch.from_numpy(u).cuda())]
        g.check()
        assert "pooled along x on the accumulators" in plans[flags] or flags == 1, plans[flags]
        st = compare(ref, *out, taps=g.read_activation if flags else None)
        if flags == 5:
            # layers 0 and 4 (pooled on their accumulators) and the ReLU'd-only input of the fc
            assert st["taps_missing"] == 3 and st["int8_compared"] > 0, st
            assert g.read_activation(5, b).shape == ref["activations"][5].shape
        g.close()
    assert plans[5] == plans[0] and plans[1] != plans[0]


def test_tensor_core_logits_layer_with_many_actions():
    """More than 32 actions: the last layer cannot run fused with the sampler, so the tensor-core
    kernel writes the fp32 logits itself and the wide sampler follows."""
    import paper_2211_15023_b200 as P
    rng = np.random.default_rng(31)
    layers = W.nature_cnn(16, 32, 32, 256, actions=40)
    params = [dict(w=(rng.standard_normal((l["out_c"], l["in_c"], l["kh"], l["kw"])) *
                      np.sqrt(2.0 / (l["in_c"] * l["kh"] * l["kw"]))).astype(np.float32),
                   bias=rng.standard_normal(l["out_c"]).astype(np.float32) * 0.05) for l in layers]
    calib = rng.integers(0, 256, (64, 4, 84, 84), dtype=np.uint8)
    pol = oracle.calibrate("u8", (4, 84, 84), layers, params, calib)
    b = 45
    obs = rng.integers(0, 256, (b, 4, 84, 84), dtype=np.uint8)
    u = rng.random(b, dtype=np.float32)
    ref = oracle.forward(pol, obs, u)
    for flags in (1, 0):
        g = P.Policy(pol, b, flags=flags)
        plan = g.info()["plan"]
        assert "tc_gemm_kernel" in plan and "sample_wide_kernel" in plan
        out = [t.cpu().numpy() for t in g.act(torch.from_numpy(obs).cuda(), torch.from_numpy(u).cuda())]
        g.check()
        compare(ref, *out, taps=g.read_activation if flags else None)
        g.close()


@pytest.mark.parametrize("name", ["nature_cnn_b160", "student_cnn_b8192"])
def test_input_stage_inside_first_conv_small_and_ragged_batches(name):
    """Without the parity taps the frames are quantised inside the first conv (no launch of their
    own): batches from one state up, none a multiple of the 256 GEMM rows of a pipeline step."""
    import paper_2211_15023_b200 as P
    pol = calibrated(name)
    g = P.Policy(pol, 61, flags=0)
    assert "frames quantised inside" in g.info()["plan"]
    for b in (1, 2, 5, 37, 61):
        obs, u = W.observations(name, b, seed=77 + b), W.uniforms(name, b, seed=78 + b)
        ref = oracle.forward(pol, obs, u, keep=False)
        out = [t.cpu().numpy() for t in g.act(torch.from_numpy(obs).cuda(), torch.from_numpy(u).cuda())]
        g.check()
        compare(ref, *out)
    g.close()


@pytest.mark.parametrize("hw,c1,peak", [((68, 100), 16, 255), ((96, 64), 32, 200), ((84, 84), 32, 140),
                                        ((44, 124), 16, 255)],
                         ids=["68x100_c16_shift", "96x64_c32_line", "84x84_c32_line_clamped", "44x124_c16"])
def test_first_conv_kernel_other_frames_and_input_tables(hw, c1, peak):
    """The first-conv kernel with the input stage inside on frames other than 84 x 84 (grid widths
    that leave idle rows in a tile, a grid height that is no multiple of the rows of a tile) and
    with input tables other than u >> 1: calibration frames whose largest byte is `peak` give
    s_input = peak / 255 / 127, a general line, with the clamp at 127 live when test frames
    exceed the calibrated range.  Production plan with and without taps, and the un-fused plan."""
    import paper_2211_15023_b200 as P
    H, Wd = hw
    rng = np.random.default_rng(H * 1000 + Wd + c1)
    h1, w1 = (H - 8) // 4 + 1, (Wd - 8) // 4 + 1
    h2, w2 = (h1 - 4) // 2 + 1, (w1 - 4) // 2 + 1
    layers = [W._conv(4, H, Wd, c1, 8, 4, 0), W._conv(c1, h1, w1, 16, 4, 2, 0) if h1 % 2 == 0 and w1 % 2 == 0
              else W._conv(c1, h1, w1, 16, 3, 1, 0)]
    if layers[1]["kh"] == 3:
        h2, w2 = h1 - 2, w1 - 2
    layers += [W._fc(16 * h2 * w2, 64), W._fc(64, 5, relu_out=False, logits=True)]
    params = W.parameters_for(layers, 11)
    calib = rng.integers(0, peak + 1, (16, 4, H, Wd), dtype=np.uint8)
    pol = oracle.calibrate("u8", (4, H, Wd), layers, params, calib)
    b = 23
    obs = rng.integers(0, 256, (b, 4, H, Wd), dtype=np.uint8)
    u = rng.random(b, dtype=np.float32)
    ref = oracle.forward(pol, obs, u)
    for flags in (0, 5, 1):
        g = P.Policy(pol, b, flags=flags)
        plan = g.info()["plan"]
        assert ("conv1_frames_kernel" in plan) == (flags != 1), plan
        out = [t.cpu().numpy() for t in g.act(torch.from_numpy(obs).cuda(), torch.from_numpy(u).cuda())]
        g.check()
        compare(ref, *out, taps=g.read_activation if flags else None)
        g.close()


@pytest.mark.parametrize("hw,c2,c3", [((68, 100), 64, 48), ((52, 84), 64, 48), ((100, 52), 64, 64)],
                         ids=["68x100_64_48", "52x84_64_48", "100x52_64_64"])
def test_strided_conv_kernel_other_grids_and_widths(hw, c2, c3):
    """The strided-conv kernel with tiles of whole grid rows on grids other than the Atari network's
    (widths that leave idle rows in a tile, 48 and 64 output channels, 128- and 64-byte rows, 2 x 2
    and 3 x 3 taps), small and ragged batches, with and without taps, against the un-fused plan's
    general kernel and the oracle."""
    import paper_2211_15023_b200 as P
    H, Wd = hw
    rng = np.random.default_rng(H * 7 + Wd + c2)
    h1, w1 = (H - 8) // 4 + 1, (Wd - 8) // 4 + 1
    h2, w2 = (h1 - 4) // 2 + 1, (w1 - 4) // 2 + 1
    h3, w3 = h2 - 2, w2 - 2
    layers = [W._conv(4, H, Wd, 32, 8, 4, 0), W._conv(32, h1, w1, c2, 4, 2, 0), W._conv(c2, h2, w2, c3, 3, 1, 0),
              W._fc(c3 * h3 * w3, 64), W._fc(64, 5, relu_out=False, logits=True)]
    params = W.parameters_for(layers, 13)
    calib = rng.integers(0, 256, (16, 4, H, Wd), dtype=np.uint8)
    pol = oracle.calibrate("u8", (4, H, Wd), layers, params, calib)
    for b in (1, 29):
        obs = rng.integers(0, 256, (b, 4, H, Wd), dtype=np.uint8)
        u = rng.random(b, dtype=np.float32)
        ref = oracle.forward(pol, obs, u)
        for flags in (0, 5, 1):
            g = P.Policy(pol, b, flags=flags)
            plan = g.info()["plan"]
            assert (plan.count("conv_rows_kernel") == 2) == (flags != 1), plan
            out = [t.cpu().numpy() for t in g.act(torch.from_numpy(obs).cuda(), torch.from_numpy(u).cuda())]
            g.check()
            compare(ref, *out, taps=g.read_activation if flags else None)
            g.close()


def test_exact_ties_on_the_tensor_core_path():
    """Power-of-two scales make many epilogue quotients land exactly on k + 0.5: the requantiser
    must round them to even exactly as the IEEE divide + rintf of the definition does."""
    import paper_2211_15023_b200 as P
    from oracle import net as ON
    name = "student_cnn_b8192"
    pol = W.drawn_int8_policy(name, seed=123)
    b = 24
    obs, u = W.observations(name, b, seed=9), W.uniforms(name, b, seed=10)
    pol["s_input"] = np.float32(2.0 ** -7)
    x = ON.ingest("u8", obs, pol["s_input"]).reshape((b,) + pol["in_shape"])
    s_prev, ties = pol["s_input"], 0
    for l in pol["layers"]:
        l["s_in"] = s_prev
        l["s_w"] = np.full(l["out_c"], 2.0 ** -7, np.float32)
        if l["kind"] == "fc":
            x = x.reshape(b, -1, 1, 1)
        acc = ON.layer_acc(l, x)
        y0 = ON.layer_float(dict(l, bias=np.zeros(l["out_c"], np.float32)), acc)
        if l["logits"]:
            break
        e = int(np.ceil(np.log2(np.abs(y0).max() / 127.0))) - 1      # some saturation on purpose
        l["s_out"] = np.float32(2.0 ** e)
        l["bias"] = (np.round(l["bias"] / (l["s_out"] / 2)) * (l["s_out"] / 2)).astype(np.float32)
        y = ON.layer_float(l, acc)
        frac = np.abs(y / l["s_out"]) % 1.0
        ties += int(((frac == 0.5) & (np.abs(y / l["s_out"]) < 127)).sum())
        x = ON.requant(y, l["s_out"])
        s_prev = l["s_out"]
    assert ties > 200, ties
    ref = oracle.forward(pol, obs, u)
    # power-of-two scales are the easy case of both division-free requantisers: the single fma is
    # exact, and so is the three-step division it replaces
    for flags, note in ((1, "single-fma requantiser verified"), (1 | P.FLAG_TEST_NO_AFFINE, "3-step divide verified")):
        g = P.Policy(pol, b, flags=flags)
        assert "tc_gemm" in g.info()["plan"]
        assert note in g.info()["plan"], g.info()["plan"]
        out = [t.cpu().numpy() for t in g.act(torch.from_numpy(obs).cuda(), torch.from_numpy(u).cuda())]
        compare(ref, *out, taps=g.read_activation)
        g.close()


def test_abi_rejects_bad_calls_without_launching():
    import paper_2211_15023_b200 as P
    pol = calibrated("cartpole_mlp")
    g = P.Policy(pol, 8)
    obs = torch.zeros((16, 4), device="cuda")
    u = torch.zeros(16, device="cuda")
    lo, ac, lp = (torch.empty((16, 2), device="cuda"), torch.empty(16, dtype=torch.int32, device="cuda"),
                  torch.empty(16, device="cuda"))
    assert g.act_raw(obs.data_ptr(), u.data_ptr(), 16, lo.data_ptr(), ac.data_ptr(), lp.data_ptr()) == 3
    assert g.act_raw(obs.data_ptr(), u.data_ptr(), 0, lo.data_ptr(), ac.data_ptr(), lp.data_ptr()) == 1
    assert g.act_raw(None, u.data_ptr(), 4, lo.data_ptr(), ac.data_ptr(), lp.data_ptr()) == 1
    assert g.act_raw(obs.data_ptr() + 4, u.data_ptr(), 4, lo.data_ptr(), ac.data_ptr(), lp.data_ptr()) == 1
    with pytest.raises(P.AccerlError):
        g.read_activation(0, 4)          # no KEEP_ACTIVATIONS flag
    g.check()
    g.close()


@pytest.mark.parametrize("name,b", [("nature_cnn_b160", 37), ("student_cnn_b8192", 21), ("impala_resnet_b16384", 5)])
def test_policies_whose_output_scales_fail_the_division_check(name, b):
    """The create-time check of the division-free requantiser can reject an output scale.  With the
    test flag every scale counts as rejected: every layer then runs the epilogue that redoes
    elements near a rounding tie with the IEEE divide -- still on tensor cores, the input stage
    still inside the first conv of the Nature-CNN plans, the residual stacks still on their
    multi-pixel rows and pooled accumulators -- and the plan says so.  Bits must not change."""
    import paper_2211_15023_b200 as P
    pol = calibrated(name, 64)
    obs, u = W.observations(name, b), W.uniforms(name, b)
    ref = oracle.forward(pol, obs, u)
    for flags in (P.FLAG_TEST_NO_FASTDIV, P.FLAG_TEST_NO_FASTDIV | 5):
        g = P.Policy(pol, b, flags=flags)
        plan = g.info()["plan"]
        assert "3-step divide verified" not in plan and "single-fma" not in plan, plan
        assert "tc_gemm_kernel" in plan and "division check failed" in plan and "note:" not in plan, plan
        if name == "impala_resnet_b16384":
            assert "dp4a" not in plan and ("pooled along x on the accumulators" in plan or flags & 1), plan
        else:
            assert "frames quantised inside" in plan, plan
        out = [t.cpu().numpy() for t in g.act(torch.from_numpy(obs).cuda(), torch.from_numpy(u).cuda())]
        g.check()
        compare(ref, *out, taps=g.read_activation if flags & 1 else None)
        g.close()


@pytest.mark.parametrize("name,b", [("nature_cnn_b8192", 200), ("student_cnn_b8192", 141), ("impala_resnet_b16384", 9),
                                    ("lunarlander_mlp", 300)])
def test_single_fma_requantiser_and_the_division_it_replaces_give_the_same_bits(name, b):
    """At create every requantising layer of a tensor-core plan searches, per output channel, the
    constants of a one-fma requantiser that equals the defining expression on every int32
    accumulator.  The workloads' conv layers find them (the plan says so); with the test flag the
    search is skipped and the verified three-step division runs instead.  Both against the oracle,
    tensor by tensor."""
    import paper_2211_15023_b200 as P
    pol = calibrated(name, 64)
    obs, u = W.observations(name, b), W.uniforms(name, b)
    ref = oracle.forward(pol, obs, u)
    for flags in (P.FLAG_KEEP_ACTIVATIONS | P.FLAG_TAP_FUSED, P.FLAG_KEEP_ACTIVATIONS | P.FLAG_TAP_FUSED | P.FLAG_TEST_NO_AFFINE, 0):
        g = P.Policy(pol, b, flags=flags)
        plan = g.info()["plan"]
        if "tc_gemm" in plan or "conv1_frames" in plan:
            if flags & P.FLAG_TEST_NO_AFFINE:
                assert "single-fma" not in plan and "3-step divide verified" in plan, plan
            else:  # the conv layers find their constants; a wide fc layer may have a channel without
                assert plan.count("single-fma requantiser verified") >= 2, plan
        out = [t.cpu().numpy() for t in g.act(torch.from_numpy(obs).cuda(), torch.from_numpy(u).cuda())]
        g.check()
        compare(ref, *out, taps=g.read_activation if flags & 1 else None)
        g.close()


@pytest.mark.parametrize("case", ["coarse_scale", "fine_scale", "bias_far_below", "bias_far_above", "tiny_weight_scale"])
def test_requantiser_constants_at_the_edges_of_their_search(case):
    """The band of accumulators the single-fma constants are checked on comes from the layer's
    scales and biases.  Scales and biases far from what calibration gives (every output saturated,
    every output in a handful of codes, bands that touch the int32 limits) must either find
    constants that still equal the defining expression or leave the layer on the division; the
    oracle decides, tensor by tensor, with and without the search."""
    import copy
    import paper_2211_15023_b200 as P
    name, b = "student_cnn_b8192", 33
    pol = copy.deepcopy(calibrated(name, 64))
    l1, l2 = pol["layers"][1], pol["layers"][2]
    if case == "coarse_scale":          # nearly everything rounds to -1, 0 or 1
        l1["s_out"] = np.float32(l1["s_out"] * 90.0)
    elif case == "fine_scale":          # nearly everything saturates
        l1["s_out"] = np.float32(l1["s_out"] / 500.0)
    elif case == "bias_far_below":      # ReLU leaves zeros only
        l1["bias"] = (l1["bias"] - np.float32(1000.0) * l1["s_out"]).astype(np.float32)
    elif case == "bias_far_above":      # every code is 127
        l1["bias"] = (l1["bias"] + np.float32(1000.0) * l1["s_out"]).astype(np.float32)
    else:                               # a band of accumulators wider than int32
        l1["s_w"] = (l1["s_w"] * np.float32(1e-7)).astype(np.float32)
    l2["s_in"] = l1["s_out"]
    obs, u = W.observations(name, b), W.uniforms(name, b)
    ref = oracle.forward(pol, obs, u)
    for flags in (1, 0, 1 | P.FLAG_TEST_NO_AFFINE):
        g = P.Policy(pol, b, flags=flags)
        out = [t.cpu().numpy() for t in g.act(torch.from_numpy(obs).cuda(), torch.from_numpy(u).cuda())]
        g.check()
        compare(ref, *out, taps=g.read_activation if flags & 1 else None)
        g.close()

