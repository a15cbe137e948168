#!/usr/bin/env python
"""Benchmark of the int8 Actor policy-inference path: states/s on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference] [--workload NAME]

A step is one `accerl_policy_act` call: input quantisation, every layer of the network and
the sampler, on one batch of synthetic states.  The default workload is the Nature-CNN policy
(the paper's "Original" network of the table "network architecture and inference time") at
batch 8192; the other workloads are timed briefly and reported under "other_workloads".
With N > 1 (torchrun) every rank runs the same batch size on its own GPU (states are
independent, there is no exchange step) and the time is the maximum over ranks.
Prints ONE JSON line on rank 0.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import workloads as W  # noqa: E402

METRIC = "int8 policy-inference states/sec"
UNIT = "states/s"
DEFAULT_WORKLOAD = "nature_cnn_b8192"
OUT_BYTES = lambda a: 4 * a + 8          # noqa: E731  logits + action + logp per state


def peaks() -> dict:
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return dict(hbm_gbs=p["hbm_gbs"], bf16_tflops=p["bf16_tflops"],
                    bf16_tflops_sustained=p.get("bf16_tflops_sustained", p["bf16_tflops"]),
                    source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, bf16_tflops_sustained=1400.0, source="fallback")


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.rows, self.proc, self.index = [], None, index

    def __enter__(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.Q,
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None
        return self

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([t.strip() for t in line.split(",")])

    def __exit__(self, *a):
        if self.proc:
            self.proc.terminate()
            try:
                self.proc.wait(timeout=5)
            except subprocess.TimeoutExpired:
                self.proc.kill()

    def summary(self) -> dict:
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            try:
                sm.append(float(r[0]))
                mx.append(float(r[1]))
            except (ValueError, IndexError):
                continue
            for n, v in zip(names, r[4:8]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        if not sm:
            return dict(sm_mhz=None, sm_max_mhz=None, reasons=[], samples=0)
        busy = [v for v in sm if v >= 0.5 * max(sm)]
        return dict(sm_mhz=statistics.median(busy), sm_max_mhz=max(mx), reasons=sorted(reasons),
                    samples=len(sm))


# plain-ALU issue peak: SMs x 4 schedulers x 32 lanes x SM clock (lane-instructions per second)
def alu_peak(sm_count: int, sm_mhz: float) -> float:
    return sm_count * 4 * 32 * sm_mhz * 1e6


def int8_probe(P) -> dict:
    """Measured cost of the int8 tensor-core instruction (M = 128, K = 32 bytes) by width N, with
    operands resident in shared memory: cycles per MMA and CTA, and chip-wide TOP/s.  The N = 256
    figure is the measured dense int8 peak the tensor roofline is taken against."""
    out = {}
    for n in (16, 32, 64, 128, 256):
        warps = 2 if n == 256 else 4
        r = P.tc_probe_i8(n, warps, 4096, 148)
        out["n%d" % n] = dict(cycles_per_mma=round(r["cycles_per_mma"], 2), tops=round(r["tops"], 1))
    return out


def latency_profile(P, torch, name: str, device: int, calls: int = 60) -> dict:
    """Latency of single act calls at the workload's batch: CUDA events around every call, one call
    at a time.  warm: the same input buffer every call; cold: a buffer larger than L2 is written
    between calls (outside the timed events), so inputs, weights and workspace come from HBM."""
    batch = W.config(name)["batch"]
    g = P.Policy(W.drawn_int8_policy(name), batch, device=device)
    dev = "cuda:%d" % device
    obs = torch.from_numpy(W.observations(name, batch)).to(dev)
    u = torch.from_numpy(W.uniforms(name, batch)).to(dev)
    out = g.act(obs, u)
    flush = torch.empty(192 << 20, dtype=torch.uint8, device=dev)
    stream = torch.cuda.current_stream(obs.device)
    res = {}
    for mode in ("warm", "cold"):
        for _ in range(10):
            g.act(obs, u, out, stream.cuda_stream)
        torch.cuda.synchronize()
        ts = []
        for _ in range(calls):
            if mode == "cold":
                flush.fill_(1)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            g.act(obs, u, out, stream.cuda_stream)
            e1.record(stream)
            torch.cuda.synchronize()
            ts.append(e0.elapsed_time(e1) * 1e3)
        ts = np.sort(np.array(ts))
        res[mode] = dict(p10_us=float(np.percentile(ts, 10)), p50_us=float(np.percentile(ts, 50)),
                         p90_us=float(np.percentile(ts, 90)))
    g.check()
    g.close()
    res["calls"] = calls
    res["batch"] = batch
    return res


def vtrace_line(P, torch, pk: dict, device: int, n_steps: int = 16, batch: int = 8192) -> dict:
    """The V-trace kernel on [n_steps, batch] rollouts: 4 input + 2 output floats per element."""
    dev = "cuda:%d" % device
    r = W.rollouts(n_steps, batch, seed=1)
    t = {k: torch.from_numpy(r[k]).to(dev) for k in ("logp_smaller", "logp_original", "rewards", "values",
                                                      "bootstrap")}
    args = (t["logp_smaller"], t["logp_original"], t["rewards"], t["values"], t["bootstrap"], r["gamma"])
    out = (torch.empty_like(t["values"]), torch.empty_like(t["values"]))
    stream = torch.cuda.current_stream(out[0].device).cuda_stream
    for _ in range(5):
        P.vtrace(*args, stream=stream, out=out, checked=False)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    reps = 200
    e0.record()
    for _ in range(reps):
        P.vtrace(*args, stream=stream, out=out, checked=False)
    e1.record()
    torch.cuda.synchronize()
    us = e0.elapsed_time(e1) / reps * 1e3
    nbytes = 4 * (6 * n_steps * batch + batch)
    gbs = nbytes / (us * 1e-6) / 1e9
    return dict(n_steps=n_steps, batch=batch, us_per_call=us, bytes=nbytes, achieved_gbs=gbs,
                frac_of_hbm=gbs / pk["hbm_gbs"],
                note="launch-latency bound at this size: %.1f MB per call" % (nbytes / 1e6))


def algorithmic(name: str, batch: int) -> dict:
    """Algorithmic work of one step: 2 x useful MACs, and input + output bytes per state.

    For a 2:4-pruned workload half of the dense MACs multiply structural zeros and are no
    algorithmic work; `ops_dense_executed` is what a dense contraction still performs."""
    a = W.n_actions(name)
    dense = 2 * W.macs_per_state(name) * batch
    return dict(ops=dense // 2 if W.config(name)["prune24"] else dense, ops_dense_executed=dense,
                bytes=(W.input_bytes_per_state(name) + 4 + OUT_BYTES(a)) * batch)


# dram__bytes_read.sum + dram__bytes_write.sum of one launch / states of that launch, from
# profiles/ncu_full_nature_cnn_b6144.md (batch 6144: 173.47 MB read + 50.96 MB written by the
# first conv with the input stage inside)
_CONV1 = "conv1_frames_kernel[single-fma requantiser verified][frames quantised inside]"
NCU_DRAM_BYTES_PER_STATE = {("nature_cnn_b8192", _CONV1): (173472000 + 50957824) / 6144}
# warp-level instructions executed per state by the dominant kernel, from the same capture
NCU_WARP_INST_PER_STATE = {("nature_cnn_b8192", _CONV1): 28499170 / 6144}


def launch_work(name: str, plan: str, batch: int) -> list:
    """Per launch of the plan: kernel name, int8 ops (2 x MACs) and algorithmic bytes."""
    c = W.config(name)
    layers = c["layers"]
    a = W.n_actions(name)

    def tensor_bytes(i):  # int8 output of layer i, or the quantised input for i = -1
        if i < 0:
            return int(np.prod(c["in_shape"]))
        oh, ow = W.out_hw(layers[i])
        return layers[i]["out_c"] * oh * ow

    out = []
    for line in plan.strip().splitlines():
        if not line.startswith("launch "):
            continue
        head, rest = line.split(" covers ", 1)
        kernel = head.split(": ", 1)[1]
        covers = rest.split(" (")[0]
        ops, nbytes, first_in, last_out = 0, 0, None, None
        for part in covers.split("+"):
            part = part.strip()
            if part == "ingest":
                nbytes += W.input_bytes_per_state(name)
                last_out = -1
            elif part == "sample":
                nbytes += 4 + 8  # uniform in, action + logp out (logits counted with their layer)
            else:
                idx = part.replace("layers", "").replace("layer", "").strip()
                lo, hi = (int(t) for t in idx.split("-")) if "-" in idx else (int(idx), int(idx))
                for i in range(lo, hi + 1):
                    l = layers[i]
                    if l["kind"] != "maxpool":
                        oh, ow = W.out_hw(l)
                        ops += 2 * oh * ow * l["out_c"] * l["in_c"] * l["kh"] * l["kw"]
                        if l["skip_from"] >= 0 and not (lo <= l["skip_from"] <= hi):
                            nbytes += tensor_bytes(l["skip_from"])
                if first_in is None and last_out is None:
                    first_in = lo - 1
                last_out = hi
        if first_in is not None:
            nbytes += tensor_bytes(first_in)
        if last_out is not None:
            nbytes += 4 * a if last_out == len(layers) - 1 else tensor_bytes(last_out)
        out.append(dict(kernel=kernel, covers=covers, ops=ops * batch, bytes=nbytes * batch))
    return out


def run_reference(args) -> None:
    """The CPU oracle, as it stands, on a bounded sample of the same workload."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    name = args.workload
    pol = W.drawn_int8_policy(name)
    sample = min(W.config(name)["batch"], args.ref_sample)
    obs, u = W.observations(name, sample), W.uniforms(name, sample)
    for _ in range(args.warmup):
        oracle.forward(pol, obs, u, keep=False)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        oracle.forward(pol, obs, u, keep=False)
    dt = (time.perf_counter() - t0) / args.steps
    cores = os.cpu_count()
    v = sample / dt
    desc = "%d states of %s per step (oracle/accerl_oracle.c, OpenMP over states)" % (sample, name)
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": v, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "int8",
        "data": "synthetic", "config": {"workload": name, "batch": sample},
        "cpu_baseline": {"value": v, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": desc},
        "e2e": {"value": v, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def max_over_ranks(ms: float, dist, device) -> float:
    """Slowest rank's time: the job's step time when every rank runs its own replica."""
    if dist is None:
        return ms
    import torch
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_value(batch_per_rank: int, world: int, ms: float) -> float:
    """Whole-job states/s: all ranks' states over the slowest rank's time."""
    return batch_per_rank * world / (ms * 1e-3)


def time_workload(P, torch, name, batch, steps, warmup, n_buffers, device, dist=None, clocks=False):
    """Times `steps` act calls with CUDA events on the launching stream; returns a dict."""
    pol = W.drawn_int8_policy(name)
    g = P.Policy(pol, batch, device=device)
    a = g.n_actions
    obs_np = W.observations(name, batch)
    # distinct device copies of the input so that consecutive steps never re-read warm lines
    obs = [torch.from_numpy(np.roll(obs_np, i, axis=0)).to("cuda:%d" % device) for i in range(n_buffers)]
    u = torch.from_numpy(W.uniforms(name, batch)).to("cuda:%d" % device)
    out = (torch.empty((batch, a), dtype=torch.float32, device=u.device),
           torch.empty(batch, dtype=torch.int32, device=u.device),
           torch.empty(batch, dtype=torch.float32, device=u.device))
    stream = torch.cuda.current_stream(u.device)
    for i in range(warmup):
        g.act(obs[i % n_buffers], u, out, stream.cuda_stream)
    torch.cuda.synchronize()
    if dist is not None:
        dist.barrier()
        torch.cuda.synchronize()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    sampler = ClockSampler(device) if clocks else None
    if sampler:
        sampler.__enter__()
        time.sleep(0.25)
    ev0.record(stream)
    for i in range(steps):
        g.act(obs[i % n_buffers], u, out, stream.cuda_stream)
    ev1.record(stream)
    torch.cuda.synchronize()
    if sampler:
        time.sleep(0.15)
        sampler.__exit__()
    ms = ev0.elapsed_time(ev1) / steps
    ms = max_over_ranks(ms, dist, u.device)
    if dist is not None:
        dist.barrier()
    g.check()
    info = g.info()
    # per-launch device times (a second pass over the same steps with events around each launch)
    per = np.zeros(info["launches_per_act"], np.float64)
    for i in range(steps):
        per += g.act_timed(obs[i % n_buffers], u, out, stream.cuda_stream)
    per /= steps
    # one more step on the un-rotated batch, outside every timed region: what the parity check reads
    g.act(obs[0], u, out, stream.cuda_stream)
    torch.cuda.synchronize()
    res = dict(ms=ms, info=info, per_launch_ms=per, policy=g, obs=obs_np, u=u, out=out,
               check_out=tuple(t.cpu().numpy() for t in out),
               clocks=sampler.summary() if sampler else None)
    return res


def main() -> None:
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD, choices=list(W.CONFIGS))
    ap.add_argument("--ref-sample", type=int, default=256)
    ap.add_argument("--cpu-sample", type=int, default=2048)
    ap.add_argument("--batch", type=int, default=0,
                    help="override the workload's batch (profiling captures on a small case only)")
    ap.add_argument("--no-cpu", action="store_true", help="skip the CPU-oracle baseline leg")
    ap.add_argument("--no-others", action="store_true", help="skip the brief runs of other workloads")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3)
    if args.impl == "reference":
        run_reference(args)
        return

    import torch
    import paper_2211_15023_b200 as P
    P.library()  # fails loudly if the CUDA library is missing
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    dist = None
    if world > 1:
        import torch.distributed as dist
        torch.cuda.set_device(local)
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    torch.cuda.set_device(local)

    name = args.workload
    batch = args.batch or W.config(name)["batch"]
    in_bytes = W.input_bytes_per_state(name) * batch
    n_buffers = 3 if in_bytes * 3 < (8 << 30) else 2
    r = time_workload(P, torch, name, batch, args.steps, args.warmup, n_buffers, local, dist,
                      clocks=(rank == 0))
    ms = r["ms"]
    g = r["policy"]
    clocks = r["clocks"]
    check_out = r["check_out"]
    value = job_value(batch, world, ms)

    # ---- end to end through the host-buffer entry point (pinned memory, copies timed)
    a = g.n_actions
    obs_pin = torch.from_numpy(r["obs"]).pin_memory()
    u_pin = r["u"].cpu().pin_memory()
    out_pin = (torch.empty((batch, a), dtype=torch.float32).pin_memory(),
               torch.empty(batch, dtype=torch.int32).pin_memory(),
               torch.empty(batch, dtype=torch.float32).pin_memory())
    stream = torch.cuda.current_stream()
    e2e_steps = max(3, min(args.steps, 10))
    for _ in range(3):
        g.act_host(obs_pin, u_pin, out_pin, stream.cuda_stream)
    if dist is not None:
        dist.barrier()
    torch.cuda.synchronize()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ev0.record(stream)
    for _ in range(e2e_steps):
        g.act_host(obs_pin, u_pin, out_pin, stream.cuda_stream)
    ev1.record(stream)
    torch.cuda.synchronize()
    e2e_ms = ev0.elapsed_time(ev1) / e2e_steps
    e2e_ms = max_over_ranks(e2e_ms, dist, "cuda")
    if rank != 0:
        if dist is not None:
            dist.barrier()
            dist.destroy_process_group()
        return

    # ---- roofline of the dominant kernel (largest share of the per-launch device time)
    pk = peaks()
    work = launch_work(name, r["info"]["plan"], batch)
    per = r["per_launch_ms"]
    top = int(np.argmax(per))
    # dense int8 peak: measured by the library's probe (N = 256 MMAs back to back, operands resident
    # in shared memory, all SMs); the nominal figure 2 x measured bf16 burst is reported beside it
    probe = int8_probe(P)
    int8_peak_nominal = 2.0 * pk["bf16_tflops"]
    int8_peak = probe["n256"]["tops"]
    t_tensor = work[top]["ops"] / (int8_peak * 1e12)
    t_hbm = work[top]["bytes"] / (pk["hbm_gbs"] * 1e9)
    if t_tensor >= t_hbm:
        achieved = work[top]["ops"] / (per[top] * 1e-3) / 1e12
        roof = dict(bound="tensor", achieved=achieved, peak=int8_peak, unit="TOP/s",
                    frac=achieved / int8_peak)
    else:
        achieved = work[top]["bytes"] / (per[top] * 1e-3) / 1e9
        roof = dict(bound="hbm", achieved=achieved, peak=pk["hbm_gbs"], unit="GB/s",
                    frac=achieved / pk["hbm_gbs"])
    # DRAM bytes per launch from the committed ncu capture of this kernel (profiles/), measured on
    # a smaller batch and scaled by the states processed; None for kernels without a capture
    per_state = NCU_DRAM_BYTES_PER_STATE.get((name, work[top]["kernel"]))
    traffic = None if per_state is None else per_state * batch
    roof.update(traffic=traffic, kernel=work[top]["kernel"], covers=work[top]["covers"],
                kernel_ms=float(per[top]), share=float(per[top] / per.sum()),
                peak_source="measured int8 probe (tcgen05.mma kind::i8, M=128 N=256)" if roof["bound"] == "tensor"
                else pk["source"])
    # third bound: plain instruction issue (warp instructions of the committed ncu capture x 32 lanes)
    wi = NCU_WARP_INST_PER_STATE.get((name, work[top]["kernel"]))
    sm_mhz = (clocks or {}).get("sm_mhz") or 1965.0
    if wi is not None:
        lane_rate = wi * 32 * batch / (per[top] * 1e-3)
        roof["alu"] = dict(warp_inst_per_state=wi, achieved_lane_inst_per_s=lane_rate,
                           peak=alu_peak(148, sm_mhz), frac=lane_rate / alu_peak(148, sm_mhz),
                           note="148 SMs x 4 schedulers x 32 lanes x SM clock")
    whole = algorithmic(name, batch)
    t_floor_tensor = whole["ops"] / (int8_peak * 1e12) * 1e3
    t_floor_hbm = whole["bytes"] / (pk["hbm_gbs"] * 1e9) * 1e3
    step_floor_ms = max(t_floor_tensor, t_floor_hbm)
    step_floor_nominal_ms = max(whole["ops"] / (int8_peak_nominal * 1e12) * 1e3, t_floor_hbm)
    launches = [dict(kernel=w["kernel"], covers=w["covers"], ms=float(m)) for w, m in zip(work, per)]

    # ---- the other workloads, briefly (kernel-resident timing only)
    others = {}
    if not args.no_others and world == 1:
        del r
        g.close()
        for other in W.CONFIGS:
            if other == name:
                continue
            ob = W.config(other)["batch"]
            nb = 3 if W.input_bytes_per_state(other) * ob * 3 < (8 << 30) else 2
            o = time_workload(P, torch, other, ob, max(5, args.steps // 2), 3, nb, local)
            w = algorithmic(other, ob)
            floor = max(w["ops"] / (int8_peak * 1e12), w["bytes"] / (pk["hbm_gbs"] * 1e9)) * 1e3
            floor_nom = max(w["ops"] / (int8_peak_nominal * 1e12), w["bytes"] / (pk["hbm_gbs"] * 1e9)) * 1e3
            others[other] = dict(batch=ob, ms_per_step=o["ms"], states_per_s=ob / (o["ms"] * 1e-3),
                                 launches=o["info"]["launches_per_act"],
                                 ops_per_state=w["ops"] // ob,
                                 ops_per_state_dense_executed=w["ops_dense_executed"] // ob,
                                 frac_of_step_roofline=floor / o["ms"],
                                 frac_of_step_roofline_nominal_int8=floor_nom / o["ms"])
            o["policy"].close()
        # latency of single calls for the small-batch configurations, and the V-trace kernel
        for small in ("cartpole_mlp", "lunarlander_mlp", "nature_cnn_b160"):
            others[small]["latency"] = latency_profile(P, torch, small, local)
        others["vtrace"] = vtrace_line(P, torch, pk, local)

    # ---- CPU oracle on a bounded sample of the same workload (reported baseline)
    # and the parity of what was timed: the GPU outputs of those states (same policy, same plan,
    # full batch) against the oracle's, outside the timed region
    cpu = parity = None
    if not args.no_cpu:
        import oracle
        sample = min(batch, args.cpu_sample)
        pol = W.drawn_int8_policy(name)
        so, su = W.observations(name, batch)[:sample], W.uniforms(name, batch)[:sample]
        oracle.forward(pol, so[:8], su[:8], keep=False)
        t0 = time.perf_counter()
        ref = oracle.forward(pol, so, su, keep=False)
        cpu_dt = time.perf_counter() - t0
        cpu = dict(value=sample / cpu_dt, unit=UNIT, cores=os.cpu_count(), kind="oracle",
                   sample="first %d states of the %d-state batch, one pass" % (sample, batch))
        # the same oracle on one thread (a smaller sample; work per state is constant)
        try:
            import ctypes
            gomp = ctypes.CDLL("libgomp.so.1")
            n_thr = gomp.omp_get_max_threads()
            gomp.omp_set_num_threads(1)
            one = max(8, sample // 32)
            t0 = time.perf_counter()
            oracle.forward(pol, so[:one], su[:one], keep=False)
            cpu["single_thread"] = dict(value=one / (time.perf_counter() - t0), unit=UNIT, sample="%d states" % one)
            gomp.omp_set_num_threads(n_thr)
            cpu["cores"] = int(n_thr)
        except OSError:
            pass
        lg, ac, lp = (a[:sample] for a in check_out)
        diff = ac != ref["actions"]
        same = ~diff
        lp_err = np.abs(lp[same].astype(np.float64) - ref["logp"][same])
        lp_tol = 1e-6 + 1e-5 * np.abs(ref["logp"][same])
        parity = dict(states=int(sample), logits_mismatch=int((lg != ref["logits"]).sum()),
                      action_mismatch=int(diff.sum()),
                      action_mismatch_near_edge=int((diff & (ref["margin"] < 1e-5)).sum()),
                      logp_out_of_tolerance=int((lp_err > lp_tol).sum()),
                      logp_max_abs_err=float(lp_err.max()) if lp_err.size else 0.0,
                      note="timed policy and plan, full batch; logits compared bit for bit")

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "int8", "data": "synthetic",
        "config": {"workload": name, "batch_per_gpu": batch,
                   "l2": "inputs larger than L2: %d input buffers of %.0f MB rotate" %
                         (n_buffers, in_bytes / 1e6),
                   "parallelism": "replicas" if world > 1 else "single"},
        "clocks": clocks,
        "e2e": {"value": job_value(batch, world, e2e_ms), "unit": UNIT, "ms_per_step": e2e_ms,
                "h2d_bytes_per_step": in_bytes + 4 * batch,
                "d2h_bytes_per_step": OUT_BYTES(a) * batch},
        "gpu_launches": int(len(per) * args.steps),
        "roofline": roof,
        "int8_probe": probe,
        "step_roofline": {"floor_ms": step_floor_ms, "frac": step_floor_ms / ms,
                          "floor_tensor_ms": t_floor_tensor, "floor_hbm_ms": t_floor_hbm,
                          "int8_peak_tops": int8_peak, "int8_peak_source": "measured probe, N=256",
                          "floor_ms_nominal_int8": step_floor_nominal_ms,
                          "frac_nominal_int8": step_floor_nominal_ms / ms,
                          "int8_peak_nominal_tops": int8_peak_nominal,
                          "ops_per_state": whole["ops"] // batch,
                          "ops_per_state_dense_executed": whole["ops_dense_executed"] // batch,
                          "bytes_per_state": whole["bytes"] // batch},
        "launches": launches,
        "cpu_baseline": cpu,
        "parity": parity,
        "other_workloads": others,
    }
    print(json.dumps(line))
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
