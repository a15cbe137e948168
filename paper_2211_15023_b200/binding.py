"""ctypes binding of libaccerl.so: same names and argument order as include/accerl.h."""
from __future__ import annotations

import ctypes as C
import os

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB = None

FLAG_KEEP_ACTIVATIONS = 1
FLAG_FORCE_GENERIC = 2
FLAG_TAP_FUSED = 4
FLAG_VALUE_HEAD = 8
FLAG_TEST_NO_FASTDIV = 16
FLAG_TEST_NO_AFFINE = 32
RELU_IN, RELU_OUT, LOGITS = 1, 2, 4
_KINDS = {"conv": 0, "fc": 1, "maxpool": 2}
STATUS = {0: "OK", 1: "INVALID_ARG", 2: "UNSUPPORTED", 3: "BATCH_TOO_LARGE", 4: "OOM", 5: "CUDA",
          6: "TIMEOUT"}


class AccerlError(RuntimeError):
    def __init__(self, status: int, message: str):
        super().__init__("accerl %s: %s" % (STATUS.get(status, status), message))
        self.status = status


class LayerDesc(C.Structure):
    _fields_ = [("kind", C.c_int32), ("flags", C.c_uint32),
                ("in_c", C.c_int32), ("in_h", C.c_int32), ("in_w", C.c_int32),
                ("out_c", C.c_int32), ("kh", C.c_int32), ("kw", C.c_int32),
                ("stride", C.c_int32), ("pad", C.c_int32),
                ("s_in", C.c_float), ("s_out", C.c_float),
                ("w", C.c_void_p), ("s_w", C.c_void_p), ("bias", C.c_void_p),
                ("skip_from", C.c_int32), ("skip_mul", C.c_void_p)]


class LayerFp32(C.Structure):
    _fields_ = [("kind", C.c_int32), ("flags", C.c_uint32),
                ("in_c", C.c_int32), ("in_h", C.c_int32), ("in_w", C.c_int32),
                ("out_c", C.c_int32), ("kh", C.c_int32), ("kw", C.c_int32),
                ("stride", C.c_int32), ("pad", C.c_int32),
                ("w", C.c_void_p), ("bias", C.c_void_p), ("skip_from", C.c_int32)]


def library_path() -> str:
    return os.path.join(_HERE, "libaccerl.so")


def library() -> C.CDLL:
    """Load libaccerl.so; there is no fallback if it has not been built."""
    global _LIB
    if _LIB is None:
        path = library_path()
        if not os.path.exists(path):
            raise ImportError("%s is missing: build it with `python -m paper_2211_15023_b200.build`"
                              % path)
        lib = C.CDLL(path)
        vp, i32, f32 = C.c_void_p, C.c_int32, C.c_float
        lib.accerl_policy_create.argtypes = [C.POINTER(vp), i32, C.POINTER(i32), f32,
                                             C.POINTER(LayerDesc), i32, i32, C.c_uint32, i32]
        lib.accerl_policy_act.argtypes = [vp, vp, vp, i32, vp, vp, vp, vp]
        lib.accerl_policy_act_timed.argtypes = [vp, vp, vp, i32, vp, vp, vp, vp, vp, i32]
        lib.accerl_policy_act_noalloc.argtypes = [vp, vp, vp, i32, vp, vp, vp, vp]
        lib.accerl_policy_act_host.argtypes = [vp, vp, vp, i32, vp, vp, vp, vp]
        lib.accerl_policy_read_activation.argtypes = [vp, i32, i32, vp, C.c_size_t]
        lib.accerl_policy_check.argtypes = [vp]
        lib.accerl_policy_info.argtypes = [vp, i32, C.POINTER(i32), C.POINTER(C.c_size_t),
                                           C.POINTER(i32), C.c_char_p, C.c_size_t]
        lib.accerl_policy_act_ex.argtypes = [vp, vp, vp, i32, vp, vp, vp, vp, vp, vp]
        lib.accerl_policy_kl.argtypes = [vp, vp, i32, i32, vp, vp, vp]
        lib.accerl_policy_act_mixed.argtypes = [vp, vp, vp, vp, vp, f32, i32, vp, vp, vp, vp, vp, vp, vp]
        lib.accerl_vtrace.argtypes = [vp, vp, vp, vp, vp, vp, i32, i32, f32, f32, f32, vp, vp, vp]
        for f in ("accerl_policy_act_ex", "accerl_policy_kl", "accerl_policy_act_mixed", "accerl_vtrace"):
            getattr(lib, f).restype = C.c_int
        lib.accerl_policy_create_fp32.argtypes = [C.POINTER(vp), i32, C.POINTER(i32), C.POINTER(LayerFp32), i32, vp,
                                                  i32, i32, i32, C.c_uint32, i32]
        lib.accerl_policy_create_fp32.restype = C.c_int
        lib.accerl_policy_export.argtypes = [vp, i32, vp, C.c_size_t, vp, vp, C.POINTER(f32), C.POINTER(f32)]
        lib.accerl_policy_export.restype = C.c_int
        lib.accerl_policy_selftest_wait.argtypes = [vp, i32, vp]
        lib.accerl_policy_selftest_wait.restype = C.c_int
        lib.accerl_tc_probe_i8.argtypes = [i32, i32, i32, i32, i32, i32, i32, i32, C.POINTER(f32), C.POINTER(f32)]
        lib.accerl_tc_probe_i8.restype = C.c_int
        lib.accerl_policy_destroy.argtypes = [vp]
        lib.accerl_policy_destroy.restype = None
        lib.accerl_last_error.restype = C.c_char_p
        lib.accerl_version.restype = C.c_char_p
        for f in ("create", "act", "act_timed", "act_noalloc", "act_host", "read_activation", "check", "info"):
            getattr(lib, "accerl_policy_" + f).restype = C.c_int
        _LIB = lib
    return _LIB


def _check(status: int):
    if status != 0:
        raise AccerlError(status, library().accerl_last_error().decode())


def _out_hw(l):
    if l["kind"] == "fc":
        return 1, 1
    return ((l["in_h"] + 2 * l["pad"] - l["kh"]) // l["stride"] + 1,
            (l["in_w"] + 2 * l["pad"] - l["kw"]) // l["stride"] + 1)


def tc_probe_i8(n: int, issuing_warps: int = 1, mmas_per_warp: int = 4096, ctas: int = 148,
                layout: int = 128, a_shift_rows: int = 0, commit_every: int = 0, device: int = 0) -> dict:
    """accerl_tc_probe_i8: cost of an M = 128, N = n int8 MMA; returns ms, cycles_per_mma, tops."""
    ms, cyc = C.c_float(), C.c_float()
    _check(library().accerl_tc_probe_i8(device, n, issuing_warps, mmas_per_warp, ctas, layout, a_shift_rows, commit_every,
                                        C.byref(ms), C.byref(cyc)))
    ops = ctas * issuing_warps * mmas_per_warp * 2.0 * 128 * n * 32
    return dict(n=n, issuing_warps=issuing_warps, mmas_per_warp=mmas_per_warp, ctas=ctas, layout=layout, a_shift_rows=a_shift_rows, commit_every=commit_every,
                ms=ms.value, cycles_per_mma=cyc.value, tops=ops / (ms.value * 1e-3) / 1e12)


def _stream_of(t, stream):
    import torch
    return torch.cuda.current_stream(t.device).cuda_stream if stream is None else stream


def kl(logits_original, logits_smaller, stream=None):
    """accerl_policy_kl on two CUDA fp32 [B, A] tensors; returns (kl [B], mean_max [2]) tensors."""
    import torch
    assert logits_original.shape == logits_smaller.shape and logits_original.is_contiguous() and \
        logits_smaller.is_contiguous() and logits_original.dtype == logits_smaller.dtype == torch.float32
    b, a = logits_original.shape
    out = torch.empty(b, dtype=torch.float32, device=logits_original.device)
    stats = torch.empty(2, dtype=torch.float32, device=logits_original.device)
    _check(library().accerl_policy_kl(logits_original.data_ptr(), logits_smaller.data_ptr(), b, a,
                                      out.data_ptr(), stats.data_ptr(), _stream_of(out, stream)))
    return out, stats


def vtrace(logp_smaller, logp_original, rewards, values, bootstrap, gamma, rho_hat=1.0, c_hat=1.0,
           discounts=None, stream=None, out=None, checked=True):
    """accerl_vtrace on CUDA fp32 time-major [n, B] tensors; returns (vs, adv) tensors [n, B]."""
    import torch
    n, b = logp_smaller.shape
    if checked:
        for t in (logp_smaller, logp_original, rewards, values):
            assert t.shape == (n, b) and t.is_contiguous() and t.dtype == torch.float32 and t.is_cuda
        assert bootstrap.shape == (b,) and bootstrap.is_contiguous() and bootstrap.dtype == torch.float32
        assert discounts is None or (discounts.shape == (n, b) and discounts.is_contiguous())
    vs, adv = (torch.empty_like(values), torch.empty_like(values)) if out is None else out
    _check(library().accerl_vtrace(logp_smaller.data_ptr(), logp_original.data_ptr(), rewards.data_ptr(),
                                   values.data_ptr(), bootstrap.data_ptr(),
                                   None if discounts is None else discounts.data_ptr(), n, b,
                                   float(gamma), float(rho_hat), float(c_hat), vs.data_ptr(),
                                   adv.data_ptr(), _stream_of(vs, stream)))
    return vs, adv


def act_mixed(smaller, original, obs, uniforms, select_uniforms, alpha, stream=None):
    """accerl_policy_act_mixed; returns dict(logits, actions, logp, entropy, use_smaller[, value])."""
    import torch
    b, dev = int(obs.shape[0]), obs.device
    out = dict(logits=torch.empty((b, smaller.n_actions), dtype=torch.float32, device=dev),
               actions=torch.empty(b, dtype=torch.int32, device=dev),
               logp=torch.empty(b, dtype=torch.float32, device=dev),
               entropy=torch.empty(b, dtype=torch.float32, device=dev),
               use_smaller=torch.empty(b, dtype=torch.uint8, device=dev))
    if smaller.value_head and original.value_head:
        out["value"] = torch.empty(b, dtype=torch.float32, device=dev)
    _check(library().accerl_policy_act_mixed(
        smaller._h, original._h, obs.data_ptr(), uniforms.data_ptr(), select_uniforms.data_ptr(),
        float(alpha), b, out["logits"].data_ptr(), out["actions"].data_ptr(), out["logp"].data_ptr(),
        out["value"].data_ptr() if "value" in out else None, out["entropy"].data_ptr(),
        out["use_smaller"].data_ptr(), _stream_of(obs, stream)))
    return out


class Policy:
    """An int8 policy resident on one GPU.

    ``policy`` is a dict with ``in_kind`` ("u8" | "f32"), ``in_shape`` (C, H, W),
    ``s_input`` and ``layers``: dicts with kind, in_c, in_h, in_w, out_c, kh, kw, stride, pad,
    relu_in, relu_out, logits, skip_from, s_in, s_out and numpy arrays w (int8 OIHW), s_w, bias,
    skip_mul (or None).
    """

    @classmethod
    def from_fp32(cls, in_kind: str, in_shape, layers, params, calib_obs, max_batch: int,
                  prune24: bool = False, flags: int = 0, device: int = 0) -> "Policy":
        """accerl_policy_create_fp32: quantise and calibrate on the device.  ``layers`` are
        architecture dicts, ``params`` the matching fp32 {w, bias} (None for max-pool)."""
        lib = library()
        self = cls.__new__(cls)
        self._h = C.c_void_p()
        n = len(layers)
        descs = (LayerFp32 * n)()
        keep = []
        for i, (l, pr) in enumerate(zip(layers, params)):
            d = descs[i]
            d.kind = _KINDS[l["kind"]]
            d.flags = (RELU_IN if l["relu_in"] else 0) | (RELU_OUT if l["relu_out"] else 0) | \
                (LOGITS if l["logits"] else 0)
            for k in ("in_c", "in_h", "in_w", "out_c", "kh", "kw", "stride", "pad", "skip_from"):
                setattr(d, k, int(l[k]))
            if pr is not None:
                w, b = np.ascontiguousarray(pr["w"], np.float32), np.ascontiguousarray(pr["bias"], np.float32)
                keep += [w, b]
                d.w, d.bias = w.ctypes.data, b.ctypes.data
        shape = (C.c_int32 * 3)(*[int(v) for v in in_shape])
        calib = np.ascontiguousarray(calib_obs, np.uint8 if in_kind == "u8" else np.float32)
        self.layers = [dict(l) for l in layers]
        self.in_kind, self.in_shape = in_kind, tuple(int(v) for v in in_shape)
        self.max_batch, self.device = int(max_batch), int(device)
        self.value_head = bool(layers[-1].get("value"))
        if self.value_head:
            flags = int(flags) | FLAG_VALUE_HEAD
        _check(lib.accerl_policy_create_fp32(C.byref(self._h), 0 if in_kind == "u8" else 1, shape, descs, n,
                                             calib.ctypes.data, int(calib.shape[0]), int(bool(prune24)),
                                             self.max_batch, int(flags), self.device))
        self.n_actions = int(layers[-1]["out_c"]) - (1 if self.value_head else 0)
        return self

    def export(self, layer: int) -> dict:
        """accerl_policy_export: the quantised parameters of one layer of a from_fp32 policy."""
        l = self.layers[layer]
        s_in, s_out = C.c_float(), C.c_float()
        if l["kind"] == "maxpool":
            _check(library().accerl_policy_export(self._h, layer, None, 0, None, None, C.byref(s_in), C.byref(s_out)))
            return dict(w=None, s_w=None, skip_mul=None, s_in=np.float32(s_in.value), s_out=np.float32(s_out.value))
        w = np.empty((l["out_c"], l["in_c"], l["kh"], l["kw"]), np.int8)
        s_w = np.empty(l["out_c"], np.float32)
        sm = np.empty(l["out_c"], np.int32) if l["skip_from"] >= 0 else None
        _check(library().accerl_policy_export(self._h, layer, w.ctypes.data, w.nbytes, s_w.ctypes.data,
                                              None if sm is None else sm.ctypes.data, C.byref(s_in),
                                              C.byref(s_out)))
        return dict(w=w, s_w=s_w, skip_mul=sm, s_in=np.float32(s_in.value), s_out=np.float32(s_out.value))

    def __init__(self, policy: dict, max_batch: int, flags: int = 0, device: int = 0):
        lib = library()
        self._h = C.c_void_p()
        self.layers = policy["layers"]
        n = len(self.layers)
        descs = (LayerDesc * n)()
        keep = []  # host arrays must outlive the create call only
        for i, l in enumerate(self.layers):
            d = descs[i]
            d.kind = _KINDS[l["kind"]]
            d.flags = (RELU_IN if l["relu_in"] else 0) | (RELU_OUT if l["relu_out"] else 0) | \
                (LOGITS if l["logits"] else 0)
            for k in ("in_c", "in_h", "in_w", "out_c", "kh", "kw", "stride", "pad", "skip_from"):
                setattr(d, k, int(l[k]))
            d.s_in, d.s_out = float(l["s_in"]), float(l["s_out"])
            for k, dt in (("w", np.int8), ("s_w", np.float32), ("bias", np.float32),
                          ("skip_mul", np.int32)):
                if l.get(k) is not None:
                    a = np.ascontiguousarray(l[k], dt)
                    keep.append(a)
                    setattr(d, k, a.ctypes.data)
        shape = (C.c_int32 * 3)(*[int(v) for v in policy["in_shape"]])
        self.in_kind = policy["in_kind"]
        self.in_shape = tuple(int(v) for v in policy["in_shape"])
        self.max_batch = int(max_batch)
        self.device = int(device)
        if self.layers[-1].get("value"):
            flags = int(flags) | FLAG_VALUE_HEAD
        _check(lib.accerl_policy_create(C.byref(self._h), 0 if self.in_kind == "u8" else 1, shape,
                                        float(policy["s_input"]), descs, n, self.max_batch,
                                        int(flags), self.device))
        self.value_head = bool(self.layers[-1].get("value"))
        self.n_actions = int(self.layers[-1]["out_c"]) - (1 if self.value_head else 0)

    # -- the hot call ---------------------------------------------------------------------
    def act(self, obs, uniforms, out=None, stream=None):
        """obs, uniforms: CUDA torch tensors.  Returns (logits, actions, logp) CUDA tensors."""
        import torch
        b = int(obs.shape[0])
        if out is None:
            dev = obs.device
            out = (torch.empty((b, self.n_actions), dtype=torch.float32, device=dev),
                   torch.empty(b, dtype=torch.int32, device=dev),
                   torch.empty(b, dtype=torch.float32, device=dev))
        if stream is None:
            stream = torch.cuda.current_stream(obs.device).cuda_stream
        assert obs.is_contiguous() and uniforms.is_contiguous() and obs.is_cuda and uniforms.is_cuda
        assert obs.dtype == (torch.uint8 if self.in_kind == "u8" else torch.float32)
        assert uniforms.dtype == torch.float32 and uniforms.numel() == b
        _check(library().accerl_policy_act(self._h, obs.data_ptr(), uniforms.data_ptr(), b,
                                           out[0].data_ptr(), out[1].data_ptr(), out[2].data_ptr(),
                                           stream))
        return out

    def act_ex(self, obs, uniforms, stream=None) -> dict:
        """accerl_policy_act_ex: dict(logits, actions, logp, entropy[, value]) of CUDA tensors."""
        import torch
        b, dev = int(obs.shape[0]), obs.device
        out = dict(logits=torch.empty((b, self.n_actions), dtype=torch.float32, device=dev),
                   actions=torch.empty(b, dtype=torch.int32, device=dev),
                   logp=torch.empty(b, dtype=torch.float32, device=dev),
                   entropy=torch.empty(b, dtype=torch.float32, device=dev))
        if self.value_head:
            out["value"] = torch.empty(b, dtype=torch.float32, device=dev)
        _check(library().accerl_policy_act_ex(
            self._h, obs.data_ptr(), uniforms.data_ptr(), b, out["logits"].data_ptr(),
            out["actions"].data_ptr(), out["logp"].data_ptr(),
            out["value"].data_ptr() if self.value_head else None, out["entropy"].data_ptr(),
            _stream_of(obs, stream)))
        return out

    def act_timed(self, obs, uniforms, out, stream=None) -> np.ndarray:
        """One step with CUDA events around every launch; returns milliseconds per launch."""
        import torch
        if stream is None:
            stream = torch.cuda.current_stream(obs.device).cuda_stream
        n = self.info()["launches_per_act"]
        ms = np.zeros(n, np.float32)
        _check(library().accerl_policy_act_timed(self._h, obs.data_ptr(), uniforms.data_ptr(),
                                                 int(obs.shape[0]), out[0].data_ptr(),
                                                 out[1].data_ptr(), out[2].data_ptr(), stream,
                                                 ms.ctypes.data, n))
        return ms

    def act_noalloc_raw(self, obs_ptr, u_ptr, batch, logits_ptr, actions_ptr, logp_ptr,
                        stream=0) -> int:
        """accerl_policy_act_noalloc with raw device addresses; returns the status code."""
        return library().accerl_policy_act_noalloc(self._h, obs_ptr, u_ptr, batch, logits_ptr,
                                                   actions_ptr, logp_ptr, stream)

    def act_raw(self, obs_ptr, u_ptr, batch, logits_ptr, actions_ptr, logp_ptr, stream=0) -> int:
        """Unchecked pass-through returning the status code (for ABI tests)."""
        return library().accerl_policy_act(self._h, obs_ptr, u_ptr, batch, logits_ptr, actions_ptr,
                                           logp_ptr, stream)

    def act_host(self, obs, uniforms, out, stream=0):
        """obs, uniforms, out=(logits, actions, logp): host tensors/arrays (pinned is faster)."""
        ptr = lambda a: a.data_ptr() if hasattr(a, "data_ptr") else a.ctypes.data  # noqa: E731
        _check(library().accerl_policy_act_host(self._h, ptr(obs), ptr(uniforms), int(obs.shape[0]),
                                                ptr(out[0]), ptr(out[1]), ptr(out[2]), stream))
        return out

    # -- parity taps and introspection --------------------------------------------------------
    def read_activation(self, layer: int, batch: int) -> np.ndarray:
        if layer < 0:
            shape = (batch,) + self.in_shape
        else:
            l = self.layers[layer]
            shape = (batch, l["out_c"]) + _out_hw(l)
        dst = np.empty(shape, np.int8)
        _check(library().accerl_policy_read_activation(self._h, layer, batch, dst.ctypes.data,
                                                       dst.nbytes))
        return dst

    def check(self):
        _check(library().accerl_policy_check(self._h))

    def selftest_wait(self, poll_limit: int = 200, stream=0):
        """accerl_policy_selftest_wait: makes a bounded device-side wait run out on purpose."""
        _check(library().accerl_policy_selftest_wait(self._h, poll_limit, stream))

    def info(self, batch: int | None = None) -> dict:
        na, ws, nl = C.c_int32(), C.c_size_t(), C.c_int32()
        buf = C.create_string_buffer(1 << 16)
        _check(library().accerl_policy_info(self._h, batch or self.max_batch, C.byref(na),
                                            C.byref(ws), C.byref(nl), buf, len(buf)))
        return dict(n_actions=na.value, workspace_bytes=ws.value, launches_per_act=nl.value,
                    plan=buf.value.decode())

    def close(self):
        if self._h:
            library().accerl_policy_destroy(self._h)
            self._h = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
