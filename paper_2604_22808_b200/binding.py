"""ctypes binding of the FreqFormer C ABI (include/freqformer.h).

Argument marshalling only: every step of the path runs inside the CUDA library.  PyTorch is
used for device memory and streams.  There is no CPU fallback: if the library has not been
built (``python -m paper_2604_22808_b200.build``) loading it raises.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Sequence

import numpy as np

from .configs import FFConfig

# FF_LIBRARY_VARIANT=debug loads the build with device-side range checks (python -m paper_2604_22808_b200.build --debug)
_LIB_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)),
                         "libfreqformer_debug.so" if os.environ.get("FF_LIBRARY_VARIANT") == "debug" else "libfreqformer.so")
_lib = None

FF_OK = 0
STATUS_NAMES = {0: "FF_OK", 1: "FF_ERR_INVALID_ARG", 2: "FF_ERR_UNSUPPORTED", 3: "FF_ERR_WORKSPACE",
                4: "FF_ERR_CUDA", 5: "FF_ERR_TIMEOUT", 6: "FF_ERR_EMPTY_BAND", 7: "FF_ERR_NOT_ROUTED"}
FF_BF16, FF_FP32 = 0, 1
FF_BAND_LOW, FF_BAND_MID, FF_BAND_HIGH = 1, 2, 4
(TAP_SPEC_LOW, TAP_SPEC_MID, TAP_SPEC_HIGH, TAP_POOLED_LOW, TAP_Y_LOW, TAP_Y_MID, TAP_Y_HIGH, TAP_SUMMARY,
 TAP_ENERGY, TAP_ALLOC, TAP_PI) = range(11)

EXPORTS = ("ff_config_validate", "ff_band_sizes", "ff_band_rank", "ff_workspace_bytes", "ff_workspace_bytes_host",
           "ff_plan_create", "ff_plan_workspace_bytes", "ff_band_info", "ff_plan_set_workspace", "ff_destroy", "ff_last_error",
           "ff_route", "ff_forward", "ff_forward_host", "ff_forward_projected", "ff_plan_device_status", "ff_plan_last_launches", "ff_plan_kernel_info",
           "ff_get_tap", "ff_plan_set_attention_impl", "ff_plan_set_profiling", "ff_plan_stage_times", "ff_high_attention_noalloc",
           "ff_plan_selftest_bounded_wait")
STAGES = ("transform", "router", "attention", "summary", "inverse")


class ff_config_t(C.Structure):
    _fields_ = [("batch", C.c_int32), ("T", C.c_int32), ("H", C.c_int32), ("W", C.c_int32), ("heads", C.c_int32),
                ("head_dim", C.c_int32), ("dtype", C.c_int32), ("low_cut", C.c_int32 * 3), ("mid_cut", C.c_int32 * 3),
                ("low_compress", C.c_int32), ("mid_block", C.c_int32), ("mid_stride", C.c_int32),
                ("high_radius", C.c_int32), ("n_summary", C.c_int32), ("router_hidden", C.c_int32),
                ("t_embed_dim", C.c_int32), ("transform", C.c_int32), ("mid_pattern", C.c_int32)]


class ff_weights_t(C.Structure):
    _fields_ = [("W1", C.c_void_p), ("b1", C.c_void_p), ("W2", C.c_void_p), ("b2", C.c_void_p), ("U", C.c_void_p)]


class FFError(RuntimeError):
    def __init__(self, status: int, message: str):
        super().__init__(f"{STATUS_NAMES.get(status, status)}: {message}")
        self.status = status


def library() -> C.CDLL:
    """Load the CUDA library; fails loudly when it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(_LIB_PATH):
            raise FFError(4, f"{_LIB_PATH} is missing: build it with `python -m paper_2604_22808_b200.build` "
                             "(there is no CPU fallback)")
        lib = C.CDLL(_LIB_PATH)
        lib.ff_last_error.restype = C.c_char_p
        lib.ff_last_error.argtypes = [C.c_void_p]
        for name in EXPORTS:
            if name != "ff_last_error":
                getattr(lib, name).restype = C.c_int32
        lib.ff_plan_create.argtypes = [C.POINTER(ff_config_t), C.POINTER(ff_weights_t), C.POINTER(C.c_void_p)]
        lib.ff_plan_workspace_bytes.argtypes = [C.c_void_p, C.POINTER(C.c_size_t)]
        lib.ff_plan_set_workspace.argtypes = [C.c_void_p, C.c_void_p, C.c_size_t]
        lib.ff_band_info.argtypes = [C.c_void_p, C.POINTER(C.c_int64)]
        lib.ff_destroy.argtypes = [C.c_void_p]
        lib.ff_route.argtypes = [C.c_void_p] + [C.c_void_p] * 3 + [C.c_void_p] * 4 + [C.c_void_p]
        lib.ff_forward.argtypes = [C.c_void_p] + [C.c_void_p] * 3 + [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
        lib.ff_forward_host.argtypes = [C.c_void_p] + [C.c_void_p] * 3 + [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
        lib.ff_forward_projected.argtypes = [C.c_void_p] + [C.c_void_p] * 3 + [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
        lib.ff_plan_device_status.argtypes = [C.c_void_p, C.c_void_p]
        lib.ff_plan_last_launches.argtypes = [C.c_void_p, C.POINTER(C.c_int64)]
        lib.ff_plan_kernel_info.argtypes = [C.c_void_p, C.POINTER(C.c_int32)]
        lib.ff_get_tap.argtypes = [C.c_void_p, C.c_int32, C.POINTER(C.c_void_p), C.POINTER(C.c_size_t)]
        lib.ff_plan_set_attention_impl.argtypes = [C.c_void_p, C.c_int32]
        lib.ff_plan_set_profiling.argtypes = [C.c_void_p, C.c_int32]
        lib.ff_plan_stage_times.argtypes = [C.c_void_p, C.POINTER(C.c_float), C.POINTER(C.c_int64)]
        lib.ff_high_attention_noalloc.argtypes = [C.c_void_p] * 4 + [C.c_int32, C.c_int64, C.c_int32, C.c_int32, C.c_void_p]
        lib.ff_plan_selftest_bounded_wait.argtypes = [C.c_void_p, C.c_int64, C.POINTER(C.c_int32), C.c_void_p]
        lib.ff_config_validate.argtypes = [C.POINTER(ff_config_t)]
        lib.ff_band_sizes.argtypes = [C.POINTER(ff_config_t), C.POINTER(C.c_int64)]
        lib.ff_band_rank.argtypes = [C.POINTER(ff_config_t), C.c_int32, C.c_int32, C.c_int32, C.POINTER(C.c_int32),
                                     C.POINTER(C.c_int64)]
        lib.ff_workspace_bytes.argtypes = [C.POINTER(ff_config_t), C.POINTER(C.c_size_t)]
        lib.ff_workspace_bytes_host.argtypes = [C.POINTER(ff_config_t), C.POINTER(C.c_size_t)]
        _lib = lib
    return _lib


def c_config(cfg: FFConfig) -> ff_config_t:
    c = ff_config_t()
    c.batch, c.T, c.H, c.W, c.heads, c.head_dim = cfg.batch, cfg.T, cfg.H, cfg.W, cfg.heads, cfg.head_dim
    c.dtype = FF_FP32 if cfg.dtype == "fp32" else FF_BF16
    c.low_cut = (C.c_int32 * 3)(*cfg.low_cut)
    c.mid_cut = (C.c_int32 * 3)(*cfg.mid_cut)
    c.low_compress, c.mid_block, c.mid_stride, c.high_radius = cfg.r, cfg.b, cfg.s, cfg.R
    c.n_summary, c.router_hidden, c.t_embed_dim = cfg.m, cfg.router_hidden, cfg.t_embed_dim
    c.transform = {"dct": 0, "haar": 1}[cfg.transform]
    c.mid_pattern = {"strided": 0, "anchor": 1}[cfg.mid_pattern]
    return c


def _check(status: int, plan=None):
    if status != FF_OK:
        raise FFError(status, library().ff_last_error(plan).decode())


# ---- host-only helpers ------------------------------------------------------------------------
def ff_config_validate(cfg: FFConfig) -> int:
    return library().ff_config_validate(C.byref(c_config(cfg)))


def ff_band_sizes(cfg: FFConfig):
    out = (C.c_int64 * 4)()
    _check(library().ff_band_sizes(C.byref(c_config(cfg)), out))
    return tuple(int(x) for x in out)


def ff_band_rank(cfg: FFConfig, kt: int, kh: int, kw: int):
    band, rank = C.c_int32(), C.c_int64()
    _check(library().ff_band_rank(C.byref(c_config(cfg)), kt, kh, kw, C.byref(band), C.byref(rank)))
    return band.value, rank.value


def ff_workspace_bytes(cfg: FFConfig, host_staging: bool = False) -> int:
    out = C.c_size_t()
    fn = library().ff_workspace_bytes_host if host_staging else library().ff_workspace_bytes
    _check(fn(C.byref(c_config(cfg)), C.byref(out)))
    return out.value


# ---- the plan -----------------------------------------------------------------------------------
def _f32(a) -> Optional[np.ndarray]:
    return None if a is None else np.ascontiguousarray(a, dtype=np.float32)


def _ptr(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


class Plan:
    """Owns an ff_plan_t and (through torch) its workspace."""

    def __init__(self, cfg: FFConfig, weights: Optional[dict] = None, U: Optional[np.ndarray] = None,
                 host_staging: bool = False, device: str = "cuda:0"):
        import torch
        self.cfg = cfg
        self._torch = torch
        self.device = torch.device(device)
        if self.device.index is None:
            self.device = torch.device("cuda", torch.cuda.current_device())
        self.handle = C.c_void_p()
        lib = library()
        w = ff_weights_t()
        keep = []
        if weights is not None:
            for name in ("W1", "b1", "W2", "b2"):
                arr = _f32(weights[name]); keep.append(arr)
                setattr(w, name, arr.ctypes.data)
        if U is not None:
            arr = _f32(U); keep.append(arr)
            w.U = arr.ctypes.data
        with torch.cuda.device(self.device):
            _check(lib.ff_plan_create(C.byref(c_config(cfg)), C.byref(w), C.byref(self.handle)))
            nbytes = ff_workspace_bytes(cfg, host_staging)
            self.workspace = torch.empty(nbytes, dtype=torch.uint8, device=self.device)
            _check(lib.ff_plan_set_workspace(self.handle, self.workspace.data_ptr(), nbytes), self.handle)
        self.workspace_bytes = nbytes

    # -- lifetime
    def destroy(self):
        if self.handle:
            library().ff_destroy(self.handle)
            self.handle = C.c_void_p()
            self.workspace = None

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass

    def band_info(self):
        """(N_low, ceil(N_low / r), N_mid, N_high) of the plan's configuration."""
        out = (C.c_int64 * 4)()
        _check(library().ff_band_info(self.handle, out), self.handle)
        return tuple(int(x) for x in out)

    def _stream(self):
        return C.c_void_p(self._torch.cuda.current_stream(self.device).cuda_stream)

    @property
    def torch_dtype(self):
        return self._torch.float32 if self.cfg.dtype == "fp32" else self._torch.bfloat16

    def _check_io(self, *tensors):
        shape = (self.cfg.batch, self.cfg.heads, self.cfg.T, self.cfg.H, self.cfg.W, self.cfg.head_dim)
        for t in tensors:
            if tuple(t.shape) != shape or t.dtype != self.torch_dtype or not t.is_contiguous():
                raise FFError(1, f"expected a contiguous {self.torch_dtype} tensor of shape {shape}")
            if not t.is_cuda or t.device != self.device:
                raise FFError(1, f"expected a tensor on {self.device}, got one on {t.device}")

    # -- the path
    def route(self, Q, K, V, timesteps: Sequence[float], alloc_out=None, want_host: bool = True):
        self._check_io(Q, K, V)
        ts = np.ascontiguousarray(timesteps, dtype=np.float32)
        assert ts.shape == (self.cfg.batch,)
        alloc_h = np.zeros(self.cfg.batch * self.cfg.heads, np.uint8) if want_host else None
        pi_h = np.zeros((self.cfg.batch, 3), np.float32) if want_host else None
        _check(library().ff_route(self.handle, Q.data_ptr(), K.data_ptr(), V.data_ptr(), _ptr(ts),
                                  None if alloc_out is None else alloc_out.data_ptr(), _ptr(alloc_h), _ptr(pi_h),
                                  self._stream()), self.handle)
        return alloc_h, pi_h

    def forward(self, Q, K, V, out, alloc=None, timesteps: Optional[Sequence[float]] = None):
        """alloc: uint8 CUDA tensor [batch*heads] of band masks, or None to route from timesteps."""
        self._check_io(Q, K, V, out)
        ts = None if timesteps is None else np.ascontiguousarray(timesteps, dtype=np.float32)
        _check(library().ff_forward(self.handle, Q.data_ptr(), K.data_ptr(), V.data_ptr(),
                                    None if alloc is None else alloc.data_ptr(), _ptr(ts), out.data_ptr(),
                                    self._stream()), self.handle)
        return out

    def forward_host(self, Qh, Kh, Vh, out_h, alloc_host: Optional[np.ndarray] = None,
                     timesteps: Optional[Sequence[float]] = None):
        """Host tensors (ideally pinned) in and out; the copies are part of the call."""
        ts = None if timesteps is None else np.ascontiguousarray(timesteps, dtype=np.float32)
        al = None if alloc_host is None else np.ascontiguousarray(alloc_host, dtype=np.uint8)
        _check(library().ff_forward_host(self.handle, Qh.data_ptr(), Kh.data_ptr(), Vh.data_ptr(), _ptr(al), _ptr(ts),
                                         out_h.data_ptr(), self._stream()), self.handle)
        return out_h

    def forward_projected(self, X, Wqkv, Wo, out, alloc=None, timesteps: Optional[Sequence[float]] = None):
        """X, out: bf16 CUDA tensors [batch][T*H*W][heads*head_dim]; Wqkv [3][D][D], Wo [D][D] (y = x W).
        The plan must have been created with host_staging=True (Q, K, V and the attention output live there)."""
        torch = self._torch
        cfg = self.cfg
        D = cfg.heads * cfg.head_dim
        for t, shape in ((X, (cfg.batch, cfg.N, D)), (out, (cfg.batch, cfg.N, D)), (Wqkv, (3, D, D)), (Wo, (D, D))):
            if (tuple(t.shape) != shape or t.dtype != torch.bfloat16 or not t.is_contiguous() or not t.is_cuda
                    or t.device != self.device):
                raise FFError(1, f"expected a contiguous bf16 tensor of shape {shape} on {self.device}")
        ts = None if timesteps is None else np.ascontiguousarray(timesteps, dtype=np.float32)
        _check(library().ff_forward_projected(self.handle, X.data_ptr(), Wqkv.data_ptr(), Wo.data_ptr(),
                                              None if alloc is None else alloc.data_ptr(), _ptr(ts), out.data_ptr(),
                                              self._stream()), self.handle)
        return out

    def device_status(self) -> int:
        return library().ff_plan_device_status(self.handle, self._stream())

    def selftest_bounded_wait(self, limit_cycles: int) -> int:
        """Runs the bounded-wait self-test; returns how many of its two waits were abandoned."""
        n = C.c_int32(-1)
        _check(library().ff_plan_selftest_bounded_wait(self.handle, int(limit_cycles), C.byref(n), self._stream()), self.handle)
        return n.value

    def kernel_info(self) -> dict:
        info = (C.c_int32 * 4)()
        _check(library().ff_plan_kernel_info(self.handle, info), self.handle)
        return {"transform_fused": bool(info[0]), "transform_cluster": int(info[1]), "attention_tensor_core": bool(info[2]),
                "low_band_tensor_core": bool(info[3])}

    def last_launches(self) -> int:
        n = C.c_int64()
        _check(library().ff_plan_last_launches(self.handle, C.byref(n)), self.handle)
        return n.value

    def set_attention_impl(self, impl: int):
        _check(library().ff_plan_set_attention_impl(self.handle, impl), self.handle)

    def set_profiling(self, enable: bool):
        _check(library().ff_plan_set_profiling(self.handle, int(enable)), self.handle)

    def stage_times(self):
        """{stage: (ms, launches)} of the last forward (profiling must be enabled)."""
        ms, n = (C.c_float * len(STAGES))(), (C.c_int64 * len(STAGES))()
        _check(library().ff_plan_stage_times(self.handle, ms, n), self.handle)
        return {name: (float(ms[i]), int(n[i])) for i, name in enumerate(STAGES)}

    # -- inspection
    def tap(self, which: int):
        """A torch view (no copy) of an intermediate buffer inside the workspace."""
        torch = self._torch
        ptr, nbytes = C.c_void_p(), C.c_size_t()
        _check(library().ff_get_tap(self.handle, which, C.byref(ptr), C.byref(nbytes)), self.handle)
        off = ptr.value - self.workspace.data_ptr()
        raw = self.workspace[off:off + nbytes.value]
        cfg = self.cfg
        n_low, n_bar, n_mid, n_high = ff_band_sizes(cfg)
        BH, d = cfg.batch * cfg.heads, cfg.head_dim
        st = self.torch_dtype
        shapes = {TAP_SPEC_LOW: (torch.float32, (3, BH, n_low, d)), TAP_SPEC_MID: (st, (3, BH, n_mid, d)),
                  TAP_SPEC_HIGH: (st, (3, BH, n_high, d)), TAP_POOLED_LOW: (torch.float32, (3, BH, n_bar, d)),
                  TAP_Y_LOW: (torch.float32, (BH, n_bar, d)), TAP_Y_MID: (st, (BH, n_mid, d)),
                  TAP_Y_HIGH: (st, (BH, n_high, d)), TAP_SUMMARY: (torch.float32, (BH, 3, cfg.m, d)),
                  TAP_ENERGY: (torch.float64, (cfg.batch, 3, d)), TAP_ALLOC: (torch.uint8, (BH,)),
                  TAP_PI: (torch.float32, (cfg.batch, 3))}
        dt, shape = shapes[which]
        return raw.view(dt).view(shape)


# Same names as the C entry points, for callers that prefer the flat API.
def ff_plan_create(cfg: FFConfig, weights=None, U=None, host_staging=False, device="cuda:0") -> Plan:
    return Plan(cfg, weights, U, host_staging, device)


def ff_route(plan: Plan, Q, K, V, timesteps, alloc_out=None):
    return plan.route(Q, K, V, timesteps, alloc_out)


def ff_forward(plan: Plan, Q, K, V, out, alloc=None, timesteps=None):
    return plan.forward(Q, K, V, out, alloc, timesteps)


def ff_forward_host(plan: Plan, Qh, Kh, Vh, out_h, alloc_host=None, timesteps=None):
    return plan.forward_host(Qh, Kh, Vh, out_h, alloc_host, timesteps)


def ff_forward_projected(plan: Plan, X, Wqkv, Wo, out, alloc=None, timesteps=None):
    return plan.forward_projected(X, Wqkv, Wo, out, alloc, timesteps)


def ff_high_attention_noalloc(q, k, v, y, radius: int, sync: bool = True):
    """High-band sliding-window attention on bf16 CUDA tensors [heads][n][128] without any device
    allocation inside the call (the kernel's scratch is a fixed array in the library): for hosts
    whose device memory is fully owned by their own pool, or that cannot tolerate the device-wide
    synchronisation of an allocation.  Calls on one device share that scratch: do not overlap them."""
    import torch
    for t in (q, k, v, y):
        if (not t.is_cuda or t.device != q.device or t.dtype != torch.bfloat16 or not t.is_contiguous() or t.dim() != 3
                or t.shape[2] != 128 or t.shape != q.shape):
            raise FFError(1, "expected contiguous bf16 CUDA tensors of one shape [heads][n][128] on one device")
    stream = C.c_void_p(torch.cuda.current_stream(q.device).cuda_stream)
    with torch.cuda.device(q.device):
        _check(library().ff_high_attention_noalloc(q.data_ptr(), k.data_ptr(), v.data_ptr(), y.data_ptr(), q.shape[0],
                                                   q.shape[1], radius, int(sync), stream))
    return y


def ff_destroy(plan: Plan):
    plan.destroy()
