"""Thin Python binding of libeora_linear (the C ABI in include/eora_linear.h).

Argument marshalling only: every step of the layer runs in the library's CUDA kernels.
torch is used for device memory and streams.  There is no CPU fallback: if the shared
library has not been built (``python -m paper_2410_21271_b200.build``) loading fails.
"""
from __future__ import annotations

import ctypes
import os
from ctypes import POINTER, Structure, byref, c_char_p, c_int, c_int32, c_int64, c_void_p

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libeora_linear.so")
HEADER_PATH = os.path.join(os.path.dirname(_HERE), "include", "eora_linear.h")

# status codes / enums (mirrors of include/eora_linear.h)
EORA_OK = 0
EORA_ERR_NULL_ARG, EORA_ERR_BAD_SHAPE, EORA_ERR_UNSUPPORTED, EORA_ERR_MISALIGNED = -1, -2, -3, -4
EORA_ERR_M_TOO_LARGE, EORA_ERR_CUDA, EORA_ERR_DEVICE_TIMEOUT = -5, -6, -7
EORA_W_QUANT, EORA_W_SPARSE24, EORA_W_SPARSE24_Q4 = 0, 1, 2
EORA_AB_F16, EORA_AB_Q4, EORA_AB_Q8, EORA_AB_Q3 = 0, 1, 2, 3
EORA_X_F16, EORA_X_BF16 = 0, 1
EORA_Y_F16, EORA_Y_BF16, EORA_Y_F32 = 0, 1, 2
EORA_PATH_GENERIC, EORA_PATH_DECODE, EORA_PATH_PREFILL = 0, 1, 2
EORA_POLICY_AUTO, EORA_POLICY_GENERIC, EORA_POLICY_TMEM_DECODE = 0, 1, 2


class eora_linear_config(Structure):
    _fields_ = [(n, c_int32) for n in ("d_in", "d_out", "rank", "w_format", "w_bits", "w_group", "ab_format",
                                       "ab_group", "x_dtype", "y_dtype", "max_m", "kernel_policy")]


class eora_linear_weights(Structure):
    _fields_ = [(n, c_void_p) for n in ("w_codes", "w_scales", "w_zeros", "a", "a_scales", "a_zeros",
                                        "b", "b_scales", "b_zeros", "w_meta")]


class eora_solve_config(Structure):
    _fields_ = [("d", c_int32), ("k", c_int32), ("n", c_int32), ("rank", c_int32), ("oversample", c_int32), ("iters", c_int32)]


class EoraError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {eora_status_string(status)} ({status})")


_lib = None


def lib() -> ctypes.CDLL:
    """The loaded C-ABI library; raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2410_21271_b200.build` "
                              "(there is no fallback path)")
        L = ctypes.CDLL(LIB_PATH)
        L.eora_linear_create.argtypes = [POINTER(eora_linear_config), POINTER(eora_linear_weights), c_void_p,
                                         POINTER(c_void_p)]
        L.eora_linear_create.restype = c_int
        L.eora_linear_forward.argtypes = [c_void_p, c_void_p, c_int32, c_void_p, c_void_p]
        L.eora_linear_forward.restype = c_int
        L.eora_linear_forward_host.argtypes = [c_void_p, c_void_p, c_int32, c_void_p, c_void_p]
        L.eora_linear_forward_host.restype = c_int
        L.eora_linear_create_fused.argtypes = [c_void_p, c_void_p, c_int32, c_void_p, c_void_p]
        L.eora_linear_create_fused.restype = c_int
        L.eora_linear_forward_fused.argtypes = [c_void_p, c_void_p, c_int32, c_void_p, c_void_p]
        L.eora_linear_forward_fused.restype = c_int
        L.eora_linear_forward_fused_host.argtypes = [c_void_p, c_void_p, c_int32, c_void_p, c_void_p]
        L.eora_linear_forward_fused_host.restype = c_int
        L.eora_linear_forward_host_async.argtypes = [c_void_p, c_void_p, c_int32, c_void_p, c_void_p]
        L.eora_linear_forward_host_async.restype = c_int
        L.eora_linear_forward_fused_host_async.argtypes = [c_void_p, c_void_p, c_int32, c_void_p, c_void_p]
        L.eora_linear_forward_fused_host_async.restype = c_int
        L.eora_linear_create_multi.argtypes = [c_void_p, c_void_p, c_int32, c_void_p, c_void_p]
        L.eora_linear_create_multi.restype = c_int
        L.eora_linear_forward_multi.argtypes = [c_void_p, c_void_p, c_int32, c_void_p, c_void_p, c_void_p]
        L.eora_linear_forward_multi.restype = c_int
        L.eora_linear_destroy.argtypes = [c_void_p]
        L.eora_linear_destroy.restype = c_int
        L.eora_linear_path.argtypes = [c_void_p, c_int32]
        L.eora_linear_path.restype = c_int
        L.eora_linear_launches.argtypes = [c_void_p, c_int32]
        L.eora_linear_launches.restype = c_int
        L.eora_linear_dump.argtypes = [c_void_p, c_int32, c_void_p, c_void_p]
        L.eora_linear_dump.restype = c_int
        L.eora_linear_last_device_status.argtypes = [c_void_p]
        L.eora_linear_last_device_status.restype = c_int
        L.eora_linear_set_wait_limit.argtypes = [c_void_p, ctypes.c_uint64]
        L.eora_linear_set_wait_limit.restype = c_int
        L.eora_linear_selftest_wait_timeout.argtypes = [c_void_p, c_void_p]
        L.eora_linear_selftest_wait_timeout.restype = c_int
        L.eora_linear_staging_bytes.argtypes = [c_void_p]
        L.eora_linear_staging_bytes.restype = ctypes.c_int64
        L.eora_linear_set_trace.argtypes = [c_void_p, c_void_p]
        L.eora_linear_set_trace.restype = c_int
        L.eora_linear_decode_grid.argtypes = [c_void_p, c_int32]
        L.eora_linear_decode_grid.restype = c_int
        L.eora_linear_forward_noalloc.argtypes = [POINTER(eora_linear_config), POINTER(eora_linear_weights), c_void_p,
                                                  c_int32, c_void_p, c_void_p]
        L.eora_linear_forward_noalloc.restype = c_int
        L.eora_linear_weight_bytes.argtypes = [c_void_p]
        L.eora_linear_weight_bytes.restype = c_int64
        L.eora_linear_scratch_bytes.argtypes = [c_void_p]
        L.eora_linear_scratch_bytes.restype = c_int64
        L.eora_solve_workspace_bytes.argtypes = [POINTER(eora_solve_config)]
        L.eora_solve_workspace_bytes.restype = ctypes.c_size_t
        L.eora_solve.argtypes = [POINTER(eora_solve_config), c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p,
                                 c_void_p, ctypes.c_size_t, c_void_p]
        L.eora_solve.restype = c_int
        L.eora_solve_loss.argtypes = [POINTER(eora_solve_config), c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p,
                                      c_void_p, ctypes.c_size_t, c_void_p]
        L.eora_solve_loss.restype = c_int
        L.eora_status_string.argtypes = [c_int]
        L.eora_status_string.restype = c_char_p
        L.eora_version.argtypes = []
        L.eora_version.restype = c_int
        _lib = L
    return _lib


def _ptr(t) -> int | None:
    """Raw address of a torch tensor / int / None."""
    if t is None:
        return None
    if isinstance(t, int):
        return t
    return t.data_ptr()


def _stream(stream) -> int | None:
    if stream is None:
        import torch
        return torch.cuda.current_stream().cuda_stream
    if isinstance(stream, int):
        return stream
    return stream.cuda_stream


def eora_status_string(status: int) -> str:
    return lib().eora_status_string(int(status)).decode()


def eora_version() -> int:
    return lib().eora_version()


def eora_linear_create(cfg: eora_linear_config, weights: eora_linear_weights, stream=None) -> int:
    """Returns the opaque handle (an address).  Raises EoraError on a non-zero status."""
    out = c_void_p()
    st = lib().eora_linear_create(byref(cfg), byref(weights), _stream(stream), byref(out))
    if st != EORA_OK:
        raise EoraError(st, "eora_linear_create")
    return out.value


def eora_linear_create_status(cfg, weights, stream=0) -> int:
    """create, returning only the status (for argument-checking tests; no handle is kept on error)."""
    out = c_void_p()
    st = lib().eora_linear_create(byref(cfg) if cfg is not None else None,
                                  byref(weights) if weights is not None else None, stream, byref(out))
    if st == EORA_OK:
        lib().eora_linear_destroy(out)
    return st


def eora_linear_forward(handle: int, x, m: int, y, stream=None, check: bool = True) -> int:
    st = lib().eora_linear_forward(handle, _ptr(x), int(m), _ptr(y), _stream(stream))
    if check and st != EORA_OK:
        raise EoraError(st, "eora_linear_forward")
    return st


def eora_linear_forward_host_async(handle: int, x_host, m: int, y_host, stream=None, check: bool = True) -> int:
    st = lib().eora_linear_forward_host_async(handle, _ptr(x_host), int(m), _ptr(y_host), _stream(stream))
    if check and st != EORA_OK:
        raise EoraError(st, "eora_linear_forward_host_async")
    return st


def eora_linear_forward_fused_host_async(handle: int, x_host, m: int, ys_host, stream=None, check: bool = True) -> int:
    arr = (c_void_p * len(ys_host))(*[_ptr(y) for y in ys_host])
    st = lib().eora_linear_forward_fused_host_async(handle, _ptr(x_host), int(m), arr, _stream(stream))
    if check and st != EORA_OK:
        raise EoraError(st, "eora_linear_forward_fused_host_async")
    return st


def eora_linear_forward_host(handle: int, x_host, m: int, y_host, stream=None, check: bool = True) -> int:
    st = lib().eora_linear_forward_host(handle, _ptr(x_host), int(m), _ptr(y_host), _stream(stream))
    if check and st != EORA_OK:
        raise EoraError(st, "eora_linear_forward_host")
    return st


def eora_linear_create_fused(cfgs, weights, stream=None, check: bool = True):
    """cfgs / weights: sequences of eora_linear_config / eora_linear_weights (one per fused layer).
    Returns the handle, or (with check=False) the status."""
    n = len(cfgs)
    carr = (eora_linear_config * n)(*cfgs)
    warr = (eora_linear_weights * n)(*weights)
    out = c_void_p()
    st = lib().eora_linear_create_fused(carr, warr, n, _stream(stream), byref(out))
    if not check:
        if st == EORA_OK:
            lib().eora_linear_destroy(out)
        return st
    if st != EORA_OK:
        raise EoraError(st, "eora_linear_create_fused")
    return out.value


def eora_linear_forward_fused(handle: int, x, m: int, ys, stream=None, check: bool = True) -> int:
    arr = (c_void_p * len(ys))(*[_ptr(y) for y in ys])
    st = lib().eora_linear_forward_fused(handle, _ptr(x), int(m), arr, _stream(stream))
    if check and st != EORA_OK:
        raise EoraError(st, "eora_linear_forward_fused")
    return st


def eora_linear_forward_fused_host(handle: int, x_host, m: int, ys_host, stream=None, check: bool = True) -> int:
    arr = (c_void_p * len(ys_host))(*[_ptr(y) for y in ys_host])
    st = lib().eora_linear_forward_fused_host(handle, _ptr(x_host), int(m), arr, _stream(stream))
    if check and st != EORA_OK:
        raise EoraError(st, "eora_linear_forward_fused_host")
    return st


def eora_linear_create_multi(cfg, weights, stream=None, check: bool = True):
    """cfg: the layer's eora_linear_config; weights: one eora_linear_weights per adapter (backbone from the
    first).  Returns the handle, or (with check=False) the status."""
    n = len(weights)
    warr = (eora_linear_weights * n)(*weights)
    out = c_void_p()
    st = lib().eora_linear_create_multi(byref(cfg), warr, n, _stream(stream), byref(out))
    if not check:
        if st == EORA_OK:
            lib().eora_linear_destroy(out)
        return st
    if st != EORA_OK:
        raise EoraError(st, "eora_linear_create_multi")
    return out.value


def eora_linear_forward_multi(handle: int, x, m: int, adapter_ids, y, stream=None, check: bool = True) -> int:
    ids = (c_int32 * int(m))(*[int(i) for i in adapter_ids])
    st = lib().eora_linear_forward_multi(handle, _ptr(x), int(m), ids, _ptr(y), _stream(stream))
    if check and st != EORA_OK:
        raise EoraError(st, "eora_linear_forward_multi")
    return st


def eora_linear_destroy(handle: int) -> int:
    return lib().eora_linear_destroy(handle)


def eora_linear_path(handle: int, m: int) -> int:
    return lib().eora_linear_path(handle, int(m))


def eora_linear_launches(handle: int, m: int) -> int:
    return lib().eora_linear_launches(handle, int(m))


def eora_linear_dump(handle: int, what: int, out, stream=None) -> int:
    st = lib().eora_linear_dump(handle, int(what), _ptr(out), _stream(stream))
    if st != EORA_OK:
        raise EoraError(st, "eora_linear_dump")
    return st


def eora_linear_last_device_status(handle: int) -> int:
    return lib().eora_linear_last_device_status(handle)


def eora_linear_set_wait_limit(handle: int, ns: int) -> int:
    return lib().eora_linear_set_wait_limit(handle, int(ns))


def eora_linear_selftest_wait_timeout(handle: int, stream=None) -> int:
    return lib().eora_linear_selftest_wait_timeout(handle, _stream(stream))


def eora_linear_staging_bytes(handle: int) -> int:
    return lib().eora_linear_staging_bytes(handle)


def eora_linear_set_trace(handle: int, buf) -> int:
    return lib().eora_linear_set_trace(handle, _ptr(buf))


def eora_linear_decode_grid(handle: int, m: int) -> int:
    return lib().eora_linear_decode_grid(handle, int(m))


EORA_NOALLOC_MAX_T_ELEMS = 65536


def eora_linear_forward_noalloc(cfg: eora_linear_config, weights: eora_linear_weights, x, m: int, y, stream=None,
                                check: bool = True) -> int:
    """Handle-free forward for callers that cannot allocate device memory: weights are read from the
    caller's interchange-layout buffers, scratch lives in a fixed array inside the library."""
    st = lib().eora_linear_forward_noalloc(byref(cfg), byref(weights), _ptr(x), int(m), _ptr(y), _stream(stream))
    if check and st != EORA_OK:
        raise EoraError(st, "eora_linear_forward_noalloc")
    return st


def eora_linear_weight_bytes(handle: int) -> int:
    return lib().eora_linear_weight_bytes(handle)


def eora_linear_scratch_bytes(handle: int) -> int:
    return lib().eora_linear_scratch_bytes(handle)


# ---------------------------------------------------------------------------------------------
# marshalling helper: numpy weight descriptions (as made by eora_inputs) -> device buffers -> handle
# ---------------------------------------------------------------------------------------------
def _dev(arr, device):
    import numpy as np
    import torch
    a = np.ascontiguousarray(arr)
    if a.dtype == np.uint32:
        a = a.view(np.int32)
    elif a.dtype == np.uint16:
        a = a.view(np.int16)
    return torch.from_numpy(a).to(device)


def _marshal(w_fmt: dict, a_fmt, b_fmt, *, max_m: int, x_dtype: str, y_dtype: str, kernel_policy: int, device):
    """Upload one layer's interchange buffers and fill the two C structs.  Returns (cfg, weights, buffers);
    the buffers must stay alive until create has returned."""
    cfg = eora_linear_config()
    wts = eora_linear_weights()
    keep = []
    cfg.d_in, cfg.d_out = w_fmt["rows"], w_fmt["cols"]
    if w_fmt["kind"] == "quant":
        cfg.w_format, cfg.w_bits, cfg.w_group = EORA_W_QUANT, w_fmt["bits"], w_fmt["group"]
        bufs = [_dev(w_fmt["codes"], device), _dev(w_fmt["scales"], device), _dev(w_fmt["zeros"], device)]
    elif w_fmt["kind"] == "sparse24":
        cfg.w_format = EORA_W_SPARSE24
        bufs = [_dev(w_fmt["values"], device), None, _dev(w_fmt["meta"], device)]
    elif w_fmt["kind"] == "sparse24q":
        cfg.w_format, cfg.w_bits, cfg.w_group = EORA_W_SPARSE24_Q4, w_fmt["bits"], w_fmt["group"]
        bufs = [_dev(w_fmt["codes"], device), _dev(w_fmt["scales"], device), _dev(w_fmt["zeros"], device)]
        meta = _dev(w_fmt["meta"], device)
        keep.append(meta)
        wts.w_meta = _ptr(meta)
    else:
        raise ValueError(w_fmt["kind"])
    keep += bufs
    wts.w_codes, wts.w_scales, wts.w_zeros = [_ptr(b) for b in bufs]
    cfg.rank = 0
    cfg.ab_format, cfg.ab_group = EORA_AB_F16, 128
    if a_fmt is not None and b_fmt is not None:
        kind = a_fmt["kind"]
        if kind == "f16":
            cfg.rank = a_fmt["data"].shape[1]
            ab = [_dev(a_fmt["data"], device), None, None, _dev(b_fmt["data"], device), None, None]
        elif kind == "quant":
            cfg.rank, cfg.ab_format, cfg.ab_group = a_fmt["cols"], {4: EORA_AB_Q4, 3: EORA_AB_Q3}[a_fmt["bits"]], a_fmt["group"]
            ab = [_dev(f[k], device) for f in (a_fmt, b_fmt) for k in ("codes", "scales", "zeros")]
        elif kind == "q8":
            cfg.rank, cfg.ab_format = a_fmt["cols"], EORA_AB_Q8
            ab = [_dev(f[k], device) for f in (a_fmt, b_fmt) for k in ("codes", "scales", "zeros")]
        else:
            raise ValueError(kind)
        keep += ab
        (wts.a, wts.a_scales, wts.a_zeros, wts.b, wts.b_scales, wts.b_zeros) = [_ptr(b) for b in ab]
    cfg.x_dtype = {"f16": EORA_X_F16, "bf16": EORA_X_BF16}[x_dtype]
    cfg.y_dtype = {"f16": EORA_Y_F16, "bf16": EORA_Y_BF16, "f32": EORA_Y_F32}[y_dtype]
    cfg.max_m, cfg.kernel_policy = max_m, kernel_policy
    return cfg, wts, keep


class Layer:
    """Owns a library handle plus nothing else (the uploaded interchange buffers are dropped after
    create).  Methods only marshal arguments."""

    def __init__(self, w_fmt: dict, a_fmt: dict | None, b_fmt: dict | None, *, max_m: int, x_dtype: str = "f16",
                 y_dtype: str = "f16", kernel_policy: int = EORA_POLICY_AUTO, device="cuda:0"):
        import torch
        cfg, wts, keep = _marshal(w_fmt, a_fmt, b_fmt, max_m=max_m, x_dtype=x_dtype, y_dtype=y_dtype,
                                  kernel_policy=kernel_policy, device=device)
        self.cfg = cfg
        self.device = torch.device(device)
        self.y_torch_dtype = {"f16": torch.float16, "bf16": torch.bfloat16, "f32": torch.float32}[y_dtype]
        with torch.cuda.device(self.device):
            self.handle = eora_linear_create(cfg, wts)
        del keep

    def forward(self, x, y=None, stream=None):
        import torch
        m = x.shape[0]
        if y is None:
            y = torch.empty((m, self.cfg.d_out), dtype=self.y_torch_dtype, device=x.device)
        eora_linear_forward(self.handle, x, m, y, stream)
        return y

    def forward_host(self, x_host, y_host, stream=None, sync: bool = True):
        (eora_linear_forward_host if sync else eora_linear_forward_host_async)(self.handle, x_host, x_host.shape[0], y_host, stream)
        return y_host

    def path(self, m: int) -> int:
        return eora_linear_path(self.handle, m)

    def launches(self, m: int) -> int:
        return eora_linear_launches(self.handle, m)

    def dump(self, what: int):
        import torch
        c = self.cfg
        shape, dt = {0: ((c.d_in, c.d_out), torch.int32), 1: ((c.d_in, c.d_out), torch.float32),
                     2: ((c.d_in, c.rank), torch.float32), 3: ((c.rank, c.d_out), torch.float32)}[what]
        out = torch.empty(shape, dtype=dt, device=self.device)
        eora_linear_dump(self.handle, what, out)
        return out

    def device_status(self) -> int:
        return eora_linear_last_device_status(self.handle)

    def close(self):
        if getattr(self, "handle", None):
            eora_linear_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


class FusedLayers:
    """Several layers that read the same X (q/k/v, gate/up) behind ONE handle and one launch per forward.
    max_m > 64 needs every d_out to be a multiple of 128 (the tensor-core family).  Methods only marshal arguments."""

    def __init__(self, layers, *, max_m: int, x_dtype: str = "f16", y_dtype: str = "f16",
                 kernel_policy: int = EORA_POLICY_AUTO, device="cuda:0"):
        import torch
        cfgs, wtss, keep = [], [], []
        for (w_fmt, a_fmt, b_fmt) in layers:
            cfg, wts, k = _marshal(w_fmt, a_fmt, b_fmt, max_m=max_m, x_dtype=x_dtype, y_dtype=y_dtype,
                                   kernel_policy=kernel_policy, device=device)
            cfgs.append(cfg); wtss.append(wts); keep.append(k)
        self.cfgs = cfgs
        self.device = torch.device(device)
        self.y_torch_dtype = {"f16": torch.float16, "bf16": torch.bfloat16, "f32": torch.float32}[y_dtype]
        with torch.cuda.device(self.device):
            self.handle = eora_linear_create_fused(cfgs, wtss)
        del keep

    def forward(self, x, ys=None, stream=None):
        import torch
        m = x.shape[0]
        if ys is None:
            ys = [torch.empty((m, c.d_out), dtype=self.y_torch_dtype, device=x.device) for c in self.cfgs]
        eora_linear_forward_fused(self.handle, x, m, ys, stream)
        return ys

    def forward_host(self, x_host, ys_host, stream=None, sync: bool = True):
        (eora_linear_forward_fused_host if sync else eora_linear_forward_fused_host_async)(self.handle, x_host, x_host.shape[0], ys_host, stream)
        return ys_host

    def launches(self, m: int) -> int:
        return eora_linear_launches(self.handle, m)

    def device_status(self) -> int:
        return eora_linear_last_device_status(self.handle)

    def close(self):
        if getattr(self, "handle", None):
            eora_linear_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


class MultiAdapterLayer:
    """One backbone with several adapters; every token of a forward names the adapter it uses (-1: none).
    max_m > 64 needs every d_out to be a multiple of 128 (the tensor-core family).  Methods only marshal arguments."""

    def __init__(self, w_fmt: dict, adapters, *, max_m: int, x_dtype: str = "f16", y_dtype: str = "f16", device="cuda:0"):
        import torch
        cfg, wtss, keep = None, [], []
        for (a_fmt, b_fmt) in adapters:
            c, wts, k = _marshal(w_fmt, a_fmt, b_fmt, max_m=max_m, x_dtype=x_dtype, y_dtype=y_dtype,
                                 kernel_policy=EORA_POLICY_AUTO, device=device)
            cfg = cfg or c
            wtss.append(wts); keep.append(k)
        self.cfg = cfg
        self.device = torch.device(device)
        self.y_torch_dtype = {"f16": torch.float16, "bf16": torch.bfloat16, "f32": torch.float32}[y_dtype]
        with torch.cuda.device(self.device):
            self.handle = eora_linear_create_multi(cfg, wtss)
        del keep

    def forward(self, x, adapter_ids, y=None, stream=None):
        import torch
        m = x.shape[0]
        if y is None:
            y = torch.empty((m, self.cfg.d_out), dtype=self.y_torch_dtype, device=x.device)
        eora_linear_forward_multi(self.handle, x, m, adapter_ids, y, stream)
        return y

    def device_status(self) -> int:
        return eora_linear_last_device_status(self.handle)

    def close(self):
        if getattr(self, "handle", None):
            eora_linear_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


# ---- offline solve (Algorithm 1 steps 1-6), include/eora_solve.h -------------------------------------------------
def eora_solve_workspace_bytes(cfg: eora_solve_config) -> int:
    return int(lib().eora_solve_workspace_bytes(ctypes.byref(cfg)))


def eora_solve(cfg: eora_solve_config, w, w_hat, x_tilde, b_prime, a, sigma, workspace, stream=None, check: bool = True) -> int:
    """Device tensors in, device tensors out (fp32, row-major); `workspace`: a device byte tensor."""
    rc = lib().eora_solve(ctypes.byref(cfg), _ptr(w), _ptr(w_hat), _ptr(x_tilde), _ptr(b_prime), _ptr(a), _ptr(sigma),
                          _ptr(workspace), workspace.numel() * workspace.element_size(), _stream(stream))
    if check and rc != EORA_OK:
        raise EoraError(rc, "eora_solve")
    return rc


def eora_solve_loss(cfg: eora_solve_config, w, w_hat, x_tilde, b_prime, a, loss_sq, workspace, stream=None, check: bool = True) -> int:
    rc = lib().eora_solve_loss(ctypes.byref(cfg), _ptr(w), _ptr(w_hat), _ptr(x_tilde), _ptr(b_prime), _ptr(a), _ptr(loss_sq),
                               _ptr(workspace), workspace.numel() * workspace.element_size(), _stream(stream))
    if check and rc != EORA_OK:
        raise EoraError(rc, "eora_solve_loss")
    return rc


def solve(w, w_hat, x_tilde, rank: int, oversample: int = 0, iters: int = 0, stream=None):
    """Convenience wrapper: device fp32 tensors W, W^ [d][k] and X~ [k][n] in, (B' [d][r], A [r][k], sigma [r]) out.
    Allocates the outputs and the workspace with torch; every step of the computation runs in the library."""
    import torch
    d, k = w.shape
    n = x_tilde.shape[1]
    cfg = eora_solve_config(d, k, n, rank, oversample, iters)
    nbytes = eora_solve_workspace_bytes(cfg)
    if nbytes == 0:
        raise EoraError(EORA_ERR_BAD_SHAPE, "eora_solve_workspace_bytes")
    ws = torch.empty(nbytes, dtype=torch.uint8, device=w.device)
    b = torch.empty((d, rank), dtype=torch.float32, device=w.device)
    a = torch.empty((rank, k), dtype=torch.float32, device=w.device)
    sigma = torch.empty(rank, dtype=torch.float32, device=w.device)
    eora_solve(cfg, w.contiguous(), w_hat.contiguous(), x_tilde.contiguous(), b, a, sigma, ws, stream)
    return b, a, sigma


def solve_loss(w, w_hat, x_tilde, b_prime, a, stream=None) -> float:
    """|| (dW - B'A) X~ ||_F computed on the device (synchronises to return the value)."""
    import torch
    d, k = w.shape
    cfg = eora_solve_config(d, k, x_tilde.shape[1], b_prime.shape[1], 0, 0)
    ws = torch.empty(eora_solve_workspace_bytes(cfg), dtype=torch.uint8, device=w.device)
    out = torch.zeros(1, dtype=torch.float64, device=w.device)
    eora_solve_loss(cfg, w.contiguous(), w_hat.contiguous(), x_tilde.contiguous(), b_prime.contiguous(), a.contiguous(), out, ws, stream)
    torch.cuda.synchronize()
    return float(out.item()) ** 0.5
