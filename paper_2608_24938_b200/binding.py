"""ctypes binding of libexfold.so: argument marshalling only.

Every function has the name and the arguments of its C counterpart in include/exfold.h;
tensors are torch tensors whose data pointers are passed through. All computation happens
in the CUDA library; there is no fallback: if the library is missing, importing fails.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libexfold.so")

EXFOLD_F32, EXFOLD_BF16 = 0, 1
EXFOLD_OK = 0
EXFOLD_ERR_INVALID_ARG = -1
EXFOLD_ERR_UNSUPPORTED = -2
EXFOLD_ERR_WORKSPACE_TOO_SMALL = -3
EXFOLD_ERR_CUDA = -4
EXFOLD_ERR_DEVICE_TIMEOUT = -5
EXFOLD_ERR_EXCEEDS_STATIC_SCRATCH = -6
EXFOLD_STATIC_SCRATCH_BYTES = 8 << 20
EXFOLD_WARN_UNOBSERVED_EXPERT = 1

EXPORTS = ["exfold_workspace_bytes", "exfold_host_staging_bytes", "exfold_calibrate", "exfold_moe_prefill",
           "exfold_moe_decode", "exfold_moe_prefill_host", "exfold_moe_decode_host", "exfold_device_status",
           "exfold_status_string", "exfold_launch_count", "exfold_profile_enable", "exfold_profile_read",
           "exfold_moe_decode_noalloc", "exfold_static_pool_build", "exfold_moe_decode_static",
           "exfold_moe_prefill_ex", "exfold_router_logits", "exfold_calibrate_layers", "exfold_device_status_noalloc",
           "exfold_static_scratch_address", "exfold_thread_release", "exfold_moe_prefill_layer", "exfold_moe_decode_layer"]
PROFILE_SLOTS = ["prefill_route", "prefill_scan", "prefill_scatter", "gemm1_gateup_swiglu", "gemm2_down_combine",
                 "convert_bf16", "decode_route", "decode_gather", "decode_gateup", "decode_down", "simt_ffn",
                 "simt_combine", "gemm1_pair_pass", "gemm2_pair_pass", "decode_ffn"]


class exfold_layer(C.Structure):
    _fields_ = [("n_experts", C.c_int32), ("n_shared", C.c_int32), ("hidden", C.c_int32), ("inter", C.c_int32),
                ("top_k", C.c_int32), ("dtype", C.c_int32)]


class exfold_tables(C.Structure):
    _fields_ = [("S", C.c_void_p), ("L", C.c_void_p), ("h", C.c_void_p), ("lnh", C.c_void_p), ("n_obs", C.c_void_p)]


class exfold_calib_opts(C.Structure):
    _fields_ = [("lambda_", C.c_float), ("clip_lo", C.c_float), ("clip_hi", C.c_float), ("eps", C.c_float),
                ("mode", C.c_int32)]


class exfold_calib_job(C.Structure):
    _fields_ = [("x_cal", C.c_void_p), ("logits_cal", C.c_void_p), ("m", C.c_int64), ("w_gate", C.c_void_p),
                ("w_up", C.c_void_p), ("w_down", C.c_void_p), ("out", C.POINTER(exfold_tables))]


class exfold_prefill_meta(C.Structure):
    _fields_ = [("ids", C.c_void_p), ("w", C.c_void_p), ("omit_src", C.c_void_p), ("omit_tgt", C.c_void_p),
                ("perm", C.c_void_p), ("offsets", C.c_void_p)]


class exfold_decode_meta(C.Structure):
    _fields_ = [("pool_ids", C.c_void_p), ("pool_size", C.c_void_p), ("pool_mask", C.c_void_p), ("ids", C.c_void_p),
                ("w", C.c_void_p), ("target", C.c_void_p), ("scale", C.c_void_p)]


class exfold_fold_opts(C.Structure):
    _fields_ = [("loss_threshold", C.c_float), ("rescale", C.c_int32), ("confidence_split", C.c_int32),
                ("gemm_path", C.c_int32)]


class exfold_static_pool(C.Structure):
    _fields_ = [("pool_ids", C.c_void_p), ("target", C.c_void_p), ("scale", C.c_void_p), ("pool_m", C.c_int32)]


def _load() -> C.CDLL:
    if not os.path.exists(LIB_PATH):
        raise ImportError(f"{LIB_PATH} is missing: run `python -m paper_2608_24938_b200.build` "
                          "(there is no CPU or PyTorch fallback)")
    lib = C.CDLL(LIB_PATH)
    vp, i64, i32, sz = C.c_void_p, C.c_int64, C.c_int32, C.c_size_t
    lib.exfold_workspace_bytes.restype = sz
    lib.exfold_workspace_bytes.argtypes = [C.POINTER(exfold_layer), i64, i32]
    lib.exfold_host_staging_bytes.restype = sz
    lib.exfold_host_staging_bytes.argtypes = [C.POINTER(exfold_layer), i64]
    lib.exfold_calibrate.restype = C.c_int
    lib.exfold_calibrate.argtypes = [C.POINTER(exfold_layer), vp, vp, i64, vp, vp, vp, C.POINTER(exfold_calib_opts),
                                     C.POINTER(exfold_tables), vp, sz, vp]
    lib.exfold_calibrate_layers.restype = C.c_int
    lib.exfold_calibrate_layers.argtypes = [C.POINTER(exfold_layer), C.POINTER(exfold_calib_job), i32,
                                            C.POINTER(exfold_calib_opts), C.POINTER(C.c_int32), vp, sz, vp]
    for fn in (lib.exfold_moe_prefill, lib.exfold_moe_prefill_host):
        fn.restype = C.c_int
        fn.argtypes = [C.POINTER(exfold_layer), vp, vp, i64, vp, vp, vp, C.POINTER(exfold_tables), i32, vp,
                       C.POINTER(exfold_prefill_meta), vp, sz, vp]
    for fn in (lib.exfold_moe_decode, lib.exfold_moe_decode_host):
        fn.restype = C.c_int
        fn.argtypes = [C.POINTER(exfold_layer), vp, vp, i64, vp, vp, vp, C.POINTER(exfold_tables), i32, vp,
                       C.POINTER(exfold_decode_meta), vp, sz, vp]
    lib.exfold_moe_prefill_layer.restype = C.c_int
    lib.exfold_moe_prefill_layer.argtypes = [C.POINTER(exfold_layer), vp, vp, i64, vp, vp, vp, C.POINTER(exfold_tables),
                                             i32, vp, vp, C.POINTER(exfold_prefill_meta), vp, sz, vp]
    lib.exfold_moe_decode_layer.restype = C.c_int
    lib.exfold_moe_decode_layer.argtypes = [C.POINTER(exfold_layer), vp, vp, i64, vp, vp, vp, C.POINTER(exfold_tables),
                                            i32, vp, vp, C.POINTER(exfold_decode_meta), vp, sz, vp]
    lib.exfold_moe_decode_noalloc.restype = C.c_int
    lib.exfold_moe_decode_noalloc.argtypes = [C.POINTER(exfold_layer), vp, vp, i64, vp, vp, vp, C.POINTER(exfold_tables),
                                              i32, vp, C.POINTER(exfold_decode_meta), vp]
    lib.exfold_moe_prefill_ex.restype = C.c_int
    lib.exfold_moe_prefill_ex.argtypes = [C.POINTER(exfold_layer), vp, vp, i64, vp, vp, vp, C.POINTER(exfold_tables), i32,
                                          C.POINTER(exfold_fold_opts), vp, C.POINTER(exfold_prefill_meta), vp, sz, vp]
    lib.exfold_router_logits.restype = C.c_int
    lib.exfold_router_logits.argtypes = [C.POINTER(exfold_layer), vp, vp, i64, vp, vp, sz, vp]
    lib.exfold_static_pool_build.restype = C.c_int
    lib.exfold_static_pool_build.argtypes = [C.POINTER(exfold_layer), C.POINTER(exfold_tables), i32,
                                             C.POINTER(exfold_static_pool), vp]
    lib.exfold_moe_decode_static.restype = C.c_int
    lib.exfold_moe_decode_static.argtypes = [C.POINTER(exfold_layer), vp, vp, i64, vp, vp, vp,
                                             C.POINTER(exfold_static_pool), vp, C.POINTER(exfold_decode_meta), vp, sz, vp]
    lib.exfold_device_status.restype = C.c_int
    lib.exfold_device_status.argtypes = [vp, vp]
    lib.exfold_device_status_noalloc.restype = C.c_int
    lib.exfold_device_status_noalloc.argtypes = [vp]
    lib.exfold_static_scratch_address.restype = C.c_int
    lib.exfold_static_scratch_address.argtypes = [C.POINTER(vp)]
    lib.exfold_thread_release.restype = C.c_int
    lib.exfold_thread_release.argtypes = []
    lib.exfold_status_string.restype = C.c_char_p
    lib.exfold_status_string.argtypes = [C.c_int]
    lib.exfold_launch_count.restype = i64
    lib.exfold_launch_count.argtypes = []
    lib.exfold_profile_enable.restype = C.c_int
    lib.exfold_profile_enable.argtypes = [C.c_int]
    lib.exfold_profile_read.restype = C.c_int
    lib.exfold_profile_read.argtypes = [C.POINTER(C.c_float), i32]
    return lib


lib = _load()


class ExfoldError(RuntimeError):
    def __init__(self, code: int, what: str):
        super().__init__(f"{what}: {exfold_status_string(code)} ({code})")
        self.code = code


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    if t is None:
        return None
    assert t.is_contiguous(), "tensors passed to the library must be contiguous"
    return t.data_ptr()


def _stream(stream: Optional[torch.cuda.Stream]) -> int:
    return (stream or torch.cuda.current_stream()).cuda_stream


def make_layer(n_experts: int, n_shared: int, hidden: int, inter: int, top_k: int, dtype) -> exfold_layer:
    if isinstance(dtype, torch.dtype):
        dtype = {torch.float32: EXFOLD_F32, torch.bfloat16: EXFOLD_BF16}[dtype]
    elif isinstance(dtype, str):
        dtype = {"f32": EXFOLD_F32, "bf16": EXFOLD_BF16}[dtype]
    return exfold_layer(n_experts, n_shared, hidden, inter, top_k, dtype)


def make_tables(S, L, h, lnh, n_obs=None) -> exfold_tables:
    for t in (S, L, h, lnh):
        assert t.dtype == torch.float32
    return exfold_tables(_ptr(S), _ptr(L), _ptr(h), _ptr(lnh), _ptr(n_obs))


def exfold_status_string(code: int) -> str:
    return lib.exfold_status_string(code).decode()


def exfold_launch_count() -> int:
    return int(lib.exfold_launch_count())


def exfold_profile_enable(enable: bool) -> int:
    return int(lib.exfold_profile_enable(1 if enable else 0))


def exfold_profile_read() -> dict:
    """Milliseconds of each kernel of the last call (kernels that did not run are left out)."""
    n = len(PROFILE_SLOTS)
    buf = (C.c_float * n)()
    rc = lib.exfold_profile_read(buf, n)
    if rc != 0:
        raise ExfoldError(rc, "exfold_profile_read")
    return {PROFILE_SLOTS[i]: float(buf[i]) for i in range(n) if buf[i] >= 0}


def exfold_workspace_bytes(layer: exfold_layer, max_tokens: int, routes_per_token: int) -> int:
    return int(lib.exfold_workspace_bytes(C.byref(layer), max_tokens, routes_per_token))


def exfold_host_staging_bytes(layer: exfold_layer, max_tokens: int) -> int:
    return int(lib.exfold_host_staging_bytes(C.byref(layer), max_tokens))


def alloc_workspace(layer: exfold_layer, max_tokens: int, routes_per_token: int, device="cuda",
                    host_staging: bool = False) -> torch.Tensor:
    n = exfold_workspace_bytes(layer, max_tokens, routes_per_token)
    if n == 0:
        raise ExfoldError(EXFOLD_ERR_INVALID_ARG, "exfold_workspace_bytes")
    if host_staging:
        n += exfold_host_staging_bytes(layer, max_tokens)
    return torch.empty(n, dtype=torch.uint8, device=device)


def exfold_router_logits(layer, x, w_router, logits, ws, stream=None) -> int:
    return int(lib.exfold_router_logits(C.byref(layer), _ptr(x), _ptr(w_router), x.shape[0], _ptr(logits), _ptr(ws),
                                        ws.numel(), _stream(stream)))


def exfold_device_status(ws: torch.Tensor, stream=None) -> int:
    return int(lib.exfold_device_status(_ptr(ws), _stream(stream)))


def exfold_device_status_noalloc(stream=None) -> int:
    return int(lib.exfold_device_status_noalloc(_stream(stream)))


def exfold_static_scratch_address() -> int:
    out = C.c_void_p()
    rc = lib.exfold_static_scratch_address(C.byref(out))
    if rc != 0:
        raise ExfoldError(rc, "exfold_static_scratch_address")
    return int(out.value)


def exfold_thread_release() -> int:
    return int(lib.exfold_thread_release())


def exfold_calibrate(layer, x_cal, logits_cal, w_gate, w_up, w_down, out: exfold_tables, ws, lam=1e-3,
                     clip_lo=-4.0, clip_hi=4.0, eps=1e-12, mode=0, stream=None) -> int:
    opts = exfold_calib_opts(lam, clip_lo, clip_hi, eps, mode)
    rc = lib.exfold_calibrate(C.byref(layer), _ptr(x_cal), _ptr(logits_cal), x_cal.shape[0], _ptr(w_gate),
                              _ptr(w_up), _ptr(w_down), C.byref(opts), C.byref(out), _ptr(ws), ws.numel(),
                              _stream(stream))
    if rc < 0:
        raise ExfoldError(rc, "exfold_calibrate")
    return rc


def exfold_calibrate_layers(layer, jobs, ws, lam=1e-3, clip_lo=-4.0, clip_hi=4.0, eps=1e-12, mode=0, stream=None):
    """jobs: sequence of (x_cal, logits_cal, w_gate, w_up, w_down, out_tables). Returns (status, unobserved per job)."""
    opts = exfold_calib_opts(lam, clip_lo, clip_hi, eps, mode)
    arr = (exfold_calib_job * len(jobs))()
    for j, (x_cal, logits_cal, w_gate, w_up, w_down, out) in enumerate(jobs):
        arr[j] = exfold_calib_job(_ptr(x_cal), _ptr(logits_cal), x_cal.shape[0], _ptr(w_gate), _ptr(w_up),
                                  _ptr(w_down), C.pointer(out))
    un = (C.c_int32 * len(jobs))()
    rc = lib.exfold_calibrate_layers(C.byref(layer), arr, len(jobs), C.byref(opts), un, _ptr(ws), ws.numel(),
                                     _stream(stream))
    if rc < 0:
        raise ExfoldError(rc, "exfold_calibrate_layers")
    return rc, list(un)


def _prefill_meta(meta: Optional[dict]):
    if not meta:
        return None
    return C.byref(exfold_prefill_meta(*[_ptr(meta.get(k)) for k in
                                         ("ids", "w", "omit_src", "omit_tgt", "perm", "offsets")]))


def _decode_meta(meta: Optional[dict]):
    if not meta:
        return None
    return C.byref(exfold_decode_meta(*[_ptr(meta.get(k)) for k in
                                        ("pool_ids", "pool_size", "pool_mask", "ids", "w", "target", "scale")]))


def exfold_moe_prefill(layer, x, logits, w_gate, w_up, w_down, tables: exfold_tables, k_pre: int, y, ws,
                       meta: Optional[dict] = None, stream=None, check: bool = True) -> int:
    rc = lib.exfold_moe_prefill(C.byref(layer), _ptr(x), _ptr(logits), x.shape[0], _ptr(w_gate), _ptr(w_up),
                                _ptr(w_down), C.byref(tables), k_pre, _ptr(y), _prefill_meta(meta), _ptr(ws),
                                ws.numel(), _stream(stream))
    if check and rc != 0:
        raise ExfoldError(rc, "exfold_moe_prefill")
    return rc


def exfold_moe_decode(layer, x, logits, w_gate, w_up, w_down, tables: exfold_tables, pool_m: int, y, ws,
                      meta: Optional[dict] = None, stream=None, check: bool = True) -> int:
    rc = lib.exfold_moe_decode(C.byref(layer), _ptr(x), _ptr(logits), x.shape[0], _ptr(w_gate), _ptr(w_up),
                               _ptr(w_down), C.byref(tables), pool_m, _ptr(y), _decode_meta(meta), _ptr(ws),
                               ws.numel(), _stream(stream))
    if check and rc != 0:
        raise ExfoldError(rc, "exfold_moe_decode")
    return rc


def exfold_moe_prefill_layer(layer, x, w_router, w_gate, w_up, w_down, tables: exfold_tables, k_pre: int, y, ws,
                             logits_out, meta: Optional[dict] = None, stream=None, check: bool = True) -> int:
    rc = lib.exfold_moe_prefill_layer(C.byref(layer), _ptr(x), _ptr(w_router), x.shape[0], _ptr(w_gate), _ptr(w_up),
                                      _ptr(w_down), C.byref(tables), k_pre, _ptr(logits_out), _ptr(y),
                                      _prefill_meta(meta), _ptr(ws), ws.numel(), _stream(stream))
    if check and rc != 0:
        raise ExfoldError(rc, "exfold_moe_prefill_layer")
    return rc


def exfold_moe_decode_layer(layer, x, w_router, w_gate, w_up, w_down, tables: exfold_tables, pool_m: int, y, ws,
                            logits_out, meta: Optional[dict] = None, stream=None, check: bool = True) -> int:
    rc = lib.exfold_moe_decode_layer(C.byref(layer), _ptr(x), _ptr(w_router), x.shape[0], _ptr(w_gate), _ptr(w_up),
                                     _ptr(w_down), C.byref(tables), pool_m, _ptr(logits_out), _ptr(y),
                                     _decode_meta(meta), _ptr(ws), ws.numel(), _stream(stream))
    if check and rc != 0:
        raise ExfoldError(rc, "exfold_moe_decode_layer")
    return rc


def exfold_moe_prefill_host(layer, x_host, logits_host, w_gate, w_up, w_down, tables, k_pre, y_host, ws,
                            meta=None, stream=None, check: bool = True) -> int:
    rc = lib.exfold_moe_prefill_host(C.byref(layer), _ptr(x_host), _ptr(logits_host), x_host.shape[0], _ptr(w_gate),
                                     _ptr(w_up), _ptr(w_down), C.byref(tables), k_pre, _ptr(y_host),
                                     _prefill_meta(meta), _ptr(ws), ws.numel(), _stream(stream))
    if check and rc != 0:
        raise ExfoldError(rc, "exfold_moe_prefill_host")
    return rc


def exfold_moe_decode_host(layer, x_host, logits_host, w_gate, w_up, w_down, tables, pool_m, y_host, ws,
                           meta=None, stream=None, check: bool = True) -> int:
    rc = lib.exfold_moe_decode_host(C.byref(layer), _ptr(x_host), _ptr(logits_host), x_host.shape[0], _ptr(w_gate),
                                    _ptr(w_up), _ptr(w_down), C.byref(tables), pool_m, _ptr(y_host),
                                    _decode_meta(meta), _ptr(ws), ws.numel(), _stream(stream))
    if check and rc != 0:
        raise ExfoldError(rc, "exfold_moe_decode_host")
    return rc


def exfold_moe_decode_noalloc(layer, x, logits, w_gate, w_up, w_down, tables: exfold_tables, pool_m: int, y,
                              meta: Optional[dict] = None, stream=None, check: bool = True) -> int:
    """Decode without a caller workspace, for hosts that may not allocate device memory: the scratch is
    the library's own fixed array (EXFOLD_STATIC_SCRATCH_BYTES per GPU). Same results as
    exfold_moe_decode. Calls on one device share that array, so keep them ordered on one stream; make
    the first call on a device outside any stream capture."""
    rc = lib.exfold_moe_decode_noalloc(C.byref(layer), _ptr(x), _ptr(logits), x.shape[0], _ptr(w_gate), _ptr(w_up),
                                       _ptr(w_down), C.byref(tables), pool_m, _ptr(y), _decode_meta(meta),
                                       _stream(stream))
    if check and rc != 0:
        raise ExfoldError(rc, "exfold_moe_decode_noalloc")
    return rc


def exfold_static_pool_build(layer, tables: exfold_tables, pool_m: int, pool_ids, target, scale,
                             stream=None) -> exfold_static_pool:
    """Fills the caller's device arrays pool_ids [M], target [N], scale [N] and returns the struct to pass to
    exfold_moe_decode_static (the tensors must stay alive as long as the struct is used)."""
    sp = exfold_static_pool(_ptr(pool_ids), _ptr(target), _ptr(scale), pool_m)
    rc = lib.exfold_static_pool_build(C.byref(layer), C.byref(tables), pool_m, C.byref(sp), _stream(stream))
    if rc != 0:
        raise ExfoldError(rc, "exfold_static_pool_build")
    return sp


def exfold_moe_decode_static(layer, x, logits, w_gate, w_up, w_down, pool: exfold_static_pool, y, ws,
                             meta: Optional[dict] = None, stream=None, check: bool = True) -> int:
    rc = lib.exfold_moe_decode_static(C.byref(layer), _ptr(x), _ptr(logits), x.shape[0], _ptr(w_gate), _ptr(w_up),
                                      _ptr(w_down), C.byref(pool), _ptr(y), _decode_meta(meta), _ptr(ws), ws.numel(),
                                      _stream(stream))
    if check and rc != 0:
        raise ExfoldError(rc, "exfold_moe_decode_static")
    return rc


def exfold_moe_prefill_ex(layer, x, logits, w_gate, w_up, w_down, tables: exfold_tables, k_pre: int, y, ws,
                          loss_threshold: float = float("inf"), rescale: bool = False, confidence_split: bool = False,
                          gemm_path: int = 0, meta: Optional[dict] = None, stream=None, check: bool = True) -> int:
    opts = exfold_fold_opts(loss_threshold, int(rescale), int(confidence_split), int(gemm_path))
    rc = lib.exfold_moe_prefill_ex(C.byref(layer), _ptr(x), _ptr(logits), x.shape[0], _ptr(w_gate), _ptr(w_up),
                                   _ptr(w_down), C.byref(tables), k_pre, C.byref(opts), _ptr(y), _prefill_meta(meta),
                                   _ptr(ws), ws.numel(), _stream(stream))
    if check and rc != 0:
        raise ExfoldError(rc, "exfold_moe_prefill_ex")
    return rc
