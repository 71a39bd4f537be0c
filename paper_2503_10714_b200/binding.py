"""ctypes binding of libzsm.so: the same entry points as include/zsm.h.

Argument marshalling only -- every step of the path runs in the library's CUDA
kernels.  There is no fallback: if the shared library is missing the import of
this module raises.  torch is used for device memory and streams.

The C library takes raw pointers and cannot know how large a tensor behind one is,
so this layer checks every tensor (device, contiguity, dtype, element count)
against the cache's configuration before it hands the pointer over, and raises
TypeError / ValueError instead of letting a wrong tensor become an out-of-bounds
access on the device.
"""
from __future__ import annotations

import ctypes as C
import os

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libzsm.so")

ZSM_OK = 0
ZSM_ERR_INVALID_ARG = 1
ZSM_ERR_BUFFER_TOO_SMALL = 2
ZSM_ERR_STATE = 3
ZSM_ERR_CUDA = 4
ZSM_ERR_UNSUPPORTED = 5
ZSM_ERR_DEVICE_CHECK = 6
ZSM_ERR_TIMEOUT = 7
ZSM_ERR_NO_MEMORY = 8
ZSM_F32, ZSM_F16, ZSM_BF16 = 0, 1, 2
DTYPE_CODE = {"f32": ZSM_F32, "f16": ZSM_F16, "bf16": ZSM_BF16,
              torch.float32: ZSM_F32, torch.float16: ZSM_F16, torch.bfloat16: ZSM_BF16}

# every symbol include/zsm.h declares
SYMBOLS = ["zsm_split_budget", "zsm_cache_bytes", "zsm_cache_create", "zsm_cache_reset",
           "zsm_cache_free", "zsm_prefill_workspace_bytes", "zsm_prefill_compress",
           "zsm_prefill_compress_static", "zsm_prefill_scores_full_workspace_bytes",
           "zsm_prefill_scores_full", "zsm_fullkv_workspace_bytes", "zsm_fullkv_decode",
           "zsm_fullkv_status",
           "zsm_decode_step", "zsm_decode_staging_bytes", "zsm_decode_step_host",
           "zsm_unit_capacity", "zsm_cache_export_unit", "zsm_cache_import_unit",
           "zsm_last_device_status", "zsm_decode_launch_info", "zsm_status_string",
           "zsm_selftest_wait_timeout", "zsm_decode_host_layout", "zsm_decode_step_host_async",
           "zsm_decode_step_host_wait", "zsm_prefill_attention"]


class ZsmConfig(C.Structure):
    _fields_ = [("n_layers", C.c_int32), ("batch", C.c_int32), ("n_q_heads", C.c_int32),
                ("n_kv_heads", C.c_int32), ("head_dim", C.c_int32), ("dtype", C.c_int32),
                ("budget_p", C.POINTER(C.c_int32)), ("budget_c", C.POINTER(C.c_int32)),
                ("budget_r", C.POINTER(C.c_int32)), ("lam", C.c_float), ("alpha", C.c_float),
                ("softmax_scale", C.c_float), ("tune_stages", C.c_int32),
                ("tune_ctas_per_sm", C.c_int32), ("tune_consumer_warps", C.c_int32),
                ("tune_split", C.c_int32), ("similarity", C.c_int32)]


class ZsmError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {zsm_status_string(status)} (status {status})")


if not os.path.exists(LIB_PATH):
    raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2503_10714_b200.build`"
                      " (there is no CPU or PyTorch fallback)")
_lib = C.CDLL(LIB_PATH)
_vp, _i32, _sz = C.c_void_p, C.c_int32, C.c_size_t
_pi32 = C.POINTER(C.c_int32)
_lib.zsm_status_string.restype = C.c_char_p
_lib.zsm_status_string.argtypes = [C.c_int]
_lib.zsm_split_budget.argtypes = [_i32, C.c_float, C.c_float, _pi32, _pi32, _pi32]
_lib.zsm_cache_bytes.argtypes = [C.POINTER(ZsmConfig), C.POINTER(_sz)]
_lib.zsm_cache_create.argtypes = [C.POINTER(ZsmConfig), _vp, _sz, C.POINTER(_vp)]
_lib.zsm_cache_reset.argtypes = [_vp, _vp]
_lib.zsm_cache_free.argtypes = [_vp]
_lib.zsm_prefill_workspace_bytes.argtypes = [_vp, _i32, _i32, C.POINTER(_sz)]
_lib.zsm_prefill_compress.argtypes = [_vp, _i32, _vp, _vp, _vp, _vp, _i32, _i32, _vp, _sz, _vp,
                                      _vp, _vp, _vp]
_lib.zsm_prefill_compress_static.argtypes = [_vp, _i32, _vp, _vp, _vp, _vp, _i32, _i32, _vp, _vp,
                                             _vp, _vp]
_lib.zsm_prefill_scores_full_workspace_bytes.argtypes = [_vp, _i32, C.POINTER(_sz)]
_lib.zsm_prefill_scores_full.argtypes = [_vp, _vp, _vp, _vp, _i32, _vp, _vp, _sz, _vp]
_lib.zsm_prefill_attention.argtypes = [_vp, _vp, _vp, _vp, _i32, _vp, _vp, _vp, _vp]
_lib.zsm_decode_step.argtypes = [_vp, _i32, _vp, _vp, _vp, _vp, _vp, _vp, _vp]
_lib.zsm_fullkv_workspace_bytes.argtypes = [_i32, _i32, _i32, _i32, C.POINTER(_sz)]
_lib.zsm_fullkv_decode.argtypes = [_i32, _i32, _i32, _i32, _i32, _vp, _vp, _vp, _vp, C.c_float, _vp,
                                   _sz, _vp]
_lib.zsm_fullkv_status.argtypes = [_vp, _vp]
_lib.zsm_decode_staging_bytes.argtypes = [_vp, _i32, C.POINTER(_sz)]
_lib.zsm_decode_step_host.argtypes = [_vp, _i32, _vp, _vp, _vp, _vp, _vp, _sz, _vp]
_lib.zsm_decode_host_layout.argtypes = [_vp, _i32] + [C.POINTER(_sz)] * 5
_lib.zsm_decode_step_host_async.argtypes = [_vp, _i32, _vp, _vp, _vp, _sz, _i32, _vp]
_lib.zsm_decode_step_host_wait.argtypes = [_vp, _i32]
_lib.zsm_unit_capacity.argtypes = [_vp, _i32, _i32, _pi32, _pi32]
_lib.zsm_cache_export_unit.argtypes = [_vp, _i32, _i32, _i32] + [_vp] * 8 + [_vp]
_lib.zsm_cache_import_unit.argtypes = [_vp, _i32, _i32, _i32] + [_vp] * 8 + [_vp]
_lib.zsm_last_device_status.argtypes = [_vp, _vp]
_lib.zsm_selftest_wait_timeout.argtypes = [_vp, C.c_uint32, _vp]
_lib.zsm_decode_launch_info.argtypes = [_vp, _i32, _pi32, _pi32, _pi32]
for _name in SYMBOLS:
    if _name != "zsm_status_string":
        getattr(_lib, _name).restype = C.c_int


def _check(status: int, where: str):
    if status != ZSM_OK:
        raise ZsmError(status, where)


def _stream(stream=None):
    if stream is None:
        stream = torch.cuda.current_stream()
    return C.c_void_p(stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream))


_TORCH_OF_CODE = {ZSM_F32: torch.float32, ZSM_F16: torch.float16, ZSM_BF16: torch.bfloat16}


class Cache:
    """What zsm_cache_create returns: the C handle (passed on wherever a `cache` argument is
    expected), the shape the checks below need, and a reference to the device buffer so that
    it outlives the handle."""

    def __init__(self, handle, cfg: ZsmConfig, dev_buf: torch.Tensor):
        self._as_parameter_ = handle
        self.buf = dev_buf
        self.device = dev_buf.device
        self.n_layers, self.batch = cfg.n_layers, cfg.batch
        self.n_q_heads, self.n_kv_heads, self.head_dim = cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim
        self.group = cfg.n_q_heads // cfg.n_kv_heads
        self.torch_dtype = _TORCH_OF_CODE[cfg.dtype]
        self._cfg = cfg  # keeps the budget arrays alive

    def units(self, layer: int) -> int:
        per_layer = self.batch * self.n_kv_heads
        return per_layer * self.n_layers if layer < 0 else per_layer


def _layer_arg(cache: "Cache", layer, allow_all: bool) -> int:
    layer = int(layer)
    if layer < (-1 if allow_all else 0) or layer >= cache.n_layers:
        raise ZsmError(ZSM_ERR_INVALID_ARG, f"layer {layer} of {cache.n_layers}")
    return layer


def _dev(t, name="tensor", dtype=None, numel=None, device=None):
    """Pointer of a device tensor after checking it is what the call will read or write."""
    if t is None:
        return None
    if not isinstance(t, torch.Tensor) or not t.is_cuda:
        raise TypeError(f"{name}: a CUDA tensor is required")
    if not t.is_contiguous():
        raise ValueError(f"{name}: tensor must be contiguous")
    if device is not None and t.device != device:
        raise ValueError(f"{name}: on {t.device}, the cache is on {device}")
    if dtype is not None and t.dtype != dtype:
        raise TypeError(f"{name}: dtype {t.dtype}, expected {dtype}")
    if numel is not None and t.numel() < numel:
        raise ValueError(f"{name}: {t.numel()} elements, the call needs {numel}")
    return C.c_void_p(t.data_ptr())


def _host(a, name="array", dtype=None, numel=None):
    if a is None:
        return None
    if isinstance(a, torch.Tensor):
        if a.is_cuda or not a.is_contiguous():
            raise ValueError(f"{name}: a contiguous host tensor is required")
        if dtype is not None and a.dtype != dtype:
            raise TypeError(f"{name}: dtype {a.dtype}, expected {dtype}")
        if numel is not None and a.numel() < numel:
            raise ValueError(f"{name}: {a.numel()} elements, the call needs {numel}")
        return C.c_void_p(a.data_ptr())
    if not a.flags["C_CONTIGUOUS"]:
        raise ValueError(f"{name}: array must be C-contiguous")
    if numel is not None and a.size < numel:
        raise ValueError(f"{name}: {a.size} elements, the call needs {numel}")
    return C.c_void_p(a.ctypes.data)


def _nbytes(t) -> int:
    return 0 if t is None else t.numel() * t.element_size()


def zsm_status_string(status: int) -> str:
    return _lib.zsm_status_string(int(status)).decode()


def zsm_split_budget(B: int, tail_ratio: float = 0.5, dense_ratio: float = 0.02):
    bp, bc, br = C.c_int32(), C.c_int32(), C.c_int32()
    _check(_lib.zsm_split_budget(int(B), float(tail_ratio), float(dense_ratio), C.byref(bp),
                                 C.byref(bc), C.byref(br)), "zsm_split_budget")
    return bp.value, bc.value, br.value


def make_config(n_layers, batch, n_q_heads, n_kv_heads, head_dim, dtype, budget_p, budget_c,
                budget_r, lam=0.98, alpha=1.0, softmax_scale=0.0, tune_stages=0,
                tune_ctas_per_sm=0, tune_consumer_warps=0, tune_split=0, similarity=0):
    """Builds a zsm_config_t; the budget arrays are kept alive on the returned object."""
    arrs = [np.ascontiguousarray(np.asarray(a, dtype=np.int32).reshape(-1))
            for a in (budget_p, budget_c, budget_r)]
    cfg = ZsmConfig(int(n_layers), int(batch), int(n_q_heads), int(n_kv_heads), int(head_dim),
                    int(DTYPE_CODE[dtype]), arrs[0].ctypes.data_as(_pi32),
                    arrs[1].ctypes.data_as(_pi32), arrs[2].ctypes.data_as(_pi32), float(lam),
                    float(alpha), float(softmax_scale), int(tune_stages), int(tune_ctas_per_sm),
                    int(tune_consumer_warps), int(tune_split), int(similarity))
    cfg._keep = arrs
    return cfg


def zsm_cache_bytes(cfg: ZsmConfig) -> int:
    n = _sz()
    _check(_lib.zsm_cache_bytes(C.byref(cfg), C.byref(n)), "zsm_cache_bytes")
    return n.value


def zsm_cache_create(cfg: ZsmConfig, dev_buf: torch.Tensor) -> Cache:
    h = _vp()
    _check(_lib.zsm_cache_create(C.byref(cfg), _dev(dev_buf, "dev_buf"), _nbytes(dev_buf), C.byref(h)),
           "zsm_cache_create")
    return Cache(h, cfg, dev_buf)


def zsm_cache_reset(cache, stream=None):
    _check(_lib.zsm_cache_reset(cache, _stream(stream)), "zsm_cache_reset")


def zsm_cache_free(cache):
    _check(_lib.zsm_cache_free(cache), "zsm_cache_free")
    if isinstance(cache, Cache):
        cache._as_parameter_ = None   # a freed handle must never reach the library again


def zsm_prefill_workspace_bytes(cache, T: int, W: int) -> int:
    n = _sz()
    _check(_lib.zsm_prefill_workspace_bytes(cache, int(T), int(W), C.byref(n)),
           "zsm_prefill_workspace_bytes")
    return n.value


def _prefill_args(cache: Cache, layer, K, V, Qw, scores, T, W, dbg_scores, dbg_evicted, dbg_targets):
    layer, T, W = _layer_arg(cache, layer, False), int(T), int(W)
    if T < 1 or (Qw is not None and not 1 <= W <= T):
        raise ZsmError(ZSM_ERR_INVALID_ARG, f"T = {T}, W = {W}")
    dt, dev, d = cache.torch_dtype, cache.device, cache.head_dim
    rows = cache.batch * cache.n_kv_heads * T
    return (layer, _dev(K, "K", dt, rows * d, dev), _dev(V, "V", dt, rows * d, dev),
            _dev(Qw, "Qw", dt, cache.batch * cache.n_q_heads * W * d, dev),
            _dev(scores, "scores", torch.float32, rows, dev), T, W,
            _dev(dbg_scores, "dbg_scores", torch.float32, rows, dev),
            _dev(dbg_evicted, "dbg_evicted", torch.uint8, rows, dev),
            _dev(dbg_targets, "dbg_targets", torch.int32, rows, dev))


def zsm_prefill_compress(cache, layer, K, V, Qw, scores, T, W, workspace, dbg_scores=None,
                         dbg_evicted=None, dbg_targets=None, stream=None):
    layer, pK, pV, pQ, pS, T, W, d1, d2, d3 = _prefill_args(cache, layer, K, V, Qw, scores, T, W,
                                                           dbg_scores, dbg_evicted, dbg_targets)
    _check(_lib.zsm_prefill_compress(cache, layer, pK, pV, pQ, pS, T, W,
                                     _dev(workspace, "workspace", device=cache.device),
                                     _nbytes(workspace), d1, d2, d3, _stream(stream)),
           "zsm_prefill_compress")


ZSM_STATIC_SCRATCH_BYTES = 16 << 20


def zsm_prefill_compress_static(cache, layer, K, V, Qw, scores, T, W, dbg_scores=None,
                                dbg_evicted=None, dbg_targets=None, stream=None):
    """zsm_prefill_compress with the library's own fixed scratch array instead of a workspace
    tensor, for callers that cannot allocate device memory at the time of the call.  Raises
    ZsmError(ZSM_ERR_BUFFER_TOO_SMALL) when the prompt needs more than
    ZSM_STATIC_SCRATCH_BYTES; calls on different streams must not overlap."""
    need = zsm_prefill_workspace_bytes(cache, T, W if Qw is not None else 0)
    if need > ZSM_STATIC_SCRATCH_BYTES:   # before any tensor is looked at, as in the library
        raise ZsmError(ZSM_ERR_BUFFER_TOO_SMALL, "zsm_prefill_compress_static")
    layer, pK, pV, pQ, pS, T, W, d1, d2, d3 = _prefill_args(cache, layer, K, V, Qw, scores, T, W,
                                                           dbg_scores, dbg_evicted, dbg_targets)
    _check(_lib.zsm_prefill_compress_static(cache, layer, pK, pV, pQ, pS, T, W, d1, d2, d3,
                                            _stream(stream)), "zsm_prefill_compress_static")


def zsm_prefill_scores_full_workspace_bytes(cache, T: int) -> int:
    n = _sz()
    _check(_lib.zsm_prefill_scores_full_workspace_bytes(cache, int(T), C.byref(n)),
           "zsm_prefill_scores_full_workspace_bytes")
    return n.value


def zsm_prefill_scores_full(cache, K, Q, T, scores, workspace=None, lse=None, stream=None):
    """Full-history prompt scores (every prompt query scores every earlier key) into `scores`
    fp32 [batch][n_kv_heads][T]; `lse` optionally supplies the rows' log-sum-exp."""
    T = int(T)
    dt, dev, d = cache.torch_dtype, cache.device, cache.head_dim
    _check(_lib.zsm_prefill_scores_full(
        cache, _dev(K, "K", dt, cache.batch * cache.n_kv_heads * T * d, dev),
        _dev(Q, "Q", dt, cache.batch * cache.n_q_heads * T * d, dev),
        _dev(lse, "lse", torch.float32, cache.batch * cache.n_q_heads * T, dev), T,
        _dev(scores, "scores", torch.float32, cache.batch * cache.n_kv_heads * T, dev),
        _dev(workspace, "workspace", device=dev), _nbytes(workspace), _stream(stream)),
        "zsm_prefill_scores_full")


def zsm_prefill_attention(cache, K, V, Q, T, out, lse, scores=None, stream=None):
    """Causal prefill attention of a prompt: writes `out` [batch][n_q_heads][T][d] (cache dtype),
    `lse` fp32 [batch][n_q_heads][T] and, if given, the full-history `scores`
    fp32 [batch][n_kv_heads][T]."""
    T = int(T)
    dt, dev, d = cache.torch_dtype, cache.device, cache.head_dim
    nk, nq = cache.batch * cache.n_kv_heads * T, cache.batch * cache.n_q_heads * T
    _check(_lib.zsm_prefill_attention(
        cache, _dev(K, "K", dt, nk * d, dev), _dev(V, "V", dt, nk * d, dev), _dev(Q, "Q", dt, nq * d, dev), T,
        _dev(out, "out", dt, nq * d, dev), _dev(lse, "lse", torch.float32, nq, dev),
        _dev(scores, "scores", torch.float32, nk, dev), _stream(stream)), "zsm_prefill_attention")


def _decode_args(cache: Cache, layer, q, k_new, v_new, out, host: bool):
    layer = _layer_arg(cache, layer, True)
    nu, d, dt = cache.units(layer), cache.head_dim, cache.torch_dtype
    if host:
        return (layer, _host(q, "q", dt, nu * cache.group * d), _host(k_new, "k_new", dt, nu * d),
                _host(v_new, "v_new", dt, nu * d), _host(out, "out", dt, nu * cache.group * d))
    dev = cache.device
    return (layer, _dev(q, "q", dt, nu * cache.group * d, dev), _dev(k_new, "k_new", dt, nu * d, dev),
            _dev(v_new, "v_new", dt, nu * d, dev), _dev(out, "out", dt, nu * cache.group * d, dev))


def zsm_decode_step(cache, layer, q, k_new, v_new, out, victim_pos=None, merge_slot=None,
                    stream=None):
    layer, pq, pk, pv, po = _decode_args(cache, layer, q, k_new, v_new, out, host=False)
    nu = cache.units(layer)
    _check(_lib.zsm_decode_step(cache, layer, pq, pk, pv, po,
                                _dev(victim_pos, "victim_pos", torch.int32, nu, cache.device),
                                _dev(merge_slot, "merge_slot", torch.int32, nu, cache.device),
                                _stream(stream)), "zsm_decode_step")


def zsm_fullkv_workspace_bytes(n_units: int, group: int, head_dim: int, T: int) -> int:
    n = _sz()
    _check(_lib.zsm_fullkv_workspace_bytes(int(n_units), int(group), int(head_dim), int(T),
                                           C.byref(n)), "zsm_fullkv_workspace_bytes")
    return n.value


def zsm_fullkv_decode(K, V, q, out, workspace, softmax_scale=0.0, stream=None):
    """Plain decode attention over an uncompressed cache: K, V [units, T, d]; q, out
    [units, G, d] device tensors of one 16-bit dtype."""
    n_units, T, d = K.shape
    G = q.shape[1]
    if tuple(V.shape) != (n_units, T, d) or tuple(q.shape) != (n_units, G, d) or \
            tuple(out.shape) != (n_units, G, d):
        raise ValueError("zsm_fullkv_decode: K, V [units, T, d] and q, out [units, G, d] disagree")
    dt, dev = K.dtype, K.device
    _check(_lib.zsm_fullkv_decode(int(DTYPE_CODE[dt]), int(n_units), int(G), int(d), int(T),
                                  _dev(K, "K"), _dev(V, "V", dt, device=dev), _dev(q, "q", dt, device=dev),
                                  _dev(out, "out", dt, device=dev), float(softmax_scale),
                                  _dev(workspace, "workspace", device=dev), _nbytes(workspace),
                                  _stream(stream)), "zsm_fullkv_decode")


def zsm_fullkv_status(workspace, stream=None) -> int:
    return int(_lib.zsm_fullkv_status(_dev(workspace, "workspace"), _stream(stream)))


def zsm_decode_staging_bytes(cache, layer) -> int:
    n = _sz()
    _check(_lib.zsm_decode_staging_bytes(cache, int(layer), C.byref(n)), "zsm_decode_staging_bytes")
    return n.value


def zsm_decode_step_host(cache, layer, q_host, k_new_host, v_new_host, out_host, staging,
                         stream=None):
    layer, pq, pk, pv, po = _decode_args(cache, layer, q_host, k_new_host, v_new_host, out_host,
                                         host=True)
    _check(_lib.zsm_decode_step_host(cache, layer, pq, pk, pv, po,
                                     _dev(staging, "staging", device=cache.device), _nbytes(staging),
                                     _stream(stream)), "zsm_decode_step_host")


def zsm_decode_host_layout(cache, layer):
    """(q_off, k_off, v_off, in_bytes, out_bytes) of the packed host input of the pipelined step."""
    v = [_sz() for _ in range(5)]
    _check(_lib.zsm_decode_host_layout(cache, _layer_arg(cache, layer, True), *[C.byref(x) for x in v]),
           "zsm_decode_host_layout")
    return tuple(x.value for x in v)


def zsm_decode_step_host_async(cache, layer, in_host, out_host, staging, slot, stream=None):
    """Enqueues one pipelined host-buffer step on staging half `slot` (0 or 1): in_host is a pinned
    uint8 tensor laid out by zsm_decode_host_layout, out_host a pinned tensor of the cache's dtype."""
    layer = _layer_arg(cache, layer, True)
    _, _, _, in_bytes, out_bytes = zsm_decode_host_layout(cache, layer)
    for name, t in (("in_host", in_host), ("out_host", out_host)):
        if not isinstance(t, torch.Tensor) or t.is_cuda or not t.is_contiguous() or not t.is_pinned():
            raise TypeError(f"{name}: a contiguous pinned host tensor is required")
    if _nbytes(in_host) < in_bytes or _nbytes(out_host) < out_bytes:
        raise ValueError("zsm_decode_step_host_async: host buffer smaller than zsm_decode_host_layout says")
    _check(_lib.zsm_decode_step_host_async(cache, layer, C.c_void_p(in_host.data_ptr()),
                                           C.c_void_p(out_host.data_ptr()),
                                           _dev(staging, "staging", device=cache.device),
                                           _nbytes(staging), int(slot), _stream(stream)),
           "zsm_decode_step_host_async")


def zsm_decode_step_host_wait(cache, slot):
    _check(_lib.zsm_decode_step_host_wait(cache, int(slot)), "zsm_decode_step_host_wait")


def zsm_unit_capacity(cache, layer, h):
    a, b = C.c_int32(), C.c_int32()
    _check(_lib.zsm_unit_capacity(cache, int(layer), int(h), C.byref(a), C.byref(b)),
           "zsm_unit_capacity")
    return a.value, b.value


def zsm_cache_export_unit(cache, layer, b, h, head_dim, stream=None):
    """Returns a dict of numpy arrays: K, V, score, pos (live rows only), Kr, Vr, w (used
    slots only), n_live, n_res, T."""
    cap, br = zsm_unit_capacity(cache, layer, h)
    K = np.empty((cap, head_dim), np.float32)
    V = np.empty((cap, head_dim), np.float32)
    score = np.empty(cap, np.float32)
    pos = np.empty(cap, np.int32)
    Kr = np.empty((br, head_dim), np.float32)
    Vr = np.empty((br, head_dim), np.float32)
    w = np.empty(br, np.uint32)
    cnt = np.zeros(3, np.int32)
    _check(_lib.zsm_cache_export_unit(cache, int(layer), int(b), int(h), _host(K), _host(V),
                                      _host(score), _host(pos), _host(Kr), _host(Vr), _host(w),
                                      _host(cnt), _stream(stream)), "zsm_cache_export_unit")
    n, r = int(cnt[0]), int(cnt[1])
    return dict(K=K[:n], V=V[:n], score=score[:n], pos=pos[:n], Kr=Kr[:r], Vr=Vr[:r], w=w[:r],
                n_live=n, n_res=r, T=int(cnt[2]))


def zsm_cache_import_unit(cache, layer, b, h, head_dim, state, stream=None):
    cap, br = zsm_unit_capacity(cache, layer, h)
    n, r = int(state["n_live"]), int(state["n_res"])

    def padded(a, rows, dtype, cols=None):
        shape = (rows,) if cols is None else (rows, cols)
        out = np.zeros(shape, dtype)
        out[: len(a)] = a
        return out
    K = padded(state["K"], cap, np.float32, head_dim)
    V = padded(state["V"], cap, np.float32, head_dim)
    score = padded(state["score"], cap, np.float32)
    pos = padded(state["pos"], cap, np.int32)
    Kr = padded(state["Kr"], br, np.float32, head_dim)
    Vr = padded(state["Vr"], br, np.float32, head_dim)
    w = padded(state["w"], br, np.uint32)
    cnt = np.array([n, r, int(state["T"])], np.int32)
    _check(_lib.zsm_cache_import_unit(cache, int(layer), int(b), int(h), _host(K), _host(V),
                                      _host(score), _host(pos), _host(Kr), _host(Vr), _host(w),
                                      _host(cnt), _stream(stream)), "zsm_cache_import_unit")


def zsm_last_device_status(cache, stream=None) -> int:
    return int(_lib.zsm_last_device_status(cache, _stream(stream)))


def zsm_selftest_wait_timeout(cache, limit_us: int, stream=None):
    """Launches the library's wait self-test: one bounded wait that can only end by its limit."""
    _check(_lib.zsm_selftest_wait_timeout(cache, int(limit_us), _stream(stream)),
           "zsm_selftest_wait_timeout")


def zsm_decode_launch_info(cache, layer):
    g, b, s = C.c_int32(), C.c_int32(), C.c_int32()
    _check(_lib.zsm_decode_launch_info(cache, int(layer), C.byref(g), C.byref(b), C.byref(s)),
           "zsm_decode_launch_info")
    return g.value, b.value, s.value
