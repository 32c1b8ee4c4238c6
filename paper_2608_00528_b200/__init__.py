"""Thin Python binding of libs4r.so (the C ABI declared in include/s4r.h).

Argument marshalling only: every step of the S4R path runs in the library's CUDA kernels.  Torch is used
for device memory and streams.  There is no CPU fallback: importing works without a GPU (the library loads
and its symbols can be inspected), but every compute call needs a B200 and raises otherwise.
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass

import torch

from . import _build

S4R_F32, S4R_BF16 = 0, 1
POOL_MAX, POOL_AVG = 0, 1
GROUP_MEAN, GROUP_MAX = 0, 1
VALUE_AUTO, VALUE_RECONSTRUCT = 0, 1
DEV_TIMEOUT, DEV_BOUNDS = 1, 2

EXPORTS = ("s4r_workspace_bytes", "s4r_workspace_bytes_windowed", "s4r_compress", "s4r_append", "s4r_decode_step",
           "s4r_decode_step_host", "s4r_decode_step_static", "s4r_append_decode_step", "s4r_decode_step_windowed", "s4r_append_decode_step_windowed", "s4r_window_init", "s4r_host_step_layout", "s4r_append_decode_step_host", "s4r_basis_workspace_bytes", "s4r_build_basis",
           "s4r_hybrid_sample_indices",
           "s4r_top_k_from_ratio", "s4r_rank_for_ratio", "s4r_last_launch_count", "s4r_stage_timing",
           "s4r_stage_times", "s4r_strerror", "s4r_last_cuda_error", "s4r_version")
STAGES = ("query_projection", "latent_scoring", "selection", "reconstruct_attend", "merge")


class S4RError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        detail = ""
        if status == -4:
            fn = load().s4r_last_cuda_error
            fn.restype = ctypes.c_char_p
            detail = ": " + fn().decode()
        super().__init__(f"{where}: {strerror(status)} ({status}){detail}")


class _Layer(ctypes.Structure):
    _fields_ = [("batch", ctypes.c_int32), ("n_q_heads", ctypes.c_int32), ("n_kv_heads", ctypes.c_int32),
                ("head_dim", ctypes.c_int32), ("rank_k", ctypes.c_int32), ("rank_v", ctypes.c_int32),
                ("sink_count", ctypes.c_int32), ("dtype", ctypes.c_int32), ("coef_capacity", ctypes.c_int64)]


class _Score(ctypes.Structure):
    _fields_ = [("score_window", ctypes.c_int32), ("pool_kernel", ctypes.c_int32), ("pool_mode", ctypes.c_int32),
                ("group_mode", ctypes.c_int32), ("value_path", ctypes.c_int32)]


class _Rope(ctypes.Structure):
    _fields_ = [("theta", ctypes.c_float), ("reserved", ctypes.c_int32)]


_lib = None


def lib_path() -> str:
    return _build.LIB


def load(build_if_missing: bool = True):
    """Load libs4r.so (building it first if the sources are newer and nvcc is present)."""
    global _lib
    if _lib is not None:
        return _lib
    if build_if_missing and _build.needs_build():
        try:
            _build.build()
        except Exception:
            if not os.path.exists(_build.LIB):
                raise
    if not os.path.exists(_build.LIB):
        raise ImportError("libs4r.so is missing; run `python -m paper_2608_00528_b200._build`")
    lib = ctypes.CDLL(_build.LIB)
    vp, i32, i64, sz = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64, ctypes.c_size_t
    lp, sp, rp = ctypes.POINTER(_Layer), ctypes.POINTER(_Score), ctypes.POINTER(_Rope)
    lib.s4r_workspace_bytes.restype = sz
    lib.s4r_workspace_bytes.argtypes = [lp, i64, i32, i32]
    lib.s4r_workspace_bytes_windowed.restype = sz
    lib.s4r_workspace_bytes_windowed.argtypes = [lp, i64, i32, i32, i32]
    lib.s4r_append_decode_step_windowed.restype = ctypes.c_int
    lib.s4r_append_decode_step_windowed.argtypes = [lp] + [vp] * 10 + [i64, i32, i32, ctypes.POINTER(_Score),
                                                    ctypes.POINTER(_Rope), vp, vp, i32, vp, vp, vp, sz, vp, vp]
    lib.s4r_window_init.restype = ctypes.c_int
    lib.s4r_window_init.argtypes = [lp, vp, i32, vp, vp, i32, vp]
    lib.s4r_decode_step_windowed.restype = ctypes.c_int
    lib.s4r_decode_step_windowed.argtypes = [lp] + [vp] * 8 + [i64, i32, i32, ctypes.POINTER(_Score), ctypes.POINTER(_Rope),
                                             vp, vp, i32, vp, vp, vp, sz, vp, vp]
    lib.s4r_compress.restype = ctypes.c_int
    lib.s4r_compress.argtypes = [lp, vp, vp, i64, vp, vp, vp, vp, vp, vp, vp, vp, vp, sz, vp, vp]
    lib.s4r_append.restype = ctypes.c_int
    lib.s4r_append.argtypes = [lp, vp, vp, vp, vp, vp, vp, vp, vp, vp]
    lib.s4r_decode_step.restype = ctypes.c_int
    lib.s4r_decode_step.argtypes = [lp, vp, vp, vp, vp, vp, vp, vp, vp, i64, i32, i32, sp, rp, vp, i32, vp, vp, vp,
                                    sz, vp, vp]
    lib.s4r_decode_step_host.restype = ctypes.c_int
    lib.s4r_decode_step_host.argtypes = [lp, vp, vp, vp, vp, vp, vp, vp, vp, vp, i64, i32, i32, sp, rp, vp, vp, i32,
                                         vp, vp, vp, vp, vp, sz, vp, vp]
    lib.s4r_basis_workspace_bytes.restype = sz
    lib.s4r_basis_workspace_bytes.argtypes = [lp, i32, i32]
    lib.s4r_build_basis.restype = ctypes.c_int
    lib.s4r_build_basis.argtypes = [lp, vp, i64, vp, i32, i32, i32, vp, vp, vp, sz, vp, vp]
    lib.s4r_hybrid_sample_indices.restype = i32
    lib.s4r_hybrid_sample_indices.argtypes = [i64, i32, ctypes.c_double, ctypes.POINTER(i32)]
    lib.s4r_host_step_layout.restype = ctypes.c_int
    lib.s4r_host_step_layout.argtypes = [lp, i32, i32, i32, ctypes.POINTER(sz), ctypes.POINTER(sz)]
    lib.s4r_append_decode_step_host.restype = ctypes.c_int
    lib.s4r_append_decode_step_host.argtypes = [lp, vp, vp, vp, vp, vp, vp, vp, vp, vp, i64, i32, i32, sp, rp, vp, vp, i32,
                                                vp, sz, vp, vp]
    lib.s4r_top_k_from_ratio.restype = i64
    lib.s4r_top_k_from_ratio.argtypes = [ctypes.c_double, i64, i32]
    lib.s4r_rank_for_ratio.restype = i32
    lib.s4r_rank_for_ratio.argtypes = [ctypes.c_double, i64, i32, i32, i32, i32, i32]
    lib.s4r_last_launch_count.restype = i32
    lib.s4r_last_launch_count.argtypes = []
    lib.s4r_stage_timing.restype = ctypes.c_int
    lib.s4r_stage_timing.argtypes = [ctypes.c_int]
    lib.s4r_stage_times.restype = ctypes.c_int
    lib.s4r_stage_times.argtypes = [ctypes.POINTER(ctypes.c_float), ctypes.c_int]
    lib.s4r_strerror.restype = ctypes.c_char_p
    lib.s4r_strerror.argtypes = [ctypes.c_int]
    lib.s4r_version.restype = ctypes.c_int
    lib.s4r_version.argtypes = []
    _lib = lib
    return lib


def strerror(status: int) -> str:
    return load().s4r_strerror(int(status)).decode()


def version() -> int:
    return load().s4r_version()


def top_k_from_ratio(rho: float, cache_len: int, window: int) -> int:
    return int(load().s4r_top_k_from_ratio(float(rho), int(cache_len), int(window)))


def rank_for_ratio(eta: float, cache_len: int, sink_count: int, d_kv: int, group: int, query_window: int,
                   multiple: int = 8) -> int:
    return int(load().s4r_rank_for_ratio(float(eta), int(cache_len), int(sink_count), int(d_kv), int(group),
                                         int(query_window), int(multiple)))


def last_launch_count() -> int:
    return int(load().s4r_last_launch_count())


def stage_timing(enable: bool) -> None:
    rc = load().s4r_stage_timing(1 if enable else 0)
    if rc != 0:
        raise S4RError(rc, "s4r_stage_timing")


def stage_times() -> dict:
    """Milliseconds per stage of the last decode step on this thread (waits for that step)."""
    buf = (ctypes.c_float * len(STAGES))()
    rc = load().s4r_stage_times(buf, len(STAGES))
    if rc < 0:
        raise S4RError(rc, "s4r_stage_times")
    return {STAGES[i]: float(buf[i]) for i in range(rc)}


@dataclass
class Layer:
    batch: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    rank_k: int
    rank_v: int
    sink_count: int
    dtype: int                 # S4R_BF16 | S4R_F32
    coef_capacity: int

    def c(self) -> _Layer:
        return _Layer(self.batch, self.n_q_heads, self.n_kv_heads, self.head_dim, self.rank_k, self.rank_v,
                      self.sink_count, self.dtype, self.coef_capacity)

    @property
    def d_kv(self) -> int:
        return self.n_kv_heads * self.head_dim

    @property
    def torch_dtype(self) -> torch.dtype:
        return torch.bfloat16 if self.dtype == S4R_BF16 else torch.float32


def _ptr(t):
    if t is None:
        return None
    if isinstance(t, int):
        return ctypes.c_void_p(t)
    assert t.is_contiguous(), "tensors passed to libs4r must be contiguous"
    return ctypes.c_void_p(t.data_ptr())


def _stream(stream):
    if stream is None:
        stream = torch.cuda.current_stream()
    return ctypes.c_void_p(stream.cuda_stream)


def _need_cuda(*tensors):
    if not torch.cuda.is_available():
        raise RuntimeError("libs4r needs a CUDA device (sm_100); there is no CPU fallback")
    for t in tensors:
        if t is not None and not isinstance(t, int) and not t.is_cuda:
            raise ValueError("expected CUDA tensors")


def workspace_bytes(layer: Layer, max_len: int, window: int, top_k: int) -> int:
    return int(load().s4r_workspace_bytes(ctypes.byref(layer.c()), int(max_len), int(window), int(top_k)))


def alloc_workspace(layer: Layer, max_len: int, window: int, top_k: int, device="cuda", score_window: int = 1) -> torch.Tensor:
    """Scratch for the decode step; with score_window > 1 sized for decode_step_windowed."""
    if score_window > 1:
        n = int(load().s4r_workspace_bytes_windowed(ctypes.byref(layer.c()), int(max_len), int(window), int(top_k),
                                                    int(score_window)))
    else:
        n = workspace_bytes(layer, max_len, window, top_k)
    if n == 0:
        raise S4RError(-1, "s4r_workspace_bytes")
    return torch.empty(n, dtype=torch.uint8, device=device)


def compress(layer: Layer, K, V, key_basis, value_basis, sink_k, sink_v, coef_k, coef_v, coef_len,
             workspace=None, dev_status=None, stream=None, norm_stats=None):
    """s4r_compress: K, V [B, T, D'] -> sinks, coefficient caches, coef_len (all preallocated by the caller)."""
    _need_cuda(K, V, key_basis, value_basis, coef_k, coef_v, coef_len)
    T = K.shape[1]
    rc = load().s4r_compress(ctypes.byref(layer.c()), _ptr(K), _ptr(V), int(T), _ptr(key_basis), _ptr(value_basis),
                             _ptr(norm_stats), _ptr(sink_k), _ptr(sink_v), _ptr(coef_k), _ptr(coef_v),
                             _ptr(coef_len), _ptr(workspace), 0 if workspace is None else workspace.numel(),
                             _ptr(dev_status), _stream(stream))
    if rc != 0:
        raise S4RError(rc, "s4r_compress")


def append(layer: Layer, k_t, v_t, key_basis, value_basis, coef_k, coef_v, coef_len, dev_status=None, stream=None):
    """s4r_append: project one new key/value row per sequence and append it to the coefficient caches."""
    _need_cuda(k_t, v_t, key_basis, value_basis, coef_k, coef_v, coef_len)
    rc = load().s4r_append(ctypes.byref(layer.c()), _ptr(k_t), _ptr(v_t), _ptr(key_basis), _ptr(value_basis),
                           _ptr(coef_k), _ptr(coef_v), _ptr(coef_len), _ptr(dev_status), _stream(stream))
    if rc != 0:
        raise S4RError(rc, "s4r_append")


def _score_rope(pool_kernel, pool_mode, group_mode, score_window, theta, value_path=0):
    return _Score(score_window, pool_kernel, pool_mode, group_mode, value_path), _Rope(float(theta), 0)


def decode_step(layer: Layer, q, sink_k, sink_v, coef_k, coef_v, coef_len, key_basis, value_basis, max_len: int,
                window: int, top_k: int, out, sel_idx, sel_count, workspace, *, pool_kernel: int = 7,
                pool_mode: int = POOL_MAX, group_mode: int = GROUP_MEAN, score_window: int = 1,
                rope_theta: float = 0.0, value_path: int = VALUE_AUTO, dev_status=None, stream=None):
    """s4r_decode_step: writes `out` [B, H_q, d_h], `sel_idx` [B, window + top_k] and `sel_count` [B]."""
    _need_cuda(q, coef_k, coef_v, coef_len, key_basis, value_basis, out, sel_idx, sel_count, workspace)
    sc, rp = _score_rope(pool_kernel, pool_mode, group_mode, score_window, rope_theta, value_path)
    out_dtype = S4R_BF16 if out.dtype == torch.bfloat16 else S4R_F32
    rc = load().s4r_decode_step(ctypes.byref(layer.c()), _ptr(q), _ptr(sink_k), _ptr(sink_v), _ptr(coef_k),
                                _ptr(coef_v), _ptr(coef_len), _ptr(key_basis), _ptr(value_basis), int(max_len),
                                int(window), int(top_k), ctypes.byref(sc), ctypes.byref(rp), _ptr(out), out_dtype,
                                _ptr(sel_idx), _ptr(sel_count), _ptr(workspace), workspace.numel(),
                                _ptr(dev_status), _stream(stream))
    if rc != 0:
        raise S4RError(rc, "s4r_decode_step")


def decode_step_windowed(layer: Layer, q, sink_k, sink_v, coef_k, coef_v, coef_len, key_basis, value_basis, max_len: int,
                         window: int, top_k: int, query_window, out, sel_idx, sel_count, workspace, *,
                         score_window: int, pool_kernel: int = 7, pool_mode: int = POOL_MAX,
                         group_mode: int = GROUP_MEAN, rope_theta: float = 0.0, value_path: int = VALUE_AUTO,
                         dev_status=None, stream=None):
    """s4r_decode_step_windowed: `query_window` [B, W_q, G, rank_k] fp32 is shifted and extended in place."""
    _need_cuda(q, coef_k, coef_v, coef_len, key_basis, value_basis, query_window, out, sel_idx, sel_count, workspace)
    if query_window.dtype != torch.float32 or tuple(query_window.shape) != (
            layer.batch, score_window, layer.n_q_heads // layer.n_kv_heads, layer.rank_k) or not query_window.is_contiguous():
        raise ValueError("query_window must be a contiguous fp32 tensor [B, W_q, G, rank_k]")
    sc, rp = _score_rope(pool_kernel, pool_mode, group_mode, score_window, rope_theta, value_path)
    out_dtype = S4R_BF16 if out.dtype == torch.bfloat16 else S4R_F32
    rc = load().s4r_decode_step_windowed(ctypes.byref(layer.c()), _ptr(q), _ptr(sink_k), _ptr(sink_v), _ptr(coef_k),
                                         _ptr(coef_v), _ptr(coef_len), _ptr(key_basis), _ptr(value_basis), int(max_len),
                                         int(window), int(top_k), ctypes.byref(sc), ctypes.byref(rp),
                                         _ptr(query_window), _ptr(out), out_dtype, _ptr(sel_idx), _ptr(sel_count),
                                         _ptr(workspace), workspace.numel(), _ptr(dev_status), _stream(stream))
    if rc != 0:
        raise S4RError(rc, "s4r_decode_step_windowed")


def append_decode_step_windowed(layer: Layer, k_t, v_t, q, sink_k, sink_v, coef_k, coef_v, coef_len, key_basis,
                                value_basis, max_len: int, window: int, top_k: int, query_window, out, sel_idx,
                                sel_count, workspace, *, score_window: int, pool_kernel: int = 7,
                                pool_mode: int = POOL_MAX, group_mode: int = GROUP_MEAN, rope_theta: float = 0.0,
                                value_path: int = VALUE_AUTO, dev_status=None, stream=None):
    """s4r_append_decode_step_windowed: the cache update and the windowed decode step as one call."""
    _need_cuda(k_t, v_t, q, coef_k, coef_v, coef_len, key_basis, value_basis, query_window, out, sel_idx, sel_count,
               workspace)
    if query_window.dtype != torch.float32 or tuple(query_window.shape) != (
            layer.batch, score_window, layer.n_q_heads // layer.n_kv_heads, layer.rank_k) or not query_window.is_contiguous():
        raise ValueError("query_window must be a contiguous fp32 tensor [B, W_q, G, rank_k]")
    sc, rp = _score_rope(pool_kernel, pool_mode, group_mode, score_window, rope_theta, value_path)
    out_dtype = S4R_BF16 if out.dtype == torch.bfloat16 else S4R_F32
    rc = load().s4r_append_decode_step_windowed(
        ctypes.byref(layer.c()), _ptr(k_t), _ptr(v_t), _ptr(q), _ptr(sink_k), _ptr(sink_v), _ptr(coef_k), _ptr(coef_v),
        _ptr(coef_len), _ptr(key_basis), _ptr(value_basis), int(max_len), int(window), int(top_k), ctypes.byref(sc),
        ctypes.byref(rp), _ptr(query_window), _ptr(out), out_dtype, _ptr(sel_idx), _ptr(sel_count), _ptr(workspace),
        workspace.numel(), _ptr(dev_status), _stream(stream))
    if rc != 0:
        raise S4RError(rc, "s4r_append_decode_step_windowed")


def window_init(layer: Layer, queries, key_basis, query_window, *, score_window: int, stream=None):
    """s4r_window_init: `queries` [B, n, H_q, d_h] (n <= W_q, oldest first; None or n = 0: an all-zero window) fill the
    last n rows of `query_window` [B, W_q, G, rank_k] fp32."""
    _need_cuda(key_basis, query_window)
    n = 0 if queries is None else int(queries.shape[1])
    if queries is not None and (not queries.is_cuda or not queries.is_contiguous()):
        raise ValueError("queries must be a contiguous CUDA tensor [B, n, H_q, d_h]")
    if query_window.dtype != torch.float32 or tuple(query_window.shape) != (
            layer.batch, score_window, layer.n_q_heads // layer.n_kv_heads, layer.rank_k) or not query_window.is_contiguous():
        raise ValueError("query_window must be a contiguous fp32 tensor [B, W_q, G, rank_k]")
    rc = load().s4r_window_init(ctypes.byref(layer.c()), _ptr(queries), n, _ptr(key_basis), _ptr(query_window),
                                int(score_window), _stream(stream))
    if rc != 0:
        raise S4RError(rc, "s4r_window_init")


def decode_step_host(layer: Layer, q_host, q_dev, sink_k, sink_v, coef_k, coef_v, coef_len, key_basis, value_basis,
                     max_len: int, window: int, top_k: int, out_host, out_dev, sel_idx_host, sel_idx_dev,
                     sel_count_host, sel_count_dev, workspace, *, pool_kernel: int = 7, pool_mode: int = POOL_MAX,
                     group_mode: int = GROUP_MEAN, score_window: int = 1, rope_theta: float = 0.0, dev_status=None,
                     stream=None):
    """s4r_decode_step_host: q / out / sel_idx / sel_count live in host memory; returns after the results landed."""
    _need_cuda(q_dev, coef_k, coef_v, coef_len, key_basis, value_basis, out_dev, sel_idx_dev, sel_count_dev, workspace)
    sc, rp = _score_rope(pool_kernel, pool_mode, group_mode, score_window, rope_theta)
    out_dtype = S4R_BF16 if out_dev.dtype == torch.bfloat16 else S4R_F32
    rc = load().s4r_decode_step_host(
        ctypes.byref(layer.c()), _ptr(q_host), _ptr(q_dev), _ptr(sink_k), _ptr(sink_v), _ptr(coef_k), _ptr(coef_v),
        _ptr(coef_len), _ptr(key_basis), _ptr(value_basis), int(max_len), int(window), int(top_k), ctypes.byref(sc),
        ctypes.byref(rp), _ptr(out_host), _ptr(out_dev), out_dtype, _ptr(sel_idx_host), _ptr(sel_idx_dev),
        _ptr(sel_count_host), _ptr(sel_count_dev), _ptr(workspace), workspace.numel(), _ptr(dev_status),
        _stream(stream))
    if rc != 0:
        raise S4RError(rc, "s4r_decode_step_host")


def hybrid_sample_indices(n_nonsink: int, n_samples: int, recent_frac: float = 0.7) -> torch.Tensor:
    """s4r_hybrid_sample_indices: the paper's sampling pattern as an int32 CPU tensor of ascending non-sink indices."""
    buf = (ctypes.c_int32 * max(int(n_samples), 1))()
    n = load().s4r_hybrid_sample_indices(int(n_nonsink), int(n_samples), float(recent_frac), buf)
    return torch.tensor(list(buf[:n]), dtype=torch.int32)


def build_basis(layer: Layer, X, sample_idx, rank: int, *, n_iter: int = 0, sigma=None, workspace=None,
                dev_status=None, stream=None) -> torch.Tensor:
    """s4r_build_basis: X [B, T, D'] (with the sink rows), sample_idx [B, n_samples] int32 non-sink indices ->
    basis [B, D', rank] in the layer dtype (returned); `sigma` [B, rank] fp32 receives the singular values."""
    _need_cuda(X, sample_idx)
    if sample_idx.dtype != torch.int32 or sample_idx.dim() != 2 or sample_idx.shape[0] != layer.batch:
        raise ValueError("sample_idx must be an int32 tensor [B, n_samples]")
    n_s = int(sample_idx.shape[1])
    if workspace is None:
        n = int(load().s4r_basis_workspace_bytes(ctypes.byref(layer.c()), int(rank), n_s))
        if n == 0:
            raise S4RError(-2, "s4r_basis_workspace_bytes")
        workspace = torch.empty(n, dtype=torch.uint8, device=X.device)
    basis = torch.empty(layer.batch, layer.d_kv, int(rank), dtype=layer.torch_dtype, device=X.device)
    rc = load().s4r_build_basis(ctypes.byref(layer.c()), _ptr(X), int(X.shape[1]), _ptr(sample_idx), n_s, int(rank),
                                int(n_iter), _ptr(basis), _ptr(sigma), _ptr(workspace), workspace.numel(),
                                _ptr(dev_status), _stream(stream))
    if rc != 0:
        raise S4RError(rc, "s4r_build_basis")
    return basis


class HostStep:
    """Packed per-step blocks of s4r_append_decode_step_host: one pinned host block and one device block for the
    inputs {q, k_t, v_t}, one of each for the results {out, sel_idx, sel_count}, with typed views into them."""

    def __init__(self, layer: Layer, window: int, top_k: int, out_dtype=torch.float32, device="cuda"):
        self.layer, self.window, self.top_k = layer, int(window), int(top_k)
        self.out_code = S4R_BF16 if out_dtype == torch.bfloat16 else S4R_F32
        io, oo = (ctypes.c_size_t * 4)(), (ctypes.c_size_t * 4)()
        rc = load().s4r_host_step_layout(ctypes.byref(layer.c()), self.window, self.top_k, self.out_code, io, oo)
        if rc != 0:
            raise S4RError(rc, "s4r_host_step_layout")
        io, oo = list(io), list(oo)
        st = torch.bfloat16 if layer.dtype == S4R_BF16 else torch.float32
        B, Hq, dh = layer.batch, layer.n_q_heads, layer.head_dim
        D = layer.n_kv_heads * dh
        self.in_host = torch.empty(io[3], dtype=torch.uint8).pin_memory()
        self.out_host = torch.empty(oo[3], dtype=torch.uint8).pin_memory()
        self.in_dev = torch.empty(io[3], dtype=torch.uint8, device=device)
        self.out_dev = torch.empty(oo[3], dtype=torch.uint8, device=device)
        esz = 2 if st == torch.bfloat16 else 4
        osz = 2 if out_dtype == torch.bfloat16 else 4

        def view(block, off, n, dtype, shape):
            return block[off:off + n].view(dtype).view(*shape)
        self.q = view(self.in_host, io[0], B * Hq * dh * esz, st, (B, Hq, dh))
        self.k_t = view(self.in_host, io[1], B * D * esz, st, (B, D))
        self.v_t = view(self.in_host, io[2], B * D * esz, st, (B, D))
        self.out = view(self.out_host, oo[0], B * Hq * dh * osz, out_dtype, (B, Hq, dh))
        self.sel_idx = view(self.out_host, oo[1], B * (self.window + self.top_k) * 4, torch.int32,
                            (B, self.window + self.top_k))
        self.sel_count = view(self.out_host, oo[2], B * 4, torch.int32, (B,))
        self.h2d_bytes, self.d2h_bytes = io[3], oo[3]


def append_decode_step_host(hs: HostStep, sink_k, sink_v, coef_k, coef_v, coef_len, key_basis, value_basis, max_len: int,
                            workspace, *, pool_kernel: int = 7, pool_mode: int = POOL_MAX, group_mode: int = GROUP_MEAN,
                            rope_theta: float = 0.0, value_path: int = VALUE_AUTO, dev_status=None, stream=None,
                            in_host=None):
    """s4r_append_decode_step_host: the caller fills hs.q / hs.k_t / hs.v_t (pinned host views); on return hs.out /
    hs.sel_idx / hs.sel_count hold the step's results.  `in_host`: another host block of the same layout to read
    the inputs from instead of hs.in_host."""
    _need_cuda(coef_k, coef_v, coef_len, key_basis, value_basis, workspace)
    src = hs.in_host if in_host is None else in_host
    if src.numel() != hs.in_host.numel() or src.is_cuda:
        raise ValueError("in_host must be a host block of hs.h2d_bytes bytes")
    sc, rp = _score_rope(pool_kernel, pool_mode, group_mode, 1, rope_theta, value_path)
    rc = load().s4r_append_decode_step_host(
        ctypes.byref(hs.layer.c()), _ptr(src), _ptr(hs.in_dev), _ptr(sink_k), _ptr(sink_v), _ptr(coef_k),
        _ptr(coef_v), _ptr(coef_len), _ptr(key_basis), _ptr(value_basis), int(max_len), hs.window, hs.top_k,
        ctypes.byref(sc), ctypes.byref(rp), _ptr(hs.out_host), _ptr(hs.out_dev), hs.out_code, _ptr(workspace),
        workspace.numel(), _ptr(dev_status), _stream(stream))
    if rc != 0:
        raise S4RError(rc, "s4r_append_decode_step_host")


STATIC_SCRATCH_BYTES = 16 << 20


def decode_step_static(layer: Layer, q, sink_k, sink_v, coef_k, coef_v, coef_len, key_basis, value_basis,
                       max_len: int, window: int, top_k: int, out, sel_idx, sel_count, *, pool_kernel: int = 7,
                       pool_mode: int = POOL_MAX, group_mode: int = GROUP_MEAN, score_window: int = 1,
                       rope_theta: float = 0.0, dev_status=None, stream=None):
    """s4r_decode_step_static: the decode step for callers that have no way to allocate a workspace.

    Same inputs and results as `decode_step`, but the scratch memory is a fixed 16 MiB array inside the
    library, so nothing is allocated by this call (not by the library, and no torch tensor is created here
    either).  Geometries that need more scratch raise S4RError(-3).  All calls on a device share that array:
    keep them ordered on the GPU, and make the first call on a device outside stream capture.
    """
    _need_cuda(q, coef_k, coef_v, coef_len, key_basis, value_basis, out, sel_idx, sel_count)
    sc, rp = _score_rope(pool_kernel, pool_mode, group_mode, score_window, rope_theta)
    out_dtype = S4R_BF16 if out.dtype == torch.bfloat16 else S4R_F32
    rc = _static_fn()(ctypes.byref(layer.c()), _ptr(q), _ptr(sink_k), _ptr(sink_v), _ptr(coef_k), _ptr(coef_v),
                      _ptr(coef_len), _ptr(key_basis), _ptr(value_basis), int(max_len), int(window), int(top_k),
                      ctypes.byref(sc), ctypes.byref(rp), _ptr(out), out_dtype, _ptr(sel_idx), _ptr(sel_count),
                      _ptr(dev_status), _stream(stream))
    if rc != 0:
        raise S4RError(rc, "s4r_decode_step_static")


def _static_fn():
    fn = load().s4r_decode_step_static
    if fn.restype is not ctypes.c_int or not fn.argtypes:
        vp, i32, i64 = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64
        fn.restype = ctypes.c_int
        fn.argtypes = [ctypes.POINTER(_Layer), vp, vp, vp, vp, vp, vp, vp, vp, i64, i32, i32, ctypes.POINTER(_Score),
                       ctypes.POINTER(_Rope), vp, i32, vp, vp, vp, vp]
    return fn


def append_decode_step(layer: Layer, k_t, v_t, q, sink_k, sink_v, coef_k, coef_v, coef_len, key_basis, value_basis,
                       max_len: int, window: int, top_k: int, out, sel_idx, sel_count, workspace, *,
                       pool_kernel: int = 7, pool_mode: int = POOL_MAX, group_mode: int = GROUP_MEAN,
                       score_window: int = 1, rope_theta: float = 0.0, dev_status=None, stream=None):
    """s4r_append_decode_step: append the new token's coefficient rows and run the decode step in one call."""
    _need_cuda(k_t, v_t, q, coef_k, coef_v, coef_len, key_basis, value_basis, out, sel_idx, sel_count, workspace)
    sc, rp = _score_rope(pool_kernel, pool_mode, group_mode, score_window, rope_theta)
    out_dtype = S4R_BF16 if out.dtype == torch.bfloat16 else S4R_F32
    fn = load().s4r_append_decode_step
    if not fn.argtypes:
        vp, i32, i64 = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64
        fn.restype = ctypes.c_int
        fn.argtypes = [ctypes.POINTER(_Layer), vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, i64, i32, i32,
                       ctypes.POINTER(_Score), ctypes.POINTER(_Rope), vp, i32, vp, vp, vp, ctypes.c_size_t, vp, vp]
    rc = fn(ctypes.byref(layer.c()), _ptr(k_t), _ptr(v_t), _ptr(q), _ptr(sink_k), _ptr(sink_v), _ptr(coef_k),
            _ptr(coef_v), _ptr(coef_len), _ptr(key_basis), _ptr(value_basis), int(max_len), int(window), int(top_k),
            ctypes.byref(sc), ctypes.byref(rp), _ptr(out), out_dtype, _ptr(sel_idx), _ptr(sel_count), _ptr(workspace),
            workspace.numel(), _ptr(dev_status), _stream(stream))
    if rc != 0:
        raise S4RError(rc, "s4r_append_decode_step")
