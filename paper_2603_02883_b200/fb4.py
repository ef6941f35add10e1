"""Python binding of libfb4 (include/fb4.h): argument marshalling only.

Every function has the name and argument order of the C entry point it calls; tensors are
torch CUDA tensors whose data pointers are handed over unchanged, and the current torch
stream is passed unless one is given.  There is no CPU fallback: if the shared library is
missing and cannot be built, importing this module raises.
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass

import torch

from . import build as _build

OK = 0
ERR_INVALID_ARG, ERR_SHAPE, ERR_ALIGN, ERR_FORMATBOOK, ERR_CUDA, ERR_NO_DEVICE = -1, -2, -3, -4, -5, -6
ERR_STATIC_LIMIT = -7
STATIC_MAX_CLUSTERS = 1024

EXPORTS = [
    "fb4_default_config", "fb4_init", "fb4_destroy", "fb4_get_tables", "fb4_block_tables", "fb4_quantize", "fb4_quantize_f32", "fb4_quantize_affine", "fb4_quantize_affine_mxfp8", "fb4_quantize_layernorm", "fb4_quantize_seda",
    "fb4_build_subformatbook", "fb4_build_subformatbook_static", "fb4_select_salient", "fb4_select_salient_topk", "fb4_quantize_decomposed", "fb4_quantize_decomposed_idx", "fb4_dequantize",
    "fb4_quantize_weights", "fb4_quantize_mxfp8", "fb4_quantize_mxfp8_decomposed", "fb4_to_mxfp8", "fb4_mxfp8_scale_bytes", "fb4_quantize_host", "fb4_set_kernel_variant", "fb4_device_status", "fb4_launch_count", "fb4_last_variant", "fb4_last_cuda_error", "fb4_strerror",
]


class Fb4Config(ctypes.Structure):
    _fields_ = [("block_size", ctypes.c_uint32), ("num_groups", ctypes.c_uint32),
                ("exp_min", ctypes.c_int32), ("exp_max", ctypes.c_int32), ("select_mode", ctypes.c_uint32)]


class Fb4Error(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        msg = lib().fb4_strerror(code).decode()
        if code == ERR_CUDA:
            msg += f" (cudaError {lib().fb4_last_cuda_error()})"
        super().__init__(f"{where}: {msg} [{code}]")


_lib = None


def library_path() -> str:
    return _build.LIB


def lib() -> ctypes.CDLL:
    """Load libfb4.so, building it first if it is missing or older than its sources."""
    global _lib
    if _lib is not None:
        return _lib
    path = _build.LIB
    if _build.stale():
        try:
            _build.build()
        except Exception as e:  # no nvcc, compile error
            if not os.path.exists(path):
                raise ImportError(f"libfb4.so is not built and could not be built: {e}") from e
            raise
    L = ctypes.CDLL(path)
    vp, i64, i32, ci = ctypes.c_void_p, ctypes.c_int64, ctypes.c_int32, ctypes.c_int
    L.fb4_default_config.argtypes = [ctypes.POINTER(Fb4Config)]
    L.fb4_default_config.restype = None
    L.fb4_init.argtypes = [ctypes.POINTER(vp), ci, vp, vp, ctypes.POINTER(Fb4Config)]
    L.fb4_destroy.argtypes = [vp]
    L.fb4_get_tables.argtypes = [vp, vp, vp, vp, vp]
    L.fb4_block_tables.argtypes = [vp, ctypes.POINTER(vp), ctypes.POINTER(ctypes.c_uint64)]
    L.fb4_block_tables.restype = ci
    L.fb4_quantize.argtypes = [vp, vp, i64, i64, i64, vp, vp, vp]
    L.fb4_quantize_f32.argtypes = [vp, vp, i64, i64, i64, vp, vp, vp]
    L.fb4_quantize_f32.restype = ci
    L.fb4_quantize_affine.argtypes = [vp, vp, i64, i64, i64, vp, vp, ci, vp, vp, i32, vp, vp, vp]
    L.fb4_quantize_affine.restype = ci
    L.fb4_quantize_layernorm.argtypes = [vp, vp, i64, i64, i64, vp, vp, ci, ctypes.c_float, vp, vp, i32, vp, vp, vp]
    L.fb4_quantize_layernorm.restype = ci
    L.fb4_quantize_affine_mxfp8.argtypes = [vp, vp, i64, i64, i64, vp, vp, ci, vp, vp, i32, vp, vp, ci, vp]
    L.fb4_quantize_affine_mxfp8.restype = ci
    L.fb4_quantize_seda.argtypes = [vp, vp, i64, i64, i64, vp, vp, i32, vp, vp, vp]
    L.fb4_build_subformatbook.argtypes = [vp, vp, i64, i64, vp, vp, i64, i32, vp, vp, vp]
    L.fb4_build_subformatbook.restype = ci
    L.fb4_build_subformatbook_static.argtypes = [vp, vp, i64, i64, vp, vp, i64, i32, vp, vp]
    L.fb4_build_subformatbook_static.restype = ci
    L.fb4_select_salient.argtypes = [vp, vp, i64, i32, vp, vp]
    L.fb4_select_salient_topk.argtypes = [vp, vp, i64, i64, vp, vp]
    L.fb4_select_salient_topk.restype = ci
    L.fb4_quantize_decomposed.argtypes = [vp, vp, i64, i64, i64, vp, i32, vp, vp, i32, vp, vp, vp, vp, vp, vp]
    L.fb4_quantize_decomposed_idx.argtypes = [vp, vp, i64, i64, i64, vp, i64, vp, vp, i32, vp, vp, vp, vp, vp]
    L.fb4_dequantize.argtypes = [vp, vp, vp, i64, i64, vp, i64, vp, vp, vp, ci, vp]
    L.fb4_quantize_weights.argtypes = [vp, vp, i64, i64, i64, vp, vp, vp]
    L.fb4_quantize_weights.restype = ci
    L.fb4_quantize_mxfp8.argtypes = [vp, vp, i64, i64, i64, vp, vp, i32, vp, vp, ci, vp]
    L.fb4_quantize_mxfp8.restype = ci
    L.fb4_quantize_mxfp8_decomposed.argtypes = [vp, vp, i64, i64, i64, vp, i32, vp, i64, vp, vp, i32, vp, vp, vp, vp,
                                                ci, vp]
    L.fb4_quantize_mxfp8_decomposed.restype = ci
    L.fb4_to_mxfp8.argtypes = [vp, vp, vp, i64, i64, vp, vp, ci, vp]
    L.fb4_to_mxfp8.restype = ci
    L.fb4_mxfp8_scale_bytes.argtypes = [i64, i64, ci]
    L.fb4_mxfp8_scale_bytes.restype = i64
    L.fb4_quantize_host.argtypes = [vp, vp, i64, i64, vp, vp, vp, vp, vp]
    for name in ("fb4_init", "fb4_destroy", "fb4_get_tables", "fb4_quantize", "fb4_quantize_f32", "fb4_quantize_seda",
                 "fb4_build_subformatbook", "fb4_build_subformatbook_static", "fb4_select_salient", "fb4_select_salient_topk", "fb4_quantize_decomposed", "fb4_quantize_decomposed_idx",
                 "fb4_dequantize", "fb4_quantize_host", "fb4_last_cuda_error"):
        getattr(L, name).restype = ci
    L.fb4_set_kernel_variant.argtypes = [vp, ci]
    L.fb4_set_kernel_variant.restype = ci
    L.fb4_device_status.argtypes = [vp, ctypes.POINTER(ctypes.c_uint32)]
    L.fb4_device_status.restype = ci
    L.fb4_launch_count.argtypes = [vp]
    L.fb4_launch_count.restype = i64
    L.fb4_last_variant.argtypes = [vp]
    L.fb4_last_variant.restype = ctypes.c_char_p
    L.fb4_strerror.argtypes = [ci]
    L.fb4_strerror.restype = ctypes.c_char_p
    _lib = L
    return L


def _ptr(t):
    if t is None:
        return None
    if isinstance(t, torch.Tensor):
        return ctypes.c_void_p(t.data_ptr())
    return ctypes.c_void_p(int(t))


def _stream(stream):
    if stream is None:
        stream = torch.cuda.current_stream()
    return ctypes.c_void_p(stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream))


def _check(rc: int, where: str):
    if rc != OK:
        raise Fb4Error(rc, where)


# ----------------------------------------------------------------------------- C-named entry points

def fb4_init(device: int = 0, formatbook=None, stage1_mask=None, config: Fb4Config | None = None) -> ctypes.c_void_p:
    """formatbook: 256 bytes (numpy uint8 [32][8]) or None; stage1_mask: numpy uint32 [32] or None."""
    import numpy as np
    fb = None if formatbook is None else np.ascontiguousarray(formatbook, dtype=np.uint8)
    s1 = None if stage1_mask is None else np.ascontiguousarray(stage1_mask, dtype=np.uint32)
    if fb is not None and fb.size != 256:
        raise ValueError("formatbook must hold 32x8 magnitudes")
    if s1 is not None and s1.size != 32:
        raise ValueError("stage1_mask must hold 32 words")
    h = ctypes.c_void_p()
    rc = lib().fb4_init(ctypes.byref(h), device, None if fb is None else fb.ctypes.data_as(ctypes.c_void_p),
                        None if s1 is None else s1.ctypes.data_as(ctypes.c_void_p),
                        None if config is None else ctypes.byref(config))
    _check(rc, "fb4_init")
    return h


def fb4_destroy(ctx) -> None:
    _check(lib().fb4_destroy(ctx), "fb4_destroy")


def fb4_get_tables(ctx):
    import numpy as np
    fb = np.zeros((32, 8), np.uint8)
    s1 = np.zeros(32, np.uint32)
    qv = np.zeros((32, 32), np.uint8)
    qe = np.zeros((32, 32), np.uint8)
    p = lambda a: a.ctypes.data_as(ctypes.c_void_p)
    _check(lib().fb4_get_tables(ctx, p(fb), p(s1), p(qv), p(qe)), "fb4_get_tables")
    return fb, s1, qv, qe


def fb4_block_tables(ctx):
    """(device pointer, size in bytes) of the table image that include/fb4_block.cuh reads"""
    ptr, n = ctypes.c_void_p(), ctypes.c_uint64(0)
    _check(lib().fb4_block_tables(ctx, ctypes.byref(ptr), ctypes.byref(n)), "fb4_block_tables")
    return int(ptr.value), int(n.value)


def fb4_quantize(ctx, x, T, C, ld_elems, codes, meta, stream=None) -> None:
    _check(lib().fb4_quantize(ctx, _ptr(x), T, C, ld_elems, _ptr(codes), _ptr(meta), _stream(stream)), "fb4_quantize")


def fb4_quantize_f32(ctx, x, T, C, ld_elems, codes, meta, stream=None) -> None:
    _check(lib().fb4_quantize_f32(ctx, _ptr(x), T, C, ld_elems, _ptr(codes), _ptr(meta), _stream(stream)),
           "fb4_quantize_f32")


def fb4_quantize_affine(ctx, x, T, C, ld_elems, gain, bias, gain_plus_one, cluster_id, cluster_mask, n_clusters, codes,
                        meta, stream=None) -> None:
    _check(lib().fb4_quantize_affine(ctx, _ptr(x), T, C, ld_elems, _ptr(gain), _ptr(bias), int(bool(gain_plus_one)),
                                     _ptr(cluster_id), _ptr(cluster_mask), n_clusters, _ptr(codes), _ptr(meta),
                                     _stream(stream)), "fb4_quantize_affine")


def fb4_quantize_layernorm(ctx, x, T, C, ld_elems, gain, bias, gain_plus_one, eps, cluster_id, cluster_mask, n_clusters,
                           codes, meta, stream=None) -> None:
    _check(lib().fb4_quantize_layernorm(ctx, _ptr(x), T, C, ld_elems, _ptr(gain), _ptr(bias), int(bool(gain_plus_one)),
                                        ctypes.c_float(eps), _ptr(cluster_id), _ptr(cluster_mask), n_clusters,
                                        _ptr(codes), _ptr(meta), _stream(stream)), "fb4_quantize_layernorm")


def fb4_quantize_affine_mxfp8(ctx, x, T, C, ld_elems, gain, bias, gain_plus_one, cluster_id, cluster_mask, n_clusters, e4m3,
                              scales, scale_layout, stream=None) -> None:
    _check(lib().fb4_quantize_affine_mxfp8(ctx, _ptr(x), T, C, ld_elems, _ptr(gain), _ptr(bias), int(bool(gain_plus_one)),
                                           _ptr(cluster_id), _ptr(cluster_mask), n_clusters, _ptr(e4m3), _ptr(scales),
                                           scale_layout, _stream(stream)), "fb4_quantize_affine_mxfp8")


def fb4_quantize_seda(ctx, x, T, C, ld_elems, cluster_id, cluster_mask, n_clusters, codes, meta, stream=None) -> None:
    _check(lib().fb4_quantize_seda(ctx, _ptr(x), T, C, ld_elems, _ptr(cluster_id), _ptr(cluster_mask), n_clusters,
                                   _ptr(codes), _ptr(meta), _stream(stream)), "fb4_quantize_seda")


def fb4_build_subformatbook(ctx, meta, T, C, anchor_token, anchor_cluster, n_anchor, n_clusters, counts, cluster_mask,
                            stream=None) -> None:
    _check(lib().fb4_build_subformatbook(ctx, _ptr(meta), T, C, _ptr(anchor_token), _ptr(anchor_cluster), n_anchor,
                                         n_clusters, _ptr(counts), _ptr(cluster_mask), _stream(stream)),
           "fb4_build_subformatbook")


def fb4_build_subformatbook_static(ctx, meta, T, C, anchor_token, anchor_cluster, n_anchor, n_clusters, cluster_mask,
                                   stream=None) -> None:
    """fb4_build_subformatbook for callers that cannot allocate: no `counts` argument, the library's
    built-in array is used (at most STATIC_MAX_CLUSTERS clusters; calls on one GPU must not overlap)."""
    _check(lib().fb4_build_subformatbook_static(ctx, _ptr(meta), T, C, _ptr(anchor_token), _ptr(anchor_cluster),
                                                n_anchor, n_clusters, _ptr(cluster_mask), _stream(stream)),
           "fb4_build_subformatbook_static")


def fb4_select_salient(ctx, score, T, tile, salient_idx, stream=None) -> None:
    _check(lib().fb4_select_salient(ctx, _ptr(score), T, tile, _ptr(salient_idx), _stream(stream)),
           "fb4_select_salient")


def fb4_select_salient_topk(ctx, score, T, k, salient_idx, stream=None) -> None:
    _check(lib().fb4_select_salient_topk(ctx, _ptr(score), T, k, _ptr(salient_idx), _stream(stream)),
           "fb4_select_salient_topk")


def fb4_quantize_decomposed(ctx, x, T, C, ld_elems, score, tile, cluster_id, cluster_mask, n_clusters, codes, meta,
                            salient_idx, res_codes, res_meta, stream=None) -> None:
    _check(lib().fb4_quantize_decomposed(ctx, _ptr(x), T, C, ld_elems, _ptr(score), tile, _ptr(cluster_id),
                                         _ptr(cluster_mask), n_clusters, _ptr(codes), _ptr(meta), _ptr(salient_idx),
                                         _ptr(res_codes), _ptr(res_meta), _stream(stream)), "fb4_quantize_decomposed")


def fb4_quantize_decomposed_idx(ctx, x, T, C, ld_elems, salient_idx, n_salient, cluster_id, cluster_mask, n_clusters,
                                codes, meta, res_codes, res_meta, stream=None) -> None:
    _check(lib().fb4_quantize_decomposed_idx(ctx, _ptr(x), T, C, ld_elems, _ptr(salient_idx), n_salient,
                                             _ptr(cluster_id), _ptr(cluster_mask), n_clusters, _ptr(codes),
                                             _ptr(meta), _ptr(res_codes), _ptr(res_meta), _stream(stream)),
           "fb4_quantize_decomposed_idx")


def fb4_dequantize(ctx, codes, meta, T, C, salient_idx, n_salient, res_codes, res_meta, out, out_dtype,
                   stream=None) -> None:
    _check(lib().fb4_dequantize(ctx, _ptr(codes), _ptr(meta), T, C, _ptr(salient_idx), n_salient, _ptr(res_codes),
                                _ptr(res_meta), _ptr(out), out_dtype, _stream(stream)), "fb4_dequantize")


def fb4_quantize_weights(ctx, w, N, K, ld_elems, codes, meta, stream=None) -> None:
    _check(lib().fb4_quantize_weights(ctx, _ptr(w), N, K, ld_elems, _ptr(codes), _ptr(meta), _stream(stream)),
           "fb4_quantize_weights")


def fb4_quantize_mxfp8(ctx, x, T, C, ld_elems, cluster_id, cluster_mask, n_clusters, e4m3, scales, scale_layout,
                       stream=None) -> None:
    _check(lib().fb4_quantize_mxfp8(ctx, _ptr(x), T, C, ld_elems, _ptr(cluster_id), _ptr(cluster_mask), n_clusters,
                                    _ptr(e4m3), _ptr(scales), scale_layout, _stream(stream)), "fb4_quantize_mxfp8")


def fb4_quantize_mxfp8_decomposed(ctx, x, T, C, ld_elems, score, tile, salient_idx, n_salient, cluster_id, cluster_mask,
                                  n_clusters, e4m3, scales, res_e4m3, res_scales, scale_layout, stream=None) -> None:
    _check(lib().fb4_quantize_mxfp8_decomposed(ctx, _ptr(x), T, C, ld_elems, _ptr(score), tile, _ptr(salient_idx),
                                               n_salient, _ptr(cluster_id), _ptr(cluster_mask), n_clusters,
                                               _ptr(e4m3), _ptr(scales), _ptr(res_e4m3), _ptr(res_scales),
                                               scale_layout, _stream(stream)), "fb4_quantize_mxfp8_decomposed")


def fb4_to_mxfp8(ctx, codes, meta, T, C, e4m3, scales, scale_layout, stream=None) -> None:
    _check(lib().fb4_to_mxfp8(ctx, _ptr(codes), _ptr(meta), T, C, _ptr(e4m3), _ptr(scales), scale_layout,
                              _stream(stream)), "fb4_to_mxfp8")


def fb4_mxfp8_scale_bytes(T, C, scale_layout) -> int:
    return int(lib().fb4_mxfp8_scale_bytes(T, C, scale_layout))


def fb4_quantize_host(ctx, x_host, T, C, d_x, d_codes, d_meta, codes_host, meta_host) -> None:
    _check(lib().fb4_quantize_host(ctx, _ptr(x_host), T, C, _ptr(d_x), _ptr(d_codes), _ptr(d_meta),
                                   _ptr(codes_host), _ptr(meta_host)), "fb4_quantize_host")


def fb4_set_kernel_variant(ctx, variant: int) -> None:
    _check(lib().fb4_set_kernel_variant(ctx, variant), "fb4_set_kernel_variant")


def fb4_device_status(ctx) -> int:
    st = ctypes.c_uint32(0)
    _check(lib().fb4_device_status(ctx, ctypes.byref(st)), "fb4_device_status")
    return int(st.value)


def fb4_launch_count(ctx) -> int:
    return int(lib().fb4_launch_count(ctx))


def fb4_last_variant(ctx) -> str:
    return lib().fb4_last_variant(ctx).decode()


# ----------------------------------------------------------------------------- convenience wrapper

@dataclass
class Quantized:
    codes: torch.Tensor                      # uint8 [T][C/2]
    meta: torch.Tensor                       # uint16 bits in an int16 tensor [T][C/B]
    salient_idx: torch.Tensor | None = None  # int32 [n_salient]
    res_codes: torch.Tensor | None = None
    res_meta: torch.Tensor | None = None


class Fb4:
    """Owns one context; allocates outputs with torch and calls the entry points above."""

    def __init__(self, device: int | None = None, formatbook=None, stage1_mask=None, block_size: int = 32,
                 num_groups: int = 8, exp_min: int = -124, exp_max: int = 127, select_mode: int = 0):
        if not torch.cuda.is_available():
            raise RuntimeError("Fb4 needs a CUDA device (there is no CPU path)")
        self.device = torch.cuda.current_device() if device is None else device
        self.config = Fb4Config(block_size, num_groups, exp_min, exp_max, select_mode)
        self.block_size = block_size
        self.ctx = fb4_init(self.device, formatbook, stage1_mask, self.config)

    def close(self):
        if getattr(self, "ctx", None) is not None:
            fb4_destroy(self.ctx)
            self.ctx = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def _outs(self, T, C, n_res=0):
        dev = torch.device("cuda", self.device)
        codes = torch.empty((T, C // 2), dtype=torch.uint8, device=dev)
        meta = torch.empty((T, C // self.block_size), dtype=torch.int16, device=dev)
        if n_res:
            rc = torch.empty((n_res, C // 2), dtype=torch.uint8, device=dev)
            rm = torch.empty((n_res, C // self.block_size), dtype=torch.int16, device=dev)
            return codes, meta, rc, rm
        return codes, meta

    @staticmethod
    def _shape(x):
        assert x.dtype in (torch.bfloat16, torch.float32) and x.dim() == 2 and x.stride(1) == 1 and x.is_cuda
        return x.shape[0], x.shape[1], (x.stride(0) if x.shape[0] > 1 else x.shape[1])

    def quantize(self, x, cluster_id=None, cluster_mask=None) -> Quantized:
        T, C, ld = self._shape(x)
        codes, meta = self._outs(T, C)
        if x.dtype == torch.float32:
            assert cluster_id is None, "fp32 input: plain quantization only"
            fb4_quantize_f32(self.ctx, x, T, C, ld, codes, meta)
        elif cluster_id is None:
            fb4_quantize(self.ctx, x, T, C, ld, codes, meta)
        else:
            fb4_quantize_seda(self.ctx, x, T, C, ld, cluster_id, cluster_mask, cluster_mask.numel(), codes, meta)
        return Quantized(codes, meta)

    def quantize_affine(self, x, gain, bias, gain_plus_one: bool = False, cluster_id=None, cluster_mask=None) -> Quantized:
        """quantize(x * g + bias) with g = gain or 1 + gain per channel, the affine step evaluated in fp32 inside the kernel"""
        assert x.dtype == torch.bfloat16 and gain.dtype == torch.bfloat16 and bias.dtype == torch.bfloat16
        T, C, ld = self._shape(x)
        assert gain.numel() == C and bias.numel() == C
        codes, meta = self._outs(T, C)
        fb4_quantize_affine(self.ctx, x, T, C, ld, gain, bias, gain_plus_one, cluster_id, cluster_mask,
                            0 if cluster_mask is None else cluster_mask.numel(), codes, meta)
        return Quantized(codes, meta)

    def quantize_layernorm(self, x, gain, bias, gain_plus_one: bool = False, eps: float = 1e-6, cluster_id=None,
                           cluster_mask=None) -> Quantized:
        """quantize(LayerNorm(x) * g + bias), g = gain or 1 + gain per channel, in one fused pass"""
        T, C, ld = self._shape(x)
        codes, meta = self._outs(T, C)
        fb4_quantize_layernorm(self.ctx, x, T, C, ld, gain, bias, gain_plus_one, eps, cluster_id, cluster_mask,
                               0 if cluster_mask is None else cluster_mask.numel(), codes, meta)
        return Quantized(codes, meta)

    def quantize_affine_mxfp8(self, x, gain, bias, gain_plus_one: bool = False, scale_layout: int = 1, cluster_id=None,
                              cluster_mask=None):
        """(e4m3 [T][C], scales) of quantize(x * g + bias): producer, quantizer and MXFP8 view in one pass"""
        T, C, ld = self._shape(x)
        e4m3 = torch.empty((T, C), dtype=torch.uint8, device=x.device)
        n = fb4_mxfp8_scale_bytes(T, C, scale_layout)
        scales = torch.empty(max(n, 1), dtype=torch.uint8, device=x.device)
        fb4_quantize_affine_mxfp8(self.ctx, x, T, C, ld, gain, bias, gain_plus_one, cluster_id, cluster_mask,
                                  0 if cluster_mask is None else cluster_mask.numel(), e4m3, scales, scale_layout)
        return e4m3, scales[:n]

    def quantize_decomposed(self, x, score=None, tile: int = 20, salient_idx=None, cluster_id=None,
                            cluster_mask=None) -> Quantized:
        assert x.dtype == torch.bfloat16
        T, C, ld = self._shape(x)
        ncl = 0 if cluster_mask is None else cluster_mask.numel()
        if salient_idx is None:
            n = -(-T // tile)
            codes, meta, rc, rm = self._outs(T, C, max(n, 1))
            sal = torch.empty(max(n, 1), dtype=torch.int32, device=x.device)
            fb4_quantize_decomposed(self.ctx, x, T, C, ld, score, tile, cluster_id, cluster_mask, ncl, codes, meta,
                                    sal, rc, rm)
            return Quantized(codes, meta, sal[:n], rc[:n], rm[:n])
        n = salient_idx.numel()
        codes, meta, rc, rm = self._outs(T, C, max(n, 1))
        fb4_quantize_decomposed_idx(self.ctx, x, T, C, ld, salient_idx, n, cluster_id, cluster_mask, ncl, codes, meta,
                                    rc, rm)
        return Quantized(codes, meta, salient_idx, rc[:n], rm[:n])

    def build_subformatbook(self, meta, anchor_token, anchor_cluster, n_clusters: int):
        """cluster masks (int32 tensor holding uint32 bit patterns) from the dialects chosen on anchor tokens"""
        T, nblk = meta.shape
        counts = torch.empty((max(n_clusters, 1), 32), dtype=torch.int32, device=meta.device)
        masks = torch.empty(max(n_clusters, 1), dtype=torch.int32, device=meta.device)
        fb4_build_subformatbook(self.ctx, meta, T, nblk * self.block_size, anchor_token, anchor_cluster,
                                anchor_token.numel(), n_clusters, counts, masks)
        return masks[:n_clusters], counts[:n_clusters]

    def select_salient(self, score, tile: int = 20):
        T = score.numel()
        out = torch.empty(max(-(-T // tile), 1), dtype=torch.int32, device=score.device)
        fb4_select_salient(self.ctx, score, T, tile, out)
        return out[:-(-T // tile)]

    def select_salient_topk(self, score, k: int):
        out = torch.empty(max(k, 1), dtype=torch.int32, device=score.device)
        fb4_select_salient_topk(self.ctx, score, score.numel(), k, out)
        return out[:k]

    def dequantize(self, q: Quantized, dtype=torch.float32):
        T, C = q.codes.shape[0], q.codes.shape[1] * 2
        out = torch.empty((T, C), dtype=dtype, device=q.codes.device)
        n = 0 if q.salient_idx is None else q.salient_idx.numel()
        fb4_dequantize(self.ctx, q.codes, q.meta, T, C, q.salient_idx if n else None, n,
                       q.res_codes if n else None, q.res_meta if n else None, out,
                       {torch.float32: 0, torch.bfloat16: 1, torch.float16: 2}[dtype])
        return out

    def quantize_weights(self, w) -> Quantized:
        """offline weight quantization: exhaustive squared-error dialect selection"""
        assert w.dtype == torch.bfloat16
        N, K, ld = self._shape(w)
        codes, meta = self._outs(N, K)
        fb4_quantize_weights(self.ctx, w, N, K, ld, codes, meta)
        return Quantized(codes, meta)

    def quantize_mxfp8(self, x, scale_layout: int = 1, cluster_id=None, cluster_mask=None):
        """quantize straight to (e4m3 bytes [T][C], E8M0 scale bytes)"""
        assert x.dtype == torch.bfloat16
        T, C, ld = self._shape(x)
        e4m3 = torch.empty((T, C), dtype=torch.uint8, device=x.device)
        n = fb4_mxfp8_scale_bytes(T, C, scale_layout)
        scales = torch.empty(max(n, 1), dtype=torch.uint8, device=x.device)
        fb4_quantize_mxfp8(self.ctx, x, T, C, ld, cluster_id, cluster_mask,
                           0 if cluster_mask is None else cluster_mask.numel(), e4m3, scales, scale_layout)
        return e4m3, scales[:n]

    def quantize_mxfp8_decomposed(self, x, score=None, tile: int = 20, salient_idx=None, scale_layout: int = 1,
                                  cluster_id=None, cluster_mask=None):
        """-> (e4m3 [T][C], scales, salient_idx, res_e4m3 [n][C], res_scales): main and residual MXFP8 operands"""
        assert x.dtype == torch.bfloat16
        T, C, ld = self._shape(x)
        n = -(-T // tile) if salient_idx is None else salient_idx.numel()
        if salient_idx is None:
            salient_idx = torch.empty(max(n, 1), dtype=torch.int32, device=x.device)
        dev = x.device
        e4m3 = torch.empty((T, C), dtype=torch.uint8, device=dev)
        scales = torch.empty(max(fb4_mxfp8_scale_bytes(T, C, scale_layout), 1), dtype=torch.uint8, device=dev)
        res = torch.empty((max(n, 1), C), dtype=torch.uint8, device=dev)
        nrs = fb4_mxfp8_scale_bytes(n, C, scale_layout)
        res_scales = torch.empty(max(nrs, 1), dtype=torch.uint8, device=dev)
        fb4_quantize_mxfp8_decomposed(self.ctx, x, T, C, ld, score, tile, salient_idx, n, cluster_id, cluster_mask,
                                      0 if cluster_mask is None else cluster_mask.numel(), e4m3, scales, res,
                                      res_scales, scale_layout)
        return (e4m3, scales[:fb4_mxfp8_scale_bytes(T, C, scale_layout)], salient_idx[:n], res[:n], res_scales[:nrs])

    def to_mxfp8(self, q: Quantized, scale_layout: int = 0):
        """(e4m3 bytes [T][C], E8M0 scale bytes) of the main tensor of q."""
        T, C = q.codes.shape[0], q.codes.shape[1] * 2
        e4m3 = torch.empty((T, C), dtype=torch.uint8, device=q.codes.device)
        scales = torch.empty(max(fb4_mxfp8_scale_bytes(T, C, scale_layout), 1), dtype=torch.uint8,
                             device=q.codes.device)
        fb4_to_mxfp8(self.ctx, q.codes, q.meta, T, C, e4m3, scales, scale_layout)
        return e4m3, scales[:fb4_mxfp8_scale_bytes(T, C, scale_layout)]

    def set_kernel_variant(self, variant: int) -> None:
        fb4_set_kernel_variant(self.ctx, variant)

    @property
    def device_status(self) -> int:
        return fb4_device_status(self.ctx)

    @property
    def launch_count(self) -> int:
        return fb4_launch_count(self.ctx)

    @property
    def last_variant(self) -> str:
        return fb4_last_variant(self.ctx)
