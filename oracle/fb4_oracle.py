"""ctypes access to the CPU oracle (oracle/fb4_oracle.c) -- TEST INFRASTRUCTURE.

Only tests, the smoke check and the benchmark's CPU-baseline / reference legs may
import this.  It imports nothing from the CUDA package and shares no code with it.
The C file is compiled with gcc on first use.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "fb4_oracle.c")
_LIB = os.path.join(_HERE, "libfb4_oracle.so")


class _Cfg(ctypes.Structure):
    _fields_ = [("block_size", ctypes.c_int), ("num_groups", ctypes.c_int),
                ("exp_min", ctypes.c_int), ("exp_max", ctypes.c_int),
                ("select_mode", ctypes.c_int)]


@dataclass(frozen=True)
class Config:
    block_size: int = 32
    num_groups: int = 8
    exp_min: int = -124
    exp_max: int = 127
    select_mode: int = 0

    def c(self) -> _Cfg:
        return _Cfg(self.block_size, self.num_groups, self.exp_min, self.exp_max, self.select_mode)


def build(force: bool = False) -> str:
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".{os.getpid()}.tmp"
        subprocess.check_call(["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-fopenmp",
                               "-ffp-contract=off", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


_libs: dict = {}
_active = None   # tests that check the pins against a deliberately broken copy set this


def use_library(path):
    """Route the functions below to another build of the oracle source (None = the real one).

    The mutation tests compile copies of fb4_oracle.c with one planted mistake each and
    check that the pins notice; nothing else should call this."""
    global _active
    _active = path


def lib():
    path = _active or build()
    if path not in _libs:
        L = ctypes.CDLL(path)
        vp, i64, i32, u32 = ctypes.c_void_p, ctypes.c_int64, ctypes.c_int32, ctypes.c_uint32
        L.fb4o_default_stage1.argtypes = [vp, vp]
        L.fb4o_default_stage1.restype = None
        L.fb4o_select_salient.argtypes = [vp, i64, i32, vp]
        L.fb4o_select_salient.restype = i64
        L.fb4o_select_salient_topk.argtypes = [vp, i64, i64, vp]
        L.fb4o_select_salient_topk.restype = i64
        L.fb4o_quantize.argtypes = [vp, i64, i64, i64, ctypes.POINTER(_Cfg), vp, vp,
                                    vp, vp, i32, vp, i64, vp, vp, vp, vp, vp]
        L.fb4o_quantize.restype = ctypes.c_int
        L.fb4o_dequantize.argtypes = [vp, vp, i64, i64, ctypes.c_int, vp, vp, i64, vp, vp, vp, ctypes.c_int]
        L.fb4o_dequantize.restype = ctypes.c_int
        L.fb4o_mse.argtypes = [vp, i64, vp, i64, i64]
        L.fb4o_mse.restype = ctypes.c_double
        L.fb4o_quantize_block_f64.argtypes = [vp, ctypes.POINTER(_Cfg), vp, vp, u32, vp, vp, vp, vp]
        L.fb4o_quantize_block_f64.restype = ctypes.c_int
        L.fb4o_quantize_f32.argtypes = [vp, i64, i64, i64, ctypes.POINTER(_Cfg), vp, vp, vp, vp, i32, vp, vp]
        L.fb4o_quantize_f32.restype = ctypes.c_int
        L.fb4o_affine_f32.argtypes = [vp, i64, i64, i64, vp, vp, ctypes.c_int, vp]
        L.fb4o_affine_f32.restype = ctypes.c_int
        L.fb4o_layernorm_f32.argtypes = [vp, i64, i64, i64, vp, vp, ctypes.c_int, ctypes.c_float, vp, vp]
        L.fb4o_layernorm_f32.restype = ctypes.c_int
        L.fb4o_to_mxfp8.argtypes = [vp, vp, i64, i64, vp, vp, vp, ctypes.c_int]
        L.fb4o_to_mxfp8.restype = ctypes.c_int
        L.fb4o_mxfp8_scale_offset.argtypes = [i64, i64, i64, ctypes.c_int]
        L.fb4o_mxfp8_scale_offset.restype = i64
        L.fb4o_mxfp8_scale_bytes.argtypes = [i64, i64, ctypes.c_int]
        L.fb4o_mxfp8_scale_bytes.restype = i64
        L.fb4o_quantize_weights.argtypes = [vp, i64, i64, i64, ctypes.POINTER(_Cfg), vp, vp, vp, vp]
        L.fb4o_quantize_weights.restype = ctypes.c_int
        L.fb4o_build_subformatbook.argtypes = [vp, i64, i64, vp, vp, i64, i32, vp, vp, vp]
        L.fb4o_build_subformatbook.restype = ctypes.c_int
        _libs[path] = L
    return _libs[path]


def _p(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _c(a, dtype):
    if a is None:
        return None
    return np.ascontiguousarray(a, dtype=dtype)


def default_stage1(formatbook) -> np.ndarray:
    F = _c(formatbook, np.uint8)
    out = np.zeros(32, dtype=np.uint32)
    lib().fb4o_default_stage1(_p(F), _p(out))
    return out


def select_salient(score, tile: int) -> np.ndarray:
    s = _c(score, np.float32)
    T = s.shape[0]
    out = np.zeros(max(1, -(-T // tile)), dtype=np.int32)
    n = lib().fb4o_select_salient(_p(s), T, tile, _p(out))
    assert n >= 0
    return out[:n].copy()


def select_salient_topk(score, k: int) -> np.ndarray:
    """the k highest-scoring tokens of the whole sequence (ties -> lowest index), ascending"""
    s = _c(score, np.float32)
    out = np.zeros(max(1, k), dtype=np.int32)
    n = lib().fb4o_select_salient_topk(_p(s), s.shape[0], k, _p(out))
    assert n == k
    return out[:k].copy()


@dataclass
class Quantized:
    codes: np.ndarray            # uint8 [T][C/2]
    meta: np.ndarray             # uint16 [T][C/B]: scale byte | did << 8
    salient_idx: np.ndarray | None = None
    res_codes: np.ndarray | None = None
    res_meta: np.ndarray | None = None
    err_q4: np.ndarray | None = None

    @property
    def did(self):
        return (self.meta >> 8).astype(np.int32)

    @property
    def exponent(self):
        return (self.meta & 0xFF).astype(np.int32) - 124


def quantize(x_bits, formatbook, cfg: Config = Config(), stage1=None, cluster_id=None,
             cluster_mask=None, salient_idx=None, want_errors: bool = False) -> Quantized:
    """x_bits: uint16 [T][C] bf16 bit patterns (a row-strided view is accepted)."""
    x = np.asarray(x_bits)
    assert x.dtype == np.uint16 and x.ndim == 2 and x.strides[1] == 2
    T, C = x.shape
    ld = x.strides[0] // 2 if T > 1 else C
    B = cfg.block_size
    F = _c(formatbook, np.uint8)
    s1 = _c(stage1, np.uint32)
    cid = _c(cluster_id, np.int32)
    cm = _c(cluster_mask, np.uint32)
    sal = _c(salient_idx, np.int32)
    ns = 0 if sal is None else sal.shape[0]
    codes = np.zeros((T, C // 2), dtype=np.uint8)
    meta = np.zeros((T, max(C // B, 0)), dtype=np.uint16)
    rc = np.zeros((max(ns, 1), C // 2), dtype=np.uint8)
    rm = np.zeros((max(ns, 1), C // B), dtype=np.uint16)
    err = np.zeros((T, C // B, 32), dtype=np.int32) if want_errors else None
    ccfg = cfg.c()
    r = lib().fb4o_quantize(x.ctypes.data_as(ctypes.c_void_p), T, C, ld, ctypes.byref(ccfg), _p(F), _p(s1),
                            _p(cid), _p(cm), 0 if cm is None else cm.shape[0], _p(sal), ns,
                            _p(codes), _p(meta), _p(rc), _p(rm), _p(err))
    if r != 0:
        raise ValueError(f"fb4o_quantize failed: {r}")
    q = Quantized(codes, meta, err_q4=err)
    if sal is not None:
        q.salient_idx, q.res_codes, q.res_meta = sal, rc[:ns], rm[:ns]
    return q


def dequantize(q: Quantized, formatbook, block_size: int = 32, out_dtype: str = "f32") -> np.ndarray:
    T, C2 = q.codes.shape
    C = C2 * 2
    F = _c(formatbook, np.uint8)
    ns = 0 if q.salient_idx is None else q.salient_idx.shape[0]
    code = {"f32": 0, "bf16": 1, "f16": 2}[out_dtype]
    out = np.zeros((T, C), dtype=np.float32 if code == 0 else np.uint16)
    r = lib().fb4o_dequantize(_p(_c(q.codes, np.uint8)), _p(_c(q.meta, np.uint16)), T, C, block_size, _p(F),
                              _p(_c(q.salient_idx, np.int32)), ns,
                              _p(_c(q.res_codes, np.uint8)), _p(_c(q.res_meta, np.uint16)),
                              _p(out), code)
    if r != 0:
        raise ValueError(f"fb4o_dequantize failed: {r}")
    return out


def mse(x_bits, recon) -> float:
    x = np.ascontiguousarray(x_bits, dtype=np.uint16)
    y = np.ascontiguousarray(recon, dtype=np.float32)
    T, C = x.shape
    return float(lib().fb4o_mse(_p(x), C, _p(y), T, C))


def quantize_block_f64(x, formatbook, cfg: Config = Config(), stage1=None, allowed: int = 0xFFFFFFFF):
    """One block of doubles -> (codes[B] with sign<<3|idx, did, e, err_q4[32])."""
    xv = np.ascontiguousarray(x, dtype=np.float64)
    assert xv.shape == (cfg.block_size,)
    F = _c(formatbook, np.uint8)
    s1 = _c(stage1, np.uint32)
    code = np.zeros(cfg.block_size, dtype=np.uint8)
    did = np.zeros(1, dtype=np.int32)
    e = np.zeros(1, dtype=np.int32)
    err = np.zeros(32, dtype=np.int32)
    ccfg = cfg.c()
    r = lib().fb4o_quantize_block_f64(_p(xv), ctypes.byref(ccfg), _p(F), _p(s1), allowed & 0xFFFFFFFF,
                                      _p(code), _p(did), _p(e), _p(err))
    if r != 0:
        raise ValueError(f"fb4o_quantize_block_f64 failed: {r}")
    return code, int(did[0]), int(e[0]), err


def build_subformatbook(meta, anchor_token, anchor_cluster, n_clusters: int, formatbook, stage1=None) -> np.ndarray:
    """meta: uint16 [T][C/B]; anchors: int32 token ids and their clusters -> uint32 [n_clusters] masks."""
    m = _c(meta, np.uint16)
    T, nblk = m.shape
    at = _c(anchor_token, np.int32)
    ac = _c(anchor_cluster, np.int32)
    assert at.shape == ac.shape
    out = np.zeros(max(n_clusters, 1), dtype=np.uint32)
    r = lib().fb4o_build_subformatbook(_p(m), T, nblk, _p(at), _p(ac), at.shape[0], n_clusters,
                                       _p(_c(formatbook, np.uint8)), _p(_c(stage1, np.uint32)), _p(out))
    if r != 0:
        raise ValueError(f"fb4o_build_subformatbook failed: {r}")
    return out[:n_clusters]


def quantize_f32(x, formatbook, cfg: Config = Config(), stage1=None, cluster_id=None, cluster_mask=None) -> Quantized:
    """x: float32 [T][C], quantized as it is (no rounding to bf16); optional SeDA tables."""
    xv = np.ascontiguousarray(x, dtype=np.float32)
    T, C = xv.shape
    codes = np.zeros((T, C // 2), dtype=np.uint8)
    meta = np.zeros((T, C // cfg.block_size), dtype=np.uint16)
    ccfg = cfg.c()
    cid, cm = _c(cluster_id, np.int32), _c(cluster_mask, np.uint32)
    r = lib().fb4o_quantize_f32(_p(xv), T, C, C, ctypes.byref(ccfg), _p(_c(formatbook, np.uint8)),
                                _p(_c(stage1, np.uint32)), _p(cid), _p(cm), 0 if cm is None else len(cm),
                                _p(codes), _p(meta))
    if r != 0:
        raise ValueError(f"fb4o_quantize_f32 failed: {r}")
    return Quantized(codes, meta)


def affine_f32(x_bits, gain_bits, bias_bits, plus_one: bool) -> np.ndarray:
    """y = x * g + bias per channel in float32 (one rounding), g = gain or 1 + gain; all inputs bf16 bit patterns."""
    x = np.asarray(x_bits)
    assert x.dtype == np.uint16 and x.ndim == 2 and x.strides[1] == 2
    T, C = x.shape
    ld = x.strides[0] // 2 if T > 1 else C
    g, b = _c(gain_bits, np.uint16), _c(bias_bits, np.uint16)
    assert g.shape == (C,) and b.shape == (C,)
    y = np.zeros((T, C), dtype=np.float32)
    r = lib().fb4o_affine_f32(_p(x), T, C, ld, _p(g), _p(b), int(bool(plus_one)), _p(y))
    if r != 0:
        raise ValueError(f"fb4o_affine_f32 failed: {r}")
    return y


def layernorm_f32(x_bits, gain_bits, bias_bits, plus_one: bool, eps: float, want_stats: bool = False):
    """LayerNorm + per-channel modulation in float32 with the stated order of operations; inputs bf16 bit patterns."""
    x = np.asarray(x_bits)
    assert x.dtype == np.uint16 and x.ndim == 2 and x.strides[1] == 2
    T, C = x.shape
    ld = x.strides[0] // 2 if T > 1 else C
    g, b = _c(gain_bits, np.uint16), _c(bias_bits, np.uint16)
    assert g.shape == (C,) and b.shape == (C,)
    y = np.zeros((T, C), dtype=np.float32)
    stats = np.zeros((T, 2), dtype=np.float32) if want_stats else None
    r = lib().fb4o_layernorm_f32(_p(x), T, C, ld, _p(g), _p(b), int(bool(plus_one)), float(np.float32(eps)), _p(y), _p(stats))
    if r != 0:
        raise ValueError(f"fb4o_layernorm_f32 failed: {r}")
    return (y, stats) if want_stats else y


def mxfp8_scale_offset(row: int, col: int, n_col: int, layout: int) -> int:
    return int(lib().fb4o_mxfp8_scale_offset(row, col, n_col, layout))


def to_mxfp8(q: Quantized, formatbook, layout: int = 0):
    """(e4m3 bytes uint8 [T][C], E8M0 scale bytes in the given layout) of a block-32 quantized tensor."""
    T, C2 = q.codes.shape
    C = C2 * 2
    out = np.zeros((T, C), dtype=np.uint8)
    n = int(lib().fb4o_mxfp8_scale_bytes(T, C, layout))
    sc = np.zeros(max(n, 1), dtype=np.uint8)
    r = lib().fb4o_to_mxfp8(_p(_c(q.codes, np.uint8)), _p(_c(q.meta, np.uint16)), T, C, _p(_c(formatbook, np.uint8)),
                            _p(out), _p(sc), layout)
    if r != 0:
        raise ValueError(f"fb4o_to_mxfp8 failed: {r}")
    return out, sc[:n]


def quantize_weights(w_bits, formatbook, cfg: Config = Config(), want_sse: bool = False):
    """w_bits: uint16 [N][K] bf16 bit patterns; exhaustive exact-squared-error dialect selection."""
    w = np.ascontiguousarray(w_bits, dtype=np.uint16)
    N, K = w.shape
    B = cfg.block_size
    codes = np.zeros((N, K // 2), dtype=np.uint8)
    meta = np.zeros((N, K // B), dtype=np.uint16)
    sse = np.zeros((N, K // B, 32), dtype=np.float64) if want_sse else None
    ccfg = cfg.c()
    r = lib().fb4o_quantize_weights(_p(w), N, K, K, ctypes.byref(ccfg), _p(_c(formatbook, np.uint8)), _p(codes),
                                    _p(meta), _p(sse))
    if r != 0:
        raise ValueError(f"fb4o_quantize_weights failed: {r}")
    q = Quantized(codes, meta)
    return (q, sse) if want_sse else q
