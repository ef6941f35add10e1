"""Seeded synthetic inputs shared by the oracle tests, the GPU parity tests and bench.py.

Nothing here belongs to the quantization method: this module only makes input
data (activation tensors as bf16 bit patterns, attention scores, SeDA cluster
tables) and names the five benchmark workloads.  The generator itself is the
small C file next to this one (counter-based, so single rows can be produced on
demand); it is compiled on first use with gcc.

The stand-in formatbook is input data as well: the paper shows its 32-dialect
formatbook only in a figure (Fig. 2a), so the table below was designed from the
four construction rules of Sec. 3.1 (cover every dynamic range 8..15, densify
small magnitudes, keep dialects that preserve large magnitudes, fewer dialects
for narrower ranges; dialect ids ascend with dynamic range as App. B states) and
can be replaced at init time.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass, field

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "fb4_synth.c")
_LIB = os.path.join(_HERE, "_fb4_synth.so")

# 32 dialects x 8 magnitudes (ints 0..15, ascending, first is 0).  Dialects per
# dynamic range (largest magnitude 8..15): 2, 2, 3, 3, 4, 5, 6, 7.
STANDIN_FORMATBOOK = np.array([
    [0, 1, 2, 3, 4, 5, 6, 8], [0, 1, 2, 4, 5, 6, 7, 8],
    [0, 1, 2, 3, 4, 5, 7, 9], [0, 1, 2, 4, 6, 7, 8, 9],
    [0, 1, 2, 3, 4, 6, 8, 10], [0, 1, 2, 3, 5, 7, 9, 10], [0, 1, 2, 4, 6, 8, 9, 10],
    [0, 1, 2, 3, 4, 6, 8, 11], [0, 1, 2, 3, 5, 7, 9, 11], [0, 1, 2, 4, 6, 8, 10, 11],
    [0, 1, 2, 3, 4, 6, 8, 12], [0, 1, 2, 3, 5, 7, 9, 12], [0, 1, 2, 4, 6, 8, 10, 12],
    [0, 2, 4, 6, 8, 10, 11, 12],
    [0, 1, 2, 3, 4, 6, 9, 13], [0, 1, 2, 3, 5, 7, 10, 13], [0, 1, 2, 4, 6, 8, 10, 13],
    [0, 1, 2, 4, 6, 9, 11, 13], [0, 2, 4, 6, 8, 10, 12, 13],
    [0, 1, 2, 3, 4, 6, 9, 14], [0, 1, 2, 3, 5, 7, 10, 14], [0, 1, 2, 4, 6, 8, 11, 14],
    [0, 1, 2, 4, 6, 9, 12, 14], [0, 1, 3, 5, 7, 9, 12, 14], [0, 2, 4, 6, 8, 10, 12, 14],
    [0, 1, 2, 3, 4, 6, 9, 15], [0, 1, 2, 3, 5, 7, 10, 15], [0, 1, 2, 4, 6, 8, 11, 15],
    [0, 1, 2, 4, 6, 9, 12, 15], [0, 1, 3, 5, 7, 9, 12, 15], [0, 1, 3, 5, 7, 10, 13, 15],
    [0, 2, 4, 6, 8, 11, 13, 15],
], dtype=np.uint8)


def build(force: bool = False) -> str:
    """Compile the generator (gcc, OpenMP) next to its source; returns the .so path."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".{os.getpid()}.tmp"
        subprocess.check_call(["gcc", "-O2", "-fPIC", "-shared", "-fopenmp", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        i64, u64, i32 = ctypes.c_int64, ctypes.c_uint64, ctypes.c_int32
        vp = ctypes.c_void_p
        lib.fb4s_outlier_channels.argtypes = [u64, i64, i64, vp]
        lib.fb4s_fill_rows.argtypes = [u64, ctypes.c_int, i64, i64, i64, vp, vp, i64]
        lib.fb4s_scores.argtypes = [u64, i64, i64, vp]
        lib.fb4s_cluster_ids.argtypes = [u64, i64, i32, vp]
        lib.fb4s_cluster_masks.argtypes = [u64, vp, i32, vp]
        for f in (lib.fb4s_outlier_channels, lib.fb4s_fill_rows, lib.fb4s_scores,
                  lib.fb4s_cluster_ids, lib.fb4s_cluster_masks):
            f.restype = ctypes.c_int
        _lib = lib
    return _lib


def _ptr(a: np.ndarray):
    return a.ctypes.data_as(ctypes.c_void_p)


@dataclass(frozen=True)
class Workload:
    """One benchmark configuration (shapes, seeds and which extensions are on)."""
    name: str
    T: int
    C: int
    seed: int
    kind: int                 # 0: N(0,1); 1: per-token log-normal scale x Student-t(3)
    n_outlier: int
    outlier_gain: float
    block_size: int = 32
    decomposed: bool = False
    tile: int = 20            # tokens per salient-token tile (top-1 of 20 = 5 %)
    score_seed: int = 0
    seda: bool = False
    n_clusters: int = 0
    cluster_seed: int = 0
    notes: str = field(default="", compare=False)


def workloads() -> dict[str, Workload]:
    """The five configurations, in order, plus the plain quantizer on the largest tensor."""
    c2 = dict(T=32760, C=3072, seed=1, kind=1, n_outlier=round(0.005 * 3072), outlier_gain=50.0)
    c5 = dict(T=75600, C=12288, seed=4, kind=1, n_outlier=round(0.005 * 12288), outlier_gain=50.0)
    return {
        "c1": Workload("c1", 256, 3072, seed=0, kind=0, n_outlier=8, outlier_gain=30.0),
        "c2": Workload("c2", **c2),
        "c3": Workload("c3", **c2, decomposed=True, score_seed=2),
        "c4": Workload("c4", **c2, seda=True, n_clusters=64, cluster_seed=3),
        "c5": Workload("c5", **c5, decomposed=True, score_seed=4, seda=True, n_clusters=256, cluster_seed=4),
        "c5_plain": Workload("c5_plain", **c5),
    }


def channel_gain(w: Workload) -> np.ndarray:
    lib = _load()
    idx = np.zeros(max(w.n_outlier, 1), dtype=np.int64)
    rc = lib.fb4s_outlier_channels(w.seed, w.C, w.n_outlier, _ptr(idx))
    assert rc == 0
    g = np.ones(w.C, dtype=np.float32)
    g[idx[:w.n_outlier]] = w.outlier_gain
    return g


def activation_rows(w: Workload, row0: int, nrows: int, out: np.ndarray | None = None) -> np.ndarray:
    """bf16 bit patterns (uint16) of rows [row0, row0+nrows) of the workload's tensor."""
    lib = _load()
    if out is None:
        out = np.empty((nrows, w.C), dtype=np.uint16)
    assert out.dtype == np.uint16 and out.shape == (nrows, w.C) and out.flags.c_contiguous
    g = channel_gain(w)
    rc = lib.fb4s_fill_rows(w.seed, w.kind, w.C, row0, nrows, _ptr(g), _ptr(out), w.C)
    assert rc == 0
    return out


def activation(w: Workload) -> np.ndarray:
    return activation_rows(w, 0, w.T)


def scores(w: Workload) -> np.ndarray:
    lib = _load()
    s = np.empty(w.T, dtype=np.float32)
    assert lib.fb4s_scores(w.score_seed, 0, w.T, _ptr(s)) == 0
    return s


def clusters(w: Workload, formatbook: np.ndarray = STANDIN_FORMATBOOK):
    """(cluster_id[T] int32, cluster_mask[n_clusters] uint32) for a SeDA workload."""
    lib = _load()
    cid = np.empty(w.T, dtype=np.int32)
    assert lib.fb4s_cluster_ids(w.cluster_seed, w.T, w.n_clusters, _ptr(cid)) == 0
    fb = np.ascontiguousarray(formatbook, dtype=np.uint8)
    mask = np.empty(w.n_clusters, dtype=np.uint32)
    assert lib.fb4s_cluster_masks(w.cluster_seed, _ptr(fb), w.n_clusters, _ptr(mask)) == 0
    return cid, mask


def anchors(cluster_id: np.ndarray, n_clusters: int, per_cluster: int = 8):
    """Anchor tokens of a SeDA workload: up to `per_cluster` tokens spread evenly over every
    cluster's token range (deterministic, no random draw).  Returns (anchor_token, anchor_cluster),
    both int32, ordered by cluster."""
    tok, clu = [], []
    for c in range(n_clusters):
        members = np.flatnonzero(cluster_id == c)
        if members.size == 0:
            continue
        pick = np.unique(members[(np.arange(per_cluster) * members.size) // per_cluster])
        tok.append(pick)
        clu.append(np.full(pick.size, c))
    if not tok:
        return np.zeros(0, np.int32), np.zeros(0, np.int32)
    return np.concatenate(tok).astype(np.int32), np.concatenate(clu).astype(np.int32)


# ---- small helpers for hand-made test inputs (format conversion only) ----

def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round float32 to bf16 (nearest even) and return the uint16 bit patterns."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32).astype(np.uint64)
    lsb = (u >> 16) & 1
    r = ((u + 0x7FFF + lsb) >> 16).astype(np.uint16)
    nan_inf = (u & 0x7F800000) == 0x7F800000
    return np.where(nan_inf, (u >> 16).astype(np.uint16), r)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << 16).view(np.float32)
