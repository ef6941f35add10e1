"""Helpers of the GPU parity tests: move seeded inputs to the device, run the library through
its binding, and compare element by element with the CPU oracle."""
from __future__ import annotations

import numpy as np
import torch

from oracle import fb4_oracle as orc
from paper_2603_02883_b200 import fb4, synth

FB = synth.STANDIN_FORMATBOOK


def to_dev_bf16(bits: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(bits.view(np.int16)).cuda().view(torch.bfloat16)


def meta_np(t: torch.Tensor) -> np.ndarray:
    return t.cpu().numpy().view(np.uint16)


def assert_same_quantized(q_gpu: fb4.Quantized, q_ref: orc.Quantized, what: str = ""):
    codes = q_gpu.codes.cpu().numpy()
    meta = meta_np(q_gpu.meta)
    bad = np.flatnonzero((meta != q_ref.meta).ravel())
    assert bad.size == 0, f"{what}: {bad.size} meta mismatches, first at block {bad[:5]}: " \
                          f"gpu {meta.ravel()[bad[:5]]} ref {q_ref.meta.ravel()[bad[:5]]}"
    badc = np.flatnonzero((codes != q_ref.codes).ravel())
    assert badc.size == 0, f"{what}: {badc.size} code byte mismatches, first at {badc[:5]}"
    if q_ref.salient_idx is not None:
        assert np.array_equal(q_gpu.salient_idx.cpu().numpy(), q_ref.salient_idx), f"{what}: salient indices"
        assert np.array_equal(meta_np(q_gpu.res_meta), q_ref.res_meta), f"{what}: residual meta"
        assert np.array_equal(q_gpu.res_codes.cpu().numpy(), q_ref.res_codes), f"{what}: residual codes"


def assert_same_bits_f32(a: torch.Tensor, b: np.ndarray, what: str = ""):
    """0 ULP: identical bit patterns, signed zeros included."""
    ga = a.cpu().numpy().view(np.uint32)
    assert np.array_equal(ga, b.view(np.uint32)), f"{what}: fp32 outputs differ in " \
                                                  f"{np.count_nonzero(ga != b.view(np.uint32))} elements"
