"""LayerNorm + modulation fused in front of the quantizer (fb4_quantize_layernorm) against the oracle: the oracle
evaluates the stated float32 order of operations and quantizes the float32 result; bit-exact."""
import numpy as np
import pytest
import torch

from gpu_util import FB, assert_same_quantized, to_dev_bf16
from oracle import fb4_oracle as orc
from paper_2603_02883_b200 import fb4, synth

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def q32():
    q = fb4.Fb4()
    yield q
    assert q.device_status == 0
    q.close()


def _inputs(T, C, seed, offset=0.0):
    w = synth.Workload("ln", T=T, C=C, seed=seed, kind=1, n_outlier=max(1, C // 200), outlier_gain=50.0)
    bits = synth.activation(w)
    rng = np.random.default_rng(seed)
    if offset:
        bits = synth.f32_to_bf16_bits(synth.bf16_bits_to_f32(bits) + np.float32(offset))
    gain = synth.f32_to_bf16_bits((0.5 * rng.standard_normal(C)).astype(np.float32))
    bias = synth.f32_to_bf16_bits(rng.standard_normal(C).astype(np.float32))
    return bits, gain, bias


@pytest.mark.parametrize("T,C,plus_one", [(1, 1024, False), (37, 1024, True), (333, 3072, True), (130, 12288, True),
                                          (50, 16384, False), (19, 5120, True), (700, 2048, False)])
def test_layernorm_quantize_matches_the_oracle(q32, T, C, plus_one):
    bits, gain, bias = _inputs(T, C, seed=100 + T, offset=0.75)
    bits[0, :32] = 0
    if T > 2:
        bits[2, :] = bits[2, 0]                       # a token of equal values: d = 0, y = bias
    eps = 1e-6
    y = orc.layernorm_f32(bits, gain, bias, plus_one, eps)
    ref = orc.quantize_f32(y, FB)
    got = q32.quantize_layernorm(to_dev_bf16(bits), to_dev_bf16(gain), to_dev_bf16(bias), plus_one, eps)
    assert q32.last_variant == "fast"
    assert_same_quantized(got, ref, f"layernorm {T}x{C}")


def test_layernorm_with_seda_masks(q32):
    T, C = 260, 3072
    bits, gain, bias = _inputs(T, C, seed=7)
    w = synth.Workload("ln", T=T, C=C, seed=7, kind=1, n_outlier=3, outlier_gain=50.0, seda=True, n_clusters=5, cluster_seed=8)
    cid, masks = synth.clusters(w)
    cid = cid.copy()
    cid[::17] = -1
    masks = masks.copy()
    masks[1] = 0x00F00F03
    y = orc.layernorm_f32(bits, gain, bias, True, 1e-5)
    ref = orc.quantize_f32(y, FB, cluster_id=cid, cluster_mask=masks)
    got = q32.quantize_layernorm(to_dev_bf16(bits), to_dev_bf16(gain), to_dev_bf16(bias), True, 1e-5,
                                 cluster_id=torch.from_numpy(cid).cuda(),
                                 cluster_mask=torch.from_numpy(masks.view(np.int32)).cuda())
    assert_same_quantized(got, ref, "layernorm seda")


def test_layernorm_full_size_rows(q32):
    """4000 tokens of the largest tensor's width (12 288 channels): several steps per CTA, ragged last step"""
    T, C = 4001, 12288
    bits, gain, bias = _inputs(T, C, seed=4)
    y = orc.layernorm_f32(bits, gain, bias, True, 1e-6)
    ref = orc.quantize_f32(y, FB)
    got = q32.quantize_layernorm(to_dev_bf16(bits), to_dev_bf16(gain), to_dev_bf16(bias), True, 1e-6)
    assert_same_quantized(got, ref, "layernorm 4001x12288")


def test_layernorm_argument_checks(q32):
    x = torch.zeros((4, 1024), dtype=torch.bfloat16, device="cuda")
    g = torch.zeros(1024, dtype=torch.bfloat16, device="cuda")
    codes = torch.zeros((4, 512), dtype=torch.uint8, device="cuda")
    meta = torch.zeros((4, 32), dtype=torch.int16, device="cuda")
    L = fb4.lib()
    p = lambda t: t.data_ptr()
    import ctypes
    call = lambda T, C, ld, eps: L.fb4_quantize_layernorm(q32.ctx, p(x), T, C, ld, p(g), p(g), 0, ctypes.c_float(eps), None,
                                                          None, 0, p(codes), p(meta), None)
    assert call(4, 1024, 1024, 1e-6) == fb4.OK
    assert call(4, 512, 512, 1e-6) == fb4.ERR_SHAPE          # not a multiple of 1024
    assert call(2, 1024, 2048, 1e-6) == fb4.ERR_SHAPE        # strided rows
    assert call(4, 1024, 1024, -1.0) == fb4.ERR_INVALID_ARG
    assert call(4, 1024, 1024, float("nan")) == fb4.ERR_INVALID_ARG
    q16 = fb4.Fb4(block_size=16)
    assert L.fb4_quantize_layernorm(q16.ctx, p(x), 4, 1024, 1024, p(g), p(g), 0, ctypes.c_float(1e-6), None, None, 0,
                                    p(codes), p(meta), None) == fb4.ERR_INVALID_ARG
    q16.close()
    torch.cuda.synchronize()


@pytest.mark.parametrize("T,C", [(1, 1024), (7, 3072), (33, 5120), (3, 16384)])
def test_layernorm_stays_inside_its_buffers(q32, T, C):
    """codes and metadata between guard bands: odd token counts leave the second token of the last step empty"""
    from test_gpu_guard_bands import Guarded
    bits, gain, bias = _inputs(T, C, seed=T)
    codes, meta = Guarded(T * C // 2), Guarded(T * (C // 32) * 2)
    fb4.fb4_quantize_layernorm(q32.ctx, to_dev_bf16(bits), T, C, C, to_dev_bf16(gain), to_dev_bf16(bias), 1, 1e-6, None, None,
                               0, codes.tensor(torch.uint8, (T, C // 2)), meta.tensor(torch.int16, (T, C // 32)))
    torch.cuda.synchronize()
    codes.check("codes, layernorm producer")
    meta.check("meta, layernorm producer")
    ref = orc.quantize_f32(orc.layernorm_f32(bits, gain, bias, True, 1e-6), FB)
    assert np.array_equal(codes.tensor(torch.uint8, (T, C // 2)).cpu().numpy(), ref.codes)
