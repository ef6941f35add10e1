"""Infinities and NaNs in the input.  The library asks for finite input; what it promises for other input is that
nothing is read or written out of bounds: every kernel saturates the magnitudes of a block that holds such a value
before it forms a table address.  Checked here on every kernel family: the call succeeds, the device status stays
clean, every block WITHOUT such a value equals the oracle bit for bit (the oracle gets the same tensor with the
offending values set to zero; blocks are independent), and the blocks WITH one carry a dialect, an exponent and
codes that decode to finite numbers."""
import numpy as np
import pytest
import torch

from gpu_util import FB, meta_np, to_dev_bf16
from oracle import fb4_oracle as orc
from paper_2603_02883_b200 import fb4, synth

pytestmark = pytest.mark.gpu

BAD = np.array([0x7F80, 0xFF80, 0x7FC0, 0xFFFF, 0x7F81, 0xFFC1], dtype=np.uint16)   # +inf, -inf, NaNs


def tensor_with_bad_values(T, C, seed, every=97):
    w = synth.Workload("n", T=T, C=C, seed=seed, kind=1, n_outlier=max(1, C // 200), outlier_gain=50.0)
    bits = synth.activation(w).copy()
    flat = bits.reshape(-1)
    pos = np.arange(seed % every, flat.size, every * 32 + 5)       # a bad value in about one block of `every`
    flat[pos] = BAD[np.arange(pos.size) % BAD.size]
    flat[-1] = 0x7F80                                               # and in the very last element
    bad = np.zeros(flat.size, dtype=bool)
    bad[pos] = True
    bad[-1] = True
    clean = bits.copy()
    clean.reshape(-1)[bad] = 0
    return bits, clean, bad.reshape(T, C)


def check(got_codes, got_meta, ref, bad_blocks, block, what):
    """ref: the oracle's result on the cleaned tensor; bad_blocks: [T][C/block] bool"""
    meta = got_meta.reshape(bad_blocks.shape)
    ok = ~bad_blocks
    assert np.array_equal(meta[ok], ref.meta.reshape(bad_blocks.shape)[ok]), f"{what}: metadata of clean blocks"
    cb = block // 2
    codes = got_codes.reshape(bad_blocks.shape + (cb,))
    assert np.array_equal(codes[ok], ref.codes.reshape(bad_blocks.shape + (cb,))[ok]), f"{what}: codes of clean blocks"
    assert np.all((meta[bad_blocks] >> 8) < 32), f"{what}: dialect ids of the other blocks"


@pytest.mark.parametrize("T,C,ld", [(700, 1024, 1024), (333, 3072, 3072 + 64), (64, 12288, 12288)])
@pytest.mark.parametrize("block", [32, 16])
def test_quantize_variants_stay_in_bounds(T, C, ld, block):
    full, clean, bad = tensor_with_bad_values(T, ld, seed=T + C + block)
    clean, bad = clean[:, :C], bad[:, :C]
    bad_blocks = bad.reshape(T, C // block, block).any(axis=2)
    assert bad_blocks.any() and not bad_blocks.all()
    cfg = orc.Config(block_size=block)
    q = fb4.Fb4(block_size=block)
    try:
        x = to_dev_bf16(full)[:, :C]
        # plain
        got = q.quantize(x)
        assert q.last_variant == "fast"
        check(got.codes.cpu().numpy(), meta_np(got.meta), orc.quantize(clean, FB, cfg), bad_blocks, block, "plain")
        dec = q.dequantize(got, torch.float32)
        assert bool(torch.isfinite(dec).all()), "decoded output of saturated blocks"
        # SeDA masks
        rng = np.random.default_rng(T)
        cid = rng.integers(-1, 4, size=T).astype(np.int32)
        masks = rng.integers(1, 2 ** 32, size=4, dtype=np.uint64).astype(np.uint32)
        got = q.quantize(x, torch.from_numpy(cid).cuda(), torch.from_numpy(masks.view(np.int32)).cuda())
        ref = orc.quantize(clean, FB, cfg, cluster_id=cid, cluster_mask=masks)
        check(got.codes.cpu().numpy(), meta_np(got.meta), ref, bad_blocks, block, "seda")
        # residual pass of salient tokens (the residual of a saturated block is infinite or NaN itself)
        sal = np.arange(0, T, 7, dtype=np.int32)
        got = q.quantize_decomposed(x, salient_idx=torch.from_numpy(sal).cuda())
        ref = orc.quantize(clean, FB, cfg, salient_idx=sal)
        check(got.codes.cpu().numpy(), meta_np(got.meta), ref, bad_blocks, block, "decomposed, main")
        check(got.res_codes.cpu().numpy(), meta_np(got.res_meta), orc.Quantized(ref.res_codes, ref.res_meta),
              bad_blocks[sal], block, "decomposed, residual")
        q.dequantize(got, torch.bfloat16)     # the sum of two saturated values may overflow: run, not compared
        if block == 32:
            e4m3, scales = q.quantize_mxfp8(x, 0)
            assert e4m3.shape[0] == T and scales.numel() >= T * C // 32
        assert q.device_status == 0
        torch.cuda.synchronize()
    finally:
        q.close()


def test_fp32_input_and_producers_stay_in_bounds():
    T, C = 500, 2048
    bits, clean, bad = tensor_with_bad_values(T, C, seed=11)
    bad_blocks = bad.reshape(T, C // 32, 32).any(axis=2)
    q = fb4.Fb4()
    try:
        # fp32 input: infinities and NaNs as float32
        xf = synth.bf16_bits_to_f32(bits)
        got = q.quantize(torch.from_numpy(xf).cuda())
        assert q.last_variant == "fast"
        ref = orc.quantize_f32(synth.bf16_bits_to_f32(clean), FB)
        check(got.codes.cpu().numpy(), meta_np(got.meta), ref, bad_blocks, 32, "fp32 input")
        # affine producer: finite input, a gain that overflows float32 in some channels -> y = +-inf there
        rng = np.random.default_rng(5)
        gain = rng.standard_normal(C).astype(np.float32)
        bias = rng.standard_normal(C).astype(np.float32)
        gain[40::257] = 3.0e38
        gb, bb = synth.f32_to_bf16_bits(gain), synth.f32_to_bf16_bits(bias)
        dev = lambda a: torch.from_numpy(a.view(np.int16)).cuda().view(torch.bfloat16)
        y = orc.affine_f32(clean, gb, bb, False)
        y_bad = ~np.isfinite(y)
        assert y_bad.any()
        y_clean = np.where(y_bad, np.float32(0), y)
        got = q.quantize_affine(to_dev_bf16(clean), dev(gb), dev(bb), False)
        assert q.last_variant == "fast"
        check(got.codes.cpu().numpy(), meta_np(got.meta), orc.quantize_f32(y_clean, FB),
              y_bad.reshape(T, C // 32, 32).any(axis=2), 32, "affine producer")
        # LayerNorm producer: a bad value poisons the statistics of its whole token
        got = q.quantize_layernorm(to_dev_bf16(bits), dev(gb), dev(bb), True, 1e-6)
        bad_tokens = bad.any(axis=1)
        yl = orc.layernorm_f32(clean, gb, bb, True, 1e-6)
        yl_bad = ~np.isfinite(yl)
        ref = orc.quantize_f32(np.where(yl_bad, np.float32(0), yl), FB)
        blocks_bad = yl_bad.reshape(T, C // 32, 32).any(axis=2) | bad_tokens[:, None]
        check(got.codes.cpu().numpy(), meta_np(got.meta), ref, blocks_bad, 32, "LayerNorm producer")
        assert q.device_status == 0
        torch.cuda.synchronize()
    finally:
        q.close()


@pytest.mark.parametrize("kw", [dict(num_groups=32), dict(select_mode=1)])
def test_selection_variants_stay_in_bounds(kw):
    T, C = 300, 2048
    bits, clean, bad = tensor_with_bad_values(T, C, seed=23)
    bad_blocks = bad.reshape(T, C // 32, 32).any(axis=2)
    q = fb4.Fb4(**kw)
    try:
        got = q.quantize(to_dev_bf16(bits))
        assert q.last_variant == "fast"
        check(got.codes.cpu().numpy(), meta_np(got.meta), orc.quantize(clean, FB, orc.Config(**kw)), bad_blocks, 32, str(kw))
        assert q.device_status == 0
        torch.cuda.synchronize()
    finally:
        q.close()
