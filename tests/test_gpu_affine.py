"""GPU parity of fb4_quantize_affine (per-channel affine producer fused in front of the quantizer, App. D.2)
against the oracle: the affine step in float32 with one rounding, then the float32 quantizer; bit-exact codes,
dialect ids and scale bytes in the TMA-staged kernel and in the generic kernel."""
import ctypes

import numpy as np
import pytest
import torch

from gpu_util import FB, assert_same_quantized, to_dev_bf16
from oracle import fb4_oracle as orc
from paper_2603_02883_b200 import fb4, synth

pytestmark = pytest.mark.gpu


def factors(C, seed, kind):
    rng = np.random.default_rng(seed)
    if kind == "layernorm":          # gamma around 1, beta small
        gain = 1.0 + 0.2 * rng.standard_normal(C)
        bias = 0.1 * rng.standard_normal(C)
    elif kind == "modulation":       # scale and shift of an adaLN block
        gain = 0.5 * rng.standard_normal(C)
        bias = rng.standard_normal(C)
    else:                            # wild: huge and tiny gains, zero and negative-zero entries
        gain = rng.standard_normal(C) * np.exp2(rng.integers(-40, 20, size=C).astype(np.float64))
        bias = rng.standard_normal(C) * np.exp2(rng.integers(-40, 20, size=C).astype(np.float64))
        gain[::7] = 0.0
        bias[::5] = 0.0
        bias[3::11] = -0.0
    return synth.f32_to_bf16_bits(gain.astype(np.float32)), synth.f32_to_bf16_bits(bias.astype(np.float32))


def run_case(q, cfg, T, C, ld, kind, plus_one, expect_variant=None, seda=False):
    w = synth.Workload("a", T=T, C=ld, seed=T + C, kind=1, n_outlier=max(1, C // 300), outlier_gain=50.0)
    bits = synth.activation(w)
    view = bits[:, :C]
    gain, bias = factors(C, C + T, kind)
    cid = masks = d_cid = d_masks = None
    if seda:
        rng = np.random.default_rng(T * 7 + C)
        n_cl = 5
        cid = rng.integers(-1, n_cl, size=T).astype(np.int32)
        masks = rng.integers(1, 2 ** 32, size=n_cl, dtype=np.uint64).astype(np.uint32)
        masks[1] = synth.clusters(synth.Workload("m", T=max(T, 8), C=C, seed=1, kind=1, n_outlier=0, outlier_gain=1.0, seda=True,
                                                 n_clusters=2, cluster_seed=T))[1][0]      # one dialect per range
        d_cid, d_masks = torch.from_numpy(cid).cuda(), torch.from_numpy(masks.view(np.int32)).cuda()
    ref = orc.quantize_f32(orc.affine_f32(view, gain, bias, plus_one), FB, cfg, cluster_id=cid, cluster_mask=masks)
    x = to_dev_bf16(bits)[:, :C]
    got = q.quantize_affine(x, torch.from_numpy(gain.view(np.int16)).cuda().view(torch.bfloat16),
                            torch.from_numpy(bias.view(np.int16)).cuda().view(torch.bfloat16), plus_one, d_cid, d_masks)
    what = f"T={T} C={C} ld={ld} {kind} plus_one={plus_one} seda={seda} kernel={q.last_variant}"
    if expect_variant:
        assert q.last_variant == expect_variant, what
    assert_same_quantized(got, ref, what)


@pytest.mark.parametrize("T,C,ld", [(1, 64, 64), (130, 3072, 3072), (300, 1024 + 64, 1024 + 64 + 8), (257, 12288 + 64, 12288 + 64),
                                    (5000, 64, 64), (2368 + 5, 2048, 2048), (37, 40 * 1024, 40 * 1024),
                                    (1600, 3072, 3072), (401, 12288, 12288)])   # the last three shapes: flat tiles
@pytest.mark.parametrize("kind,plus_one", [("layernorm", False), ("modulation", True), ("wild", False), ("wild", True)])
def test_tma_staged_kernel(T, C, ld, kind, plus_one):
    q = fb4.Fb4()
    try:
        run_case(q, orc.Config(), T, C, ld, kind, plus_one, "fast")
        run_case(q, orc.Config(), T, C, ld, kind, plus_one, "fast", seda=True)
        assert q.device_status == 0
    finally:
        q.close()


@pytest.mark.parametrize("cfg,T,C", [(dict(), 50, 96), (dict(block_size=16), 33, 48), (dict(block_size=16), 64, 1024),
                                     (dict(select_mode=1), 40, 256), (dict(num_groups=32), 40, 256),
                                     (dict(exp_min=-15, exp_max=16), 40, 1024)])
@pytest.mark.parametrize("plus_one", [False, True])
def test_other_configurations_run_in_the_generic_kernel(cfg, T, C, plus_one):
    q = fb4.Fb4(**cfg)
    try:
        run_case(q, orc.Config(**cfg), T, C, C, "wild" if plus_one else "modulation", plus_one, "generic")
        run_case(q, orc.Config(**cfg), T, C, C, "modulation", plus_one, "generic", seda=True)
        assert q.device_status == 0
    finally:
        q.close()


def test_both_kernels_agree_and_identity_equals_the_plain_quantizer():
    q = fb4.Fb4()
    try:
        run_case(q, orc.Config(), 200, 2048, 2048, "modulation", True, "fast")
        q.set_kernel_variant(1)
        run_case(q, orc.Config(), 200, 2048, 2048, "modulation", True, "generic")
        q.set_kernel_variant(0)
        # gain 1, bias -0: y = x bit for bit, so the result is the plain quantizer's
        w = synth.Workload("a", T=300, C=3072, seed=5, kind=1, n_outlier=9, outlier_gain=50.0)
        x = to_dev_bf16(synth.activation(w))
        one = torch.ones(3072, dtype=torch.bfloat16, device="cuda")
        nzero = torch.full((3072,), -0.0, dtype=torch.bfloat16, device="cuda")
        a, b = q.quantize_affine(x, one, nzero), q.quantize(x)
        assert torch.equal(a.codes, b.codes) and torch.equal(a.meta, b.meta)
        a = q.quantize_affine(x, torch.zeros_like(one), nzero, True)
        assert torch.equal(a.codes, b.codes) and torch.equal(a.meta, b.meta)
    finally:
        q.close()


def test_argument_checks():
    q = fb4.Fb4()
    L = fb4.lib()
    x = torch.zeros((4, 64), dtype=torch.bfloat16, device="cuda")
    v = torch.zeros(64, dtype=torch.bfloat16, device="cuda")
    out = torch.zeros(4096, dtype=torch.uint8, device="cuda")
    p = lambda t: ctypes.c_void_p(t.data_ptr())
    f = L.fb4_quantize_affine
    assert f(q.ctx, p(x), 4, 64, 64, p(v), p(v), 0, None, None, 0, p(out), p(out), None) == fb4.OK
    assert f(q.ctx, p(x), 4, 64, 64, None, p(v), 0, None, None, 0, p(out), p(out), None) == fb4.ERR_INVALID_ARG
    assert f(q.ctx, p(x), 4, 64, 64, p(v), p(v), 2, None, None, 0, p(out), p(out), None) == fb4.ERR_INVALID_ARG
    assert f(q.ctx, p(x), 4, 48, 64, p(v), p(v), 0, None, None, 0, p(out), p(out), None) == fb4.ERR_SHAPE
    assert f(q.ctx, p(x), 4, 64, 60, p(v), p(v), 0, None, None, 0, p(out), p(out), None) == fb4.ERR_SHAPE
    assert f(q.ctx, p(x), 4, 64, 64, ctypes.c_void_p(v.data_ptr() + 1), p(v), 0, None, None, 0, p(out), p(out), None) == fb4.ERR_ALIGN
    assert f(q.ctx, None, 0, 64, 64, None, None, 0, None, None, 0, None, None, None) == fb4.OK
    # gain / bias not 16-byte aligned: the generic kernel takes the call
    v2 = torch.zeros(72, dtype=torch.bfloat16, device="cuda")[1:65]
    assert f(q.ctx, p(x), 4, 64, 64, p(v2), p(v2), 0, None, None, 0, p(out), p(out), None) == fb4.OK
    assert q.last_variant == "generic"
    assert q.device_status == 0
    q.close()


@pytest.mark.parametrize("T,C", [(1, 64), (130, 3072), (300, 1024 + 64), (257, 128), (2368 + 5, 2048), (1600, 3072)])
@pytest.mark.parametrize("plus_one", [False, True])
def test_affine_producer_straight_to_mxfp8(T, C, plus_one):
    """fb4_quantize_affine_mxfp8 = affine producer (oracle, fp32) -> fp32 quantizer (oracle) -> MXFP8 view (oracle),
    byte for byte, both scale layouts, with and without SeDA."""
    w = synth.Workload("a", T=T, C=C, seed=T + C, kind=1, n_outlier=max(1, C // 300), outlier_gain=50.0, seda=True,
                       n_clusters=min(4, T), cluster_seed=3)
    bits = synth.activation(w)
    cid, masks = synth.clusters(w)
    gain, bias = factors(C, T, "modulation" if plus_one else "layernorm")
    dev = lambda a: torch.from_numpy(a.view(np.int16)).cuda().view(torch.bfloat16)
    y = orc.affine_f32(bits, gain, bias, plus_one)
    q = fb4.Fb4()
    try:
        for seda in (False, True):
            ref = orc.quantize_f32(y, FB, cluster_id=cid if seda else None, cluster_mask=masks if seda else None)
            for layout in (0, 1):
                e_ref, s_ref = orc.to_mxfp8(ref, FB, layout)
                e4m3, scales = q.quantize_affine_mxfp8(
                    to_dev_bf16(bits), dev(gain), dev(bias), plus_one, layout,
                    torch.from_numpy(cid).cuda() if seda else None,
                    torch.from_numpy(masks.view(np.int32)).cuda() if seda else None)
                what = f"seda {seda} layout {layout}"
                assert np.array_equal(e4m3.cpu().numpy(), e_ref), what
                assert np.array_equal(scales.cpu().numpy(), s_ref), what
        assert q.device_status == 0
        # other configurations are refused, not approximated
        L = fb4.lib()
        x = to_dev_bf16(bits)
        g, b = dev(gain), dev(bias)
        p = lambda t: ctypes.c_void_p(t.data_ptr())
        out = torch.zeros(T * C + 4096, dtype=torch.uint8, device="cuda")
        q16 = fb4.Fb4(block_size=16)
        assert L.fb4_quantize_affine_mxfp8(q16.ctx, p(x), T, C, C, p(g), p(b), 0, None, None, 0, p(out), p(out), 0,
                                           None) == fb4.ERR_INVALID_ARG
        q16.close()
        assert L.fb4_quantize_affine_mxfp8(q.ctx, p(x), T, C, C, p(g), p(b), 0, None, None, 0, p(out), p(out), 2,
                                           None) == fb4.ERR_INVALID_ARG
        assert L.fb4_quantize_affine_mxfp8(q.ctx, p(x), T, C, C, p(g), None, 0, None, None, 0, p(out), p(out), 0,
                                           None) == fb4.ERR_INVALID_ARG
        assert L.fb4_quantize_affine_mxfp8(q.ctx, p(x), T, 32, C, p(g), p(b), 0, None, None, 0, p(out), p(out), 0,
                                           None) == fb4.ERR_SHAPE
    finally:
        q.close()
