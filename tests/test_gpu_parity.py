"""GPU parity: the CUDA library (through its C-ABI binding) against the CPU oracle, bit for bit,
on the same seeded inputs.  Sizes span several tiles and ragged tails; the five workloads run at
full size (the largest on sampled rows).  Run with -m gpu on a B200."""
import numpy as np
import pytest
import torch

from gpu_util import FB, assert_same_bits_f32, assert_same_quantized, meta_np, to_dev_bf16
from oracle import fb4_oracle as orc
from paper_2603_02883_b200 import fb4, synth

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", params=["auto", "generic"])
def q32(request):
    """Default-configuration context; 'auto' takes the TMA-staged kernel whenever the call
    qualifies, 'generic' forces the fallback kernel, so both are checked on every case."""
    q = fb4.Fb4()
    q.set_kernel_variant(1 if request.param == "generic" else 0)
    yield q
    assert q.device_status == 0
    q.close()


def test_kernel_choice():
    q = fb4.Fb4()
    x = torch.zeros((8, 1024), dtype=torch.bfloat16, device="cuda")
    q.quantize(x)
    assert q.last_variant == "fast"
    q.quantize(x[:, :96])            # 96 channels: not a multiple of 64
    assert q.last_variant == "generic"
    q.set_kernel_variant(1)
    q.quantize(x)
    assert q.last_variant == "generic"
    assert q.device_status == 0
    q.close()


def heavy(T, C, seed, kind=1):
    w = synth.Workload("t", T=T, C=C, seed=seed, kind=kind, n_outlier=max(1, C // 200), outlier_gain=50.0)
    return synth.activation(w)


def edge_blocks():
    """Hand-made blocks: zeros, -0, subnormals, extreme exponents, exact rounding ties, dialect ties."""
    f = np.zeros((40, 64), dtype=np.float32)
    f[1, :] = -0.0
    f[2, 5] = 1e-40
    f[2, 6] = -3e-39                       # bf16 subnormals
    f[3, :32] = 2.0 ** -126
    f[3, 32:] = 2.0 ** -130
    f[4, 0] = 3.0e38
    f[4, 1:8] = 1.5e38                     # top of the bf16 range
    f[5, :] = 2.0 ** 127
    f[6, :32] = np.arange(32) / 2.0        # every half-integer: exact ties at v = k/2 (max 15.5 -> e = 3)
    f[6, 32:] = -np.arange(32) / 4.0
    f[7, :] = 1.0                          # all equal: every element is the block maximum
    f[8, ::4] = [8, 9, 10, 11, 12, 13, 14, 15, 8.5, 9.5, 10.5, 11.5, 12.5, 13.5, 14.5, 15.5]
    f[9, 0], f[9, 33] = 12.0, -12.0
    f[9, 1:32] = 0.25
    rng = np.random.default_rng(11)
    f[10:] = rng.standard_normal((30, 64)).astype(np.float32) * (2.0 ** rng.integers(-140, 120, size=(30, 1)))
    bits = synth.f32_to_bf16_bits(f)
    bits[11, :] = 0x0001                   # smallest subnormal everywhere
    bits[12, 3] = 0x7F7F                   # largest finite bf16
    bits[12, 4] = 0xFF7F
    return bits


CONFIGS = [dict(block_size=32, num_groups=8), dict(block_size=16, num_groups=8),
           dict(block_size=32, num_groups=32), dict(block_size=16, num_groups=16),
           dict(block_size=32, num_groups=8, select_mode=1),
           dict(block_size=32, num_groups=8, exp_min=-15, exp_max=16),
           dict(block_size=16, num_groups=8, exp_min=-8, exp_max=3, select_mode=1)]


@pytest.mark.parametrize("cfg", CONFIGS, ids=lambda c: "-".join(f"{k[:3]}{v}" for k, v in c.items()))
def test_edge_blocks_and_random_small(cfg):
    q = fb4.Fb4(**cfg)
    ocfg = orc.Config(**cfg)
    for bits in (edge_blocks(), heavy(37, 96, 5), heavy(3, 2048 + 64, 6), heavy(130, 1024, 7, kind=0)):
        ref = orc.quantize(bits, FB, ocfg)
        got = q.quantize(to_dev_bf16(bits))
        assert_same_quantized(got, ref, f"{cfg}")
        out = q.dequantize(got)
        assert_same_bits_f32(out, orc.dequantize(ref, FB, cfg["block_size"]), f"{cfg} dequant")
        outb = q.dequantize(got, torch.bfloat16)
        refb = orc.dequantize(ref, FB, cfg["block_size"], out_dtype="bf16")
        assert np.array_equal(outb.view(torch.int16).cpu().numpy().view(np.uint16), refb)
        outh = q.dequantize(got, torch.float16)                      # IEEE half: overflow to inf, gradual underflow
        refh = orc.dequantize(ref, FB, cfg["block_size"], out_dtype="f16")
        assert np.array_equal(outh.view(torch.int16).cpu().numpy().view(np.uint16), refh)
    q.close()


def test_tables_match_direct_rounding(q32):
    """Qvalue/Qerror built at init against exhaustive direct rounding over every bf16 v in [0,16)."""
    fbk, s1, qv, qe = fb4.fb4_get_tables(q32.ctx)
    assert np.array_equal(fbk, FB)
    assert np.array_equal(s1, orc.default_stage1(FB))
    pats = np.arange(0, 0x4180, dtype=np.uint16)                 # 0 .. 16.0 (exclusive)
    v = synth.bf16_bits_to_f32(pats).astype(np.float64)
    assert v.max() < 16
    bins = np.floor(2 * v).astype(int)
    for d in range(32):
        mags = FB[d].astype(np.float64)
        dist = np.abs(v[:, None] - mags[None, :])
        near = 7 - np.argmin(dist[:, ::-1], axis=1)             # ties -> larger magnitude
        assert np.array_equal(qv[d][bins], near)
        mid = np.arange(32) / 2 + 0.25
        assert np.array_equal(qe[d], (4 * np.min(np.abs(mid[:, None] - mags[None, :]), axis=1)).astype(int))


def test_strided_rows(q32):
    bits = heavy(50, 256 + 64, 8)
    x = to_dev_bf16(bits)
    view = x[:, :256]                                            # ld = 320
    ref = orc.quantize(bits[:, :256], FB)
    assert_same_quantized(q32.quantize(view), ref, "strided")


def test_seda_masks(q32):
    bits = heavy(64, 512, 9)
    rng = np.random.default_rng(3)
    w = synth.Workload("t", T=64, C=512, seed=9, kind=1, n_outlier=0, outlier_gain=1.0, seda=True, n_clusters=6,
                       cluster_seed=12)
    cid, masks = synth.clusters(w)
    masks = masks.copy()
    masks[1] = rng.integers(1, 2 ** 32)          # arbitrary masks: partial / empty stage-1 intersections
    masks[2] = 1 << 31
    masks[3] = 0x00000003                        # only the narrowest dynamic range
    cid = cid.copy()
    cid[5:9] = -1                                # unconstrained tokens
    ref = orc.quantize(bits, FB, cluster_id=cid, cluster_mask=masks)
    got = q32.quantize(to_dev_bf16(bits), torch.from_numpy(cid).cuda(),
                       torch.from_numpy(masks.view(np.int32)).cuda())
    assert_same_quantized(got, ref, "seda")
    did = meta_np(got.meta) >> 8
    for t in range(64):
        if cid[t] >= 0:
            assert np.all((int(masks[cid[t]]) >> did[t].astype(np.int64)) & 1)


@pytest.mark.parametrize("T,tile", [(40, 20), (47, 20), (7, 20), (64, 1), (100, 7)])
def test_decomposed_small(q32, T, tile):
    bits = heavy(T, 256, 10 + T)
    w = synth.Workload("t", T=T, C=256, seed=1, kind=1, n_outlier=0, outlier_gain=1.0, score_seed=T)
    score = synth.scores(w)
    score[T // 2:T // 2 + 3] = score[T // 2]                    # ties inside a tile
    sal = orc.select_salient(score, tile)
    ref = orc.quantize(bits, FB, salient_idx=sal)
    got = q32.quantize_decomposed(to_dev_bf16(bits), torch.from_numpy(score).cuda(), tile)
    assert_same_quantized(got, ref, "decomposed")
    assert np.array_equal(q32.select_salient(torch.from_numpy(score).cuda(), tile).cpu().numpy(), sal)
    assert_same_bits_f32(q32.dequantize(got), orc.dequantize(ref, FB), "decomposed dequant")
    for dt, name in ((torch.bfloat16, "bf16"), (torch.float16, "f16")):
        o = q32.dequantize(got, dt)
        assert np.array_equal(o.view(torch.int16).cpu().numpy().view(np.uint16), orc.dequantize(ref, FB, out_dtype=name))
    # caller-given salient set (reused from an earlier step): arbitrary ascending list
    mine = np.unique(np.random.default_rng(T).integers(0, T, size=max(1, T // 3))).astype(np.int32)
    ref2 = orc.quantize(bits, FB, salient_idx=mine)
    got2 = q32.quantize_decomposed(to_dev_bf16(bits), salient_idx=torch.from_numpy(mine).cuda())
    assert_same_quantized(got2, ref2, "decomposed idx")
    assert_same_bits_f32(q32.dequantize(got2), orc.dequantize(ref2, FB), "decomposed idx dequant")


@pytest.mark.parametrize("T,C,tile", [(300, 8192, 1), (257, 8192 + 32, 3), (500, 12288, 20), (130, 16384 + 64, 2)])
def test_decode_adds_residual_rows_in_the_same_pass(q32, T, C, tile):
    """At 256 or more blocks per row the decode adds the residual of salient rows inside its one kernel
    (steps with several salient rows, runs of consecutive salient rows, ragged last step); every output
    type against the oracle, and one launch per call."""
    bits = heavy(T, C, T + C)
    w = synth.Workload("t", T=T, C=C, seed=1, kind=1, n_outlier=0, outlier_gain=1.0, score_seed=T + tile)
    score = synth.scores(w)
    lists = [orc.select_salient(score, tile),
             np.array(sorted(set(range(5, 12)) | {0, T // 2, T - 2, T - 1}), dtype=np.int32),
             np.array([T - 1], dtype=np.int32)]
    x = to_dev_bf16(bits)
    for sal in lists:
        ref = orc.quantize(bits, FB, salient_idx=sal)
        got = q32.quantize_decomposed(x, salient_idx=torch.from_numpy(sal).cuda())
        assert_same_quantized(got, ref, "given set")
        before = q32.launch_count
        assert_same_bits_f32(q32.dequantize(got), orc.dequantize(ref, FB), "fp32 decode with residual rows")
        assert q32.launch_count == before + 1          # fp32 output: residual rows inside the one kernel
        for dt, name in ((torch.bfloat16, "bf16"), (torch.float16, "f16")):
            o = q32.dequantize(got, dt)
            assert np.array_equal(o.view(torch.int16).cpu().numpy().view(np.uint16),
                                  orc.dequantize(ref, FB, out_dtype=name)), name


def test_decomposed_with_seda_and_b16():
    q = fb4.Fb4(block_size=16)
    bits = heavy(60, 128, 21)
    w = synth.Workload("t", T=60, C=128, seed=1, kind=1, n_outlier=0, outlier_gain=1.0, score_seed=3, seda=True,
                       n_clusters=5, cluster_seed=4)
    score = synth.scores(w)
    cid, masks = synth.clusters(w)
    sal = orc.select_salient(score, 20)
    ref = orc.quantize(bits, FB, orc.Config(block_size=16), cluster_id=cid, cluster_mask=masks, salient_idx=sal)
    got = q.quantize_decomposed(to_dev_bf16(bits), torch.from_numpy(score).cuda(), 20,
                                cluster_id=torch.from_numpy(cid).cuda(),
                                cluster_mask=torch.from_numpy(masks.view(np.int32)).cuda())
    assert_same_quantized(got, ref, "decomposed+seda b16")
    assert_same_bits_f32(q.dequantize(got), orc.dequantize(ref, FB, 16), "b16 dequant")
    q.close()


def test_argument_checks(q32):
    x = torch.zeros((4, 64), dtype=torch.bfloat16, device="cuda")
    codes = torch.empty((4, 32), dtype=torch.uint8, device="cuda")
    meta = torch.empty((4, 2), dtype=torch.int16, device="cuda")
    L = fb4.lib()
    import ctypes
    p = lambda t, off=0: ctypes.c_void_p(t.data_ptr() + off)
    assert L.fb4_quantize(q32.ctx, p(x), 4, 48, 64, p(codes), p(meta), None) == fb4.ERR_SHAPE       # C % B
    assert L.fb4_quantize(q32.ctx, p(x), 4, 64, 32, p(codes), p(meta), None) == fb4.ERR_SHAPE       # ld < C
    assert L.fb4_quantize(q32.ctx, p(x), -1, 64, 64, p(codes), p(meta), None) == fb4.ERR_SHAPE
    assert L.fb4_quantize(q32.ctx, p(x, 2), 3, 64, 64, p(codes), p(meta), None) == fb4.ERR_ALIGN
    assert L.fb4_quantize(q32.ctx, p(x), 4, 32, 36, p(codes), p(meta), None) == fb4.ERR_ALIGN       # ld % 8
    assert L.fb4_quantize(q32.ctx, p(x), 4, 64, 64, None, p(meta), None) == fb4.ERR_INVALID_ARG
    assert L.fb4_quantize(q32.ctx, None, 0, 64, 64, None, None, None) == fb4.OK                      # empty
    assert L.fb4_quantize_seda(q32.ctx, p(x), 4, 64, 64, None, None, 0, p(codes), p(meta), None) == fb4.ERR_INVALID_ARG
    assert L.fb4_dequantize(q32.ctx, p(codes), p(meta), 4, 64, None, 0, None, None, p(x), 7, None) == fb4.ERR_INVALID_ARG
    assert L.fb4_select_salient(q32.ctx, p(x), 4, 0, p(meta), None) == fb4.ERR_INVALID_ARG
    torch.cuda.synchronize()


def test_host_buffer_entry_point(q32):
    w = synth.workloads()["c1"]
    bits = synth.activation(w)
    ref = orc.quantize(bits, FB)
    xh = torch.from_numpy(bits.view(np.int16)).pin_memory()
    ch = torch.empty((w.T, w.C // 2), dtype=torch.uint8).pin_memory()
    mh = torch.empty((w.T, w.C // 32), dtype=torch.int16).pin_memory()
    dx = torch.empty((w.T, w.C), dtype=torch.int16, device="cuda")
    dc = torch.empty((w.T, w.C // 2), dtype=torch.uint8, device="cuda")
    dm = torch.empty((w.T, w.C // 32), dtype=torch.int16, device="cuda")
    fb4.fb4_quantize_host(q32.ctx, xh, w.T, w.C, dx, dc, dm, ch, mh)
    assert np.array_equal(ch.numpy(), ref.codes) and np.array_equal(mh.numpy().view(np.uint16), ref.meta)


def f32_inputs():
    rng = np.random.default_rng(23)
    yield "edge", synth.bf16_bits_to_f32(edge_blocks())           # bf16-valued fp32, all the edge cases
    x = (rng.standard_normal((67, 1024 + 96)) * np.exp2(rng.integers(-40, 40, size=(67, 1)))).astype(np.float32)
    x[3, 40:80] = 0.0
    x[5, :] = np.float32(1e-41)                                    # fp32 subnormals
    x[6, 7] = np.float32(3.4e38)
    x[7, :64] = np.nextafter(np.float32(2.5), np.float32(0), dtype=np.float32)   # just below a rounding boundary
    x[7, 0] = 8.0
    yield "random", x
    yield "student-t", synth.bf16_bits_to_f32(heavy(130, 2048, 31)) * np.float32(1.0009765625)   # not bf16 values


@pytest.mark.parametrize("cfg", [dict(), dict(block_size=16), dict(select_mode=1), dict(exp_min=-15, exp_max=16)],
                         ids=["default", "b16", "select-all", "exp5"])
def test_f32_input(cfg):
    q = fb4.Fb4(**cfg)
    ocfg = orc.Config(**cfg)
    for name, x in f32_inputs():
        ref = orc.quantize_f32(x, FB, ocfg)
        xd = torch.from_numpy(x).cuda()
        for variant in (0, 1):
            q.set_kernel_variant(variant)
            got = q.quantize(xd)
            assert_same_quantized(got, ref, f"f32 {name} {cfg} variant {variant}")
        if not cfg:
            q.set_kernel_variant(0)
            q.quantize(xd)
            assert q.last_variant == "fast"
            # strided rows
            view = xd[:, :64]
            assert_same_quantized(q.quantize(view), orc.quantize_f32(np.ascontiguousarray(x[:, :64]), FB), "f32 strided")
    assert q.device_status == 0
    q.close()


def test_block16_fast_kernel_plain_and_seda():
    """Block size 16 in the TMA-staged kernel (two blocks per lane), plain, SeDA and with a residual
    pass, against the oracle and the generic kernel."""
    q = fb4.Fb4(block_size=16)
    ocfg = orc.Config(block_size=16)
    w = synth.Workload("t", T=300, C=3072, seed=51, kind=1, n_outlier=15, outlier_gain=50.0, seda=True, n_clusters=9,
                       cluster_seed=52, score_seed=53)
    bits = synth.activation(w)
    cid, masks = synth.clusters(w)
    masks = masks.copy()
    masks[2] = 0x0000F0F3                      # cuts stage-1 groups
    masks[5] = 1 << 30
    cid = cid.copy()
    cid[10:20] = -1
    x = to_dev_bf16(bits)
    dcid, dmask = torch.from_numpy(cid).cuda(), torch.from_numpy(masks.view(np.int32)).cuda()
    ref_plain = orc.quantize(bits, FB, ocfg)
    ref_seda = orc.quantize(bits, FB, ocfg, cluster_id=cid, cluster_mask=masks)
    for variant, name in ((0, "fast"), (1, "generic")):
        q.set_kernel_variant(variant)
        assert_same_quantized(q.quantize(x), ref_plain, f"b16 plain {name}")
        assert q.last_variant == name
        assert_same_quantized(q.quantize(x, dcid, dmask), ref_seda, f"b16 seda {name}")
        assert q.last_variant == name
    sal = orc.select_salient(synth.scores(w), 20)
    ref_dec = orc.quantize(bits, FB, ocfg, salient_idx=sal)
    ref_dec_seda = orc.quantize(bits, FB, ocfg, cluster_id=cid, cluster_mask=masks, salient_idx=sal)
    for variant, name in ((0, "fast"), (1, "generic")):
        q.set_kernel_variant(variant)
        got = q.quantize_decomposed(x, torch.from_numpy(synth.scores(w)).cuda(), 20)
        assert q.last_variant == name
        assert_same_quantized(got, ref_dec, f"b16 decomposed {name}")
        got = q.quantize_decomposed(x, torch.from_numpy(synth.scores(w)).cuda(), 20, cluster_id=dcid, cluster_mask=dmask)
        assert_same_quantized(got, ref_dec_seda, f"b16 decomposed seda {name}")
        assert_same_bits_f32(q.dequantize(got), orc.dequantize(ref_dec_seda, FB, 16), "b16 decomposed dequant")
    q.set_kernel_variant(0)
    assert_same_bits_f32(q.dequantize(q.quantize(x)), orc.dequantize(ref_plain, FB, 16), "b16 dequant")
    assert q.device_status == 0
    q.close()


@pytest.mark.parametrize("cfg", [dict(exp_min=-15, exp_max=16), dict(block_size=16, exp_min=-15, exp_max=16),
                                 dict(exp_min=-3, exp_max=2), dict(block_size=16, exp_min=0, exp_max=0)],
                         ids=["exp5", "b16-exp5", "narrow", "b16-single-exponent"])
def test_clamped_exponent_fast_kernel(cfg):
    """The paper's 5-bit shared exponent (and narrower clamps, which saturate many elements) in the
    TMA-staged kernel, plain, SeDA and with a residual pass, against the oracle and the generic kernel."""
    q = fb4.Fb4(**cfg)
    ocfg = orc.Config(**cfg)
    w = synth.Workload("t", T=200, C=1024 + 128, seed=61, kind=1, n_outlier=6, outlier_gain=50.0, seda=True,
                       n_clusters=4, cluster_seed=62)
    cid, masks = synth.clusters(w)
    for bits in (synth.activation(w), np.tile(edge_blocks(), (5, 18))[:200]):
        x = to_dev_bf16(bits)
        ref = orc.quantize(bits, FB, ocfg)
        ref_seda = orc.quantize(bits, FB, ocfg, cluster_id=cid, cluster_mask=masks)
        sal = np.arange(3, 200, 7, dtype=np.int32)
        ref_dec = orc.quantize(bits, FB, ocfg, cluster_id=cid, cluster_mask=masks, salient_idx=sal)
        for variant, name in ((0, "fast"), (1, "generic")):
            q.set_kernel_variant(variant)
            got = q.quantize_decomposed(x, salient_idx=torch.from_numpy(sal).cuda(), cluster_id=torch.from_numpy(cid).cuda(),
                                        cluster_mask=torch.from_numpy(masks.view(np.int32)).cuda())
            assert q.last_variant == name
            assert_same_quantized(got, ref_dec, f"clamped decomposed {cfg} {name}")
            assert_same_bits_f32(q.dequantize(got), orc.dequantize(ref_dec, FB, cfg.get("block_size", 32)),
                                 "clamped decomposed dequant")
            got = q.quantize(x)
            assert q.last_variant == name
            assert_same_quantized(got, ref, f"clamped {cfg} {name}")
            got = q.quantize(x, torch.from_numpy(cid).cuda(), torch.from_numpy(masks.view(np.int32)).cuda())
            assert_same_quantized(got, ref_seda, f"clamped seda {cfg} {name}")
        assert_same_bits_f32(q.dequantize(got), orc.dequantize(ref_seda, FB, cfg.get("block_size", 32)), "clamped dequant")
    assert q.device_status == 0
    q.close()


def _random_formatbook(rng, tops):
    """32 dialects, strictly ascending from 0, largest magnitude as listed"""
    fb = np.zeros((32, 8), dtype=np.uint8)
    seen = set()
    for d, top in enumerate(tops):
        while True:
            inner = np.sort(rng.choice(np.arange(1, top), size=6, replace=False))
            row = (0, *inner.tolist(), top)
            if row not in seen:
                seen.add(row)
                fb[d] = row
                break
    return fb


def test_custom_formatbooks():
    """The formatbook is init-time data: another table whose dynamic-range groups fit the packed
    tables runs in the TMA-staged kernel, one with a group of 12 dialects falls back to the generic
    kernel; both match the oracle run with the same table (quantize, SeDA, residual, decode, MXFP8)."""
    rng = np.random.default_rng(99)
    fits = _random_formatbook(rng, [8] * 3 + [9] * 3 + [10] * 4 + [11] * 4 + [12] * 4 + [13] * 4 + [14] * 5 + [15] * 5)
    wide = _random_formatbook(rng, [8] * 2 + [9] * 2 + [10] * 2 + [11] * 2 + [12] * 4 + [13] * 4 + [14] * 4 + [15] * 12)
    w = synth.Workload("t", T=160, C=1024, seed=81, kind=1, n_outlier=5, outlier_gain=50.0, seda=True, n_clusters=5,
                       cluster_seed=82, score_seed=83)
    bits = synth.activation(w)
    x = to_dev_bf16(bits)
    score = synth.scores(w)
    sal = orc.select_salient(score, 20)
    for fbk, want in ((fits, "fast"), (wide, "generic")):
        cid, masks = synth.clusters(w, fbk)
        q = fb4.Fb4(formatbook=fbk)
        got = q.quantize(x)
        assert q.last_variant == want
        ref = orc.quantize(bits, fbk)
        assert_same_quantized(got, ref, f"custom formatbook plain ({want})")
        got = q.quantize_decomposed(x, torch.from_numpy(score).cuda(), 20, cluster_id=torch.from_numpy(cid).cuda(),
                                    cluster_mask=torch.from_numpy(masks.view(np.int32)).cuda())
        ref = orc.quantize(bits, fbk, cluster_id=cid, cluster_mask=masks, salient_idx=sal)
        assert_same_quantized(got, ref, f"custom formatbook decomposed+seda ({want})")
        assert np.array_equal(q.dequantize(got).cpu().numpy().view(np.uint32), orc.dequantize(ref, fbk).view(np.uint32))
        e4m3, sc = q.to_mxfp8(got, 1)
        e_ref, s_ref = orc.to_mxfp8(orc.Quantized(ref.codes, ref.meta), fbk, 1)
        assert np.array_equal(e4m3.cpu().numpy(), e_ref) and np.array_equal(sc.cpu().numpy(), s_ref)
        qw = q.quantize_weights(x)
        assert_same_quantized(qw, orc.quantize_weights(bits, fbk), f"custom formatbook weights ({want})")
        assert q.device_status == 0
        q.close()


@pytest.mark.parametrize("cfg", [dict(num_groups=32), dict(select_mode=1)], ids=["every_element_a_group", "all_dialects_scored"])
def test_selection_variants_in_both_kernels(cfg):
    """num_groups = block size (the paper's Table 2 setting) and select_mode 1: the TMA-staged kernel and the generic
    kernel both against the oracle, plain, with SeDA masks (paper-structured, arbitrary, one dialect, all ones) and
    with a residual pass."""
    ocfg = orc.Config(**cfg)
    T, C = 150, 1536
    bits = heavy(T, C, 21)
    bits[3, :64] = 0
    w = synth.Workload("t", T=T, C=C, seed=9, kind=1, n_outlier=0, outlier_gain=1.0, seda=True, n_clusters=6, cluster_seed=12,
                       score_seed=5)
    cid, masks = synth.clusters(w)
    rng = np.random.default_rng(4)
    masks = masks.copy()
    masks[1] = rng.integers(1, 2 ** 32)
    masks[2] = 1 << 31
    masks[3] = 0xFFFFFFFF
    cid = cid.copy()
    cid[5:9] = -1
    score = synth.scores(w)
    sal = orc.select_salient(score, 20)
    refs = {"plain": orc.quantize(bits, FB, ocfg),
            "seda": orc.quantize(bits, FB, ocfg, cluster_id=cid, cluster_mask=masks),
            "decomposed+seda": orc.quantize(bits, FB, ocfg, cluster_id=cid, cluster_mask=masks, salient_idx=sal)}
    x = to_dev_bf16(bits)
    dcid, dmask = torch.from_numpy(cid).cuda(), torch.from_numpy(masks.view(np.int32)).cuda()
    for variant, name in ((0, "fast"), (1, "generic")):
        q = fb4.Fb4(**cfg)
        q.set_kernel_variant(variant)
        assert_same_quantized(q.quantize(x), refs["plain"], f"{cfg} plain {name}")
        assert q.last_variant == name
        assert_same_quantized(q.quantize(x, dcid, dmask), refs["seda"], f"{cfg} seda {name}")
        got = q.quantize_decomposed(x, torch.from_numpy(score).cuda(), 20, cluster_id=dcid, cluster_mask=dmask)
        assert q.last_variant == name
        assert_same_quantized(got, refs["decomposed+seda"], f"{cfg} decomposed {name}")
        assert q.device_status == 0
        q.close()
    # a strided view takes the generic kernel and still agrees
    q = fb4.Fb4(**cfg)
    wide = torch.zeros((T, C + 64), dtype=torch.bfloat16, device="cuda")
    wide[:, :C] = x
    assert_same_quantized(q.quantize(wide[:, :C]), refs["plain"], f"{cfg} strided")
    assert q.last_variant == "generic"
    q.close()
