"""GPU parity of the MXFP8 view (e4m3 bytes + E8M0 scale bytes, both scale layouts) against the CPU
oracle, byte for byte, padding of the tiled layout included."""
import ctypes

import numpy as np
import pytest
import torch

from gpu_util import FB, to_dev_bf16
from oracle import fb4_oracle as orc
from paper_2603_02883_b200 import fb4, synth

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def q32():
    q = fb4.Fb4()
    yield q
    assert q.device_status == 0
    q.close()


@pytest.mark.parametrize("T,C", [(1, 32), (130, 96), (300, 320), (257, 1024 + 64), (128, 128)])
def test_random_codes_every_dialect(q32, T, C):
    rng = np.random.default_rng(T + C)
    codes = rng.integers(0, 256, size=(T, C // 2), dtype=np.uint8)
    meta = (rng.integers(0, 252, size=(T, C // 32)) | (rng.integers(0, 32, size=(T, C // 32)) << 8)).astype(np.uint16)
    ref = orc.Quantized(codes, meta)
    got = fb4.Quantized(torch.from_numpy(codes).cuda(), torch.from_numpy(meta.view(np.int16)).cuda())
    for layout in (0, 1):
        e_ref, s_ref = orc.to_mxfp8(ref, FB, layout)
        e4m3, scales = q32.to_mxfp8(got, layout)
        scales_before = scales.clone()
        assert np.array_equal(e4m3.cpu().numpy(), e_ref), f"e4m3 bytes, layout {layout}"
        assert np.array_equal(scales.cpu().numpy(), s_ref), f"scale bytes, layout {layout}"
        assert scales.numel() == fb4.fb4_mxfp8_scale_bytes(T, C, layout) == len(s_ref)
        del scales_before


def test_c2_workload_and_decoded_value(q32):
    w = synth.workloads()["c2"]
    bits = synth.activation(w)
    q = q32.quantize(to_dev_bf16(bits))
    ref = orc.quantize(bits, FB)
    e_ref, s_ref = orc.to_mxfp8(ref, FB, 1)
    e4m3, scales = q32.to_mxfp8(q, 1)
    assert np.array_equal(e4m3.cpu().numpy(), e_ref) and np.array_equal(scales.cpu().numpy(), s_ref)
    # e4m3 * 2^(scale-127) is the decoded value (torch's own e4m3 decoder on a slab of rows)
    rows = slice(1000, 1256)
    vals = e4m3[rows].view(torch.float8_e4m3fn).float().view(256, w.C // 32, 32)
    e0, s0 = q32.to_mxfp8(fb4.Quantized(q.codes[rows].contiguous(), q.meta[rows].contiguous()), 0)
    sc = torch.exp2(s0.view(256, w.C // 32, 1).float() - 127.0)
    want = q32.dequantize(fb4.Quantized(q.codes[rows].contiguous(), q.meta[rows].contiguous()))
    assert torch.equal((vals * sc).view(256, w.C), want)


def test_argument_checks(q32):
    L = fb4.lib()
    t = torch.zeros(4096, dtype=torch.uint8, device="cuda")
    p = ctypes.c_void_p(t.data_ptr())
    assert L.fb4_to_mxfp8(q32.ctx, p, p, 4, 48, p, p, 0, None) == fb4.ERR_SHAPE
    assert L.fb4_to_mxfp8(q32.ctx, p, p, 4, 64, p, p, 2, None) == fb4.ERR_INVALID_ARG
    assert L.fb4_to_mxfp8(q32.ctx, p, p, 4, 64, None, p, 0, None) == fb4.ERR_INVALID_ARG
    assert L.fb4_to_mxfp8(q32.ctx, None, None, 0, 64, None, None, 0, None) == fb4.OK
    assert L.fb4_mxfp8_scale_bytes(300, 320, 1) == 3 * 3 * 512 and L.fb4_mxfp8_scale_bytes(300, 320, 0) == 3000
    assert L.fb4_mxfp8_scale_bytes(300, 330, 0) == -1
    q16 = fb4.Fb4(block_size=16)
    assert L.fb4_to_mxfp8(q16.ctx, p, p, 4, 64, p, p, 0, None) == fb4.ERR_INVALID_ARG
    q16.close()


@pytest.mark.parametrize("T,C", [(1, 64), (130, 3072), (300, 1024 + 64), (257, 128), (2368, 64)])
def test_fused_quantize_to_mxfp8(q32, T, C):
    """fb4_quantize_mxfp8 equals quantize followed by the MXFP8 view (oracle), plain and SeDA, both layouts."""
    w = synth.Workload("m", T=T, C=C, seed=T + C, kind=1, n_outlier=2, outlier_gain=50.0, seda=True,
                       n_clusters=min(4, T), cluster_seed=5)
    bits = synth.activation(w)
    cid, masks = synth.clusters(w)
    x = to_dev_bf16(bits)
    ref_plain = orc.quantize(bits, FB)
    ref_seda = orc.quantize(bits, FB, cluster_id=cid, cluster_mask=masks)
    for layout in (0, 1):
        e4m3, scales = q32.quantize_mxfp8(x, layout)
        e_ref, s_ref = orc.to_mxfp8(ref_plain, FB, layout)
        assert np.array_equal(e4m3.cpu().numpy(), e_ref) and np.array_equal(scales.cpu().numpy(), s_ref)
        e4m3, scales = q32.quantize_mxfp8(x, layout, torch.from_numpy(cid).cuda(),
                                          torch.from_numpy(masks.view(np.int32)).cuda())
        e_ref, s_ref = orc.to_mxfp8(ref_seda, FB, layout)
        assert np.array_equal(e4m3.cpu().numpy(), e_ref) and np.array_equal(scales.cpu().numpy(), s_ref)


def test_fused_quantize_to_mxfp8_rejects_other_configurations():
    import ctypes
    q16 = fb4.Fb4(block_size=16)
    x = torch.zeros((4, 64), dtype=torch.bfloat16, device="cuda")
    out = torch.zeros(4096, dtype=torch.uint8, device="cuda")
    p = lambda t: ctypes.c_void_p(t.data_ptr())
    L = fb4.lib()
    assert L.fb4_quantize_mxfp8(q16.ctx, p(x), 4, 64, 64, None, None, 0, p(out), p(out), 0, None) == fb4.ERR_INVALID_ARG
    q16.close()
    q = fb4.Fb4()
    assert L.fb4_quantize_mxfp8(q.ctx, p(x), 4, 32, 64, None, None, 0, p(out), p(out), 0, None) == fb4.ERR_SHAPE
    assert L.fb4_quantize_mxfp8(q.ctx, p(x), 4, 64, 64, None, None, 0, ctypes.c_void_p(out.data_ptr() + 16), p(out), 0,
                                None) == fb4.ERR_ALIGN
    assert L.fb4_quantize_mxfp8(q.ctx, p(x), 4, 64, 64, None, None, 0, p(out), p(out), 3, None) == fb4.ERR_INVALID_ARG
    q.close()


@pytest.mark.parametrize("T,N,K", [(256, 256, 3072), (300, 144, 1088), (130, 16, 96)])
def test_library_block_scaled_gemm_consumes_the_view(q32, T, N, K):
    """External pin of the tiled scale layout (Sec. 4.1: FB4 mapped to MXFP8): the library's block-scaled
    e4m3 GEMM, given FB4 activations and FB4 weights in the MXFP8 view, reproduces the product of the two
    dequantized matrices to bf16 rounding; with the scales in the other (row-major) order it does not."""
    if not hasattr(torch, "_scaled_mm") or not hasattr(torch, "float8_e8m0fnu"):
        pytest.skip("this torch build has no block-scaled GEMM")
    a_bits = synth.activation(synth.Workload("a", T=T, C=K, seed=T + K, kind=1, n_outlier=2, outlier_gain=50.0))
    w_bits = synth.activation(synth.Workload("w", T=N, C=K, seed=N + K + 1, kind=1, n_outlier=0, outlier_gain=1.0))
    qa = q32.quantize(to_dev_bf16(a_bits))
    qw = q32.quantize_weights(to_dev_bf16(w_bits))
    ea, sa = q32.to_mxfp8(qa, 1)
    ew, sw = q32.to_mxfp8(qw, 1)
    da, dw = q32.dequantize(qa).double(), q32.dequantize(qw).double()
    want, bound = da @ dw.T, da.abs() @ dw.abs().T

    def gemm(scale_a, scale_w):
        return torch._scaled_mm(ea.view(torch.float8_e4m3fn), ew.view(torch.float8_e4m3fn).t(),
                                scale_a=scale_a.view(torch.float8_e8m0fnu), scale_b=scale_w.view(torch.float8_e8m0fnu),
                                out_dtype=torch.bfloat16).double()

    tol = want.abs() * 2.0 ** -8 + bound * 1e-5      # one bf16 rounding + fp32 accumulation
    assert bool(((gemm(sa, sw) - want).abs() <= tol).all())
    # negative control: the same scale bytes, row-major, zero-padded to the tiled size
    sa_rm = torch.zeros_like(sa)
    sa_rm[: T * (K // 32)] = q32.to_mxfp8(qa, 0)[1]
    if not torch.equal(sa_rm, sa):
        assert not bool(((gemm(sa_rm, sw) - want).abs() <= tol).all())


@pytest.mark.parametrize("T,C", [(130, 96), (300, 320), (257, 1024 + 64), (129, 32 * 33)])
def test_tiled_scales_at_an_odd_address(q32, T, C):
    """The tiled scale order goes through a CTA-staged kernel when the scale buffer is 16-byte aligned and
    through the byte-store kernel otherwise: both give the oracle's bytes."""
    rng = np.random.default_rng(T * C)
    codes = rng.integers(0, 256, size=(T, C // 2), dtype=np.uint8)
    meta = (rng.integers(0, 252, size=(T, C // 32)) | (rng.integers(0, 32, size=(T, C // 32)) << 8)).astype(np.uint16)
    e_ref, s_ref = orc.to_mxfp8(orc.Quantized(codes, meta), FB, 1)
    d_codes, d_meta = torch.from_numpy(codes).cuda(), torch.from_numpy(meta.view(np.int16)).cuda()
    n = fb4.fb4_mxfp8_scale_bytes(T, C, 1)
    for shift in (0, 1, 8):
        e4m3 = torch.zeros((T, C), dtype=torch.uint8, device="cuda")
        buf = torch.full((n + 64,), 0xEE, dtype=torch.uint8, device="cuda")
        fb4.fb4_to_mxfp8(q32.ctx, d_codes, d_meta, T, C, e4m3, buf[shift:], 1)
        assert np.array_equal(e4m3.cpu().numpy(), e_ref), f"e4m3 bytes, shift {shift}"
        got = buf.cpu().numpy()
        assert np.array_equal(got[shift:shift + n], s_ref), f"scale bytes, shift {shift}"
        assert (got[:shift] == 0xEE).all() and (got[shift + n:] == 0xEE).all(), "bytes outside the scale array"


@pytest.mark.parametrize("T,C,tile", [(1, 64, 20), (130, 3072, 20), (300, 1024 + 64, 7), (257, 128, 1), (2368, 64, 20)])
def test_fused_quantize_to_mxfp8_with_decomposition(q32, T, C, tile):
    """fb4_quantize_mxfp8_decomposed equals the decomposed quantizer (oracle) followed by the MXFP8 view of the main
    and of the residual tensor: per-tile selection and a given salient set, with and without SeDA, both layouts."""
    w = synth.Workload("m", T=T, C=C, seed=T + C, kind=1, n_outlier=2, outlier_gain=50.0, seda=True,
                       n_clusters=min(4, T), cluster_seed=5, score_seed=T)
    bits = synth.activation(w)
    cid, masks = synth.clusters(w)
    score = synth.scores(w)
    x = to_dev_bf16(bits)
    d_cid, d_masks = torch.from_numpy(cid).cuda(), torch.from_numpy(masks.view(np.int32)).cuda()
    sal = orc.select_salient(score, tile)
    mine = np.unique(np.random.default_rng(T).integers(0, T, size=max(1, T // 3))).astype(np.int32)
    for seda in (False, True):
        kw = dict(cluster_id=cid, cluster_mask=masks) if seda else {}
        dkw = dict(cluster_id=d_cid, cluster_mask=d_masks) if seda else {}
        for layout in (0, 1):
            for given in (False, True):
                want_idx = mine if given else sal
                ref = orc.quantize(bits, FB, salient_idx=want_idx, **kw)
                e_ref, s_ref = orc.to_mxfp8(orc.Quantized(ref.codes, ref.meta), FB, layout)
                re_ref, rs_ref = orc.to_mxfp8(orc.Quantized(ref.res_codes, ref.res_meta), FB, layout)
                if given:
                    out = q32.quantize_mxfp8_decomposed(x, salient_idx=torch.from_numpy(mine).cuda(),
                                                        scale_layout=layout, **dkw)
                else:
                    out = q32.quantize_mxfp8_decomposed(x, score=torch.from_numpy(score).cuda(), tile=tile,
                                                        scale_layout=layout, **dkw)
                e4m3, scales, idx, res, res_scales = out
                what = f"seda {seda} layout {layout} given {given}"
                assert np.array_equal(idx.cpu().numpy(), want_idx), what
                assert np.array_equal(e4m3.cpu().numpy(), e_ref), what
                assert np.array_equal(scales.cpu().numpy(), s_ref), what
                assert np.array_equal(res.cpu().numpy(), re_ref), what
                assert np.array_equal(res_scales.cpu().numpy(), rs_ref), what


def test_library_block_scaled_gemm_with_residual_operand(q32):
    """(Q(Act) + Q(Delta)) W (Sec. 3.3) as two block-scaled library GEMMs on the operands of
    fb4_quantize_mxfp8_decomposed: the main one over all tokens, the residual one over the salient tokens, added
    into their rows; compared with the product of the decoded sum and the decoded weights."""
    if not hasattr(torch, "_scaled_mm") or not hasattr(torch, "float8_e8m0fnu"):
        pytest.skip("this torch build has no block-scaled GEMM")
    T, N, K, tile = 320, 128, 1024, 20
    wl = synth.Workload("a", T=T, C=K, seed=3, kind=1, n_outlier=2, outlier_gain=50.0, score_seed=9)
    a_bits, score = synth.activation(wl), synth.scores(wl)
    w_bits = synth.activation(synth.Workload("w", T=N, C=K, seed=4, kind=1, n_outlier=0, outlier_gain=1.0))
    x = to_dev_bf16(a_bits)
    e4m3, scales, idx, res, res_scales = q32.quantize_mxfp8_decomposed(x, score=torch.from_numpy(score).cuda(), tile=tile)
    qw = q32.quantize_weights(to_dev_bf16(w_bits))
    ew, sw = q32.to_mxfp8(qw, 1)
    f8, e8 = torch.float8_e4m3fn, torch.float8_e8m0fnu

    def gemm(a, sa):
        return torch._scaled_mm(a.view(f8), ew.view(f8).t(), scale_a=sa.view(e8), scale_b=sw.view(e8),
                                out_dtype=torch.float32)

    y = gemm(e4m3, scales)
    y.index_add_(0, idx.long(), gemm(res.contiguous(), res_scales))
    qa = q32.quantize_decomposed(x, score=torch.from_numpy(score).cuda(), tile=tile)
    da, dw = q32.dequantize(qa).double(), q32.dequantize(qw).double()
    want, bound = da @ dw.T, da.abs() @ dw.abs().T
    assert bool(((y.double() - want).abs() <= bound * 2e-5).all())      # fp32 accumulation, two partial products
    # the residual operand matters: without it the salient rows are off by more than that
    y0 = gemm(e4m3, scales).double()
    rows = idx.long()
    assert not bool(((y0[rows] - want[rows]).abs() <= bound[rows] * 2e-5).all())


def test_fused_decomposed_argument_checks(q32):
    L = fb4.lib()
    x = torch.zeros((8, 64), dtype=torch.bfloat16, device="cuda")
    out = torch.zeros(8192, dtype=torch.uint8, device="cuda")
    idx = torch.zeros(8, dtype=torch.int32, device="cuda")
    sc = torch.zeros(8, dtype=torch.float32, device="cuda")
    p = lambda t: ctypes.c_void_p(t.data_ptr())
    f = L.fb4_quantize_mxfp8_decomposed
    ok = (q32.ctx, p(x), 8, 64, 64, p(sc), 4, p(idx), 0, None, None, 0, p(out), p(out), p(out), p(out), 0, None)
    assert f(*ok) == fb4.OK

    def call(**kw):
        a = list(ok)
        names = ["ctx", "x", "T", "C", "ld", "score", "tile", "idx", "n", "cid", "cmask", "ncl", "e", "s", "re", "rs",
                 "layout", "stream"]
        for k, v in kw.items():
            a[names.index(k)] = v
        return f(*a)

    assert call(tile=0) == fb4.ERR_INVALID_ARG
    assert call(score=None, n=9) == fb4.ERR_INVALID_ARG          # more salient tokens than tokens
    assert call(score=None, n=-1) == fb4.ERR_INVALID_ARG
    assert call(score=None, n=2, re=None) == fb4.ERR_INVALID_ARG
    assert call(score=None, n=0, idx=None, re=None, rs=None) == fb4.OK     # no salient tokens: plain call
    assert call(C=32) == fb4.ERR_SHAPE
    assert call(layout=2) == fb4.ERR_INVALID_ARG
    assert call(cid=p(idx)) == fb4.ERR_INVALID_ARG               # cluster ids without masks
    assert call(re=ctypes.c_void_p(out.data_ptr() + 16)) == fb4.ERR_ALIGN
    assert call(T=0, x=None) == fb4.OK
    q16 = fb4.Fb4(block_size=16)
    assert call(ctx=q16.ctx) == fb4.ERR_INVALID_ARG
    q16.close()
