"""The five benchmark workloads at full size against the oracle (bit-exact codes, dialect ids,
scale bytes, salient indices; decoded fp32 at 0 ULP; MSE within 1e-6 relative), every row of every
tensor; the decoded tensors of the largest one are compared in row slabs."""
import numpy as np
import pytest
import torch

from gpu_util import FB, assert_same_bits_f32, assert_same_quantized, meta_np, to_dev_bf16
from oracle import fb4_oracle as orc
from paper_2603_02883_b200 import fb4, synth

pytestmark = pytest.mark.gpu

MSE_RTOL = 1e-6


@pytest.fixture(scope="module")
def q32():
    q = fb4.Fb4()
    yield q
    assert q.last_variant == "fast" and q.device_status == 0
    q.close()


@pytest.fixture(scope="module")
def c2_bits():
    return synth.activation(synth.workloads()["c2"])


def gpu_mse(x: torch.Tensor, recon: torch.Tensor, chunk: int = 4096) -> float:
    acc = 0.0
    for r in range(0, x.shape[0], chunk):
        d = x[r:r + chunk].double() - recon[r:r + chunk].double()
        acc += float((d * d).sum())
    return acc / x.numel()


def test_c1_quantize_dequantize(q32):
    w = synth.workloads()["c1"]
    bits = synth.activation(w)
    ref = orc.quantize(bits, FB)
    x = to_dev_bf16(bits)
    got = q32.quantize(x)
    assert_same_quantized(got, ref, "c1")
    out = q32.dequantize(got)
    ref_out = orc.dequantize(ref, FB)
    assert_same_bits_f32(out, ref_out, "c1 dequant")
    m_ref = orc.mse(bits, ref_out)
    assert abs(gpu_mse(x, out) - m_ref) <= MSE_RTOL * m_ref


def test_c2_plain(q32, c2_bits):
    ref = orc.quantize(c2_bits, FB)
    x = to_dev_bf16(c2_bits)
    got = q32.quantize(x)
    assert_same_quantized(got, ref, "c2")
    out = q32.dequantize(got)
    ref_out = orc.dequantize(ref, FB)
    assert_same_bits_f32(out, ref_out, "c2 dequant")
    m_ref = orc.mse(c2_bits, ref_out)
    assert abs(gpu_mse(x, out) - m_ref) <= MSE_RTOL * m_ref


def test_c3_decomposed(q32, c2_bits):
    w = synth.workloads()["c3"]
    score = synth.scores(w)
    sal = orc.select_salient(score, w.tile)
    assert len(sal) == 1638
    ref = orc.quantize(c2_bits, FB, salient_idx=sal)
    x = to_dev_bf16(c2_bits)
    got = q32.quantize_decomposed(x, torch.from_numpy(score).cuda(), w.tile)
    assert_same_quantized(got, ref, "c3")
    out = q32.dequantize(got)
    ref_out = orc.dequantize(ref, FB)
    assert_same_bits_f32(out, ref_out, "c3 dequant")
    m_ref = orc.mse(c2_bits, ref_out)
    assert abs(gpu_mse(x, out) - m_ref) <= MSE_RTOL * m_ref


def test_c4_seda(q32, c2_bits):
    w = synth.workloads()["c4"]
    cid, masks = synth.clusters(w)
    ref = orc.quantize(c2_bits, FB, cluster_id=cid, cluster_mask=masks)
    got = q32.quantize(to_dev_bf16(c2_bits), torch.from_numpy(cid).cuda(),
                       torch.from_numpy(masks.view(np.int32)).cuda())
    assert_same_quantized(got, ref, "c4")
    did = (meta_np(got.meta) >> 8).astype(np.int64)
    allowed = masks[cid][:, None].astype(np.int64)
    assert np.all((allowed >> did) & 1)
    x = to_dev_bf16(c2_bits)
    out = q32.dequantize(got)
    ref_out = orc.dequantize(ref, FB)
    assert_same_bits_f32(out, ref_out, "c4 dequant")
    m_ref = orc.mse(c2_bits, ref_out)
    assert abs(gpu_mse(x, out) - m_ref) <= MSE_RTOL * m_ref
    ref_b = orc.dequantize(ref, FB, out_dtype="bf16")
    assert np.array_equal(q32.dequantize(got, torch.bfloat16).view(torch.int16).cpu().numpy().view(np.uint16), ref_b)


def _row_slab(q: orc.Quantized, r0: int, r1: int) -> orc.Quantized:
    """rows [r0, r1) of an oracle result as a tensor of its own (salient indices rebased)"""
    if q.salient_idx is None:
        return orc.Quantized(q.codes[r0:r1], q.meta[r0:r1])
    s0, s1 = np.searchsorted(q.salient_idx, [r0, r1])
    return orc.Quantized(q.codes[r0:r1], q.meta[r0:r1], salient_idx=(q.salient_idx[s0:s1] - r0).astype(np.int32),
                         res_codes=q.res_codes[s0:s1], res_meta=q.res_meta[s0:s1])


def test_c5_decomposed_seda_and_plain_every_row(q32):
    """The largest tensor (75 600 x 12 288), decomposition and SeDA together, and the plain quantizer on
    the same tensor: every row of every output against the oracle.  The decoded tensors (fp32 at 0 ULP,
    bf16) are produced by one full-size call each and compared in row slabs to bound host memory."""
    w = synth.workloads()["c5"]
    bits = synth.activation(w)                       # 1.86 GB on the host
    score = synth.scores(w)
    cid, masks = synth.clusters(w)
    sal = orc.select_salient(score, w.tile)
    assert len(sal) == 3780
    x = to_dev_bf16(bits)
    got = q32.quantize_decomposed(x, torch.from_numpy(score).cuda(), w.tile,
                                  cluster_id=torch.from_numpy(cid).cuda(),
                                  cluster_mask=torch.from_numpy(masks.view(np.int32)).cuda())
    ref = orc.quantize(bits, FB, cluster_id=cid, cluster_mask=masks, salient_idx=sal)
    assert_same_quantized(got, ref, "c5")
    plain = q32.quantize(x)
    refp = orc.quantize(bits, FB)
    assert_same_quantized(plain, refp, "c5 plain")
    # decode: fp32 bit patterns, MSE, then bf16
    out = q32.dequantize(got)
    n_slab = 12
    edges = [w.T * i // n_slab for i in range(n_slab + 1)]
    sse_ref = 0.0
    for r0, r1 in zip(edges[:-1], edges[1:]):
        ref_out = orc.dequantize(_row_slab(ref, r0, r1), FB)
        assert_same_bits_f32(out[r0:r1], ref_out, f"c5 dequant rows {r0}..{r1}")
        sse_ref += orc.mse(bits[r0:r1], ref_out) * (r1 - r0) * w.C
    m_ref = sse_ref / (w.T * w.C)
    assert abs(gpu_mse(x, out) - m_ref) <= MSE_RTOL * m_ref
    del out
    outp = q32.dequantize(plain)
    sse_p = 0.0
    for r0, r1 in zip(edges[:-1], edges[1:]):
        ref_out = orc.dequantize(_row_slab(refp, r0, r1), FB)
        assert_same_bits_f32(outp[r0:r1], ref_out, f"c5 plain dequant rows {r0}..{r1}")
        sse_p += orc.mse(bits[r0:r1], ref_out) * (r1 - r0) * w.C
    m_p = sse_p / (w.T * w.C)
    assert abs(gpu_mse(x, outp) - m_p) <= MSE_RTOL * m_p
    del outp
    outb = q32.dequantize(got, torch.bfloat16)
    for r0, r1 in zip(edges[:-1], edges[1:]):
        ref_b = orc.dequantize(_row_slab(ref, r0, r1), FB, out_dtype="bf16")
        assert np.array_equal(outb[r0:r1].view(torch.int16).cpu().numpy().view(np.uint16), ref_b), f"bf16 rows {r0}..{r1}"
    # SeDA choices inside the mask (a property, beside the element-wise comparison)
    did = (meta_np(got.meta) >> 8).astype(np.int64)
    assert np.all((masks[cid][:, None].astype(np.int64) >> did) & 1)


def test_c3_global_top5_percent_reading(q32, c2_bits):
    """Config 3 read literally ("top 5 % by score" over the whole sequence instead of one token per
    tile of 20): global top-k selection feeding the decomposition with a given salient set."""
    w = synth.workloads()["c3"]
    score = synth.scores(w)
    k = -(-w.T * 5 // 100)
    assert k == 1638
    sal = orc.select_salient_topk(score, k)
    got_sal = q32.select_salient_topk(torch.from_numpy(score).cuda(), k)
    assert np.array_equal(got_sal.cpu().numpy(), sal)
    ref = orc.quantize(c2_bits, FB, salient_idx=sal)
    got = q32.quantize_decomposed(to_dev_bf16(c2_bits), salient_idx=got_sal)
    assert_same_quantized(got, ref, "c3 global")
    assert_same_bits_f32(q32.dequantize(got), orc.dequantize(ref, FB), "c3 global dequant")


@pytest.mark.parametrize("T,k", [(1, 1), (7, 0), (7, 7), (1000, 50), (1024, 1), (5000, 4999), (75600, 3780), (8192, 1),
                                 (8192, 8192), (8193, 4000), (100001, 5000), (300000, 299999), (1 << 20, 52429)])
def test_topk_selection_with_ties(q32, T, k):
    rng = np.random.default_rng(T + k)
    s = rng.random(T).astype(np.float32)
    if T > 4:
        s[rng.integers(0, T, size=T // 3)] = s[T // 2]           # a large tie group, likely at the threshold
        s[rng.integers(0, T, size=3)] = -0.0
        s[rng.integers(0, T, size=3)] = 0.0
        s[rng.integers(0, T, size=T // 10)] *= -1                 # negative scores
    want = orc.select_salient_topk(s, k) if T <= 5000 else np.sort(np.argsort(-s.astype(np.float64), kind="stable")[:k])
    got = q32.select_salient_topk(torch.from_numpy(s).cuda(), k)
    assert np.array_equal(got.cpu().numpy(), want)


@pytest.mark.parametrize("variant", [0, 1])      # 0: several launches over many CTAs, 1: one CTA
def test_topk_degenerate_scores_and_both_kernels(variant):
    """All scores equal (every key ties at the threshold: the lowest indices win), two values only, and a
    descending ramp; the many-CTA path and the single-CTA kernel give the same indices."""
    q = fb4.Fb4()
    try:
        q.set_kernel_variant(variant)
        T = 50000
        for name, s in (("equal", np.full(T, 0.25, np.float32)),
                        ("two values", (np.arange(T) % 3 == 0).astype(np.float32)),
                        ("ramp", np.linspace(1.0, -1.0, T).astype(np.float32)),
                        ("tiny differences", np.float32(1.0) + np.arange(T, dtype=np.float32) * np.float32(2.0 ** -23))):
            for k in (1, 2500, T - 1):
                want = np.sort(np.argsort(-s.astype(np.float64), kind="stable")[:k])
                got = q.select_salient_topk(torch.from_numpy(s).cuda(), k)
                assert np.array_equal(got.cpu().numpy(), want), f"{name} k={k}"
        assert q.device_status == 0
    finally:
        q.close()

