"""Index arguments that point outside their tables are caught by the kernels' own bounds checks: a
cluster id outside [-1, n_clusters) counts as -1 (unconstrained), a salient token index outside
[0, T) is skipped on decode, and either raises bit 1 of the context's status word.  The expected
outputs are the oracle's on the same inputs with the offending entries replaced / dropped on the CPU."""
import numpy as np
import pytest
import torch

from gpu_util import FB, assert_same_bits_f32, assert_same_quantized, to_dev_bf16
from oracle import fb4_oracle as orc
from paper_2603_02883_b200 import fb4, synth

pytestmark = pytest.mark.gpu


def _workload(T, C):
    return synth.Workload("idx", T=T, C=C, seed=T + C, kind=1, n_outlier=2, outlier_gain=50.0, seda=True,
                          n_clusters=4, cluster_seed=9)


@pytest.mark.parametrize("variant", [0, 1])          # 0 = TMA-staged kernel, 1 = generic kernel
@pytest.mark.parametrize("T,C", [(300, 1024), (64, 64)])
def test_cluster_ids_out_of_range_are_unconstrained_and_reported(variant, T, C):
    w = _workload(T, C)
    bits = synth.activation(w)
    cid, masks = synth.clusters(w)
    bad = cid.copy()
    bad[1::7] = len(masks)              # first id past the table
    bad[2::11] = 1_000_000
    bad[3::13] = -7
    bad[5::17] = np.iinfo(np.int32).min
    clean = np.where((bad >= 0) & (bad < len(masks)), bad, -1).astype(np.int32)
    ref = orc.quantize(bits, FB, cluster_id=clean, cluster_mask=masks)
    q = fb4.Fb4()
    try:
        q.set_kernel_variant(variant)
        x = to_dev_bf16(bits)
        d_masks = torch.from_numpy(masks.view(np.int32)).cuda()
        got = q.quantize(x, torch.from_numpy(bad).cuda(), d_masks)
        assert_same_quantized(got, ref, "ids out of range")
        assert q.last_variant == ("generic" if variant else "fast")
        assert q.device_status == 2
        if variant == 0:
            e4m3, scales = q.quantize_mxfp8(x, 0, torch.from_numpy(bad).cuda(), d_masks)
            e_ref, s_ref = orc.to_mxfp8(ref, FB, 0)
            assert np.array_equal(e4m3.cpu().numpy(), e_ref) and np.array_equal(scales.cpu().numpy(), s_ref)
    finally:
        q.close()
    # the same call with ids in range leaves the status word alone
    q = fb4.Fb4()
    try:
        q.set_kernel_variant(variant)
        q.quantize(to_dev_bf16(bits), torch.from_numpy(clean).cuda(), torch.from_numpy(masks.view(np.int32)).cuda())
        assert q.device_status == 0
    finally:
        q.close()


@pytest.mark.parametrize("block_size,C", [(32, 8192), (32, 1024), (32, 96), (16, 48)])
def test_decode_skips_salient_rows_outside_the_tensor(block_size, C):
    T = 200
    w = synth.Workload("idx", T=T, C=C, seed=C, kind=1, n_outlier=1, outlier_gain=50.0)
    bits = synth.activation(w)
    cfg = orc.Config(block_size=block_size)
    keep = np.array([3, 50, 51, 199], dtype=np.int32)
    ref = orc.quantize(bits, FB, cfg, salient_idx=keep)
    want = orc.dequantize(ref, FB, block_size)
    q = fb4.Fb4(block_size=block_size)
    try:
        got = q.quantize_decomposed(to_dev_bf16(bits), salient_idx=torch.from_numpy(keep).cuda())
        assert_same_quantized(got, ref, "given set")
        # the same residual rows in a list (still ascending) that also has entries outside [0, T)
        idx = np.array([np.iinfo(np.int32).min, -1, 3, 50, 51, 199, T, np.iinfo(np.int32).max], dtype=np.int32)
        pos = [2, 3, 4, 5]
        nblk = C // block_size
        rc = torch.zeros((len(idx), C // 2), dtype=torch.uint8, device="cuda")
        rm = torch.zeros((len(idx), nblk), dtype=torch.int16, device="cuda")
        rc[pos] = got.res_codes
        rm[pos] = got.res_meta
        padded = fb4.Quantized(got.codes, got.meta, torch.from_numpy(idx).cuda(), rc, rm)
        assert q.device_status == 0
        out = q.dequantize(padded)
        assert_same_bits_f32(out, want, "decode with entries outside the tensor")
        assert q.device_status == 2
    finally:
        q.close()


@pytest.mark.parametrize("variant", [0, 1])
def test_affine_entry_checks_cluster_ids_too(variant):
    T, C = 150, 1024
    w = _workload(T, C)
    bits = synth.activation(w)
    cid, masks = synth.clusters(w)
    bad = cid.copy()
    bad[::9] = 77
    bad[4::13] = -3
    clean = np.where((bad >= 0) & (bad < len(masks)), bad, -1).astype(np.int32)
    gain = synth.f32_to_bf16_bits(np.linspace(-0.5, 0.5, C).astype(np.float32))
    bias = synth.f32_to_bf16_bits(np.linspace(1.0, -1.0, C).astype(np.float32))
    ref = orc.quantize_f32(orc.affine_f32(bits, gain, bias, True), FB, cluster_id=clean, cluster_mask=masks)
    q = fb4.Fb4()
    try:
        q.set_kernel_variant(variant)
        dev = lambda a: torch.from_numpy(a.view(np.int16)).cuda().view(torch.bfloat16)
        got = q.quantize_affine(to_dev_bf16(bits), dev(gain), dev(bias), True, torch.from_numpy(bad).cuda(),
                                torch.from_numpy(masks.view(np.int32)).cuda())
        assert_same_quantized(got, ref, "affine, ids out of range")
        assert q.device_status == 2
    finally:
        q.close()
