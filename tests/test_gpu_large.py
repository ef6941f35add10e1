"""A tensor with more than 2^32 elements: element, byte and block offsets leave 32 bits.  The input
is made on the device in slabs (seeded), quantized and decoded in full, and compared with the oracle
on sampled rows from the start, the 2^32-element boundary and the end."""
import numpy as np
import pytest
import torch

from gpu_util import FB, meta_np
from oracle import fb4_oracle as orc
from paper_2603_02883_b200 import fb4

pytestmark = pytest.mark.gpu


def test_more_than_2_to_32_elements():
    T, C = 70000, 65536                               # 4.59 G elements: 9.2 GB in, 2.3 GB of codes
    free, _ = torch.cuda.mem_get_info()
    if free < 40e9:
        pytest.skip("needs 40 GB of free device memory")
    g = torch.Generator(device="cuda").manual_seed(77)
    x = torch.empty((T, C), dtype=torch.bfloat16, device="cuda")
    for r in range(0, T, 5000):
        slab = torch.randn((min(5000, T - r), C), generator=g, device="cuda")
        slab *= torch.exp2(torch.randint(-8, 8, (slab.shape[0], 1), generator=g, device="cuda").float())
        x[r:r + slab.shape[0]] = slab.to(torch.bfloat16)
        del slab
    q = fb4.Fb4()
    got = q.quantize(x)
    assert q.last_variant == "fast"
    out = q.dequantize(got, torch.bfloat16)
    rows = np.unique(np.concatenate([np.arange(0, 40), np.arange(65530, 65545), np.arange(T - 40, T),
                                     np.random.default_rng(1).integers(0, T, 60)]))   # 65536 rows = 2^32 elements
    ridx = torch.from_numpy(rows).cuda()
    bits = x[ridx].view(torch.int16).cpu().numpy().view(np.uint16)
    ref = orc.quantize(bits, FB)
    assert np.array_equal(got.codes[ridx].cpu().numpy(), ref.codes)
    assert np.array_equal(meta_np(got.meta[ridx]), ref.meta)
    ref_out = orc.dequantize(ref, FB, out_dtype="bf16")
    assert np.array_equal(out[ridx].view(torch.int16).cpu().numpy().view(np.uint16), ref_out)
    # a property over the whole tensor: every scale byte is the exponent of its block maximum
    for r in range(0, T, 10000):
        amax = x[r:r + 10000].view(-1, C // 32, 32).abs().amax(dim=2).float()
        e = torch.floor(torch.log2(amax.clamp_min(2.0 ** -124))).to(torch.int32)
        sb = got.meta[r:r + 10000].to(torch.int32) & 0xFF
        assert bool((sb == e + 124).all())
    e4m3, scales = q.to_mxfp8(fb4.Quantized(got.codes, got.meta), 1)
    e_ref, s_ref = orc.to_mxfp8(ref, FB, 0)
    assert np.array_equal(e4m3[ridx].cpu().numpy(), e_ref)
    # scale bytes of a few sampled rows, through the tiled scale order
    for t in (0, 39, 65536, T - 1):
        k = int(np.searchsorted(rows, t))
        for c in (0, 5, C // 32 - 1):
            off = orc.mxfp8_scale_offset(t, c, C // 32, 1)
            assert int(scales[off]) == int(s_ref[k * (C // 32) + c])
    assert q.device_status == 0
    q.close()
