"""include/fb4_block.cuh: a producer kernel that is not part of the library includes the header, evaluates
y = (x + 1) * 0.75 in fp32 and quantizes y from its registers; the result must equal the oracle's
quantization of the same fp32 values, bit for bit."""
import ctypes
import os
import subprocess

import numpy as np
import pytest
import torch

from gpu_util import FB
from oracle import fb4_oracle as orc
from paper_2603_02883_b200 import fb4, synth

pytestmark = pytest.mark.gpu

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
SRC = os.path.join(HERE, "producer", "producer_kernel.cu")


@pytest.fixture(scope="module")
def producer(tmp_path_factory):
    so = str(tmp_path_factory.mktemp("producer") / "libproducer.so")
    subprocess.check_call([os.environ.get("NVCC", "nvcc"), "-O3", "-std=c++17", "-gencode", "arch=compute_100a,code=sm_100a",
                           "-Xcompiler", "-fPIC", "-shared", "-I", os.path.join(ROOT, "include"), "-o", so, SRC,
                           "-cudart", "shared"])
    L = ctypes.CDLL(so)
    vp = ctypes.c_void_p
    L.producer_launch.argtypes = [vp, vp, ctypes.c_int64, vp, vp, vp]
    L.producer_table_bytes.restype = ctypes.c_uint64
    return L


def test_producer_kernel_with_the_block_header_matches_the_oracle(producer):
    q = fb4.Fb4()
    image, nbytes = fb4.fb4_block_tables(q.ctx)
    assert nbytes == producer.producer_table_bytes() and image % 16 == 0
    w = synth.Workload("p", T=203, C=1536, seed=31, kind=1, n_outlier=7, outlier_gain=50.0)
    bits = synth.activation(w)
    bits[5, :64] = 0
    bits[6, 3] = 0x8000                                        # -0: (x + 1) * 0.75 = 0.75
    bits[7, :32] = synth.f32_to_bf16_bits(np.full(32, -1.0, np.float32))   # y = +0 everywhere in that block
    xf = synth.bf16_bits_to_f32(bits)
    y = ((xf + np.float32(1.0)) * np.float32(0.75)).astype(np.float32)     # two IEEE single operations
    ref = orc.quantize_f32(y, FB)
    x = torch.from_numpy(bits.view(np.int16)).cuda()
    codes = torch.zeros((w.T, w.C // 2), dtype=torch.uint8, device="cuda")
    meta = torch.zeros((w.T, w.C // 32), dtype=torch.int16, device="cuda")
    rc = producer.producer_launch(image, x.data_ptr(), w.T * w.C // 32, codes.data_ptr(), meta.data_ptr(),
                                  torch.cuda.current_stream().cuda_stream)
    assert rc == 0
    torch.cuda.synchronize()
    assert np.array_equal(meta.cpu().numpy().view(np.uint16), ref.meta)
    assert np.array_equal(codes.cpu().numpy(), ref.codes)
    # the library's own fp32 entry point agrees (it is built on the same routine)
    got = q.quantize(torch.from_numpy(y).cuda())
    assert np.array_equal(got.codes.cpu().numpy(), ref.codes)
    q.close()


def test_no_image_for_other_configurations():
    q16 = fb4.Fb4(block_size=16)
    with pytest.raises(fb4.Fb4Error) as e:
        fb4.fb4_block_tables(q16.ctx)
    assert e.value.code == fb4.ERR_INVALID_ARG
    q16.close()
