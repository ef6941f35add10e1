"""GPU parity of the offline weight quantizer (exhaustive squared-error dialect selection) against
the CPU oracle, bit for bit, and the properties that tie it to the online quantizer."""
import numpy as np
import pytest
import torch

from gpu_util import FB, assert_same_quantized, meta_np, to_dev_bf16
from oracle import fb4_oracle as orc
from paper_2603_02883_b200 import fb4, synth
from test_gpu_parity import edge_blocks, heavy

pytestmark = pytest.mark.gpu


def weight_like(N, K, seed):
    rng = np.random.default_rng(seed)
    w = rng.standard_normal((N, K)).astype(np.float32) * 0.02
    w[:, rng.integers(0, K, size=max(1, K // 100))] *= 8.0        # a few heavy input channels
    return synth.f32_to_bf16_bits(w)


@pytest.mark.parametrize("cfg", [dict(), dict(block_size=16), dict(exp_min=-15, exp_max=16),
                                 dict(block_size=16, exp_min=-8, exp_max=3)],
                         ids=["default", "b16", "exp5", "b16-clamped"])
def test_weights_match_oracle(cfg):
    q = fb4.Fb4(**cfg)
    ocfg = orc.Config(**cfg)
    for bits in (weight_like(96, 512, 1), edge_blocks(), heavy(33, 96, 41), weight_like(7, 2048 + 32, 2)):
        ref = orc.quantize_weights(bits, FB, ocfg)
        got = q.quantize_weights(to_dev_bf16(bits))
        assert_same_quantized(got, ref, f"weights {cfg}")
    x = to_dev_bf16(weight_like(40, 320, 3))
    ref = orc.quantize_weights(weight_like(40, 320, 3)[:, :256], FB, ocfg)
    assert_same_quantized(q.quantize_weights(x[:, :256]), ref, "weights strided")
    assert q.device_status == 0
    q.close()


def test_exhaustive_choice_never_worse_than_online_choice():
    q = fb4.Fb4()
    bits = weight_like(512, 3072, 5)
    x = to_dev_bf16(bits)
    qw, qa = q.quantize_weights(x), q.quantize(x)
    assert np.array_equal(meta_np(qw.meta) & 0xFF, meta_np(qa.meta) & 0xFF)        # same scale
    xf = x.float().view(512, -1, 32)
    ew = ((q.dequantize(qw).view(512, -1, 32) - xf).double() ** 2).sum(-1)
    ea = ((q.dequantize(qa).view(512, -1, 32) - xf).double() ** 2).sum(-1)
    assert bool((ew <= ea * (1 + 1e-12)).all())
    assert float(ew.sum()) < float(ea.sum())
    q.close()
