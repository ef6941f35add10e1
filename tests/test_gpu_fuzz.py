"""Seeded differential test: random shapes, configurations and extensions through the library, every
output compared with the CPU oracle bit for bit.  Each seed draws block size, group count, selection
mode, exponent clamp, token and channel counts (some reach the TMA-staged kernel, some the generic
one), a row stride, arbitrary SeDA masks, per-tile or caller-given salient tokens, and the scale of the
data (zeros, subnormal blocks and huge rows included); then checks codes, metadata, salient indices,
residual tensors and the decoded fp32 / bf16 / half values."""
import numpy as np
import pytest
import torch

from gpu_util import FB, assert_same_bits_f32, assert_same_quantized
from oracle import fb4_oracle as orc
from paper_2603_02883_b200 import fb4, synth

pytestmark = pytest.mark.gpu


def draw(seed):
    rng = np.random.default_rng(1000 + seed)
    B = int(rng.choice([32, 32, 16]))
    cfg = dict(block_size=B, num_groups=int(rng.choice([8, 8, 8, B])), select_mode=int(rng.random() < 0.2))
    clamp = rng.random()
    if clamp < 0.2:
        cfg.update(exp_min=-15, exp_max=16)
    elif clamp < 0.3:
        cfg.update(exp_min=int(rng.integers(-6, 0)), exp_max=int(rng.integers(0, 6)))
    T = int(rng.choice([1, 2, 19, 20, 21, 64, 127, 129, 300]))
    if rng.random() < 0.6:
        C = 64 * int(rng.integers(1, 40))          # the TMA-staged kernel takes multiples of 64
    else:
        C = B * int(rng.integers(1, 50))
    ld = C + 8 * int(rng.integers(0, 4)) if T > 1 else C
    return rng, cfg, T, C, ld


@pytest.mark.parametrize("seed", range(48))
def test_random_configuration_against_the_oracle(seed):
    rng, cfg, T, C, ld = draw(seed)
    B = cfg["block_size"]
    # data: heavy-tailed rows with per-row scales over the whole exponent range, some rows zero or tiny
    f = rng.standard_t(3, size=(T, ld)).astype(np.float32)
    f *= np.exp2(rng.integers(-60, 60, size=(T, 1))).astype(np.float32)
    f[rng.random(T) < 0.1] = 0.0
    f[rng.random(T) < 0.1] *= np.float32(2.0 ** -100)
    f[rng.random((T, ld)) < 0.02] = 0.0
    f[rng.random((T, ld)) < 0.01] *= -1.0
    bits = synth.f32_to_bf16_bits(f)
    view = bits[:, :C]
    seda = rng.random() < 0.5
    n_cl = int(rng.integers(1, 6))
    cid = rng.integers(-1, n_cl, size=T).astype(np.int32) if seda else None
    masks = rng.integers(1, 2 ** 32, size=n_cl, dtype=np.uint64).astype(np.uint32) if seda else None
    if seda and rng.random() < 0.5:        # paper-structured masks: one dialect per dynamic range
        masks = synth.clusters(synth.Workload("f", T=T, C=C, seed=seed, kind=1, n_outlier=0, outlier_gain=1.0,
                                              seda=True, n_clusters=n_cl, cluster_seed=seed))[1]
    mode = rng.choice(["plain", "tile", "given"])
    tile = int(rng.choice([1, 3, 20]))
    score = rng.random(T).astype(np.float32)
    if mode == "tile":
        sal = orc.select_salient(score, tile)
    elif mode == "given":
        sal = np.unique(rng.integers(0, T, size=max(1, T // 4))).astype(np.int32)
    else:
        sal = None
    ocfg = orc.Config(**cfg)
    ref = orc.quantize(view, FB, ocfg, cluster_id=cid, cluster_mask=masks, salient_idx=sal)

    q = fb4.Fb4(**cfg)
    try:
        x = torch.from_numpy(bits.view(np.int16)).cuda().view(torch.bfloat16)[:, :C]
        d_cid = None if cid is None else torch.from_numpy(cid).cuda()
        d_masks = None if masks is None else torch.from_numpy(masks.view(np.int32)).cuda()
        if mode == "plain":
            got = q.quantize(x, d_cid, d_masks)
        elif mode == "tile":
            got = q.quantize_decomposed(x, torch.from_numpy(score).cuda(), tile, cluster_id=d_cid, cluster_mask=d_masks)
        else:
            got = q.quantize_decomposed(x, salient_idx=torch.from_numpy(sal).cuda(), cluster_id=d_cid,
                                        cluster_mask=d_masks)
        what = f"seed {seed}: {cfg} T={T} C={C} ld={ld} seda={seda} mode={mode} kernel={q.last_variant}"
        assert_same_quantized(got, ref, what)
        assert_same_bits_f32(q.dequantize(got), orc.dequantize(ref, FB, B), what)
        for dt, name in ((torch.bfloat16, "bf16"), (torch.float16, "f16")):
            o = q.dequantize(got, dt).view(torch.int16).cpu().numpy().view(np.uint16)
            assert np.array_equal(o, orc.dequantize(ref, FB, B, out_dtype=name)), f"{what} {name}"
        assert q.device_status == 0
    finally:
        q.close()
