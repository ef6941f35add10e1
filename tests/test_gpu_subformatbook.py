"""GPU parity of the SeDA sub-formatbook construction (Sec. 3.4 bin-count profiling) against the
CPU oracle: cluster masks and per-cluster dialect counts, bit for bit."""
import ctypes

import numpy as np
import pytest
import torch

from gpu_util import FB, meta_np, to_dev_bf16
from oracle import fb4_oracle as orc
from paper_2603_02883_b200 import fb4, synth

pytestmark = pytest.mark.gpu


def dev_i32(a):
    return torch.from_numpy(np.ascontiguousarray(a, dtype=np.int32)).cuda()


def expected_counts(meta, tok, clu, n_clusters):
    T = meta.shape[0]
    cnt = np.zeros((n_clusters, 32), dtype=np.int64)
    for t, c in zip(tok, clu):
        if 0 <= t < T and 0 <= c < n_clusters:
            cnt[c] += np.bincount((meta[t] >> 8) & 31, minlength=32)
    return cnt


@pytest.fixture(scope="module")
def q32():
    q = fb4.Fb4()
    yield q
    assert q.device_status == 0
    q.close()


def run(q, meta_dev, tok, clu, n_clusters):
    masks, counts = q.build_subformatbook(meta_dev, dev_i32(tok), dev_i32(clu), n_clusters)
    torch.cuda.synchronize()
    return masks.cpu().numpy().view(np.uint32), counts.cpu().numpy().view(np.uint32)


def test_c4_workload_closes_the_seda_loop(q32):
    """Quantize unconstrained, build every cluster's sub-formatbook from its anchors, quantize the
    tensor again under those sub-formatbooks: both steps equal the oracle's."""
    w = synth.workloads()["c4"]
    bits = synth.activation(w)
    cid, _ = synth.clusters(w)
    tok, clu = synth.anchors(cid, w.n_clusters, per_cluster=16)
    x = to_dev_bf16(bits)
    free = q32.quantize(x)
    ref_free = orc.quantize(bits, FB)
    assert np.array_equal(meta_np(free.meta), ref_free.meta)
    masks, counts = run(q32, free.meta, tok, clu, w.n_clusters)
    want = orc.build_subformatbook(ref_free.meta, tok, clu, w.n_clusters, FB)
    assert np.array_equal(masks, want)
    assert np.array_equal(counts.astype(np.int64), expected_counts(ref_free.meta, tok, clu, w.n_clusters))
    for m in masks:
        assert sorted(int(FB[d, 7]) for d in range(32) if (int(m) >> d) & 1) == list(range(8, 16))
    got = q32.quantize(x, torch.from_numpy(cid).cuda(), torch.from_numpy(masks.view(np.int32)).cuda())
    ref = orc.quantize(bits, FB, cluster_id=cid, cluster_mask=want)
    assert np.array_equal(meta_np(got.meta), ref.meta) and np.array_equal(got.codes.cpu().numpy(), ref.codes)


def test_edge_cases(q32):
    rng = np.random.default_rng(5)
    T, nblk, n_clusters = 300, 37, 9              # ragged row length
    meta = (rng.integers(0, 252, size=(T, nblk)) | (rng.integers(0, 32, size=(T, nblk)) << 8)).astype(np.uint16)
    meta[:40, :] = (meta[:40, :] & 0xFF) | (5 << 8)             # a block of rows with one dialect only
    md = torch.from_numpy(meta.view(np.int16)).cuda()
    tok = rng.integers(-3, T + 3, size=500)       # duplicates, and ids outside the tensor
    clu = rng.integers(-1, n_clusters + 1, size=500)
    clu[clu == 4] = 3                             # cluster 4 has no anchors
    masks, counts = run(q32, md, tok, clu, n_clusters)
    assert np.array_equal(masks, orc.build_subformatbook(meta, tok, clu, n_clusters, FB))
    assert np.array_equal(counts.astype(np.int64), expected_counts(meta, tok, clu, n_clusters))
    lowest = sum(1 << d for d in (0, 2, 4, 7, 10, 14, 19, 25))
    assert int(masks[4]) == lowest
    # no anchors at all; a second call on the same scratch must not see the first call's counts
    masks0, counts0 = run(q32, md, np.zeros(0, np.int32), np.zeros(0, np.int32), n_clusters)
    assert np.all(masks0 == lowest) and not counts0.any()
    L = fb4.lib()
    p = lambda t: ctypes.c_void_p(t.data_ptr())
    c32 = torch.empty((n_clusters, 32), dtype=torch.int32, device="cuda")
    m32 = torch.empty(n_clusters, dtype=torch.int32, device="cuda")
    a = dev_i32([1, 2])
    assert L.fb4_build_subformatbook(q32.ctx, p(md), T, nblk * 32, p(a), p(a), 2, n_clusters, None, p(m32), None) \
        == fb4.ERR_INVALID_ARG
    assert L.fb4_build_subformatbook(q32.ctx, p(md), T, nblk * 32 + 8, p(a), p(a), 2, n_clusters, p(c32), p(m32), None) \
        == fb4.ERR_SHAPE
    assert L.fb4_build_subformatbook(q32.ctx, p(md), T, nblk * 32, p(a), p(a), -1, n_clusters, p(c32), p(m32), None) \
        == fb4.ERR_INVALID_ARG
    assert L.fb4_build_subformatbook(q32.ctx, None, T, nblk * 32, None, None, 0, 0, None, None, None) == fb4.OK


def test_custom_stage1_and_block16():
    s1 = np.array([0x0000FFFF] * 16 + [0xFFFF0000] * 16, dtype=np.uint32)
    q = fb4.Fb4(block_size=16, stage1_mask=s1)
    w = synth.Workload("t", T=200, C=256, seed=3, kind=1, n_outlier=1, outlier_gain=50.0, seda=True, n_clusters=5,
                       cluster_seed=6)
    bits = synth.activation(w)
    cid, _ = synth.clusters(w)
    tok, clu = synth.anchors(cid, 5, per_cluster=6)
    ref = orc.quantize(bits, FB, orc.Config(block_size=16), stage1=s1)
    got = q.quantize(to_dev_bf16(bits))
    assert np.array_equal(meta_np(got.meta), ref.meta)
    masks, _ = run(q, got.meta, tok, clu, 5)
    assert np.array_equal(masks, orc.build_subformatbook(ref.meta, tok, clu, 5, FB, stage1=s1))
    assert all(bin(int(m)).count("1") == 2 for m in masks)
    q.close()
