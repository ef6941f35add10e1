"""Row sharding over two ranks (gloo, CPU): every rank runs the quantizer's definition (the CPU
oracle) on its shard with decomposition and SeDA on; gathered, the shards must equal the
unsharded result bit for bit.  This is the host-side logic of the multi-GPU path; there is no
collective on the data path itself (the gather below only serves the comparison)."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from oracle import fb4_oracle as orc
from paper_2603_02883_b200 import shard, synth

FB = synth.STANDIN_FORMATBOOK
W = synth.Workload("shard", T=250, C=256, seed=11, kind=1, n_outlier=2, outlier_gain=50.0, decomposed=True, tile=20,
                   score_seed=12, seda=True, n_clusters=7, cluster_seed=13)


def test_row_shard_covers_and_aligns():
    for T, world, align in [(250, 2, 20), (75600, 8, 20), (7, 4, 20), (0, 3, 1), (100, 3, 1), (41, 2, 20)]:
        cuts = [shard.row_shard(T, world, r, align) for r in range(world)]
        assert cuts[0][0] == 0 and cuts[-1][1] == T
        for (a0, a1), (b0, b1) in zip(cuts, cuts[1:]):
            assert a1 == b0 and a0 <= a1
        assert all(c0 % align == 0 for c0, c1 in cuts if c1 > c0)
        sizes = [c1 - c0 for c0, c1 in cuts]
        assert max(sizes) - min(sizes) < 2 * align
    with pytest.raises(ValueError):
        shard.row_shard(10, 2, 2)


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        r0, r1 = shard.row_shard(W.T, world, rank, W.tile)
        bits = synth.activation_rows(W, r0, r1 - r0)           # each rank makes only its own rows
        score = synth.scores(W)[r0:r1]
        cid, masks = synth.clusters(W)
        sal = orc.select_salient(score, W.tile)
        q = orc.quantize(bits, FB, cluster_id=cid[r0:r1], cluster_mask=masks, salient_idx=sal)
        mine = dict(r0=r0, codes=q.codes, meta=q.meta, sal=shard.local_salient_to_global(sal, r0),
                    res_codes=q.res_codes, res_meta=q.res_meta)
        gathered = [None] * world
        dist.all_gather_object(gathered, mine)
        if rank == 0:
            torch.save(gathered, out)
    finally:
        dist.destroy_process_group()


def test_two_rank_shards_equal_the_unsharded_result(tmp_path):
    world = 2
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    out = str(tmp_path / "gathered.pt")
    mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
    parts = sorted(torch.load(out, weights_only=False), key=lambda p: p["r0"])
    bits = synth.activation(W)
    cid, masks = synth.clusters(W)
    sal = orc.select_salient(synth.scores(W), W.tile)
    ref = orc.quantize(bits, FB, cluster_id=cid, cluster_mask=masks, salient_idx=sal)
    assert np.array_equal(np.concatenate([p["codes"] for p in parts]), ref.codes)
    assert np.array_equal(np.concatenate([p["meta"] for p in parts]), ref.meta)
    assert np.array_equal(np.concatenate([p["sal"] for p in parts]), sal)
    assert np.array_equal(np.concatenate([p["res_codes"] for p in parts]), ref.res_codes)
    assert np.array_equal(np.concatenate([p["res_meta"] for p in parts]), ref.res_meta)
