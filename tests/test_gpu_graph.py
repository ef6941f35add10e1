"""The entry points only enqueue work on the caller's stream (no synchronisation, no allocation per
call), so a whole SeDA + decomposition step can be recorded once into a CUDA graph and replayed on new
data: the replay must equal the oracle on that data."""
import numpy as np
import pytest
import torch

from gpu_util import FB, assert_same_bits_f32, meta_np, to_dev_bf16
from oracle import fb4_oracle as orc
from paper_2603_02883_b200 import fb4, synth

pytestmark = pytest.mark.gpu


def test_recorded_step_replays_on_new_data():
    q = fb4.Fb4()
    T, C, tile, ncl = 240, 2048, 20, 6
    ws = [synth.Workload("g", T=T, C=C, seed=s, kind=1, n_outlier=10, outlier_gain=50.0, seda=True, n_clusters=ncl,
                         cluster_seed=70, score_seed=s + 1) for s in (71, 72)]
    cid_np, _ = synth.clusters(ws[0])
    tok_np, clu_np = synth.anchors(cid_np, ncl, per_cluster=5)
    dev = lambda a: torch.from_numpy(np.ascontiguousarray(a)).cuda()
    x, score = torch.empty((T, C), dtype=torch.bfloat16, device="cuda"), torch.empty(T, dtype=torch.float32, device="cuda")
    cid, tok, clu = dev(cid_np), dev(tok_np), dev(clu_np)
    ns = T // tile
    free_codes = torch.empty((T, C // 2), dtype=torch.uint8, device="cuda")
    free_meta = torch.empty((T, C // 32), dtype=torch.int16, device="cuda")
    counts = torch.empty((ncl, 32), dtype=torch.int32, device="cuda")
    masks = torch.empty(ncl, dtype=torch.int32, device="cuda")
    codes, meta = torch.empty_like(free_codes), torch.empty_like(free_meta)
    sal = torch.empty(ns, dtype=torch.int32, device="cuda")
    rc, rm = torch.empty((ns, C // 2), dtype=torch.uint8, device="cuda"), torch.empty((ns, C // 32), dtype=torch.int16, device="cuda")
    out = torch.empty((T, C), dtype=torch.float32, device="cuda")
    e4m3 = torch.empty((T, C), dtype=torch.uint8, device="cuda")
    sf = torch.empty(fb4.fb4_mxfp8_scale_bytes(T, C, 1), dtype=torch.uint8, device="cuda")

    def step():
        # unconstrained pass -> sub-formatbooks from the anchors -> constrained, decomposed pass -> decode, MXFP8 view
        fb4.fb4_quantize(q.ctx, x, T, C, C, free_codes, free_meta)
        fb4.fb4_build_subformatbook(q.ctx, free_meta, T, C, tok, clu, tok.numel(), ncl, counts, masks)
        fb4.fb4_quantize_decomposed(q.ctx, x, T, C, C, score, tile, cid, masks, ncl, codes, meta, sal, rc, rm)
        fb4.fb4_dequantize(q.ctx, codes, meta, T, C, sal, ns, rc, rm, out, 0)
        fb4.fb4_to_mxfp8(q.ctx, codes, meta, T, C, e4m3, sf, 1)

    x.copy_(to_dev_bf16(synth.activation(ws[0])))
    score.copy_(dev(synth.scores(ws[0])))
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        step()                                   # warm-up outside the capture (first-use set-up)
    torch.cuda.current_stream().wait_stream(side)
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        step()
    for w in ws[::-1]:                            # replay on the second tensor first, then the first again
        bits, sc = synth.activation(w), synth.scores(w)
        x.copy_(to_dev_bf16(bits))
        score.copy_(dev(sc))
        graph.replay()
        torch.cuda.synchronize()
        ref_free = orc.quantize(bits, FB)
        ref_masks = orc.build_subformatbook(ref_free.meta, tok_np, clu_np, ncl, FB)
        ref_sal = orc.select_salient(sc, tile)
        ref = orc.quantize(bits, FB, cluster_id=cid_np, cluster_mask=ref_masks, salient_idx=ref_sal)
        assert np.array_equal(masks.cpu().numpy().view(np.uint32), ref_masks)
        assert np.array_equal(sal.cpu().numpy(), ref_sal)
        assert np.array_equal(codes.cpu().numpy(), ref.codes) and np.array_equal(meta_np(meta), ref.meta)
        assert np.array_equal(rc.cpu().numpy(), ref.res_codes) and np.array_equal(meta_np(rm), ref.res_meta)
        assert_same_bits_f32(out, orc.dequantize(ref, FB), "replayed decode")
        e_ref, s_ref = orc.to_mxfp8(orc.Quantized(ref.codes, ref.meta), FB, 1)
        assert np.array_equal(e4m3.cpu().numpy(), e_ref) and np.array_equal(sf.cpu().numpy(), s_ref)
    assert q.device_status == 0
    q.close()
