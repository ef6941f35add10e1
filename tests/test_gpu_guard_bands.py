"""Out-of-bounds writes: every output buffer of every entry point sits between two guard bands
filled with a known byte; after the call the bands must be untouched.  Shapes are chosen ragged
(odd token counts, channel counts that end inside a tile, strided rows)."""
import numpy as np
import pytest
import torch

from paper_2603_02883_b200 import fb4, synth

pytestmark = pytest.mark.gpu

GUARD = 4096          # bytes on either side
FILL = 0xA5


class Guarded:
    """A device buffer of `nbytes` usable bytes, 256-byte aligned, between two guard bands."""

    def __init__(self, nbytes: int):
        self.n = nbytes
        self.raw = torch.full((GUARD + nbytes + GUARD + 256,), FILL, dtype=torch.uint8, device="cuda")
        off = (-self.raw.data_ptr() - GUARD) % 256
        self.lo = off
        self.view = self.raw[off + GUARD: off + GUARD + nbytes]
        assert self.view.data_ptr() % 256 == 0

    def tensor(self, dtype, shape):
        return self.view.view(dtype).view(shape)

    def check(self, what):
        a = self.raw[: self.lo + GUARD]
        b = self.raw[self.lo + GUARD + self.n:]
        assert bool((a == FILL).all()) and bool((b == FILL).all()), f"guard band of {what} was written"


SHAPES = [(1, 32), (3, 96), (37, 64), (19, 1024), (5, 1024 + 64), (130, 3072), (7, 12288 + 128), (2368, 64),
          (2373, 2048)]      # the last one is large enough for the grids of the flat producer kernels


@pytest.mark.parametrize("T,C", SHAPES)
@pytest.mark.parametrize("B", [32, 16])
def test_all_entry_points_stay_inside_their_buffers(T, C, B):
    if C % B:
        pytest.skip("C not a multiple of the block size")
    q = fb4.Fb4(block_size=B)
    w = synth.Workload("g", T=T, C=C, seed=T + C, kind=1, n_outlier=1, outlier_gain=50.0, seda=True,
                       n_clusters=min(3, T), cluster_seed=1, score_seed=2)
    x = torch.from_numpy(synth.activation(w).view(np.int16)).cuda().view(torch.bfloat16)
    score = torch.from_numpy(synth.scores(w)).cuda()
    cid_np, mask_np = synth.clusters(w)
    cid, cmask = torch.from_numpy(cid_np).cuda(), torch.from_numpy(mask_np.view(np.int32)).cuda()
    tile = 4
    ns = -(-T // tile)
    codes, meta = Guarded(T * C // 2), Guarded(T * (C // B) * 2)
    rc, rm, sal = Guarded(ns * C // 2), Guarded(ns * (C // B) * 2), Guarded(ns * 4)
    c_t, m_t = codes.tensor(torch.uint8, (T, C // 2)), meta.tensor(torch.int16, (T, C // B))
    rc_t, rm_t, sal_t = rc.tensor(torch.uint8, (ns, C // 2)), rm.tensor(torch.int16, (ns, C // B)), sal.tensor(torch.int32, (ns,))
    outs = [codes, meta, rc, rm, sal]

    def check(what):
        torch.cuda.synchronize()
        for g, n in zip(outs, ("codes", "meta", "res_codes", "res_meta", "salient_idx")):
            g.check(f"{n} after {what}")

    for variant in (0, 1):
        q.set_kernel_variant(variant)
        fb4.fb4_quantize(q.ctx, x, T, C, C, c_t, m_t)
        check(f"quantize v{variant}")
        fb4.fb4_quantize_seda(q.ctx, x, T, C, C, cid, cmask, cmask.numel(), c_t, m_t)
        check(f"quantize_seda v{variant}")
        fb4.fb4_quantize_decomposed(q.ctx, x, T, C, C, score, tile, cid, cmask, cmask.numel(), c_t, m_t, sal_t, rc_t, rm_t)
        check(f"quantize_decomposed v{variant}")
        xf = x.float()
        fb4.fb4_quantize_f32(q.ctx, xf, T, C, C, c_t, m_t)
        check(f"quantize_f32 v{variant}")
    fb4.fb4_quantize_weights(q.ctx, x, T, C, C, c_t, m_t)
    check("quantize_weights")
    if C >= 128:      # strided rows: only the first half of the channels
        h = C // 2 // B * B
        if h:
            hc, hm = Guarded(T * h // 2), Guarded(T * (h // B) * 2)
            fb4.fb4_quantize(q.ctx, x, T, h, C, hc.tensor(torch.uint8, (T, h // 2)), hm.tensor(torch.int16, (T, h // B)))
            torch.cuda.synchronize()
            hc.check("codes, strided input")
            hm.check("meta, strided input")
    vec = torch.randn(C, device="cuda").to(torch.bfloat16)
    ac, am = Guarded(T * C // 2), Guarded(T * (C // B) * 2)
    fb4.fb4_quantize_affine(q.ctx, x, T, C, C, vec, vec, 1, cid, cmask, cmask.numel(),
                            ac.tensor(torch.uint8, (T, C // 2)), am.tensor(torch.int16, (T, C // B)))
    torch.cuda.synchronize()
    ac.check("codes, affine producer")
    am.check("meta, affine producer")
    fb4.fb4_quantize_decomposed(q.ctx, x, T, C, C, score, tile, None, None, 0, c_t, m_t, sal_t, rc_t, rm_t)
    for dt, bpe in ((torch.float32, 4), (torch.bfloat16, 2)):
        out = Guarded(T * C * bpe)
        fb4.fb4_dequantize(q.ctx, c_t, m_t, T, C, sal_t, ns, rc_t, rm_t, out.tensor(dt, (T, C)), 0 if bpe == 4 else 1)
        torch.cuda.synchronize()
        out.check(f"dequantize {dt}")
    if B == 32:
        for layout in (0, 1):
            e8, sc = Guarded(T * C), Guarded(fb4.fb4_mxfp8_scale_bytes(T, C, layout))
            fb4.fb4_to_mxfp8(q.ctx, c_t, m_t, T, C, e8.view, sc.view, layout)
            torch.cuda.synchronize()
            e8.check(f"e4m3 layout {layout}")
            sc.check(f"scales layout {layout}")
            if C % 64 == 0 and B == 32:   # producer + quantizer + MXFP8 view in one pass (default configuration only)
                e8, sc = Guarded(T * C), Guarded(fb4.fb4_mxfp8_scale_bytes(T, C, layout))
                fb4.fb4_quantize_affine_mxfp8(q.ctx, x, T, C, C, vec, vec, 1, cid, cmask, cmask.numel(), e8.view, sc.view,
                                              layout)
                torch.cuda.synchronize()
                e8.check(f"affine MXFP8, e4m3, layout {layout}")
                sc.check(f"affine MXFP8, scales, layout {layout}")
            if C % 64 == 0 and B == 32:   # the one-pass form with residual rows (default configuration only)
                e8, sc = Guarded(T * C), Guarded(fb4.fb4_mxfp8_scale_bytes(T, C, layout))
                r8, rs = Guarded(ns * C), Guarded(fb4.fb4_mxfp8_scale_bytes(ns, C, layout))
                si = Guarded(ns * 4)
                fb4.fb4_quantize_mxfp8_decomposed(q.ctx, x, T, C, C, score, tile, si.tensor(torch.int32, (ns,)), 0,
                                                  cid, cmask, cmask.numel(), e8.view, sc.view, r8.view, rs.view, layout)
                torch.cuda.synchronize()
                for g, what in ((e8, "e4m3"), (sc, "scales"), (r8, "residual e4m3"), (rs, "residual scales"),
                                (si, "salient indices")):
                    g.check(f"one-pass decomposed MXFP8, {what}, layout {layout}")
    ncl = cmask.numel()
    cnt, msk = Guarded(ncl * 32 * 4), Guarded(ncl * 4)
    tok = torch.arange(0, T, max(1, T // 5), dtype=torch.int32, device="cuda")
    fb4.fb4_build_subformatbook(q.ctx, m_t, T, C, tok, cid[tok.long()].contiguous(), tok.numel(), ncl,
                                cnt.tensor(torch.int32, (ncl, 32)), msk.tensor(torch.int32, (ncl,)))
    torch.cuda.synchronize()
    cnt.check("subformatbook counts")
    msk.check("subformatbook masks")
    assert q.device_status == 0
    q.close()
