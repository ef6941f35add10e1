"""Input generator: deterministic, row-addressable, and shaped as the workloads state."""
import numpy as np

from paper_2603_02883_b200 import synth


def test_rows_are_counter_based():
    w = synth.workloads()["c2"]
    a = synth.activation_rows(w, 100, 4)
    b = synth.activation_rows(w, 102, 1)
    assert np.array_equal(a[2], b[0])
    assert np.array_equal(a, synth.activation_rows(w, 100, 4))


def test_workload_shapes():
    ws = synth.workloads()
    assert (ws["c1"].T, ws["c1"].C) == (256, 3072)
    assert (ws["c2"].T, ws["c2"].C, ws["c2"].n_outlier) == (32760, 3072, 15)
    assert (ws["c5"].T, ws["c5"].C, ws["c5"].n_outlier) == (75600, 12288, 61)
    assert ws["c3"].decomposed and ws["c4"].seda and ws["c5"].decomposed and ws["c5"].seda
    assert ws["c4"].n_clusters == 64 and ws["c5"].n_clusters == 256


def test_c1_distribution_and_outliers():
    w = synth.workloads()["c1"]
    x = synth.bf16_bits_to_f32(synth.activation(w))
    g = synth.channel_gain(w)
    out = np.flatnonzero(g != 1)
    assert len(out) == 8 and np.all(g[out] == 30.0)
    normal = np.delete(x, out, axis=1)
    assert abs(normal.mean()) < 0.01 and abs(normal.std() - 1.0) < 0.01
    assert abs(x[:, out].std() - 30.0) < 1.5


def test_c2_is_heavy_tailed_with_token_scales():
    w = synth.workloads()["c2"]
    x = synth.bf16_bits_to_f32(synth.activation_rows(w, 0, 512)).astype(np.float64)
    g = synth.channel_gain(w)
    x = x[:, g == 1]
    row_scale = np.median(np.abs(x), axis=1) / 0.7649      # median |t_3| = 0.7649
    logs = np.log(row_scale)
    assert abs(logs.mean()) < 0.15 and abs(logs.std() - 1.0) < 0.15
    z = x / row_scale[:, None]
    assert 3.0 < np.mean(np.abs(z) > 3.182) * 100 < 7.0       # P(|t_3| > 3.182) = 5 %


def test_scores_and_clusters():
    w = synth.workloads()["c5"]
    s = synth.scores(w)
    assert s.dtype == np.float32 and s.min() >= 0 and s.max() < 1 and abs(s.mean() - 0.5) < 0.01
    cid, mask = synth.clusters(w)
    assert cid[0] == 0 and cid[-1] == 255 and np.all(np.diff(cid) >= 0) and len(np.unique(cid)) == 256
    fb = synth.STANDIN_FORMATBOOK
    for m in mask:
        tops = sorted(int(fb[d, 7]) for d in range(32) if (int(m) >> d) & 1)
        assert tops == list(range(8, 16))


def test_standin_formatbook_follows_the_rules():
    fb = synth.STANDIN_FORMATBOOK
    assert fb.shape == (32, 8) and np.all(fb[:, 0] == 0) and np.all(np.diff(fb.astype(int), axis=1) > 0)
    tops = fb[:, 7].astype(int)
    assert np.all(np.diff(tops) >= 0)                      # lower id = narrower dynamic range
    counts = [int(np.sum(tops == b)) for b in range(8, 16)]
    assert counts == sorted(counts) and min(counts) >= 1 and sum(counts) == 32
    assert len({tuple(r) for r in fb}) == 32
