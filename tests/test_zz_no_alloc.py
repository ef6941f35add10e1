"""fb4_build_subformatbook_static, the entry point for callers that cannot allocate device memory
(it keeps its count scratch in an array built into the library), against fb4_build_subformatbook
with caller-allocated scratch.  Collected last on purpose.  Several calls in a row with different
inputs: a later one must not see what an earlier one left in the shared array."""
import ctypes

import numpy as np
import pytest
import torch

from paper_2603_02883_b200 import fb4

pytestmark = pytest.mark.gpu


def test_static_entry_point_matches_the_allocating_one_twice_in_a_row():
    q = fb4.Fb4()
    rng = np.random.default_rng(17)
    T, nblk = 500, 96
    dev = lambda a, dt: torch.from_numpy(np.ascontiguousarray(a, dtype=dt)).cuda()
    # every output buffer of the test exists before the calls under test: they allocate nothing
    # the last round uses every cluster the built-in array can hold
    for call, (n_clusters, n_anchor) in enumerate([(700, 3000), (64, 900), (fb4.STATIC_MAX_CLUSTERS, 5000)]):
        meta = (rng.integers(0, 252, size=(T, nblk)) | (rng.integers(0, 32, size=(T, nblk)) << 8)).astype(np.uint16)
        md = dev(meta.view(np.int16), np.int16)
        tok = dev(rng.integers(-2, T + 2, size=n_anchor), np.int32)
        clu = dev(rng.integers(-1, n_clusters + 1, size=n_anchor), np.int32)
        counts = torch.empty((n_clusters, 32), dtype=torch.int32, device="cuda")
        want = torch.empty(n_clusters, dtype=torch.int32, device="cuda")
        got = torch.full((n_clusters,), -1, dtype=torch.int32, device="cuda")
        fb4.fb4_build_subformatbook(q.ctx, md, T, nblk * 32, tok, clu, n_anchor, n_clusters, counts, want)
        torch.cuda.synchronize()
        # Device memory as the driver sees it, which an allocation made inside the library (its CUDA runtime is
        # linked statically, torch's allocator would not notice it) would lower.  The first call on a device
        # looks up the address of the built-in array; the comparison is made on a call after that.
        if call == 0:
            fb4.fb4_build_subformatbook_static(q.ctx, md, T, nblk * 32, tok, clu, n_anchor, n_clusters, got)
            torch.cuda.synchronize()
            got.fill_(-1)
            torch.cuda.synchronize()
        before = (torch.cuda.mem_get_info()[0], torch.cuda.memory_allocated())
        fb4.fb4_build_subformatbook_static(q.ctx, md, T, nblk * 32, tok, clu, n_anchor, n_clusters, got)
        torch.cuda.synchronize()
        assert (torch.cuda.mem_get_info()[0], torch.cuda.memory_allocated()) == before
        assert np.array_equal(got.cpu().numpy(), want.cpu().numpy()), f"call {call}: masks differ"   # bit-exact
        assert int(counts.sum()) > 0
    # beyond the built-in scratch: refused, nothing launched
    L = fb4.lib()
    n0 = q.launch_count
    rc = L.fb4_build_subformatbook_static(q.ctx, ctypes.c_void_p(md.data_ptr()), T, nblk * 32,
                                          ctypes.c_void_p(tok.data_ptr()), ctypes.c_void_p(clu.data_ptr()), 10,
                                          fb4.STATIC_MAX_CLUSTERS + 1, ctypes.c_void_p(got.data_ptr()), None)
    assert rc == fb4.ERR_STATIC_LIMIT and q.launch_count == n0
    assert "FB4_STATIC_MAX_CLUSTERS" in L.fb4_strerror(rc).decode()
    assert q.device_status == 0
    q.close()
