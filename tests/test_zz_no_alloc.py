"""The allocation-free global-mask entry point, obc_select_global_mask_static.

Some users of the library may not allocate device memory when they need the global step: their host application
gave the whole GPU to its own pool at start-up, or a cudaMalloc in their running loop is not acceptable.  For them
the library carries a fixed scratch array in its device image.  This test calls that entry point through the C ABI
twice in a row (the array keeps the first call's contents, so the second call checks that nothing stale leaks
through) and requires bit-identical results to the workspace-taking entry point.  This file sorts last so that a
run stopping at the first failure has already exercised every other test.
"""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu


def _case(rng, R, d):
    L = rng.exponential(size=(R, d)).astype(np.float32)
    L[rng.uniform(size=L.shape) < 0.15] = np.float32(0.25)      # exact ties across rows
    P = np.stack([rng.permutation(d) for _ in range(R)]).astype(np.int32)
    return torch.from_numpy(L).cuda(), torch.from_numpy(P).cuda()


def test_static_scratch_matches_workspace_entry_point_twice_in_a_row():
    import paper_2208_11580_b200 as obc
    obc.load_library()
    rng = np.random.default_rng(123)
    # two different problems back to back: the second is smaller, so stale keys of the first lie beyond it
    for R, d, frac in [(300, 577, 0.6), (64, 96, 0.35), (300, 577, 0.0), (7, 9, 1.0)]:
        L, P = _case(rng, R, d)
        k = int(round(frac * R * d))
        want_c = torch.full((R,), -1, dtype=torch.int32, device="cuda")
        want_m = torch.full((R, d), 7, dtype=torch.uint8, device="cuda")
        obc.obc_select_global_mask(L, P, k, want_c, want_m)
        for rep in range(2):
            got_c = torch.full((R,), -2, dtype=torch.int32, device="cuda")
            got_m = torch.full((R, d), 9, dtype=torch.uint8, device="cuda")
            torch.cuda.synchronize()
            free_before = torch.cuda.mem_get_info()[0]
            obc.obc_select_global_mask_static(L, P, k, got_c, got_m)
            torch.cuda.synchronize()
            if rep == 1:      # (the very first call on a device may load the device image; later calls take nothing)
                assert torch.cuda.mem_get_info()[0] == free_before
            assert torch.equal(got_c, want_c) and torch.equal(got_m, want_m)
        assert int(want_c.sum()) == k


def test_static_scratch_rejects_sizes_beyond_its_limit():
    import paper_2208_11580_b200 as obc
    R, d = 2049, 2048                     # 2049 * 2048 entries > OBC_SELECT_STATIC_MAX_KEYS
    L = torch.zeros(R, d, dtype=torch.float32, device="cuda")
    P = torch.zeros(R, d, dtype=torch.int32, device="cuda")
    c = torch.full((R,), -5, dtype=torch.int32, device="cuda")
    m = torch.full((R, d), 3, dtype=torch.uint8, device="cuda")
    with pytest.raises(obc.OBCError) as ei:
        obc.obc_select_global_mask_static(L, P, 10, c, m)
    assert ei.value.status == 9 and "scratch" in str(ei.value)
    torch.cuda.synchronize()
    assert int((c != -5).sum()) == 0 and int((m != 3).sum()) == 0       # nothing was launched or written
