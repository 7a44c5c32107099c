"""ap_mask_to_tiles_static: the tile-list builder whose scratch space is a fixed
device array inside the library, for callers that are not allowed to allocate
device memory (plugins inside another framework's pool, allocator-free loops).

It must give exactly the tile list ap_mask_to_tiles gives, also on a second call
that finds the previous call's leftovers in the shared array.  This file is
collected last on purpose, so a stop-at-first-failure run has already run every
other test when it gets here.
"""
import ctypes

import numpy as np
import pytest
import torch

from paper_2012_02030_b200 import inputs

FAKE = 0x10000


def test_static_variant_rejects_shapes_beyond_its_scratch_before_touching_a_device():
    from paper_2012_02030_b200 import binding as ap

    t = ap.ap_tiles(16, 4096, 4096, 32, 32, 16384, *([FAKE] * 9))
    assert 16 * 32 * 32 > ap.AP_STATIC_MAX_TILES
    st = ap.lib.ap_mask_to_tiles_static(FAKE, 16, 4096, 4096, ctypes.byref(t), None)
    assert st == ap.AP_ERR_WORKSPACE
    assert "capacity" in ap.status_string(st) or "workspace" in ap.status_string(st)
    assert ap.lib.ap_mask_to_tiles_static(None, 1, 8, 8, ctypes.byref(t), None) == ap.AP_ERR_INVALID_ARG


def test_static_variant_rejects_misaligned_tile_arrays_like_the_workspace_variant():
    """The kernels behind both entry points store 16-byte vectors to bitmap, round_bitmap and
    round_rows and 32-bit words to row_ptr, col_idx and round_ptr: a misaligned array must come back as
    an argument error from the host, not as a misaligned-address fault from the device."""
    from paper_2012_02030_b200 import binding as ap

    names = [f[0] for f in ap.ap_tiles._fields_]
    for field, off in (("bitmap", 8), ("round_bitmap", 4), ("round_rows", 8), ("row_ptr", 2), ("col_idx", 1),
                       ("round_ptr", 2)):
        t = ap.ap_tiles(1, 128, 128, 1, 1, 4, *([FAKE] * 9))
        assert field in names
        setattr(t, field, FAKE + off)
        assert ap.lib.ap_mask_to_tiles_static(FAKE, 1, 128, 128, ctypes.byref(t), None) == ap.AP_ERR_INVALID_ARG, field
        assert ap.lib.ap_mask_to_tiles(FAKE, 1, 128, 128, ctypes.byref(t), FAKE, 1 << 30, None) == \
            ap.AP_ERR_INVALID_ARG, field


@pytest.mark.gpu
def test_static_variant_matches_workspace_variant_on_two_calls_in_a_row():
    from paper_2012_02030_b200 import binding as ap

    # two different shapes and masks back to back: the second call starts from
    # an array that still holds the first call's bitmaps, counts and positions
    cases = [(4, 1024, 1024, 0.02, 101), (3, 300, 700, 0.3, 102), (4, 1024, 1024, 0.001, 103)]
    for call, (H, Lq, Lk, density, seed) in enumerate(cases):
        mask = inputs.random_mask(H, Lq, Lk, density, seed=seed).cuda()
        mask[0, :128, :128] = 1
        want = ap.Tiles(H, Lq, Lk)
        ap.ap_mask_to_tiles(mask, want)
        got = ap.Tiles(H, Lq, Lk)
        before = ap.ap_launch_count()
        torch.cuda.synchronize()
        free_before = torch.cuda.mem_get_info()[0]
        ap.ap_mask_to_tiles_static(mask, got)
        torch.cuda.synchronize()
        # The call takes no device memory.  (Not asserted for the very first call in a process: that
        # one resolves the array's address, and the driver may load the library's code and the array
        # itself onto the device at that moment, which is not an allocation the call makes.)
        if call > 0:
            assert torch.cuda.mem_get_info()[0] == free_before
        assert ap.ap_launch_count() - before == 6  # bitmaps, scan, gather; rounds: count, scan, fill
        assert ap.ap_device_status() == ap.AP_OK
        a, b = got.to_host(), want.to_host()
        for key in ("row_ptr", "col_idx", "flags", "bitmap", "groups", "round_ptr", "round_rows", "round_info",
                    "round_bitmap"):
            np.testing.assert_array_equal(a[key], b[key], err_msg=key)
        assert got.n_tiles() > 0
    # exactly at the limit is accepted, one tile more is refused
    H = ap.AP_STATIC_MAX_TILES // 4
    mask = torch.ones((H, 256, 256), dtype=torch.uint8, device="cuda")
    full = ap.Tiles(H, 256, 256)
    ap.ap_mask_to_tiles_static(mask, full)
    assert ap.ap_device_status() == ap.AP_OK and full.n_tiles() == ap.AP_STATIC_MAX_TILES
    with pytest.raises(ap.ApError) as e:
        ap.ap_mask_to_tiles_static(torch.ones((H + 1, 256, 256), dtype=torch.uint8, device="cuda"),
                                   ap.Tiles(H + 1, 256, 256))
    assert e.value.status == ap.AP_ERR_WORKSPACE
