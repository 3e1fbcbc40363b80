"""rr_random_read_static: the read entry point for callers that cannot allocate device memory
(a plugin inside another framework's memory pool, code loaded after the application has taken
all of HBM).  Its scratch is a fixed array inside the library, so what has to be shown is that
it gives bit-identical checksums to rr_random_read, and still does on a second call that finds
the first call's claims and records in that array.  Collected last on purpose."""
import ctypes

import numpy as np
import pytest

from paper_2405_11425_b200 import binding as rr
from paper_2405_11425_b200 import build as rr_build

FAKE = 0x7F0000000000


def test_requests_beyond_the_built_in_scratch_are_refused_before_any_launch():
    rr_build.build()
    lib = rr._load()
    g = np.zeros(200, np.uint16)
    p = rr.ReadParams(FAKE, 1 << 20, warps_per_sm=8, reads_per_warp=4, nsm=200, group_of_sm=g,
                      windows=[[0, 8]])
    assert lib.rr_random_read_static(ctypes.byref(p.c), FAKE, None, 0) == rr.RR_ERR_STATIC_LIMIT
    p = rr.ReadParams(FAKE, 1 << 20, W=3, reads_per_warp=4)
    assert lib.rr_random_read_static(ctypes.byref(p.c), FAKE, None, 0) == rr.RR_ERR_ARG
    assert "192 SMs" in rr.rr_strerror(rr.RR_ERR_STATIC_LIMIT)


@pytest.mark.gpu
def test_static_scratch_read_equals_the_allocating_entry_point_twice_in_a_row():
    import torch

    import rr_inputs
    rr_build.build()
    torch.cuda.set_device(0)
    nsm = rr.rr_device_info()["nsm_prop"]
    region = 256 << 20
    buf = torch.empty(region, dtype=torch.uint8, device="cuda")
    rr.rr_fill(buf, region // 4)
    scratch = torch.zeros(rr.rr_scratch_bytes(), dtype=torch.uint8, device="cuda")

    def both(params, n):
        ref = torch.full((n, 2), 0x11111111, dtype=torch.int32, device="cuda")
        got = torch.full((n, 2), 0x22222222, dtype=torch.int32, device="cuda")
        r_ref = rr.rr_random_read(params, ref, scratch)
        r_got = rr.rr_random_read_static(params, got)
        assert torch.equal(ref, got)                      # integer checksums: bit exact
        assert r_got.bytes == r_ref.bytes and r_got.sms_covered == r_ref.sms_covered
        assert r_got.blocks_run == r_ref.blocks_run and r_got.status == 0
        assert r_got.seconds_event == 0.0 and r_got.seconds_device > 0
        return got

    # call 1: grouped per-SM read with some SMs inactive
    groups = rr_inputs.synthetic_group_map(nsm, 5, seed=3, inactive_frac=0.2)
    windows, _ = rr.rr_make_windows(region, 1, region // 5, 5)
    p1 = rr.ReadParams(buf, region, W=1, warps_per_sm=16, reads_per_warp=77, seed=23,
                       group_of_sm=groups, windows=windows)
    both(p1, nsm * 16)
    # call 2, straight after: every SM active, other width; stale claims would leave SMs unserved
    p2 = rr.ReadParams(buf, region, W=4, warps_per_sm=32, reads_per_warp=40, seed=7)
    both(p2, nsm * 32)
    # call 3: logical mode, queued without a report, then read back
    p3 = rr.ReadParams(buf, region, W=2, mode=rr.RR_MODE_LOGICAL, n_warps=3000, reads_per_warp=19,
                       seed=1)
    ref = torch.zeros((3000, 2), dtype=torch.int32, device="cuda")
    got = torch.zeros((3000, 2), dtype=torch.int32, device="cuda")
    rr.rr_random_read(p3, ref, scratch)
    assert rr.rr_random_read_static(p3, got, report=False) is None
    torch.cuda.synchronize()
    assert torch.equal(ref, got)
