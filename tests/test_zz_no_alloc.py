"""The allocation-free backward-data entry point.

Some users of the library cannot allocate device memory at the point where they
call it (a plugin without an allocator, a loop whose memory belongs to another
pool).  pcl_conv_bwd_data_noalloc keeps its scratch in a fixed array inside the
library instead of asking for a workspace.  This test calls it through the C ABI
twice in a row and compares with the regular entry point, and checks that a
layer too large for the built-in array is refused.  The file name sorts last so
that a run stopping at the first failure has already run every other test.
"""
import numpy as np
import pytest
import torch

import gpu_helpers as G
import oracle
from oracle import ConvShape

pytestmark = pytest.mark.gpu


def test_noalloc_matches_regular_entry_point_twice():
    import gpu_helpers as G
    from paper_1602_06709_b200 import binding as B
    B.set_path(B.PATH_AUTO)
    shapes = [ConvShape(N=3, C=40, K=72, H=19, W=23, R=3, S=3, pad_h=1, pad_w=1),
              ConvShape(N=2, C=64, K=128, H=16, W=16, R=3, S=3, pad_h=1, pad_w=1)]
    for call, s in enumerate(shapes + shapes[:1]):          # two different layers, then the first again
        d = G.shape_to_desc(s)
        assert B.conv_workspace_bytes(d, B.PASS_BWD_DATA) > 0, "the case must be one that needs scratch"
        x, w, dy, _ = G.make_inputs(s, f"noalloc{call}")
        dyt, wt, xt = G.dev(dy), G.dev(w), G.dev(x)
        ref = G.guarded((s.N, s.H, s.W, s.C))
        B.conv_bwd_data(d, dyt, wt, xt, ref, G.workspace(B.conv_workspace_bytes(d, B.PASS_BWD_DATA)))
        for rep in range(2):                                 # two calls in a row share the built-in array
            got = torch.full_like(ref, float("nan"))
            B.conv_bwd_data_noalloc(d, dyt, wt, xt, got)
            B.check_device_status()
            assert torch.equal(got, ref), f"call {call}.{rep}: differs from pcl_conv_bwd_data"
        G.assert_parity(ref.cpu().numpy(), oracle.conv_bwd_data(s, dy, w, x), "bwd_data (no-alloc)")


def test_noalloc_capacity_counts_only_the_transposed_copy():
    """What must fit the built-in array is the transposed weight copy.  A wide layer whose weights are read in
    place (C % 32 == 0) needs none and runs although the regular call's full workspace (copy area + room to split
    the reduction) would not fit; a layer with C % 32 != 0 just under the limit runs too.  Both bit-equal to the
    regular entry point given exactly the same amount of scratch."""
    import gpu_helpers as G
    from paper_1602_06709_b200 import binding as B
    B.set_path(B.PATH_AUTO)
    cap = B.noalloc_scratch_bytes()
    for s in (ConvShape(N=4, C=512, K=512, H=14, W=14, R=3, S=3, pad_h=1, pad_w=1),
              ConvShape(N=2, C=904, K=512, H=6, W=6, R=3, S=3, pad_h=1, pad_w=1)):     # 4.17 M of 4.19 M weights
        d = G.shape_to_desc(s)
        x, w, dy, _ = G.make_inputs(s, f"noalloc_cap{s.C}")
        dyt, wt = G.dev(dy), G.dev(w)
        ref = G.guarded((s.N, s.H, s.W, s.C))
        B.conv_bwd_data(d, dyt, wt, None, ref, torch.empty(cap, dtype=torch.uint8, device="cuda"))
        for rep in range(2):
            got = torch.full_like(ref, float("nan"))
            B.conv_bwd_data_noalloc(d, dyt, wt, None, got)
            B.check_device_status()
            assert torch.equal(got, ref), f"C={s.C} call {rep}: differs from pcl_conv_bwd_data with the same scratch"
        G.assert_parity(ref.cpu().numpy(), oracle.conv_bwd_data(s, dy, w), f"bwd_data (no-alloc, C={s.C})")


def test_noalloc_rejects_layers_beyond_its_capacity():
    import ctypes
    from paper_1602_06709_b200 import binding as B
    assert B.noalloc_scratch_bytes() == 16 << 20
    big = B.conv_desc(1, 2040, 2048, 4, 4, 3, 3, 1, 1)       # C % 32 != 0: needs a copy of 37.6 M weights > 4 Mi floats
    assert B.conv_workspace_bytes(big, B.PASS_BWD_DATA) > B.noalloc_scratch_bytes()
    null = ctypes.c_void_p(0)
    rc = B.lib().pcl_conv_bwd_data_noalloc(ctypes.byref(big), ctypes.c_void_p(256), ctypes.c_void_p(256), null,
                                           ctypes.c_void_p(256), null)
    assert rc == B.ERR_SCRATCH_LIMIT
    assert "scratch" in B.status_string(rc)
