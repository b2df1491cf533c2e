"""wush_calib_moments_static: the workspace-free variant of the calibration-moment call.

Some hosts cannot give this library scratch memory at call time (an allocator that owns all
of HBM, allocation switched off after start-up).  For them the library carries a fixed 4 MiB
scratch array and this entry point uses it.  The test calls it through the C ABI twice in a
row - the array is shared and keeps the previous call's contents, so the second call proves
that stale contents do no harm - and compares with the ordinary entry point.  It lives in a
file that sorts last so that a run stopping at the first failure has already run the rest.
"""
import ctypes

import numpy as np
import pytest
import torch

from paper_2512_00956_b200 import synth, wush
from parity_util import dev_bf16, rel_fro

pytestmark = pytest.mark.gpu


# the last case needs more sets of partial sums (6 x 1 MiB) than the 4 MiB array holds: the call then runs
# with 4 token splits on the register-staged kernels
@pytest.mark.parametrize("g,B,K", [(32, 700, 2048), (16, 333, 4096), (32, 2000, 8192)])
def test_static_scratch_matches_workspace_entry_point_twice(g, B, K):
    cfg = synth.CONFIGS[2]
    Xa = dev_bf16(synth.calibration(cfg, B=B, K=K))
    Xb = dev_bf16(synth.activations(cfg, M=B, K=K))            # different data for the second call
    for X in (Xa, Xb):
        ref, ref_cnt = wush.calib_moments(X, g)
        mom = torch.zeros_like(ref)
        cnt = torch.zeros(2, dtype=torch.int64, device="cuda")
        wush.calib_moments_static(X, g, mom, cnt)
        torch.cuda.synchronize()
        assert int(cnt[0].item()) == int(ref_cnt[0].item()) == B
        assert rel_fro(mom.cpu().numpy(), ref.cpu().numpy()) <= 1e-5
        assert float(mom.abs().max()) > 0
    # accumulate-in-place semantics are kept: a second pass over the same tokens doubles the sums
    wush.calib_moments_static(Xb, g, mom, cnt)
    torch.cuda.synchronize()
    assert int(cnt[0].item()) == 2 * B
    assert rel_fro(mom.cpu().numpy(), 2 * ref.cpu().numpy()) <= 1e-5


def test_static_scratch_rejects_oversized_problems():
    L = wush.lib()
    p = ctypes.c_void_p(0x1000)
    # K * g * 4 bytes = 8 MiB > the 4 MiB built-in scratch: refused on the host, nothing launched
    assert L.wush_calib_moments_static(p, 16, 65536, 32, p, p, None) == -5
    assert L.wush_calib_moments_static(p, 16, 64, 24, p, p, None) == -3
    assert L.wush_calib_moments_static(None, 16, 64, 32, p, p, None) == -1
    assert wush.STATIC_SCRATCH_BYTES == 4 << 20
