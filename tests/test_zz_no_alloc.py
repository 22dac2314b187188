"""heart_drift_static: the drift decision for callers that cannot allocate device memory.

Some users of this library run where cudaMalloc is not an option (inside another framework's
allocator-managed region, in a callback that must not block on the driver, or as a plugin that is
given tensors but no scratch).  For them the library carries its own fixed 16 MiB scratch array.
This test drives that entry point through the C ABI and checks that it gives exactly what the
ordinary, caller-allocated heart_drift gives -- on two calls in a row, because the built-in array
is shared by every call and keeps the previous call's contents.

Collected last on purpose (file name), so a failure here cannot hide the other tests in a run
that stops at the first failure.  It passes alone in a fresh process and after the other tests.
"""
import ctypes as C

import numpy as np
import pytest
import torch

from paper_2605_14513_b200 import inputs

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def heart():
    from paper_2605_14513_b200 import heart as h

    h.lib()
    assert torch.cuda.is_available()
    return h


def test_static_scratch_drift_matches_workspace_drift_twice(heart):
    wl = inputs.small_workload(H=3, grid=(3, 10, 14), block=64, seed=31, eps=[0.005, 0.05, 0.3],
                               delta=[0.6, 0.6, 0.6])
    seq = inputs.Sequence(wl, "cuda")
    cfg = heart.make_config(wl.B, wl.H, wl.N, wl.block)
    assert heart.workspace_bytes(cfg) <= heart.STATIC_SCRATCH_BYTES
    st_ws, st_static = heart.State(cfg), heart.State(cfg)
    ws = heart.new_workspace(cfg)
    delta = torch.tensor(wl.delta, dtype=torch.float64, device="cuda")
    seen = []
    for call in range(2):  # two calls in a row: the second one finds the first one's leftovers
        Q, K, _ = seq.bf16()
        d_ws = torch.full((wl.R,), -1.0, dtype=torch.float64, device="cuda")
        d_st = torch.full((wl.R,), -2.0, dtype=torch.float64, device="cuda")
        r_ws = torch.full((wl.R,), 7, dtype=torch.uint8, device="cuda")
        r_st = torch.full((wl.R,), 9, dtype=torch.uint8, device="cuda")
        heart.heart_drift(cfg, Q, K, delta, st_ws, ws, drift_out=d_ws, refresh_out=r_ws)
        heart.heart_drift_static(cfg, Q, K, delta, st_static, drift_out=d_st, refresh_out=r_st)
        torch.cuda.synchronize()
        # same kernels, same order of operations: the two paths must agree to the last bit,
        # which is well inside the 1e-6 relative band the drift tests use
        assert torch.equal(d_ws, d_st), (d_ws, d_st)
        assert torch.equal(r_ws, r_st)
        assert torch.equal(st_ws.anchor_q, st_static.anchor_q) and torch.equal(st_ws.anchor_k, st_static.anchor_k)
        assert torch.equal(st_ws.has_anchor, st_static.has_anchor)
        seen.append((d_st.cpu().numpy().copy(), r_st.cpu().numpy().copy()))
        seq.advance()
    assert np.all(np.isinf(seen[0][0])) and np.all(seen[0][1] == 1)   # first call: no anchors yet
    assert np.all(np.isfinite(seen[1][0])) and np.all(seen[1][0] > 0)  # second call: real drifts
    assert 0 < seen[1][1].sum() < wl.R                                  # a mix of reuse and refresh


def test_static_scratch_rejects_shapes_beyond_its_maximum(heart):
    big = heart.make_config(1, 40, 32760, 64)  # 40 heads x 512 blocks needs ~42 MB of scratch
    assert heart.workspace_bytes(big) > heart.STATIC_SCRATCH_BYTES
    st = heart.StateStruct(256, 256, 256, 0, 0, 0)
    fake = C.c_void_p(256)  # never dereferenced: the size check comes first
    rc = heart.lib().heart_drift_static(C.byref(big), fake, fake, fake, C.byref(st), None, None, None)
    assert rc == heart.ERR_TOO_LARGE
    assert b"scratch" in heart.lib().heart_strerror(rc)
