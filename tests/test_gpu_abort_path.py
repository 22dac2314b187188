"""The attention kernel's time-out path, taken once under test without faulting or hanging anything.

Every wait in the kernel is bounded; when one runs out the CTA raises an abort flag, its roles
drain (copies and tensor-core products in flight are waited for, with a bound), tensor memory is
released, the CTA exits and the workspace's status word reports HEART_ERR_DEVICE_CHECK.  The
test-hook build of the library (same sources, HEART_TEST_HOOKS, a wait limit of 2e6 clocks) has one
reserved flag bit that makes the V producer of CTA 0 leave out one copy -- neither the byte count is
announced nor the copy issued -- so the waits that depend on that tile run out after about a
millisecond.  Nothing traps and nothing waits without a bound.
"""
import time

import numpy as np
import pytest
import torch

from paper_2605_14513_b200 import build as heart_build
from paper_2605_14513_b200 import inputs

pytestmark = pytest.mark.gpu

TEST_SKIP_V = 0x80000000


def dense_attention(h, flags, Q, K, V, wl):
    cfg = h.make_config(wl.B, wl.H, wl.N, wl.block, flags=h.FORCE_DENSE | flags)
    ws = h.new_workspace(cfg)
    O = torch.full_like(Q, float("nan"))
    t0 = time.perf_counter()
    h.heart_block_sparse_attn(cfg, Q, K, V, None, None, O, ws)
    status = h.heart_get_status(ws)  # synchronises
    return O, status, time.perf_counter() - t0, (cfg, ws)


def test_a_wait_that_runs_out_is_reported_and_the_context_stays_usable():
    from paper_2605_14513_b200 import heart as h

    assert torch.cuda.is_available()
    product = h.lib()
    hooks = h.load(heart_build.build_test_hooks())
    wl = inputs.small_workload(H=2, grid=(3, 10, 14), block=64, seed=41)  # N = 420: 4 query tiles a head, 7 key steps
    Q, K, V = inputs.Sequence(wl, "cuda").bf16()
    try:
        h._lib = hooks
        O_ref, status, _, _ = dense_attention(h, 0, Q, K, V, wl)
        assert status == 0
        O_bad, status, seconds, (cfg, ws) = dense_attention(h, TEST_SKIP_V, Q, K, V, wl)
        assert status == h.ERR_DEVICE_CHECK          # the wait ran out and said so
        assert seconds < 5.0                          # ... after milliseconds, not the product's 2 s limit
        assert h.heart_get_status(ws) == 0            # the status word is cleared by the read
        # CTA 0 (head 0, query rows 0..127) gave up without writing; every other tile is complete
        ref, bad = O_ref.view(wl.R, wl.N, wl.D), O_bad.view(wl.R, wl.N, wl.D)
        assert torch.isnan(bad[0, :128].float()).all()
        assert torch.equal(bad[0, 128:].view(torch.int16), ref[0, 128:].view(torch.int16))
        assert torch.equal(bad[1].view(torch.int16), ref[1].view(torch.int16))
        # the same workspace and the same context serve a normal call right after, bit for bit
        cfg.flags = h.FORCE_DENSE
        O_again = torch.full_like(Q, float("nan"))
        h.heart_block_sparse_attn(cfg, Q, K, V, None, None, O_again, ws)
        assert h.heart_get_status(ws) == 0
        assert torch.equal(O_again.view(torch.int16), O_ref.view(torch.int16))
    finally:
        h._lib = product
    # the product library has no such hook: the reserved bit changes nothing there
    O_prod, status, _, _ = dense_attention(h, TEST_SKIP_V, Q, K, V, wl)
    assert status == 0
    assert torch.equal(O_prod.view(torch.int16), O_ref.view(torch.int16))
