"""GPU parity: the CUDA path (through the C ABI) against the CPU oracle on the same seeded bytes.

Bars: refresh flags and block masks bit-exact (outside the near-threshold bands counted by the
checkers); drift inside the 1e-6 relative decision band; attention output within max-abs 2e-2 and relative-L2 1e-2.
"""
import numpy as np
import pytest
import torch

from paper_2605_14513_b200 import inputs

from parity import (Pair, check_attention, check_decisions, check_masks, mask_bits_u32, sample_rows,
                    to_np)

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def heart():
    from paper_2605_14513_b200 import heart as h

    h.lib()
    assert torch.cuda.is_available()
    return h


def widen(t):
    return to_np(t.to(torch.float32)).astype(np.float64)


def run_sweep(pair, steps, full_attention=True, n_sample=0, seed=0):
    """Drive both sides `steps` denoising steps; compare everything at every step."""
    wl = pair.wl
    rs = np.random.RandomState(seed)
    exempt_rows = exempt_flags = 0
    max_drift_err = 0.0
    seen_refresh = []
    for t in range(steps):
        O, lse, drift, refresh = pair.gpu_step()
        Oo, lse_o, drift_o, refresh_o = pair.oracle_step(want_O=full_attention)
        exempt_flags += check_decisions(drift, refresh, drift_o, refresh_o, wl.delta)
        assert np.array_equal(refresh, refresh_o), "flag exemption would desynchronise the sweep"
        seen_refresh.append(refresh_o.copy())
        assert np.array_equal(to_np(pair.gst.has_anchor), pair.ost.has_anchor)
        # means: fp64 on both sides except the GPU's fp32 partial sums of <= 8 bf16 values
        for a, b in ((pair.gst.anchor_q, pair.ost.anchor_q), (pair.gst.anchor_k, pair.ost.anchor_k)):
            err = np.abs(to_np(a) - b).max()
            assert err <= 1e-8, f"anchor mean differs by {err}"
        fin = np.isfinite(drift_o)
        if fin.any():
            max_drift_err = max(max_drift_err, float((np.abs(drift[fin] - drift_o[fin]) / np.maximum(drift_o[fin], 1e-300)).max()))
        exempt_rows += check_masks(pair.gst, pair.ost, range(wl.R), wl.tau, pair.probs_row)
        assert np.array_equal(to_np(pair.gst.kv_cnt), pair.ost.kv_cnt), "mask exemption would change the attention"
        Ov = O.view(wl.R, wl.N, wl.D)
        if full_attention:
            check_attention(widen(Ov), Oo)
            assert np.allclose(to_np(lse), lse_o, rtol=2e-3, atol=2e-3)
        elif n_sample:
            rr, II = sample_rows(rs, wl.R, wl.n_blocks, pair.ost.kv_cnt, n_sample)
            ref = pair.oracle.attn_rows(pair.Qb, pair.Kb, pair.Vb, wl.block, pair.ost.kv_idx, pair.ost.kv_cnt, rr, II)
            got = np.full_like(ref, np.nan)
            for n, (r, I) in enumerate(zip(rr, II)):
                rows = widen(Ov[int(r), int(I) * wl.block:(int(I) + 1) * wl.block])
                got[n, :rows.shape[0]] = rows
            valid = ~np.isnan(ref)
            assert np.array_equal(valid, ~np.isnan(got)), "rows past N must stay unwritten"
            check_attention(got, ref, valid)
        if t + 1 < steps:
            pair.advance()
    print(f"[{wl.name}] steps={steps} max rel drift err={max_drift_err:.2e} exempt rows={exempt_rows} flags={exempt_flags}")
    return seen_refresh, exempt_rows, exempt_flags


# ------------------------------------------------------------------ small cases, compared in full
@pytest.mark.parametrize("block,grid,H,B", [
    (64, (3, 10, 14), 3, 1),    # N = 420: 6 full blocks + 36 ragged tokens
    (128, (3, 10, 14), 2, 1),   # N = 420: 3 full blocks + 36
    (64, (2, 9, 13), 2, 2),     # two batch entries (guidance branches), N = 234
    (128, (1, 5, 11), 1, 1),    # N = 55: a single ragged block, one head
    (64, (4, 16, 16), 2, 1),    # N = 1024: exact multiple
])
def test_small_sweeps(heart, oracle, block, grid, H, B):
    wl = inputs.small_workload(H=H, grid=grid, block=block, seed=11 + block + H, steps=4, B=B,
                               eps=np.tile([0.005, 0.3, 0.05], 4)[:B * H],
                               delta=np.full(B * H, 0.8 * np.sqrt(420.0 / (grid[0] * grid[1] * grid[2]))))
    pair = Pair(wl, heart, oracle, idx_pad=5)
    seen, ex_rows, ex_flags = run_sweep(pair, 4)
    assert np.all(seen[0] == 1)
    assert ex_rows == 0 and ex_flags == 0


def test_random_small_shapes(heart, oracle):
    """24 seeded random shapes (both block sizes, ragged token counts, 1-3 heads, one or two batch
    entries, gate on or off, padded index pitch), three steps each, everything compared in full."""
    rs = np.random.RandomState(20260514)
    for case in range(24):
        block = int(rs.choice([64, 128]))
        grid = (int(rs.randint(1, 7)), int(rs.randint(3, 30)), int(rs.randint(3, 44)))
        N = grid[0] * grid[1] * grid[2]
        H, B = int(rs.randint(1, 4)), int(rs.choice([1, 1, 2]))
        R = B * H
        wl = inputs.small_workload(H=H, grid=grid, block=block, seed=int(rs.randint(1, 10000)), steps=3, B=B,
                                   eps=np.exp(rs.uniform(np.log(0.003), np.log(0.3), R)),
                                   tau=rs.uniform(0.3, 0.995, R), delta=np.full(R, 0.8 * np.sqrt(420.0 / N)),
                                   pos_scale=float(rs.choice([0.5, 1.5, 2.0, 2.5, 3.0])))  # 3.0: outputs beyond 4
        pair = Pair(wl, heart, oracle, idx_pad=int(rs.randint(0, 7)),
                    gate=(0.0, 1.0) if rs.rand() < 0.5 else (0.4, 0.8))
        _, ex_rows, ex_flags = run_sweep(pair, 3)
        assert ex_rows == 0 and ex_flags == 0, (case, block, grid, H, B)


def test_tiny_config_in_full(heart, oracle):
    """Config 1: H=2, N=2048, block 64; step 0 both refresh, step 1 only head 1."""
    pair = Pair(inputs.workload("tiny"), heart, oracle)
    seen, ex_rows, ex_flags = run_sweep(pair, 2)
    assert np.array_equal(seen[0], [1, 1]) and np.array_equal(seen[1], [0, 1])
    assert ex_rows == 0 and ex_flags == 0


def test_step_equals_three_calls_and_checkpoint(heart, oracle):
    wl = inputs.small_workload(H=3, grid=(3, 10, 14), block=64, seed=21, steps=4, eps=[0.005, 0.05, 0.3],
                               delta=[1.0, 1.0, 1.0])
    a = Pair(wl, heart, oracle)
    b = Pair(wl, heart, oracle)
    ckpt = None
    for t in range(4):
        O, lse, drift, refresh = a.gpu_step()
        # the same step as three separate calls on the second state
        d2 = torch.empty(wl.R, dtype=torch.float64, device="cuda")
        r2 = torch.empty(wl.R, dtype=torch.uint8, device="cuda")
        heart.heart_drift(b.cfg, b.Q, b.K, b.delta, b.gst, b.ws, drift_out=d2, refresh_out=r2)
        # odd steps reuse the block means heart_drift left in the workspace, even steps recompute them
        heart.heart_predict_mask(b.cfg, b.Q, b.K, b.tau, b.gst, b.ws, refresh=r2, means_valid=bool(t & 1))
        assert heart.heart_get_status(b.ws) == 0
        O2 = torch.full_like(b.Q, float("nan"))
        heart.heart_block_sparse_attn(b.cfg, b.Q, b.K, b.V, b.gst.kv_idx, b.gst.kv_cnt, O2, b.ws)
        assert np.array_equal(drift, to_np(d2)) and np.array_equal(refresh, to_np(r2))
        for x, y in zip(a.gst.tensors(), b.gst.tensors()):
            assert torch.equal(x, y)
        assert torch.equal(O[~O.isnan()], O2[~O2.isnan()]) and torch.equal(O.isnan(), O2.isnan())
        if t == 1:  # checkpoint = copies of the state tensors; resume in a fresh State
            ckpt = a.gst.state_dict()
            fresh = heart.State(a.cfg)
            fresh.load_state_dict(ckpt)
            a.gst = fresh
        a.advance()
        b.advance()


@pytest.mark.parametrize("B,H,flags", [(1, 3, 0), (2, 5, 0), (1, 2, 2), (1, 19, 0)])  # 19 heads: 16 uneven head groups
def test_host_buffer_step_equals_device_step(heart, oracle, B, H, flags):
    """heart_step_host (uploads, per-head-group pipeline, downloads) against heart_step on the same
    bytes: identical O, drift, refresh and state at every step; the last row of flags runs the dense
    warm-up mode."""
    rs = np.random.RandomState(B * 10 + H)
    wl = inputs.small_workload(H=H, B=B, grid=(3, 10, 14), block=64, seed=33, steps=3,
                               eps=list(np.exp(rs.uniform(np.log(0.005), np.log(0.3), B * H))),
                               delta=[0.6] * (B * H))
    a = Pair(wl, heart, oracle)
    b = Pair(wl, heart, oracle)
    staging = tuple(torch.empty_like(b.Q) for _ in range(4))
    for t in range(3):
        O, _, drift, refresh = a.gpu_step(flags=flags, want_lse=False)
        b.cfg.flags = flags
        host = [x.cpu().contiguous().pin_memory() for x in (b.Q, b.K, b.V)]
        Oh = torch.full(b.Q.shape, float("nan"), dtype=torch.bfloat16).pin_memory()
        dh = torch.full((wl.R,), float("nan"), dtype=torch.float64).pin_memory()
        rh = torch.full((wl.R,), 7, dtype=torch.uint8).pin_memory()
        heart.heart_step_host(b.cfg, host[0], host[1], host[2], b.delta, b.tau, b.gst, Oh, staging, b.ws,
                              drift_host=dh, refresh_host=rh)
        torch.cuda.current_stream().synchronize()  # the call's own ordering: no device-wide sync
        assert heart.heart_get_status(b.ws) == 0
        assert np.array_equal(drift, dh.numpy()) and np.array_equal(refresh, rh.numpy())
        Oc = O.cpu()
        assert torch.equal(Oc.view(torch.int16), Oh.view(torch.int16))
        for x, y in zip(a.gst.tensors(), b.gst.tensors()):
            assert torch.equal(x, y)
        a.advance()
        b.advance()


def test_run_to_run_bit_reproducible(heart, oracle):
    wl = inputs.small_workload(H=2, grid=(3, 10, 14), block=64, seed=5)
    outs = []
    for _ in range(2):
        p = Pair(wl, heart, oracle)
        O, lse, drift, refresh = p.gpu_step()
        p.gst_copy = [t.clone() for t in p.gst.tensors()]
        outs.append((O.clone(), drift.copy(), p.gst_copy))
    assert np.array_equal(outs[0][1], outs[1][1])
    assert torch.equal(outs[0][0].view(torch.int16), outs[1][0].view(torch.int16))
    for x, y in zip(outs[0][2], outs[1][2]):
        assert torch.equal(x, y)


def test_identical_inputs_have_exactly_zero_drift(heart, oracle):
    wl = inputs.small_workload(H=2, grid=(3, 10, 14), block=128, seed=6, delta=[0.0, 0.0])
    p = Pair(wl, heart, oracle)
    _, _, d0, r0 = p.gpu_step()
    _, _, d1, r1 = p.gpu_step()  # same tensors again, delta = 0
    assert np.all(np.isinf(d0)) and np.all(r0 == 1)
    assert np.array_equal(d1, [0.0, 0.0]) and np.array_equal(r1, [0, 0])


def test_block_means_valid_flag_is_checked_on_the_device(heart, oracle):
    """HEART_BLOCK_MEANS_VALID with block means that belong to other tensors (or to none): nothing is
    predicted, the state keeps its old masks and the status word reports the mismatch."""
    wl = inputs.small_workload(H=2, grid=(3, 10, 14), block=64, seed=17)
    p = Pair(wl, heart, oracle)
    # a fresh (zeroed) workspace holds no block means at all
    heart.heart_predict_mask(p.cfg, p.Q, p.K, p.tau, p.gst, p.ws, means_valid=True)
    assert heart.heart_get_status(p.ws) == heart.ERR_DEVICE_CHECK
    assert int(p.gst.kv_cnt.sum()) == 0
    # means of (Q, K) are there after heart_drift; claiming them for another K tensor is caught
    heart.heart_drift(p.cfg, p.Q, p.K, p.delta, p.gst, p.ws)
    K2 = p.K.clone()
    heart.heart_predict_mask(p.cfg, p.Q, K2, p.tau, p.gst, p.ws, means_valid=True)
    assert heart.heart_get_status(p.ws) == heart.ERR_DEVICE_CHECK
    assert int(p.gst.kv_cnt.sum()) == 0
    # the honest call works and equals the recomputing call
    heart.heart_predict_mask(p.cfg, p.Q, p.K, p.tau, p.gst, p.ws, means_valid=True)
    assert heart.heart_get_status(p.ws) == 0
    a = [t.clone() for t in p.gst.tensors()]
    heart.heart_predict_mask(p.cfg, p.Q, p.K, p.tau, p.gst, p.ws)
    for x, y in zip(a, p.gst.tensors()):
        assert torch.equal(x, y)
    assert int(p.gst.kv_cnt.min()) >= 1
    # the full-token drift uses the block-mean area as scratch: the means are gone afterwards
    d = torch.empty(wl.R, dtype=torch.float64, device="cuda")
    heart.heart_full_token_drift(p.cfg, p.Q, p.K, p.Q, p.K, d, p.ws)
    heart.heart_predict_mask(p.cfg, p.Q, p.K, p.tau, p.gst, p.ws, means_valid=True)
    assert heart.heart_get_status(p.ws) == heart.ERR_DEVICE_CHECK


# ------------------------------------------------------------------ degenerate thresholds / flags
def test_tau_extremes_and_force_flags(heart, oracle):
    wl = inputs.small_workload(H=5, grid=(3, 10, 14), block=64, seed=8, tau=[1.0, 1e-9, 0.5, 0.0, -1.0])
    p = Pair(wl, heart, oracle)
    O, _, _, _ = p.gpu_step()
    p.oracle_step(want_O=False)
    nb = wl.n_blocks
    cnt = to_np(p.gst.kv_cnt)
    assert np.all(cnt[0] == nb)               # tau = 1 -> dense mask
    assert np.all(cnt[1] == 1)                # tau -> 0+ -> exactly one block
    assert np.all(cnt[3] == 1) and np.all(cnt[4] == 1)  # tau <= 0: still the one largest block
    assert np.array_equal(cnt, p.ost.kv_cnt)
    assert check_masks(p.gst, p.ost, range(5), wl.tau, p.probs_row) == 0
    # dense warm-up step: state untouched, output = dense attention
    before = [t.clone() for t in p.gst.tensors()]
    O, lse, drift, refresh = p.gpu_step(flags=heart.FORCE_DENSE)
    for x, y in zip(before, p.gst.tensors()):
        assert torch.equal(x, y)
    assert np.all(np.isinf(drift)) and np.all(refresh == 0)
    check_attention(widen(O).reshape(wl.R, wl.N, wl.D), oracle.dense_attn(p.Qb, p.Kb, p.Vb))
    # forced refresh overrides a huge delta
    p.delta.fill_(1e30)
    _, _, _, refresh = p.gpu_step(flags=heart.FORCE_REFRESH)
    assert np.all(refresh == 1)
    _, _, _, refresh = p.gpu_step()
    assert np.all(refresh == 0)


def test_uniform_scores_keep_lowest_indices(heart, oracle):
    """Q = 0 makes every block score equal: 32 blocks, tau = 0.9 must keep blocks 0..28."""
    wl = inputs.workload("tiny")
    p = Pair(wl, heart, oracle)
    p.Q = torch.zeros_like(p.Q)
    p.tau.fill_(0.9)
    heart.heart_predict_mask(p.cfg, p.Q, p.K, p.tau, p.gst, p.ws)
    cnt, idx = to_np(p.gst.kv_cnt), to_np(p.gst.kv_idx)
    assert np.all(cnt == 29)
    assert np.array_equal(idx[:, :, :29], np.broadcast_to(np.arange(29), (2, 32, 29)))
    assert np.all(mask_bits_u32(p.gst.mask_bits)[:, :, 0] == (1 << 29) - 1)


def test_many_tied_blocks_around_the_threshold(heart, oracle):
    """100 key blocks of which 90 have identical keys (identical pooled means, so identical weights
    down to the last bit): the threshold falls inside the tie group for the larger tau, more candidates
    share its leading bits than the direct evaluation takes, and ties must enter lowest index first."""
    wl = inputs.small_workload(H=3, grid=(5, 16, 80), block=64, seed=21, tau=[0.3, 0.9, 0.995], pos_scale=0.5)
    assert wl.n_blocks == 100
    p = Pair(wl, heart, oracle)
    K = p.K.clone()
    K[:, :, 640:, :] = K[:, :, 640:704, :].repeat(1, 1, 90, 1)
    p.K, p.Kb = K, inputs.bits(K)
    p.gpu_step(want_lse=False)
    p.oracle_step(want_O=False)
    assert check_masks(p.gst, p.ost, range(wl.R), wl.tau, p.probs_row) == 0
    cnt = to_np(p.gst.kv_cnt)
    assert cnt.min() >= 1 and cnt.max() > 64  # some rows cut inside the tie group, beyond 64 candidates


def test_layer_gate_on_gpu(heart, oracle):
    wl = inputs.small_workload(H=5, grid=(2, 9, 13), block=64, seed=9, eps=[0.3, 0.001, 0.001, 0.001, 0.001],
                               delta=np.full(5, 1.0))
    p = Pair(wl, heart, oracle, gate=(0.4, 0.8))
    seen, _, _ = run_sweep(p, 3, full_attention=False)
    assert np.all(seen[0] == 1)
    assert np.all(seen[1] == 0)  # 1 of 5 heads drifting = 0.2 < 0.4: whole layer reuses
    wl2 = inputs.small_workload(H=5, grid=(2, 9, 13), block=64, seed=9, eps=[0.3, 0.3, 0.3, 0.3, 0.001],
                                delta=np.full(5, 1.0))
    p2 = Pair(wl2, heart, oracle, gate=(0.4, 0.79))
    seen, _, _ = run_sweep(p2, 2, full_attention=False)
    assert np.all(seen[1] == 1)  # 4 of 5 = 0.8 > 0.79: whole layer refreshes


# ------------------------------------------------------------------ attention entry point on its own
def test_attention_with_arbitrary_lists_strides_and_bad_entries(heart, oracle):
    rs = np.random.RandomState(3)
    B, H, N, D, b = 1, 2, 300, 128, 64  # 4 full blocks + 44
    nb = 5
    # [B, N, H, D] storage viewed as [B, H, N, D]: non-contiguous strides
    store = [torch.randn(B, N, H, D, device="cuda").to(torch.bfloat16) for _ in range(3)]
    Q, K, V = (s.permute(0, 2, 1, 3) for s in store)
    cfg = heart.config_for(Q, b, idx_stride=nb + 2)
    ws = heart.new_workspace(cfg)
    idx = np.full((H, nb, nb + 2), -1, np.int32)
    cnt = np.zeros((H, nb), np.int32)
    for r in range(H):
        for I in range(nb):
            k = int(rs.randint(0, nb + 1)) if (r, I) != (0, 0) else 0  # (0,0): empty list
            sel = np.sort(rs.choice(nb, k, replace=False))
            idx[r, I, :k], cnt[r, I] = sel, k
    O = torch.full((B, N, H, D), float("nan"), device="cuda", dtype=torch.bfloat16).permute(0, 2, 1, 3)
    lse = torch.full((H, N), float("nan"), device="cuda")
    heart.heart_block_sparse_attn(cfg, Q, K, V, torch.from_numpy(idx).cuda(), torch.from_numpy(cnt).cuda(), O, ws, lse=lse)
    assert heart.heart_get_status(ws) == 0
    Qb, Kb, Vb = (inputs.bits(t.contiguous()) for t in (Q, K, V))
    ref, lse_ref = oracle.block_sparse_attn(Qb, Kb, Vb, b, idx, cnt, want_lse=True)
    got = widen(O.contiguous()).reshape(H, N, D)
    check_attention(got, ref)
    assert np.all(got[0, :64] == 0) and np.all(np.isneginf(to_np(lse)[0, :64]))
    fin = np.isfinite(lse_ref)
    assert np.allclose(to_np(lse)[fin], lse_ref[fin], rtol=2e-3, atol=2e-3)
    # an out-of-range entry is skipped and reported, nothing faults
    idx[1, 2, 0], cnt[1, 2] = nb + 7, max(cnt[1, 2], 1)
    heart.heart_block_sparse_attn(cfg, Q, K, V, torch.from_numpy(idx).cuda(), torch.from_numpy(cnt).cuda(), O, ws)
    assert heart.heart_get_status(ws) == heart.ERR_DEVICE_CHECK
    assert heart.heart_get_status(ws) == 0  # cleared by the read


def test_state_reset(heart, oracle):
    wl = inputs.small_workload(H=2, grid=(2, 9, 13), block=64, seed=4, delta=[1e9, 1e9])
    p = Pair(wl, heart, oracle)
    p.gpu_step()
    _, _, _, r = p.gpu_step()
    assert np.all(r == 0)
    heart.heart_state_reset(p.cfg, p.gst)
    _, _, d, r = p.gpu_step()
    assert np.all(r == 1) and np.all(np.isinf(d))


# ------------------------------------------------------------------ the benchmark configurations
@pytest.mark.parametrize("name,steps,n_sample", [
    ("wan1.3b-480p", 8, 64),   # eight steps: heads that never, sometimes and always refresh
    ("wan14b-480p", 2, 64),
    ("wan14b-720p", 2, 64),
    ("hunyuan-720p", 2, 64),
])
def test_full_size_configs(heart, oracle, name, steps, n_sample):
    """Full shapes, the launch configuration the benchmark times: drift, decisions and masks in
    full; attention on a seeded sample of query blocks (row 0, the ragged last block, the densest
    and the sparsest row, random others)."""
    wl = inputs.workload(name)
    pair = Pair(wl, heart, oracle)
    seen, ex_rows, ex_flags = run_sweep(pair, steps, full_attention=False, n_sample=n_sample, seed=1)
    assert np.all(seen[0] == 1)
    total_rows = wl.R * wl.n_blocks * steps
    print(f"[{name}] exempt mask rows: {ex_rows} of {total_rows}")
    assert ex_rows <= max(1, int(1e-3 * total_rows)) and ex_flags == 0
    dens = pair.ost.kv_cnt.mean() / wl.n_blocks
    assert 0.03 < dens < 0.5


# ------------------------------------------------------------------ size limits
def test_maximum_block_count(heart, oracle):
    """n_b = 1024 (the largest supported): N = 64 * 1024 - 9 tokens at block 64, one head.  Masks and
    decisions in full, attention on sampled query blocks."""
    wl = inputs.small_workload(H=1, grid=(1, 1, 64 * 1024 - 9), block=64, seed=13, tau=[0.9], eps=[0.05],
                               delta=[0.01])
    assert wl.n_blocks == heart.MAX_BLOCKS
    pair = Pair(wl, heart, oracle)
    seen, ex_rows, ex_flags = run_sweep(pair, 2, full_attention=False, n_sample=6, seed=2)
    assert ex_rows == 0 and ex_flags == 0
    cfg = heart.make_config(1, 1, 64 * 1024 + 1, 64)  # one block too many
    assert heart.workspace_bytes(cfg) == 0


@pytest.mark.parametrize("N,block", [(1, 64), (63, 64), (65, 128), (129, 128)])
def test_tiny_token_counts(heart, oracle, N, block):
    """Fewer tokens than a block, one token more than a block: ragged tiles everywhere."""
    wl = inputs.small_workload(H=2, grid=(1, 1, N), block=block, seed=N, tau=[0.7, 1.0], eps=[0.3, 0.3],
                               delta=[0.0, 0.0])
    pair = Pair(wl, heart, oracle)
    seen, ex_rows, ex_flags = run_sweep(pair, 2)
    assert np.all(seen[0] == 1) and np.all(seen[1] == 1)  # delta = 0 and moving inputs: always refresh
    assert ex_rows == 0 and ex_flags == 0
