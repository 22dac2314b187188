"""GPU parity of the strided antidiagonal block-importance estimator (HEART_ESTIMATOR_ANTIDIAG):
masks against the oracle's definition, bit-exact outside the near-threshold bands of the checker."""
import numpy as np
import pytest
import torch

from paper_2605_14513_b200 import inputs

from parity import Pair, check_attention, check_differing_row, check_masks, mask_bits_u32, to_np

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def heart():
    from paper_2605_14513_b200 import heart as h

    h.lib()
    assert torch.cuda.is_available()
    return h


def antidiag_pair(wl, heart, oracle):
    """A Pair whose config and workspace carry the estimator flag."""
    p = Pair(wl, heart, oracle)
    p.cfg.flags = heart.ESTIMATOR_ANTIDIAG
    p.ws = heart.new_workspace(p.cfg)
    return p


@pytest.mark.parametrize("block,grid,H,B", [
    (64, (3, 10, 14), 3, 1),    # N = 420: 26 full groups + 4 unsampled tokens, ragged last block
    (128, (3, 10, 14), 2, 1),
    (64, (4, 16, 16), 2, 2),    # N = 1024: exact multiple, two batch entries
    (128, (1, 3, 43), 2, 1),    # N = 129: the second block has no full group
    (64, (1, 5, 19), 1, 1),     # N = 95: 5 groups, the last block holds one
    (64, (1, 1, 9), 2, 1),      # N = 9: no full group at all
    (128, (5, 20, 33), 2, 1),   # N = 3300: several column tiles of 256 groups? no: 206 groups, one tile, two row tiles
    (64, (6, 25, 40), 1, 1),    # N = 6000: 375 groups: two column tiles, three row tiles
])
def test_masks_match_the_oracle_in_full(heart, oracle, block, grid, H, B):
    wl = inputs.small_workload(H=H, grid=grid, block=block, seed=3 + block + H, B=B,
                               tau=np.linspace(0.5, 0.97, B * H))
    p = antidiag_pair(wl, heart, oracle)
    heart.heart_predict_mask(p.cfg, p.Q, p.K, p.tau, p.gst, p.ws)
    assert heart.heart_get_status(p.ws) == 0
    oracle.predict_mask_antidiag(p.Qb, p.Kb, wl.block, wl.tau, p.ost)
    ex = check_masks(p.gst, p.ost, range(wl.R), wl.tau,
                     lambda r, I: oracle.antidiag_probs_row(p.Qb, p.Kb, wl.block, r, I))
    assert ex <= max(1, wl.R * wl.n_blocks // 200), ex
    assert int(to_np(p.gst.kv_cnt).min()) >= 1


def test_refresh_flags_and_the_fused_step(heart, oracle):
    """Heads with refresh = 0 keep their masks; heart_step with the flag = drift + this predictor +
    attention over the lists it wrote."""
    wl = inputs.small_workload(H=3, grid=(3, 10, 14), block=64, seed=19, tau=[0.6, 0.8, 0.9])
    p = antidiag_pair(wl, heart, oracle)
    refresh = torch.tensor([1, 0, 1], dtype=torch.uint8, device="cuda")
    heart.heart_predict_mask(p.cfg, p.Q, p.K, p.tau, p.gst, p.ws, refresh=refresh)
    cnt = to_np(p.gst.kv_cnt)
    assert np.all(cnt[1] == 0) and cnt[0].min() >= 1 and cnt[2].min() >= 1
    # the fused step: first step, every head refreshes
    heart.heart_state_reset(p.cfg, p.gst)
    O = torch.full_like(p.Q, float("nan"))
    heart.heart_step(p.cfg, p.Q, p.K, p.V, p.delta, p.tau, p.gst, O, p.ws)
    assert heart.heart_get_status(p.ws) == 0
    oracle.predict_mask_antidiag(p.Qb, p.Kb, wl.block, wl.tau, p.ost)
    assert check_masks(p.gst, p.ost, range(wl.R), wl.tau,
                       lambda r, I: oracle.antidiag_probs_row(p.Qb, p.Kb, wl.block, r, I)) <= 1
    ref = oracle.block_sparse_attn(p.Qb, p.Kb, p.Vb, wl.block, to_np(p.gst.kv_idx), to_np(p.gst.kv_cnt))
    check_attention(to_np(O.float()).astype(np.float64).reshape(wl.R, wl.N, wl.D), ref)
    # the pooled predictor on the same workspace still works (the flag only adds to the workspace)
    p.cfg.flags = 0
    before = to_np(p.gst.kv_cnt).copy()
    heart.heart_predict_mask(p.cfg, p.Q, p.K, p.tau, p.gst, p.ws)
    assert heart.heart_get_status(p.ws) == 0 and not np.array_equal(before, to_np(p.gst.kv_cnt))


@pytest.mark.parametrize("name,n_sample", [("wan1.3b-480p", 96), ("wan14b-720p", 64), ("hunyuan-720p", 64)])
def test_full_size_shapes_on_sampled_rows(heart, oracle, name, n_sample):
    """The benchmark shapes: the GPU predicts every row; the oracle recomputes a seeded sample of
    (head, query block) rows one by one -- first and last block, both block sizes' ragged tails."""
    wl = inputs.workload(name)
    p = antidiag_pair(wl, heart, oracle)
    heart.heart_predict_mask(p.cfg, p.Q, p.K, p.tau, p.gst, p.ws)
    assert heart.heart_get_status(p.ws) == 0
    bits, cnt, idx = mask_bits_u32(p.gst.mask_bits), to_np(p.gst.kv_cnt), to_np(p.gst.kv_idx)
    nb = wl.n_blocks
    rs = np.random.RandomState(5)
    picks = {(0, 0), (wl.R - 1, nb - 1), (0, nb - 1), (wl.R - 1, 0)}
    while len(picks) < n_sample:
        picks.add((int(rs.randint(wl.R)), int(rs.randint(nb))))
    differing = 0
    for r, I in sorted(picks):
        P = oracle.antidiag_probs_row(p.Qb, p.Kb, wl.block, r, I)
        keep, k, _, _ = oracle.top_p(P, wl.tau[r])
        G = set(idx[r, I, :cnt[r, I]].tolist())
        assert len(G) == cnt[r, I]
        assert sum(bin(int(x)).count("1") for x in bits[r, I]) == cnt[r, I]
        Rf = set(np.nonzero(keep)[0].tolist())
        if G != Rf:
            check_differing_row(G, Rf, P, wl.tau[r], nb, (r, I))
            differing += 1
    print(f"[{name}] antidiagonal estimator: {differing} of {len(picks)} sampled rows differ inside the bands; "
          f"density {cnt.mean() / nb:.3f}")
    assert differing <= max(1, n_sample // 16)


def test_strided_layout_and_padded_index_pitch(heart, oracle):
    """Q and K stored [B, N, H, D] and viewed as [B, H, N, D]: the estimator's 5-D tensor maps take
    the strides from the config; the index lists get a padded row pitch."""
    rs = np.random.RandomState(23)
    B, H, N, D, b = 2, 3, 700, 128, 64   # 43 full groups + 12 unsampled tokens
    nb = (N + b - 1) // b
    store = [(torch.randn(B, N, H, D, device="cuda") * 1.5).to(torch.bfloat16) for _ in range(2)]
    Q, K = (s.permute(0, 2, 1, 3) for s in store)
    cfg = heart.config_for(Q, b, idx_stride=nb + 3, flags=heart.ESTIMATOR_ANTIDIAG)
    st, ws = heart.State(cfg), heart.new_workspace(cfg)
    tau_np = rs.uniform(0.5, 0.95, B * H)
    tau = torch.tensor(tau_np, dtype=torch.float64, device="cuda")
    heart.heart_predict_mask(cfg, Q, K, tau, st, ws)
    assert heart.heart_get_status(ws) == 0
    Qb, Kb = (inputs.bits(t.contiguous()) for t in (Q, K))
    ost = oracle.State(B, H, N, D, b, idx_stride=nb + 3)
    oracle.predict_mask_antidiag(Qb, Kb, b, tau_np, ost)
    assert check_masks(st, ost, range(B * H), tau_np, lambda r, I: oracle.antidiag_probs_row(Qb, Kb, b, r, I)) <= 1


def test_host_buffer_step_with_this_estimator(heart, oracle):
    """heart_step_host honours the flag: identical masks, flags and output to heart_step."""
    wl = inputs.small_workload(H=3, grid=(3, 10, 14), block=128, seed=29, steps=2, eps=[0.01, 0.1, 0.3],
                               delta=[0.6, 0.6, 0.6])
    a, b = antidiag_pair(wl, heart, oracle), antidiag_pair(wl, heart, oracle)
    staging = tuple(torch.empty_like(b.Q) for _ in range(4))
    for t in range(2):
        O = torch.full_like(a.Q, float("nan"))
        r1 = torch.empty(wl.R, dtype=torch.uint8, device="cuda")
        heart.heart_step(a.cfg, a.Q, a.K, a.V, a.delta, a.tau, a.gst, O, a.ws, refresh_out=r1)
        host = [x.cpu().contiguous().pin_memory() for x in (b.Q, b.K, b.V)]
        Oh = torch.full(b.Q.shape, float("nan"), dtype=torch.bfloat16).pin_memory()
        rh = torch.full((wl.R,), 7, dtype=torch.uint8).pin_memory()
        heart.heart_step_host(b.cfg, host[0], host[1], host[2], b.delta, b.tau, b.gst, Oh, staging, b.ws, refresh_host=rh)
        torch.cuda.current_stream().synchronize()
        assert heart.heart_get_status(a.ws) == 0 and heart.heart_get_status(b.ws) == 0
        assert np.array_equal(to_np(r1), rh.numpy())
        assert torch.equal(O.cpu().view(torch.int16), Oh.view(torch.int16))
        for x, y in zip(a.gst.tensors(), b.gst.tensors()):
            assert torch.equal(x, y)
        a.advance()
        b.advance()


def test_maximum_block_count_with_this_estimator(heart, oracle):
    """n_b = 1024 at block 64 (4095 groups, 16 column tiles dealt to several CTAs per row tile): sampled rows."""
    wl = inputs.small_workload(H=1, grid=(1, 1, 64 * 1024 - 9), block=64, seed=13, tau=[0.9])
    assert wl.n_blocks == heart.MAX_BLOCKS
    p = antidiag_pair(wl, heart, oracle)
    heart.heart_predict_mask(p.cfg, p.Q, p.K, p.tau, p.gst, p.ws)
    assert heart.heart_get_status(p.ws) == 0
    cnt, idx = to_np(p.gst.kv_cnt), to_np(p.gst.kv_idx)
    differing = 0
    for I in (0, 1, 255, 256, 511, 777, 1022, 1023):
        P = oracle.antidiag_probs_row(p.Qb, p.Kb, wl.block, 0, I)
        keep, k, _, _ = oracle.top_p(P, 0.9)
        G, Rf = set(idx[0, I, :cnt[0, I]].tolist()), set(np.nonzero(keep)[0].tolist())
        if G != Rf:
            check_differing_row(G, Rf, P, 0.9, wl.n_blocks, (0, I))
            differing += 1
    assert differing <= 1
