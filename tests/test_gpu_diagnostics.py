"""GPU parity of the two analysis quantities (full-token drift, block-mask IoU) against the oracle."""
import numpy as np
import pytest
import torch

from paper_2605_14513_b200 import inputs

from parity import DRIFT_RTOL, Pair, to_np

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def heart():
    from paper_2605_14513_b200 import heart as h

    h.lib()
    assert torch.cuda.is_available()
    return h


def two_steps(wl, device="cuda"):
    seq = inputs.Sequence(wl, device)
    a = [t.to(device) for t in seq.bf16()]
    seq.advance()
    b = [t.to(device) for t in seq.bf16()]
    return a, b


def gpu_full_drift(heart, cfg, ws, Qa, Ka, Qb, Kb, R):
    out = torch.full((R,), float("nan"), dtype=torch.float64, device="cuda")
    heart.heart_full_token_drift(cfg, Qa, Ka, Qb, Kb, out, ws)
    torch.cuda.synchronize()
    return to_np(out)


@pytest.mark.parametrize("block,grid,H,B", [
    (64, (3, 10, 14), 3, 1),   # N = 420, ragged
    (128, (1, 5, 11), 1, 1),   # N = 55 < one row tile pair
    (64, (2, 9, 13), 2, 2),    # two batch entries
    (64, (1, 1, 1), 2, 1),     # a single token
    (128, (6, 32, 40), 4, 1),  # N = 7680: several CTAs per head
])
def test_full_token_drift_small(heart, oracle, block, grid, H, B):
    wl = inputs.small_workload(H=H, B=B, grid=grid, block=block, seed=31, eps=[0.01 * (h + 1) for h in range(B * H)])
    (Qa, Ka, _), (Qb, Kb, _) = two_steps(wl)
    cfg = heart.make_config(wl.B, wl.H, wl.N, wl.block)
    ws = heart.new_workspace(cfg)
    got = gpu_full_drift(heart, cfg, ws, Qa, Ka, Qb, Kb, wl.R)
    ref = oracle.full_token_drift(*(inputs.bits(t) for t in (Qa, Ka, Qb, Kb)))
    assert np.all(ref > 0)
    assert np.allclose(got, ref, rtol=DRIFT_RTOL, atol=0)
    # identical tensors: exactly zero; and bit-reproducible
    assert np.all(gpu_full_drift(heart, cfg, ws, Qa, Ka, Qa, Ka, wl.R) == 0)
    assert np.array_equal(gpu_full_drift(heart, cfg, ws, Qa, Ka, Qb, Kb, wl.R), got)


def test_full_token_drift_strided_layout(heart, oracle):
    B, H, N, D = 2, 3, 333, 128
    gen = torch.Generator(device="cuda").manual_seed(5)
    store = [torch.randn(B, N, H, D, device="cuda", generator=gen).to(torch.bfloat16) for _ in range(4)]
    Qa, Ka, Qb, Kb = (s.permute(0, 2, 1, 3) for s in store)
    cfg = heart.config_for(Qa, 64)
    ws = heart.new_workspace(cfg)
    got = gpu_full_drift(heart, cfg, ws, Qa, Ka, Qb, Kb, B * H)
    ref = oracle.full_token_drift(*(inputs.bits(t.contiguous()) for t in (Qa, Ka, Qb, Kb)))
    assert np.allclose(got, ref, rtol=DRIFT_RTOL, atol=0)


def test_full_token_drift_bounds_the_pooled_drift_at_full_size(heart, oracle):
    """wan1.3b-480p shape: against the oracle in full, and the pooled drift the step reports never
    exceeds it (triangle inequality, up to the decision band)."""
    wl = inputs.workload("wan1.3b-480p")
    pair = Pair(wl, heart, oracle)
    pair.gpu_step()  # every head refreshes: anchors = step 0
    Qa, Ka = pair.Q, pair.K
    Qa_b, Ka_b = pair.Qb, pair.Kb
    pair.advance()
    _, _, pooled, _ = pair.gpu_step(want_lse=False)
    got = gpu_full_drift(heart, pair.cfg, pair.ws, Qa, Ka, pair.Q, pair.K, wl.R)
    ref = oracle.full_token_drift(Qa_b, Ka_b, pair.Qb, pair.Kb)
    assert np.allclose(got, ref, rtol=DRIFT_RTOL, atol=0)
    assert np.all(pooled <= got * (1 + 1e-6))


def test_mask_iou_matches_oracle(heart, oracle):
    """Masks of two consecutive steps as the predictor writes them; counts and IoU bit-exact."""
    wl = inputs.small_workload(H=4, grid=(4, 20, 30), block=64, seed=23, eps=[0.002, 0.05, 0.3, 0.8],
                               tau=[0.9, 0.8, 0.9, 0.6], delta=[0.0] * 4)
    pair = Pair(wl, heart, oracle)
    pair.gpu_step(want_lse=False)
    pair.oracle_step(want_O=False)
    A, A_o = pair.gst.mask_bits.clone(), pair.ost.mask_bits.copy()
    pair.advance()
    pair.gpu_step(want_lse=False)
    pair.oracle_step(want_O=False)
    B_, B_o = pair.gst.mask_bits, pair.ost.mask_bits
    assert np.array_equal(to_np(A).view(np.uint32).reshape(A_o.shape), A_o)
    iou = torch.empty(wl.R, dtype=torch.float64, device="cuda")
    counts = torch.empty(wl.R, 2, dtype=torch.int64, device="cuda")
    heart.heart_mask_iou(pair.cfg, A, B_, iou, counts)
    iou_o, counts_o = oracle.mask_iou(A_o, B_o, wl.n_blocks)
    assert np.array_equal(to_np(counts), counts_o)
    assert np.array_equal(to_np(iou), iou_o)
    assert iou_o[0] > iou_o[3]  # the slow head keeps its mask, the fast one does not
    # identical and empty masks
    heart.heart_mask_iou(pair.cfg, A, A, iou)
    assert np.all(to_np(iou) == 1.0)
    Z = torch.zeros_like(A)
    heart.heart_mask_iou(pair.cfg, Z, Z, iou, counts)
    assert np.all(to_np(iou) == 1.0) and np.all(to_np(counts) == 0)
    heart.heart_mask_iou(pair.cfg, A, Z, iou)
    assert np.all(to_np(iou) == 0.0)


def test_mask_iou_random_bits_at_maximum_size(heart, oracle):
    nb, R = heart.MAX_BLOCKS, 3
    W = nb // 32
    rs = np.random.RandomState(9)
    a = rs.randint(0, 2**32, size=(R, nb, W), dtype=np.uint64).astype(np.uint32)
    b = rs.randint(0, 2**32, size=(R, nb, W), dtype=np.uint64).astype(np.uint32)
    b[1] = a[1] & b[1]  # a subset: IoU = |B| / |A|
    cfg = heart.make_config(1, R, nb * 64, 64)
    iou = torch.empty(R, dtype=torch.float64, device="cuda")
    counts = torch.empty(R, 2, dtype=torch.int64, device="cuda")
    ta = torch.from_numpy(a.view(np.int32)).cuda()
    tb = torch.from_numpy(b.view(np.int32)).cuda()
    heart.heart_mask_iou(cfg, ta, tb, iou, counts)
    iou_o, counts_o = oracle.mask_iou(a, b, nb)
    assert np.array_equal(to_np(counts), counts_o) and np.array_equal(to_np(iou), iou_o)


# ----------------------------------------------------------------------------- calibration error
@pytest.mark.parametrize("shape", [
    (2, 5, 6, 9),        # odd and even axes, tiny
    (1, 8, 8, 12),       # the single-frequency grid of the oracle pins
    (3, 7, 20, 33),      # several thousand elements per channel
    (16, 21, 30, 52),    # a 480P latent at half resolution: 524k elements
])
def test_band_error_matches_oracle(heart, oracle, shape):
    gen = torch.Generator(device="cuda").manual_seed(sum(shape))
    yd = torch.randn(shape, device="cuda", generator=gen)
    # error with structure in every band: smooth part + white noise
    C, T, H, W = shape
    t = torch.arange(T, device="cuda").view(1, T, 1, 1) / T
    h = torch.arange(H, device="cuda").view(1, 1, H, 1) / H
    smooth = 0.3 * torch.cos(2 * np.pi * (t + h))
    ys = (yd + smooth + 0.05 * torch.randn(shape, device="cuda", generator=gen)).contiguous()
    out = to_np(heart.heart_band_error(ys, yd))
    e, bands, denom = oracle.band_error(to_np(ys), to_np(yd))
    total = bands.sum()
    assert np.allclose(out[1:5], bands, rtol=1e-9, atol=1e-12 * total)
    assert np.isclose(out[5], denom, rtol=1e-12)
    assert np.isclose(out[0], e, rtol=1e-9)
    # run to run bit-reproducible
    assert np.array_equal(to_np(heart.heart_band_error(ys, yd)), out)


def test_band_error_single_frequencies_on_gpu(heart, oracle):
    C, T, H, W = 1, 8, 8, 12
    t, h, w = np.meshgrid(np.arange(T), np.arange(H), np.arange(W), indexing="ij")
    yd = torch.ones((C, T, H, W), device="cuda")
    for (kt, kh, kw), band in [((0, 0, 0), 0), ((2, 2, 3), 0), ((1, 3, 0), 1), ((2, 0, 4), 1), ((3, 1, 1), 2),
                               ((4, 2, 3), 2), ((3, 3, 0), 3), ((4, 0, 6), 3)]:
        wave = np.cos(2 * np.pi * (kt * t / T + kh * h / H + kw * w / W))[None].astype(np.float32)
        ys = yd + torch.from_numpy(wave).cuda()
        out = to_np(heart.heart_band_error(ys.contiguous(), yd))
        e, bands, _ = oracle.band_error(to_np(ys), to_np(yd))
        assert int(np.argmax(out[1:5])) == band
        assert np.allclose(out[1:5], bands, rtol=1e-9, atol=1e-9 * bands.sum()) and np.isclose(out[0], e, rtol=1e-9)
    # identical tensors: zero error; zero reference: the stabiliser alone in the denominator
    out = to_np(heart.heart_band_error(yd, yd))
    assert np.all(out[:5] == 0)
    z = torch.zeros_like(yd)
    out = to_np(heart.heart_band_error(yd * 1e-3, z))
    assert out[5] == 1e-10
