"""Pins of the oracle's strided antidiagonal block-importance estimator (the estimator family of the
paper's main backbone: anti-diagonal scoring, stride 16, 128-token blocks; the definition is this
build's own, so what is pinned is the definition, not fidelity to that backbone)."""
import numpy as np
import pytest
import torch

from oracle import heart_oracle as oracle


def bf16_bits(x):
    t = torch.from_numpy(np.asarray(x, np.float32)).to(torch.bfloat16)
    return t.view(torch.int16).numpy().view(np.uint16), t.to(torch.float64).numpy()


def make(rs, R, N, D=128, amp=1.0):
    Qb, Q = bf16_bits(rs.standard_normal((R, N, D)) * amp)
    Kb, K = bf16_bits(rs.standard_normal((R, N, D)) * amp)
    return Qb, Kb, Q, K


def brute_force(Q, K, b, s, r, I, scale):
    """From the token-level logit matrix: the antidiagonal of every s x s tile, averaged."""
    N = Q.shape[1]
    nb, Ns, g = -(-N // b), N // s, b // s
    L = (Q[r] @ K[r].T) * scale                      # all N x N token-level logits
    rows = [a for a in range(I * g, (I + 1) * g) if a < Ns]
    if not rows:
        return np.full(nb, 1.0 / nb)
    P = np.zeros(nb)
    for a in rows:
        srow = np.array([np.mean([L[a * s + t, c * s + s - 1 - t] for t in range(s)]) for c in range(Ns)])
        e = np.exp(srow - srow.max())
        e /= e.sum()
        for c in range(Ns):
            P[c // g] += e[c]
    return P / len(rows)


@pytest.mark.parametrize("N,b,s", [(256, 64, 16), (300, 128, 16), (200, 64, 8), (129, 128, 16), (95, 64, 16)])
def test_matches_the_token_level_definition(N, b, s):
    rs = np.random.RandomState(N + s)
    Qb, Kb, Q, K = make(rs, 2, N, amp=1.5)
    scale = 1.0 / np.sqrt(128.0)
    nb = -(-N // b)
    for r in range(2):
        for I in range(nb):
            got = oracle.antidiag_probs_row(Qb, Kb, b, r, I, s=s)
            ref = brute_force(Q, K, b, s, r, I, scale)
            assert np.allclose(got, ref, rtol=1e-11, atol=1e-15), (r, I)
            assert got.sum() == pytest.approx(1.0, abs=1e-12)


def test_stride_one_is_the_block_sum_of_dense_softmax_attention():
    sp = pytest.importorskip("scipy.special")
    rs = np.random.RandomState(7)
    N, b = 192, 64
    Qb, Kb, Q, K = make(rs, 1, N)
    A = sp.softmax(Q[0] @ K[0].T / np.sqrt(128.0), axis=1)   # textbook attention probabilities
    for I in range(3):
        ref = A[I * b:(I + 1) * b].reshape(b, 3, b).sum(axis=2).mean(axis=0)
        assert np.allclose(oracle.antidiag_probs_row(Qb, Kb, b, 0, I, s=1), ref, rtol=1e-11)


def test_only_the_antidiagonal_pairs_count():
    """One non-zero query token (offset t0 in its group) and one non-zero key token (offset t1):
    the pair contributes iff t1 = s - 1 - t0; then S' = scale/s * <q, k> for that one tile."""
    s, b, N, D = 16, 64, 128, 128
    for t0, t1 in [(3, 12), (3, 3), (0, 15), (15, 0), (7, 9)]:
        Q = np.zeros((1, N, D), np.float32)
        K = np.zeros((1, N, D), np.float32)
        Q[0, 2 * s + t0, 5] = 4.0      # group a = 2 (query block 0)
        K[0, 5 * s + t1, 5] = 8.0      # group c = 5 (key block 1)
        Qb, _ = bf16_bits(Q)
        Kb, _ = bf16_bits(K)
        P = oracle.antidiag_probs_row(Qb, Kb, b, 0, 0, s=s)
        Ns, g = N // s, b // s
        if t1 == s - 1 - t0:
            x = 32.0 / np.sqrt(128.0) / s
            # the one group (2) that sees the pair puts e^x on column 5 and 1 elsewhere; the other three
            # groups of the query block are uniform
            hot = np.full(Ns, 1.0)
            hot[5] = np.exp(x)
            hot /= hot.sum()
            uni = np.full(Ns, 1.0 / Ns)
            ref = (hot.reshape(2, g).sum(1) + 3 * uni.reshape(2, g).sum(1)) / 4
            assert np.allclose(P, ref, rtol=1e-12)
            assert P[1] > P[0]
        else:
            assert np.allclose(P, [0.5, 0.5], rtol=1e-12)


def test_zero_queries_give_importance_proportional_to_the_sampled_groups():
    rs = np.random.RandomState(9)
    N, b, s = 200, 64, 16          # 12 full groups: blocks hold 4, 4, 4, 0 of them (block 3 = tokens 192..199)
    Qb, Kb, _, _ = make(rs, 1, N)
    Qb[:] = 0
    for I in range(3):
        assert np.allclose(oracle.antidiag_probs_row(Qb, Kb, b, 0, I, s=s), [1 / 3, 1 / 3, 1 / 3, 0.0], rtol=1e-12)
    # the last query block has no full group: uniform over all four key blocks
    assert np.allclose(oracle.antidiag_probs_row(Qb, Kb, b, 0, 3, s=s), [0.25] * 4)


def test_a_common_key_offset_and_the_unsampled_tail_change_nothing():
    rs = np.random.RandomState(11)
    N, b, s = 200, 64, 8
    Qb, Kb, Q, K = make(rs, 1, N)
    base = [oracle.antidiag_probs_row(Qb, Kb, b, 0, I, s=s) for I in range(4)]
    # adding one vector to every key shifts all logits of a strided row by the same amount
    v = np.round(rs.standard_normal(128) * 4) / 4          # exactly representable after the add
    K2b, _ = bf16_bits(np.round(K * 8) / 8 + v)
    K1b, _ = bf16_bits(np.round(K * 8) / 8)
    for I in range(3):
        a = oracle.antidiag_probs_row(Qb, K1b, b, 0, I, s=s)
        c = oracle.antidiag_probs_row(Qb, K2b, b, 0, I, s=s)
        assert np.allclose(a, c, rtol=1e-9, atol=1e-14)
    # tokens past the last full group (here none at s = 8: 200 = 25 * 8; use s = 16: 192..199) are not seen
    base16 = [oracle.antidiag_probs_row(Qb, Kb, b, 0, I, s=16) for I in range(4)]
    Q3, K3 = Qb.copy(), Kb.copy()
    Q3[0, 192:] = 0x4120  # 10.0 in bf16
    K3[0, 192:] = 0xC120  # -10.0
    for I in range(4):
        assert np.array_equal(oracle.antidiag_probs_row(Q3, K3, b, 0, I, s=16), base16[I])
    assert all(abs(p.sum() - 1) < 1e-12 for p in base)


def test_mask_prediction_applies_the_same_top_p_rule():
    rs = np.random.RandomState(13)
    N, b = 512, 64
    Qb, Kb, _, _ = make(rs, 2, N, amp=2.0)
    st = oracle.State(1, 2, N, 128, b)
    tau = np.array([0.6, 1.0])
    oracle.predict_mask_antidiag(Qb, Kb, b, tau, st)
    nb = 8
    assert np.all(st.kv_cnt[1] == nb)
    for I in range(nb):
        P = oracle.antidiag_probs_row(Qb, Kb, b, 0, I)
        keep, k, c_at, c_before = oracle.top_p(P, 0.6)
        assert st.kv_cnt[0, I] == k and c_at >= 0.6 > c_before
        assert np.array_equal(np.nonzero(keep)[0], st.kv_idx[0, I, :k])
        assert int(st.mask_bits[0, I, 0]) == sum(1 << int(j) for j in np.nonzero(keep)[0])
