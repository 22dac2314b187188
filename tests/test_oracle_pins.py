"""Pins of the CPU oracle against what the paper and the mathematics fix.

Each test checks an oracle function against something other than itself: a
closed form, a brute-force enumeration, a textbook special case, a library
routine used as a second opinion, a figure printed in the paper
(tests/golden/*.txt), or the control flow of Algorithm 1 written as a table.
No GPU is involved.
"""
import itertools
import math
import os

import numpy as np
import pytest
import torch

from paper_2605_14513_b200 import inputs

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def bf16_bits(a):
    """float array -> (raw bf16 bits uint16, the bf16-rounded values as float64)."""
    t = torch.as_tensor(np.asarray(a, dtype=np.float32)).to(torch.bfloat16)
    return t.view(torch.int16).numpy().view(np.uint16).copy(), t.to(torch.float64).numpy()


def rand_bf16(rs, shape, scale=1.0):
    return bf16_bits(rs.standard_normal(shape) * scale)


def read_golden(name):
    vals = {}
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            line = line.split("#")[0].strip()
            if line:
                k, v = line.split("=")
                vals[k.strip()] = float(v)
    return vals


# ----------------------------------------------------------------------------- O1 / O2
def test_cache_size_example_from_paper(oracle):
    """The paper's worked memory example fixes the shape of the statistic: one pooled
    D-vector for Q and one for K per (layer, head, guidance branch)."""
    g = read_golden("cache_size_example.txt")
    L, H, D, N = int(g["L"]), int(g["H"]), int(g["D"]), int(g["N"])
    st = oracle.State(1, H, N, D, 64)
    pooled_elems = st.anchor_q.size + st.anchor_k.size  # per layer, per branch
    pooled_bytes = pooled_elems * L * int(g["cfg_branches"]) * int(g["bytes_fp16"])
    token_bytes = 2 * H * N * D * L * int(g["cfg_branches"]) * int(g["bytes_fp16"])
    assert abs(pooled_bytes / 2**20 - g["pooled_MB"]) < 0.01
    assert abs(token_bytes / 2**30 - g["token_GB"]) < 0.06
    assert N == 21 * 30 * 52


def test_token_mean_closed_form(oracle):
    # X[r,i,d] = (i mod 8) + (d mod 3) + r  (small integers: exact in bf16)
    R, N, D = 2, 64, 6
    i = np.arange(N)[None, :, None]
    d = np.arange(D)[None, None, :]
    r = np.arange(R)[:, None, None]
    X, _ = bf16_bits((i % 8) + (d % 3) + r)
    m = oracle.token_mean(X)
    expect = 3.5 + (np.arange(D) % 3)[None, :] + np.arange(R)[:, None]
    assert np.array_equal(m, expect)


def test_token_mean_ragged_n_and_library(oracle):
    rs = np.random.RandomState(0)
    X, Xv = rand_bf16(rs, (3, 77, 16))
    m = oracle.token_mean(X)
    assert np.allclose(m, Xv.mean(axis=1), rtol=1e-13, atol=1e-15)


def test_drift_constant_shift_closed_form(oracle):
    # Q_b = Q_a + c with c and all values exactly representable -> drift = D*|cq| + D*|ck|
    rs = np.random.RandomState(1)
    R, N, D = 2, 40, 128
    base = np.round(rs.standard_normal((R, N, D)) * 4) / 8.0  # multiples of 1/8, |x| < 4
    Qa, _ = bf16_bits(base)
    Qb, _ = bf16_bits(base + 0.125)
    Ka, _ = bf16_bits(base)
    Kb, _ = bf16_bits(base - 0.25)
    d = oracle.pooled_drift(oracle.token_mean(Qa), oracle.token_mean(Ka), oracle.token_mean(Qb), oracle.token_mean(Kb))
    assert np.allclose(d, D * 0.125 + D * 0.25, rtol=1e-12)


def test_drift_metric_properties(oracle):
    rs = np.random.RandomState(2)
    R, N, D = 3, 50, 32
    T = [rand_bf16(rs, (R, N, D))[0] for _ in range(6)]
    ma, ka, mb, kb, mc, kc = [oracle.token_mean(t) for t in T]
    dab = oracle.pooled_drift(ma, ka, mb, kb)
    dba = oracle.pooled_drift(mb, kb, ma, ka)
    dbc = oracle.pooled_drift(mb, kb, mc, kc)
    dac = oracle.pooled_drift(ma, ka, mc, kc)
    assert np.array_equal(dab, dba)  # symmetry
    assert np.all(dac <= dab + dbc + 1e-12)  # triangle inequality
    assert np.array_equal(oracle.pooled_drift(ma, ka, ma, ka), np.zeros(R))  # identity -> exactly 0
    # homogeneity for a power-of-two factor (exact in bf16)
    Xa2 = [bf16_bits(bf16_to_float(t) * 4.0)[0] for t in T[:4]]
    m2 = [oracle.token_mean(t) for t in Xa2]
    assert np.allclose(oracle.pooled_drift(*[m2[0], m2[1], m2[2], m2[3]]), 4.0 * dab, rtol=1e-13)
    # no division by D and Q-part + K-part unweighted: the K term alone
    assert np.allclose(oracle.pooled_drift(ma, ka, ma, kb), np.abs(ka - kb).sum(axis=1), rtol=1e-13)


def bf16_to_float(bits):
    return torch.from_numpy(bits.view(np.int16).copy()).view(torch.bfloat16).to(torch.float64).numpy()


def test_pooled_drift_bounded_by_full_token_drift(oracle):
    # |mean of differences| <= mean of |differences|, dimension by dimension
    rs = np.random.RandomState(3)
    R, N, D = 2, 60, 16
    Qa, Ka, Qb, Kb = [rand_bf16(rs, (R, N, D))[0] for _ in range(4)]
    pooled = oracle.pooled_drift(oracle.token_mean(Qa), oracle.token_mean(Ka), oracle.token_mean(Qb), oracle.token_mean(Kb))
    full = oracle.full_token_drift(Qa, Ka, Qb, Kb)
    assert np.all(pooled <= full + 1e-12)
    # and the full-token drift of a constant shift equals the pooled one
    base = np.round(rs.standard_normal((R, N, D)) * 4) / 8.0
    A, _ = bf16_bits(base)
    Bq, _ = bf16_bits(base + 0.5)
    f = oracle.full_token_drift(A, A, Bq, A)
    assert np.allclose(f, D * 0.5)


def test_drift_random_walk_statistics(oracle):
    # Q_{t+k} = Q_t + sum of k steps eps*N(0,1): each pooled coordinate is N(0, k eps^2/N), so
    # E[drift] = 2 D eps sqrt(2k/(pi N)).  fp32 (not bf16) increments via exactly-representable trick:
    # use large eps so bf16 rounding of the sums is negligible relative to the walk.
    rs = np.random.RandomState(4)
    R, N, D, eps, k = 4, 2048, 128, 0.5, 3
    X0 = np.zeros((R, N, D))
    Xk = sum(rs.standard_normal((R, N, D)) * eps for _ in range(k))
    Z, _ = bf16_bits(X0)
    W, _ = bf16_bits(Xk)
    d = oracle.pooled_drift(oracle.token_mean(Z), oracle.token_mean(Z), oracle.token_mean(W), oracle.token_mean(W))
    expect = 2 * D * eps * math.sqrt(2 * k / (math.pi * N))
    assert abs(d.mean() / expect - 1) < 0.05


# ----------------------------------------------------------------------------- O3
def _decide_once(oracle, st, mq, mk, delta, **kw):
    return oracle.decide(mq, mk, delta, st, **kw)


def test_algorithm1_state_table(oracle):
    """no anchor / drift<delta / drift==delta / drift>delta, as Algorithm 1 branches."""
    D = 4
    st = oracle.State(1, 4, 64, D, 64)
    m0 = np.zeros((4, D))
    drift, refresh = oracle.decide(m0, m0, np.full(4, 1.0), st)
    assert np.all(np.isinf(drift)) and np.all(refresh == 1) and np.all(st.has_anchor == 1)
    # head0: no change; head1: below; head2: exactly delta; head3: above.  delta = 1.0
    mq = np.zeros((4, D))
    mk = np.zeros((4, D))
    mq[1, 0], mk[1, 1] = 0.25, -0.5          # 0.75
    mq[2, 0], mk[2, 3] = 0.5, 0.5            # 1.0 exactly
    mq[3, :] = 0.25
    mk[3, 0] = 0.125                          # 1.125
    drift, refresh = oracle.decide(mq, mk, np.full(4, 1.0), st)
    assert np.array_equal(drift, [0.0, 0.75, 1.0, 1.125])
    assert np.array_equal(refresh, [0, 0, 0, 1])  # strict: drift == delta reuses
    assert np.array_equal(st.anchor_q[3], mq[3]) and np.array_equal(st.anchor_k[3], mk[3])
    assert np.array_equal(st.anchor_q[1], np.zeros(D))  # reuse keeps the anchor


def test_zero_drift_never_refreshes_and_delta0_refreshes_on_any_change(oracle):
    D = 8
    st = oracle.State(1, 2, 64, D, 64)
    m = np.random.RandomState(5).standard_normal((2, D))
    oracle.decide(m, m, np.zeros(2), st)
    for _ in range(3):
        drift, refresh = oracle.decide(m, m, np.zeros(2), st)
        assert np.array_equal(drift, [0.0, 0.0]) and np.array_equal(refresh, [0, 0])
    m2 = m.copy()
    m2[1, 0] += 1e-9
    drift, refresh = oracle.decide(m2, m, np.zeros(2), st)
    assert np.array_equal(refresh, [0, 1])


def test_drift_is_against_the_anchor_not_the_previous_step(oracle):
    """A monotone walk of +0.4*delta per step must refresh on every third step."""
    D, delta = 2, 1.0
    st = oracle.State(1, 1, 64, D, 64)
    pattern = []
    for t in range(10):
        mq = np.array([[0.4 * delta * t, 0.0]])
        _, refresh = oracle.decide(mq, np.zeros((1, D)), np.array([delta]), st)
        pattern.append(int(refresh[0]))
    assert pattern == [1, 0, 0, 1, 0, 0, 1, 0, 0, 1]


def test_layer_gate(oracle):
    g = read_golden("tmr_constants.txt")
    lo, hi = g["gate_lo"], g["gate_hi"]
    H, D = 10, 2

    def run(n_drifting, n_without_anchor=0):
        st = oracle.State(1, H, 64, D, 64)
        z = np.zeros((H, D))
        oracle.decide(z, z, np.ones(H), st)
        if n_without_anchor:
            st.has_anchor[H - n_without_anchor:] = 0
        mq = z.copy()
        mq[:n_drifting, 0] = 5.0
        _, refresh = oracle.decide(mq, z, np.ones(H), st, gate_lo=lo, gate_hi=hi)
        return refresh, st

    assert run(3)[0].sum() == 0          # 0.3 < 0.4: whole layer reuses
    r, st = run(3)
    assert np.array_equal(st.anchor_q[:3, 0], np.zeros(3))  # forced reuse keeps the anchors
    assert run(4)[0].sum() == 4          # 0.4 is not below 0.4: head-wise
    assert run(8)[0].sum() == 8          # 0.8 does not exceed 0.8: head-wise
    assert run(9)[0].sum() == 10         # 0.9 > 0.8: whole layer refreshes
    r, st = run(9)
    assert np.all(st.anchor_q[:9, 0] == 5.0) and st.anchor_q[9, 0] == 0.0  # forced refresh moves anchors
    # heads without an anchor refresh even when the gate says reuse
    r, _ = run(1, n_without_anchor=2)    # 3 of 10 marked -> gate says reuse
    assert np.array_equal(r, [0] * 8 + [1, 1])
    # gate (0,1) never fires
    st = oracle.State(1, H, 64, D, 64)
    z = np.zeros((H, D))
    oracle.decide(z, z, np.ones(H), st)
    mq = z.copy()
    mq[0, 0] = 5
    _, r = oracle.decide(mq, z, np.ones(H), st, gate_lo=0.0, gate_hi=1.0)
    assert r.sum() == 1
    mq[:, 0] = 5
    st2 = oracle.State(1, H, 64, D, 64)
    oracle.decide(z, z, np.ones(H), st2)
    _, r = oracle.decide(mq, z, np.ones(H), st2)
    assert r.sum() == H


def test_gate_is_per_batch_entry(oracle):
    H, D = 5, 2
    st = oracle.State(2, H, 64, D, 64)
    z = np.zeros((2 * H, D))
    oracle.decide(z, z, np.ones(2 * H), st)
    mq = z.copy()
    mq[0, 0] = 5          # batch 0: 1/5 = 0.2 < 0.4 -> reuse all
    mq[H:2 * H, 0] = 5    # batch 1: 5/5 -> all refresh
    _, r = oracle.decide(mq, z, np.ones(2 * H), st, gate_lo=0.4, gate_hi=0.8)
    assert np.array_equal(r, [0] * H + [1] * H)


# ----------------------------------------------------------------------------- O4
def test_block_pool_ragged_last_block(oracle):
    R, N, D, b = 1, 150, 4, 64  # blocks of 64, 64, 22 real tokens
    X = np.zeros((R, N, D))
    X[0, :64] = 1.0
    X[0, 64:128] = np.arange(64)[:, None] % 4  # mean 1.5
    X[0, 128:] = 3.0
    bits, _ = bf16_bits(X)
    p = oracle.block_pool(bits, b)
    assert p.shape == (1, 3, D)
    assert np.array_equal(p[0, 0], np.full(D, 1.0))
    assert np.array_equal(p[0, 1], np.full(D, 1.5))
    assert np.array_equal(p[0, 2], np.full(D, 3.0))  # divides by 22, not 64


def test_block_pool_weighted_average_is_token_mean(oracle):
    rs = np.random.RandomState(6)
    X, _ = rand_bf16(rs, (2, 200, 8))
    p = oracle.block_pool(X, 64)
    cnt = np.array([64, 64, 64, 8])[None, :, None]
    assert np.allclose((p * cnt).sum(1) / 200, oracle.token_mean(X), rtol=1e-13, atol=1e-15)


# ----------------------------------------------------------------------------- O5
def test_block_probs_softmax_properties(oracle):
    from scipy.special import softmax as sp_softmax

    rs = np.random.RandomState(7)
    nb, D = 37, 16
    qp, Kp = rs.standard_normal(D), rs.standard_normal((nb, D))
    P = oracle.block_probs(qp, Kp, 0.25)
    assert abs(P.sum() - 1) < 1e-14 and np.all(P > 0)
    assert np.allclose(P, sp_softmax(0.25 * Kp @ qp), rtol=1e-12)
    # shift invariance: adding a constant logit via one extra feature
    qp2 = np.append(qp, 1.0)
    Kp2 = np.concatenate([Kp, np.full((nb, 1), 40.0)], axis=1)
    assert np.allclose(oracle.block_probs(qp2, Kp2, 0.25), P, rtol=1e-10)
    # one-hot limit
    P3 = oracle.block_probs(qp, Kp, 1e4)
    assert P3.argmax() == (Kp @ qp).argmax() and P3.max() > 1 - 1e-12
    # transposed operands would fail this: scores are <qp, Kp[J]> for each J
    e = np.zeros(D)
    e[3] = 1.0
    P4 = oracle.block_probs(e, Kp, 1.0)
    assert np.allclose(P4, sp_softmax(Kp[:, 3]), rtol=1e-12)


# ----------------------------------------------------------------------------- O6
def brute_force_min_set(P, tau):
    n = len(P)
    for k in range(1, n + 1):
        best = None
        for sub in itertools.combinations(range(n), k):
            m = sum(P[j] for j in sub)
            if m >= tau and (best is None or m > best[0]):
                best = (m, sub)
        if best is not None:
            return k, set(best[1])
    return n, set(range(n))


@pytest.mark.parametrize("seed", range(6))
def test_top_p_against_subset_enumeration(oracle, seed):
    rs = np.random.RandomState(seed)
    n = int(rs.randint(2, 12))
    P = rs.dirichlet(np.ones(n) * 0.5)
    for tau in (0.05, 0.3, 0.6, 0.9, 0.99):
        keep, k, c_at, c_before = oracle.top_p(P, tau)
        kb, sb = brute_force_min_set(P, tau)
        assert k == kb == keep.sum()
        assert set(np.nonzero(keep)[0]) == sb  # no ties in a Dirichlet draw
        kept, dropped = P[keep == 1], P[keep == 0]
        assert kept.sum() >= tau - 1e-15
        assert kept.sum() - kept.min() < tau  # minimal
        assert dropped.size == 0 or kept.min() >= dropped.max()
        assert abs(c_at - kept.sum()) < 1e-12 and abs(c_before - (kept.sum() - kept.min())) < 1e-12


def test_top_p_uniform_row_closed_form(oracle):
    """n = 32 equal probabilities of 2^-5 (exact): tau = 0.9 needs ceil(28.8) = 29 blocks, and
    the tie-break (lower index first) makes them blocks 0..28.  Pins >=, minimality, tie order."""
    P = np.full(32, 2.0**-5)
    keep, k, _, _ = oracle.top_p(P, 0.9)
    assert k == 29 and np.array_equal(np.nonzero(keep)[0], np.arange(29))
    keep, k, _, _ = oracle.top_p(P, 0.5)  # reaches exactly 0.5 at k = 16: ">=" keeps 16, not 17
    assert k == 16 and np.array_equal(np.nonzero(keep)[0], np.arange(16))


def test_top_p_limits_and_monotonicity(oracle):
    rs = np.random.RandomState(11)
    P = rs.dirichlet(np.ones(40))
    keep, k, _, _ = oracle.top_p(P, 1.0)
    assert k == 40 and keep.all()          # tau = 1 -> dense
    keep, k, _, _ = oracle.top_p(P, 1.5)
    assert k == 40 and keep.all()
    keep, k, _, _ = oracle.top_p(P, 1e-12)
    assert k == 1 and keep.argmax() == P.argmax()  # tau -> 0+: exactly the argmax block
    prev = set()
    for tau in np.linspace(0.05, 0.999, 25):
        keep, _, _, _ = oracle.top_p(P, tau)
        cur = set(np.nonzero(keep)[0])
        assert prev <= cur
        prev = cur
    # underflowed tail: mass never reaches tau numerically -> keep all
    P2 = np.array([0.5, 0.25, 0.0, 0.0])
    keep, k, _, _ = oracle.top_p(P2, 0.9)
    assert k == 4


def test_predict_mask_outputs_consistent(oracle):
    wl = inputs.small_workload(H=2, grid=(2, 9, 13), block=64, seed=3)
    seq = inputs.Sequence(wl)
    Q, K, V = seq.bf16()
    Qb, Kb = inputs.bits(Q), inputs.bits(K)
    st = oracle.State(1, wl.H, wl.N, 128, 64, idx_stride=wl.n_blocks + 3)
    oracle.predict_mask(Qb, Kb, 64, wl.tau, st, refresh=np.array([1, 0], np.uint8))
    nb = wl.n_blocks
    assert np.all(st.kv_cnt[1] == 0) and np.all(st.mask_bits[1] == 0)  # head 1 untouched
    Qp, Kp = oracle.block_pool(Qb, 64), oracle.block_pool(Kb, 64)
    for I in range(nb):
        P = oracle.block_probs(Qp[0, I], Kp[0], 1 / math.sqrt(128))
        assert np.allclose(P, oracle.probs_row(Qb, Kb, 64, 0, I))
        keep, k, _, _ = oracle.top_p(P, wl.tau[0])
        lst = st.kv_idx[0, I, :k]
        assert st.kv_cnt[0, I] == k and np.array_equal(lst, np.nonzero(keep)[0])
        assert np.all(np.diff(lst) > 0)
        bits = [(int(st.mask_bits[0, I, J // 32]) >> (J % 32)) & 1 for J in range(nb)]
        assert np.array_equal(bits, keep)
    # tau = 1 gives the dense mask
    st2 = oracle.State(1, wl.H, wl.N, 128, 64)
    oracle.predict_mask(Qb, Kb, 64, np.ones(2), st2)
    assert np.all(st2.kv_cnt == nb)
    assert np.array_equal(st2.kv_idx, np.broadcast_to(np.arange(nb), st2.kv_idx.shape))


# ----------------------------------------------------------------------------- O7
def _full_lists(R, nb):
    idx = np.broadcast_to(np.arange(nb, dtype=np.int32), (R, nb, nb)).copy()
    cnt = np.full((R, nb), nb, np.int32)
    return idx, cnt


def test_attention_full_mask_equals_dense_definitions(oracle):
    rs = np.random.RandomState(12)
    R, N, D, b = 2, 150, 128, 64  # ragged: 64 + 64 + 22
    Q, Qv = rand_bf16(rs, (R, N, D))
    K, Kv = rand_bf16(rs, (R, N, D))
    V, Vv = rand_bf16(rs, (R, N, D))
    idx, cnt = _full_lists(R, 3)
    O, lse = oracle.block_sparse_attn(Q, K, V, b, idx, cnt, want_lse=True)
    # (a) textbook loop in C with no block structure at all
    assert np.allclose(O, oracle.dense_attn(Q, K, V), rtol=1e-12, atol=1e-14)
    # (b) library attention in fp64
    ref = torch.nn.functional.scaled_dot_product_attention(
        torch.from_numpy(Qv), torch.from_numpy(Kv), torch.from_numpy(Vv)).numpy()
    assert np.allclose(O, ref, rtol=1e-10, atol=1e-12)
    # (c) log-sum-exp of the scaled logits
    logits = np.einsum("rid,rjd->rij", Qv, Kv) / math.sqrt(D)
    assert np.allclose(lse, torch.logsumexp(torch.from_numpy(logits), -1).numpy(), rtol=1e-12)


def test_attention_closed_forms(oracle):
    rs = np.random.RandomState(13)
    R, N, D, b = 1, 200, 128, 64  # blocks 64,64,64,8
    K, Kv = rand_bf16(rs, (R, N, D))
    V, Vv = rand_bf16(rs, (R, N, D))
    Q, Qv = rand_bf16(rs, (R, N, D))
    idx = np.full((1, 4, 4), -1, np.int32)
    cnt = np.zeros((1, 4), np.int32)
    idx[0, 0, :2], cnt[0, 0] = [1, 3], 2      # includes the ragged block (8 real keys)
    idx[0, 1, :1], cnt[0, 1] = [2], 1
    idx[0, 2, :3], cnt[0, 2] = [0, 1, 2], 3
    idx[0, 3, :1], cnt[0, 3] = [3], 1
    # Q = 0 -> plain mean of V over the retained real keys
    Z = np.zeros_like(Q)
    O = oracle.block_sparse_attn(Z, K, V, b, idx, cnt)
    keys0 = np.r_[64:128, 192:200]
    assert np.allclose(O[0, :64], Vv[0, keys0].mean(0)[None], rtol=1e-12, atol=1e-14)
    assert np.allclose(O[0, 192:200], Vv[0, 192:200].mean(0)[None], rtol=1e-12, atol=1e-14)
    # V constant -> O constant
    Vc, _ = bf16_bits(np.full((R, N, D), 0.75))
    assert np.allclose(oracle.block_sparse_attn(Q, K, Vc, b, idx, cnt), 0.75, rtol=1e-13)
    # a single retained block == dense attention restricted to that block's keys
    O = oracle.block_sparse_attn(Q, K, V, b, idx, cnt)
    ref = torch.nn.functional.scaled_dot_product_attention(
        torch.from_numpy(Qv[:, 64:128]), torch.from_numpy(Kv[:, 128:192]), torch.from_numpy(Vv[:, 128:192])).numpy()
    assert np.allclose(O[0, 64:128], ref[0], rtol=1e-10, atol=1e-12)
    # two retained blocks incl. ragged one == dense attention over the union of their real keys
    ref = torch.nn.functional.scaled_dot_product_attention(
        torch.from_numpy(Qv[:, :64]), torch.from_numpy(Kv[:, keys0]), torch.from_numpy(Vv[:, keys0])).numpy()
    assert np.allclose(O[0, :64], ref[0], rtol=1e-10, atol=1e-12)
    # order of the list does not matter beyond rounding
    idx2 = idx.copy()
    idx2[0, 2, :3] = [2, 0, 1]
    assert np.allclose(oracle.block_sparse_attn(Q, K, V, b, idx2, cnt), O, rtol=1e-12, atol=1e-14)
    # empty list -> zeros and lse = -inf
    cnt2 = cnt.copy()
    cnt2[0, 1] = 0
    O2, lse2 = oracle.block_sparse_attn(Q, K, V, b, idx, cnt2, want_lse=True)
    assert np.all(O2[0, 64:128] == 0) and np.all(np.isneginf(lse2[0, 64:128]))


def test_attention_logit_shift_invariance_with_large_logits(oracle):
    """Adding ~45 to every logit of a row (one extra feature pair) changes nothing:
    exercises the max subtraction at the logit magnitudes the synthetic workloads reach."""
    rs = np.random.RandomState(14)
    R, N, D, b = 1, 128, 128, 64
    Qf = rs.standard_normal((R, N, D))
    Kf = rs.standard_normal((R, N, D))
    Qf[..., -1] = 0.0
    Kf[..., -1] = 0.0
    V, _ = rand_bf16(rs, (R, N, D))
    Q0, _ = bf16_bits(Qf)
    K0, _ = bf16_bits(Kf)
    Qf[..., -1] = 16.0
    Kf[..., -1] = 32.0  # adds 16*32/sqrt(128) = 45.25 to every logit
    Q1, _ = bf16_bits(Qf)
    K1, _ = bf16_bits(Kf)
    idx, cnt = _full_lists(R, 2)
    A = oracle.block_sparse_attn(Q0, K0, V, b, idx, cnt)
    Bo = oracle.block_sparse_attn(Q1, K1, V, b, idx, cnt)
    assert np.allclose(A, Bo, rtol=1e-9, atol=1e-12)


def test_attn_rows_matches_full(oracle):
    wl = inputs.small_workload(H=2, grid=(2, 9, 13), block=64, seed=5)
    Q, K, V = (inputs.bits(t) for t in inputs.Sequence(wl).bf16())
    st = oracle.State(1, wl.H, wl.N, 128, 64)
    oracle.predict_mask(Q, K, 64, wl.tau, st)
    O = oracle.block_sparse_attn(Q, K, V, 64, st.kv_idx, st.kv_cnt)
    nb = wl.n_blocks
    rows_r, rows_I = np.array([0, 1, 1]), np.array([nb - 1, 0, 2])
    out = oracle.attn_rows(Q, K, V, 64, st.kv_idx, st.kv_cnt, rows_r, rows_I)
    last = wl.N - (nb - 1) * 64
    assert np.array_equal(out[0, :last], O[0, (nb - 1) * 64:])
    assert np.all(np.isnan(out[0, last:]))  # rows past N are never written
    assert np.array_equal(out[1], O[1, :64]) and np.array_equal(out[2], O[1, 128:192])


# ----------------------------------------------------------------------------- O8
def test_step_equals_separate_calls_and_state_roundtrip(oracle):
    wl = inputs.small_workload(H=3, grid=(2, 9, 13), block=64, seed=9, steps=4, eps=[0.005, 0.05, 0.3],
                               delta=[1.0, 1.0, 1.0])
    seq = inputs.Sequence(wl)
    st_a = oracle.State(1, wl.H, wl.N, 128, 64)
    st_b = oracle.State(1, wl.H, wl.N, 128, 64)
    refreshes = []
    for t in range(4):
        Q, K, V = (inputs.bits(x) for x in seq.bf16())
        O, _, drift, refresh = oracle.step(Q, K, V, wl.delta, wl.tau, st_a)
        d2, r2 = oracle.decide(oracle.token_mean(Q), oracle.token_mean(K), wl.delta, st_b)
        oracle.predict_mask(Q, K, 64, wl.tau, st_b, refresh=r2)
        O2 = oracle.block_sparse_attn(Q, K, V, 64, st_b.kv_idx, st_b.kv_cnt)
        assert np.array_equal(drift, d2) and np.array_equal(refresh, r2)
        assert np.array_equal(st_a.kv_idx, st_b.kv_idx) and np.array_equal(st_a.mask_bits, st_b.mask_bits)
        assert np.array_equal(O, O2)
        refreshes.append(refresh.copy())
        if t == 1:  # checkpoint = plain copies of the state arrays
            st_a = st_a.copy()
        seq.advance()
    assert np.all(refreshes[0] == 1)
    assert 0 < sum(int(r.sum()) for r in refreshes[1:]) < 3 * wl.H  # a mix of reuse and refresh


def test_force_dense_step_leaves_state_alone(oracle):
    wl = inputs.small_workload(H=2, grid=(2, 9, 13), block=64, seed=10)
    Q, K, V = (inputs.bits(x) for x in inputs.Sequence(wl).bf16())
    st = oracle.State(1, wl.H, wl.N, 128, 64)
    O, _, drift, refresh = oracle.step(Q, K, V, wl.delta, wl.tau, st, flags=oracle.FORCE_DENSE)
    assert np.all(st.has_anchor == 0) and np.all(st.kv_cnt == 0) and np.all(refresh == 0)
    assert np.allclose(O, oracle.dense_attn(Q, K, V), rtol=1e-12, atol=1e-14)


def test_tiny_config_refresh_pattern(oracle):
    """Config 1: both heads refresh at step 0; at step 1 exactly head 1 (eps = 0.3) refreshes."""
    wl = inputs.workload("tiny")
    seq = inputs.Sequence(wl)
    st = oracle.State(1, wl.H, wl.N, 128, wl.block)
    Q, K, V = (inputs.bits(x) for x in seq.bf16())
    _, _, d0, r0 = oracle.step(Q, K, V, wl.delta, wl.tau, st, want_O=False)
    cnt0 = st.kv_cnt.copy()
    seq.advance()
    Q, K, V = (inputs.bits(x) for x in seq.bf16())
    _, _, d1, r1 = oracle.step(Q, K, V, wl.delta, wl.tau, st, want_O=False)
    assert np.array_equal(r0, [1, 1]) and np.array_equal(r1, [0, 1])
    assert d1[0] < wl.delta[0] < d1[1]
    assert np.array_equal(st.kv_cnt[0], cnt0[0])  # reused head keeps its mask
    dens = st.kv_cnt.mean(axis=1) / wl.n_blocks
    assert np.all(dens > 0.1) and np.all(dens < 0.8)


# ----------------------------------------------------------------------------- diagnostics
def test_mask_iou_closed_forms(oracle):
    nb, W = 40, 2
    a = np.zeros((3, nb, W), np.uint32)
    b = np.zeros((3, nb, W), np.uint32)
    # head 0: identical masks (every row keeps blocks 0..9) -> IoU 1
    a[0, :, 0] = b[0, :, 0] = (1 << 10) - 1
    # head 1: A keeps blocks 0..9, B keeps 5..14 -> |A&B| = 5, |A|B| = 15 per row -> 1/3
    a[1, :, 0] = (1 << 10) - 1
    b[1, :, 0] = ((1 << 15) - 1) ^ ((1 << 5) - 1)
    # head 2: disjoint, B in the second word (blocks 32..39) -> 0
    a[2, :, 0] = 0xff
    b[2, :, 1] = 0xff
    iou, counts = oracle.mask_iou(a, b, nb)
    assert np.array_equal(iou, [1.0, 5.0 / 15.0, 0.0])
    assert np.array_equal(counts, [[10 * nb, 10 * nb], [5 * nb, 15 * nb], [0, 16 * nb]])
    # both empty -> 1 by convention; symmetric
    z = np.zeros_like(a)
    assert np.array_equal(oracle.mask_iou(z, z, nb)[0], [1.0, 1.0, 1.0])
    assert np.array_equal(oracle.mask_iou(b, a, nb)[0], iou)


def test_mask_iou_of_predicted_masks_drops_with_drift(oracle):
    """Small drift keeps the predicted mask (IoU near 1), large drift changes it: the relation the
    paper's reuse rule relies on, on the synthetic tensors."""
    wl = inputs.small_workload(H=2, grid=(3, 10, 14), block=64, seed=17, eps=[0.002, 0.6], tau=[0.9, 0.9])
    seq = inputs.Sequence(wl)
    Q, K, _ = (inputs.bits(x) for x in seq.bf16())
    s0 = oracle.State(1, 2, wl.N, 128, 64)
    oracle.predict_mask(Q, K, 64, wl.tau, s0)
    seq.advance()
    Q1, K1, _ = (inputs.bits(x) for x in seq.bf16())
    s1 = oracle.State(1, 2, wl.N, 128, 64)
    oracle.predict_mask(Q1, K1, 64, wl.tau, s1)
    iou, _ = oracle.mask_iou(s0.mask_bits, s1.mask_bits, wl.n_blocks)
    full = oracle.full_token_drift(Q, K, Q1, K1)
    assert iou[0] > 0.9 and iou[1] < iou[0] and full[1] > 50 * full[0]


def test_full_token_drift_bounds_the_interaction_change(oracle):
    """Stability bound of the appendix: the mean absolute change of the scaled query-key logits is
    at most max(B_q, B_k)/sqrt(D) times the full-token drift -- with equality when the keys are a
    constant vector of magnitude B_k >= B_q that does not move and every query coordinate grows."""
    rs = np.random.RandomState(21)
    R, N, D = 2, 24, 16
    # general case: inequality
    Qa, fa = rand_bf16(rs, (R, N, D))
    Ka, ka = rand_bf16(rs, (R, N, D))
    Qb, fb = rand_bf16(rs, (R, N, D))
    Kb, kb = rand_bf16(rs, (R, N, D))
    d = oracle.full_token_drift(Qa, Ka, Qb, Kb)
    for r in range(R):
        ga = fa[r] @ ka[r].T / math.sqrt(D)
        gb = fb[r] @ kb[r].T / math.sqrt(D)
        Bq = max(np.abs(fa[r]).max(), np.abs(fb[r]).max())
        Bk = max(np.abs(ka[r]).max(), np.abs(kb[r]).max())
        assert np.abs(gb - ga).mean() <= max(Bq, Bk) / math.sqrt(D) * d[r] + 1e-12
    # equality case (all values exactly representable in bf16)
    qa = np.round(rs.uniform(-1, 1, (R, N, D)) * 8) / 8.0
    inc = np.round(rs.uniform(0, 1, (R, N, D)) * 8) / 8.0
    k = np.full((R, N, D), 2.0)
    A, _ = bf16_bits(qa)
    Bm, _ = bf16_bits(qa + inc)
    Kc, _ = bf16_bits(k)
    d = oracle.full_token_drift(A, Kc, Bm, Kc)
    for r in range(R):
        delta_qk = np.abs((qa[r] + inc[r]) @ k[r].T - qa[r] @ k[r].T).mean() / math.sqrt(D)
        assert np.isclose(delta_qk, 2.0 / math.sqrt(D) * d[r], rtol=1e-13)


# ----------------------------------------------------------------------------- calibration error
def _brute_dft3(x):
    """Direct O(n^2) 3-D DFT of one [T, H, W] array (separable, from the definition of the DFT)."""
    out = x.astype(np.complex128)
    for ax in range(3):
        n = out.shape[ax]
        k = np.arange(n)
        F = np.exp(-2j * np.pi * np.outer(k, k) / n)
        out = np.moveaxis(np.tensordot(F, np.moveaxis(out, ax, 0), axes=(1, 0)), 0, ax)
    return out


def test_band_error_against_direct_dft_and_parseval(oracle):
    rs = np.random.RandomState(31)
    C, T, H, W = 2, 5, 6, 9
    yd = rs.standard_normal((C, T, H, W))
    ys = yd + 0.1 * rs.standard_normal((C, T, H, W))
    e, bands, denom = oracle.band_error(ys, yd)
    # Parseval: the four bands partition the spectrum
    assert np.isclose(bands.sum(), T * H * W * ((ys - yd) ** 2).sum(), rtol=1e-12)
    assert np.isclose(denom, T * H * W * (yd ** 2).sum() + 1e-10, rtol=1e-12)
    # band membership spelled out per unshifted frequency index: k is low iff min(k, n-k) <= n//4
    # (the fftshift-ed distance to the centre n//2 is k for k < ceil(n/2) and n-k above, which for
    # even n makes the Nyquist index n/2 lie at distance n/2)
    def low(n):
        k = np.arange(n)
        return np.minimum(k, n - k) <= n // 4
    lt, lh, lw = low(T), low(H), low(W)
    ref = np.zeros(4)
    for c in range(C):
        P = np.abs(_brute_dft3(ys[c] - yd[c])) ** 2
        for t in range(T):
            for h in range(H):
                for w in range(W):
                    q = (0 if lt[t] else 2) + (0 if (lh[h] and lw[w]) else 1)
                    ref[q] += P[t, h, w]
    assert np.allclose(bands, ref, rtol=1e-10)
    assert np.isclose(e, (1.0 * ref[0] + 0.5 * ref[1] + 0.01 * ref[2] + 0.01 * ref[3]) / denom, rtol=1e-10)


@pytest.mark.parametrize("n,expected_low", [
    (8, [0, 1, 2, 6, 7]),          # floor(8/4) = 2: |k| <= 2
    (9, [0, 1, 2, 7, 8]),          # floor(9/4) = 2
    (21, [0, 1, 2, 3, 4, 5, 16, 17, 18, 19, 20]),  # floor(21/4) = 5
    (4, [0, 1, 3]),
    (3, [0]),                      # floor(3/4) = 0: only the zero frequency
])
def test_band_low_frequency_rule(oracle, n, expected_low):
    m = np.fft.ifftshift(oracle.low_frequency_mask(n))  # back to the unshifted index
    assert sorted(np.nonzero(m)[0].tolist()) == expected_low


def test_band_error_single_frequencies_and_weights(oracle):
    C, T, H, W = 1, 8, 8, 12
    t, h, w = np.meshgrid(np.arange(T), np.arange(H), np.arange(W), indexing="ij")
    yd = np.ones((C, T, H, W))
    N = T * H * W

    def wave(kt, kh, kw):
        return np.cos(2 * np.pi * (kt * t / T + kh * h / H + kw * w / W))[None]

    # (kt, kh, kw) -> band; thresholds: T,H: |k| <= 2 low; W: |k| <= 3 low
    for (kt, kh, kw), band in [((0, 0, 0), 0), ((2, 2, 3), 0), ((1, 3, 0), 1), ((2, 0, 4), 1),
                               ((3, 1, 1), 2), ((4, 2, 3), 2), ((3, 3, 0), 3), ((4, 0, 6), 3)]:
        e, bands, denom = oracle.band_error(yd + wave(kt, kh, kw), yd)
        assert np.argmax(bands) == band and np.isclose(bands[band], bands.sum(), rtol=1e-12)
        energy = N * (wave(kt, kh, kw) ** 2).sum()
        assert np.isclose(e, oracle.BAND_WEIGHTS[band] * energy / (N * N + 1e-10), rtol=1e-12)
    # homogeneity in the error, and the stabiliser when the reference is zero
    e1, _, _ = oracle.band_error(yd + 0.5 * wave(1, 0, 0), yd)
    e2, _, _ = oracle.band_error(yd + 1.5 * wave(1, 0, 0), yd)
    assert np.isclose(e2, 9 * e1, rtol=1e-12)
    e0, bands0, denom0 = oracle.band_error(wave(0, 0, 0) * 1e-3, np.zeros((C, T, H, W)))
    assert denom0 == 1e-10 and np.isclose(e0, bands0[0] / 1e-10)
