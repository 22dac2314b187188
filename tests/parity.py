"""Helpers shared by the GPU parity tests: run both sides on the same bytes and compare.

The CUDA path is reached only through the C-ABI binding (paper_2605_14513_b200.heart);
the oracle only through oracle.heart_oracle.  Neither side sees the other's results.
"""
import math

import numpy as np
import torch

from paper_2605_14513_b200 import inputs

ATTN_MAX_ABS = 2e-2   # bf16 in / fp32 accumulate / bf16 out, identical masks
ATTN_REL_L2 = 1e-2
DRIFT_RTOL = 1e-6     # the decision band; fp64 both sides except fp32 partials of <= 8 bf16 values on the GPU
DECISION_BAND = 1e-6  # a refresh flag may differ only if |drift - delta| <= 1e-6 * delta
MASS_BAND = 1e-5      # a mask row may differ only if the cumulative mass is within 1e-5 of tau


def to_np(t):
    return t.detach().cpu().numpy()


def mask_bits_u32(t):
    return to_np(t).view(np.uint32)


def check_decisions(drift_gpu, refresh_gpu, drift_ref, refresh_ref, delta):
    """Drift within DRIFT_RTOL; flags identical outside the near-threshold band. Returns #exempt."""
    fin = np.isfinite(drift_ref)
    assert np.array_equal(np.isfinite(drift_gpu), fin)
    assert np.allclose(drift_gpu[fin], drift_ref[fin], rtol=DRIFT_RTOL, atol=1e-300), (drift_gpu, drift_ref)
    diff = np.nonzero(refresh_gpu != refresh_ref)[0]
    for r in diff:
        assert abs(drift_ref[r] - delta[r]) <= DECISION_BAND * abs(delta[r]), (r, drift_ref[r], delta[r])
    return len(diff)


def check_masks(gpu_state, ref_state, heads, tau, probs_row_fn):
    """Bit masks / lists / counts of `heads` identical, except rows whose cumulative mass sits within
    MASS_BAND of tau, or whose swapped boundary blocks are tied to within 1e-5 relative AND whose
    retained mass equals the oracle's within MASS_BAND (judged with the oracle's fp64 probabilities).
    Returns the number of exempted rows."""
    gb, rb = mask_bits_u32(gpu_state.mask_bits), ref_state.mask_bits
    gc, rc = to_np(gpu_state.kv_cnt), ref_state.kv_cnt
    gi, ri = to_np(gpu_state.kv_idx), ref_state.kv_idx
    nb = rb.shape[1]
    exempt = 0
    for r in heads:
        # the index list, the count and the bit mask of the GPU must agree with each other
        pop = np.zeros(nb, np.int64)
        for w in range(gb.shape[2]):
            pop += np.array([bin(int(x)).count("1") for x in gb[r, :, w]])
        assert np.array_equal(pop, gc[r]), f"head {r}: popcount(mask) != kv_cnt"
        bad_rows = np.nonzero((gb[r] != rb[r]).any(axis=1) | (gc[r] != rc[r]))[0]
        same = np.setdiff1d(np.arange(nb), bad_rows)
        for I in same:
            k = rc[r, I]
            assert np.array_equal(gi[r, I, :k], ri[r, I, :k]), f"list mismatch at ({r},{I})"
        for I in bad_rows:
            G = set(gi[r, I, :gc[r, I]].tolist())
            Rf = set(ri[r, I, :rc[r, I]].tolist())
            assert len(G) == gc[r, I]
            check_differing_row(G, Rf, probs_row_fn(r, I), tau[r], nb, (r, I))
            exempt += 1
    return exempt


def check_differing_row(G, Rf, P, t, nb, where=None):
    """A mask row on which the GPU (set G) and the oracle (set Rf) disagree is acceptable only inside
    the near-threshold bands, judged with the oracle's fp64 importances P: the GPU's set must itself be
    a valid top-p set up to MASS_BAND, and every block the two sets disagree on must either be tied
    with the boundary block (1e-5 relative) at equal retained mass, or the oracle's cumulative mass
    must sit within MASS_BAND of tau on one side of the cut."""
    assert G and all(0 <= j < nb for j in G), where
    mass = sum(P[j] for j in G)
    pmin = min(P[j] for j in G)
    p_edge = min(P[j] for j in Rf)
    assert mass >= t - MASS_BAND and mass - pmin < t + MASS_BAND, (where, mass, t)
    mass_ref = sum(P[x] for x in Rf)
    for j in G ^ Rf:
        tied = abs(P[j] - p_edge) <= 1e-6 * P.max() + 1e-5 * p_edge and abs(mass - mass_ref) <= MASS_BAND
        assert tied or abs(mass_ref - t) <= MASS_BAND or \
            abs(mass_ref - p_edge - t) <= MASS_BAND, (where, j, P[j], p_edge)


def attention_abs_bound(O_ref):
    """Element-wise absolute bound on |O_gpu - O_ref|.  The output is stored as bf16 (8 significant
    bits), so rounding alone costs up to half a unit in the last place: 2^(e-8) for |O| in
    [2^e, 2^(e+1)), i.e. 0.0078 on [2, 4) and 0.0156 on [4, 8).  Below 4 the flat 2e-2 of the
    acceptance bar covers that rounding plus the ~5e-3 the fp32 accumulation of bf16-rounded weights
    contributes; from 4 up the bound is that same 5e-3 on top of the half-ulp of the value itself."""
    mag = np.abs(np.asarray(O_ref, np.float64))
    half_ulp = np.exp2(np.floor(np.log2(np.maximum(mag, 1e-30))) - 8.0)
    return np.where(mag < 4.0, ATTN_MAX_ABS, half_ulp + 5e-3)


def check_attention(O_gpu, O_ref, valid=None):
    """O_gpu: float array widened from bf16; O_ref: fp64 oracle; both [..., D]."""
    a = np.asarray(O_gpu, np.float64)
    b = np.asarray(O_ref, np.float64)
    if valid is not None:
        a, b = a[valid], b[valid]
    assert np.isfinite(a).all()
    err = np.abs(a - b)
    max_abs = err.max()
    rel_l2 = math.sqrt(((a - b) ** 2).sum() / max((b ** 2).sum(), 1e-300))
    over = err > attention_abs_bound(b)
    assert not over.any(), f"max-abs {max_abs} (worst excess {(err - attention_abs_bound(b)).max()})"
    assert rel_l2 <= ATTN_REL_L2, f"rel-L2 {rel_l2}"
    return max_abs, rel_l2


class Pair:
    """The same workload driven through the CUDA library and through the oracle."""

    def __init__(self, wl, heart, oracle, device="cuda", gate=(0.0, 1.0), idx_pad=0, gen_device=None):
        self.wl, self.heart, self.oracle = wl, heart, oracle
        self.seq = inputs.Sequence(wl, gen_device or device)
        nb = wl.n_blocks
        self.cfg = heart.make_config(wl.B, wl.H, wl.N, wl.block, gate_lo=gate[0], gate_hi=gate[1],
                                     idx_stride=nb + idx_pad)
        self.gate = gate
        self.gst = heart.State(self.cfg, device)
        self.ws = heart.new_workspace(self.cfg, device)
        self.ost = oracle.State(wl.B, wl.H, wl.N, wl.D, wl.block, idx_stride=nb + idx_pad)
        self.delta = torch.tensor(wl.delta, dtype=torch.float64, device=device)
        self.tau = torch.tensor(wl.tau, dtype=torch.float64, device=device)
        self.device = device
        self.load()

    def load(self):
        self.Q, self.K, self.V = (t.to(self.device) for t in self.seq.bf16())
        self.Qb, self.Kb, self.Vb = (inputs.bits(t) for t in (self.Q, self.K, self.V))

    def advance(self):
        self.seq.advance()
        self.load()

    def probs_row(self, r, I):
        return self.oracle.probs_row(self.Qb, self.Kb, self.wl.block, r, I)

    def gpu_step(self, flags=0, want_lse=True):
        h, wl = self.heart, self.wl
        self.cfg.flags = flags
        O = torch.full_like(self.Q, float("nan"))
        lse = torch.full((wl.R, wl.N), float("nan"), dtype=torch.float32, device=self.device) if want_lse else None
        drift = torch.empty(wl.R, dtype=torch.float64, device=self.device)
        refresh = torch.empty(wl.R, dtype=torch.uint8, device=self.device)
        h.heart_step(self.cfg, self.Q, self.K, self.V, self.delta, self.tau, self.gst, O, self.ws, lse=lse,
                     drift_out=drift, refresh_out=refresh)
        assert h.heart_get_status(self.ws) == 0
        return O, lse, to_np(drift), to_np(refresh)

    def oracle_step(self, flags=0, want_O=True):
        return self.oracle.step(self.Qb, self.Kb, self.Vb, self.wl.delta, self.wl.tau, self.ost,
                                gate_lo=self.gate[0], gate_hi=self.gate[1], flags=flags, want_O=want_O,
                                want_lse=want_O)


def sample_rows(rs, R, nb, kv_cnt, n):
    """(r, I) sample: row 0, the ragged last block, the densest and the sparsest row; two adjacent query
    blocks (the two halves of one 128-row tile at block 64) of the first head, whose tiles run in index
    order, and of the last head, whose tiles the attention launch orders longest-first; then random."""
    flat = kv_cnt.reshape(-1)
    picks = {(0, 0), (R - 1, nb - 1), divmod(int(flat.argmax()), nb), divmod(int(flat.argmin()), nb)}
    if nb >= 4:
        picks |= {(0, 0), (0, 1), (R - 1, 2), (R - 1, 3)}
    while len(picks) < n:
        picks.add((int(rs.randint(R)), int(rs.randint(nb))))
    picks = sorted(picks)
    return np.array([p[0] for p in picks], np.int32), np.array([p[1] for p in picks], np.int32)
