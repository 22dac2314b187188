"""ctypes front end of the CPU oracle (oracle/heart_oracle.c).

TEST INFRASTRUCTURE ONLY: imported by the tests, the smoke check and the
benchmark's CPU-baseline leg.  For the layer-step path this file holds no
arithmetic of its own -- every number comes from the C functions; it only builds
the shared object with gcc, marshals numpy arrays and allocates outputs.  The one
exception is at the end: band_error (the offline calibration's four-band
spectral error) is written here, in numpy, straight from its definition.

bf16 tensors are passed as numpy uint16 arrays holding the raw bf16 bits,
contiguous [R, N, D] (R = batch * heads).
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "heart_oracle.c")
_LIB = os.path.join(_HERE, "libheart_oracle.so")

FORCE_REFRESH = 1
FORCE_DENSE = 2

_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (-O2 -fopenmp).  Returns the library path."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        subprocess.check_call(
            ["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c99", "-o", _LIB, _SRC, "-lm"]
        )
    return _LIB


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.oracle_top_p.restype = C.c_int
    return _lib


def _p(a, t=None):
    if a is None:
        return None
    return a.ctypes.data_as(C.c_void_p)


def _u16(x):
    x = np.ascontiguousarray(x)
    assert x.dtype == np.uint16, "bf16 tensors are passed as raw uint16 bits"
    return x


def n_blocks(N, b):
    return (N + b - 1) // b


def token_mean(X):
    X = _u16(X)
    R, N, D = X.shape
    out = np.empty((R, D), np.float64)
    lib().oracle_token_mean(_p(X), R, N, D, _p(out))
    return out


def pooled_drift(aq, ak, mq, mk):
    aq, ak, mq, mk = (np.ascontiguousarray(a, np.float64) for a in (aq, ak, mq, mk))
    R, D = aq.shape
    out = np.empty(R, np.float64)
    lib().oracle_pooled_drift(_p(aq), _p(ak), _p(mq), _p(mk), R, D, _p(out))
    return out


def full_token_drift(Qa, Ka, Qb, Kb):
    Qa, Ka, Qb, Kb = map(_u16, (Qa, Ka, Qb, Kb))
    R, N, D = Qa.shape
    out = np.empty(R, np.float64)
    lib().oracle_full_token_drift(_p(Qa), _p(Ka), _p(Qb), _p(Kb), R, N, D, _p(out))
    return out


class State:
    """TMR state of one layer: anchors, has_anchor, cached masks (Algorithm 1)."""

    def __init__(self, B, H, N, D, block, idx_stride=None):
        self.B, self.H, self.N, self.D, self.block = B, H, N, D, block
        R, nb = B * H, n_blocks(N, block)
        self.R, self.nb, self.W = R, nb, (nb + 31) // 32
        self.idx_stride = idx_stride or nb
        self.anchor_q = np.zeros((R, D), np.float64)
        self.anchor_k = np.zeros((R, D), np.float64)
        self.has_anchor = np.zeros(R, np.uint8)
        self.mask_bits = np.zeros((R, nb, self.W), np.uint32)
        self.kv_idx = np.full((R, nb, self.idx_stride), -1, np.int32)
        self.kv_cnt = np.zeros((R, nb), np.int32)

    def copy(self):
        s = State(self.B, self.H, self.N, self.D, self.block, self.idx_stride)
        for k in ("anchor_q", "anchor_k", "has_anchor", "mask_bits", "kv_idx", "kv_cnt"):
            setattr(s, k, getattr(self, k).copy())
        return s


def decide(mq, mk, delta, st: State, gate_lo=0.0, gate_hi=1.0, flags=0):
    mq = np.ascontiguousarray(mq, np.float64)
    mk = np.ascontiguousarray(mk, np.float64)
    delta = np.ascontiguousarray(delta, np.float64)
    drift = np.empty(st.R, np.float64)
    refresh = np.empty(st.R, np.uint8)
    lib().oracle_decide(_p(mq), _p(mk), _p(delta), st.B, st.H, st.D, C.c_double(gate_lo),
                        C.c_double(gate_hi), C.c_uint32(flags), _p(st.anchor_q), _p(st.anchor_k),
                        _p(st.has_anchor), _p(drift), _p(refresh))
    return drift, refresh


def block_pool(X, b):
    X = _u16(X)
    R, N, D = X.shape
    out = np.empty((R, n_blocks(N, b), D), np.float64)
    lib().oracle_block_pool(_p(X), R, N, D, b, _p(out))
    return out


def block_probs(qp, Kp, scale):
    qp = np.ascontiguousarray(qp, np.float64)
    Kp = np.ascontiguousarray(Kp, np.float64)
    nb, D = Kp.shape
    P = np.empty(nb, np.float64)
    lib().oracle_block_probs(_p(qp), _p(Kp), nb, D, C.c_double(scale), _p(P))
    return P


def top_p(P, tau):
    """Returns (keep[n] uint8, k*, c_{k*}, c_{k*-1})."""
    P = np.ascontiguousarray(P, np.float64)
    n = P.shape[0]
    keep = np.empty(n, np.uint8)
    ca, cb = C.c_double(0), C.c_double(0)
    k = lib().oracle_top_p(_p(P), n, C.c_double(tau), _p(keep), C.byref(ca), C.byref(cb))
    return keep, k, ca.value, cb.value


def predict_mask(Q, K, b, tau, st: State, refresh=None, scale=0.0, flags=0):
    Q, K = _u16(Q), _u16(K)
    R, N, D = Q.shape
    tau = np.ascontiguousarray(tau, np.float64)
    if refresh is not None:
        refresh = np.ascontiguousarray(refresh, np.uint8)
    lib().oracle_predict_mask(_p(Q), _p(K), R, N, D, b, C.c_double(scale), _p(tau), _p(refresh),
                              C.c_uint32(flags), _p(st.mask_bits), _p(st.kv_idx), _p(st.kv_cnt),
                              st.idx_stride)


ANTIDIAG_STRIDE = 16


def antidiag_probs_row(Q, K, b, r, I, s=ANTIDIAG_STRIDE, scale=0.0):
    """Block importances of query block I of head r under the strided antidiagonal estimator."""
    Q, K = _u16(Q), _u16(K)
    R, N, D = Q.shape
    assert b % s == 0
    P = np.empty(n_blocks(N, b), np.float64)
    lib().oracle_antidiag_probs_row(_p(Q), _p(K), N, D, b, int(s), C.c_double(scale), int(r), int(I), _p(P))
    return P


def predict_mask_antidiag(Q, K, b, tau, st: State, refresh=None, s=ANTIDIAG_STRIDE, scale=0.0, flags=0):
    Q, K = _u16(Q), _u16(K)
    R, N, D = Q.shape
    assert b % s == 0
    tau = np.ascontiguousarray(tau, np.float64)
    if refresh is not None:
        refresh = np.ascontiguousarray(refresh, np.uint8)
    lib().oracle_predict_mask_antidiag(_p(Q), _p(K), R, N, D, b, int(s), C.c_double(scale), _p(tau), _p(refresh),
                                       C.c_uint32(flags), _p(st.mask_bits), _p(st.kv_idx), _p(st.kv_cnt),
                                       st.idx_stride)


def probs_row(Q, K, b, r, I, scale=0.0):
    Q, K = _u16(Q), _u16(K)
    R, N, D = Q.shape
    P = np.empty(n_blocks(N, b), np.float64)
    lib().oracle_probs_row(_p(Q), _p(K), N, D, b, C.c_double(scale), int(r), int(I), _p(P))
    return P


def attn_rows(Q, K, V, b, kv_idx, kv_cnt, rows_r, rows_I, scale=0.0, want_lse=False):
    """O7 on the listed (r, I) query blocks -> out [n, b, D] fp64 (rows past N are NaN)."""
    Q, K, V = _u16(Q), _u16(K), _u16(V)
    R, N, D = Q.shape
    kv_idx = np.ascontiguousarray(kv_idx, np.int32)
    kv_cnt = np.ascontiguousarray(kv_cnt, np.int32)
    rows_r = np.ascontiguousarray(rows_r, np.int32)
    rows_I = np.ascontiguousarray(rows_I, np.int32)
    n = rows_r.shape[0]
    out = np.full((n, b, D), np.nan, np.float64)
    lse = np.full((n, b), np.nan, np.float64) if want_lse else None
    lib().oracle_attn_rows(_p(Q), _p(K), _p(V), N, D, b, C.c_double(scale), _p(kv_idx), _p(kv_cnt),
                           kv_idx.shape[-1], _p(rows_r), _p(rows_I), n, _p(out), _p(lse))
    return (out, lse) if want_lse else out


def block_sparse_attn(Q, K, V, b, kv_idx, kv_cnt, scale=0.0, want_lse=False):
    Q, K, V = _u16(Q), _u16(K), _u16(V)
    R, N, D = Q.shape
    kv_idx = np.ascontiguousarray(kv_idx, np.int32)
    kv_cnt = np.ascontiguousarray(kv_cnt, np.int32)
    O = np.empty((R, N, D), np.float64)
    lse = np.empty((R, N), np.float64) if want_lse else None
    lib().oracle_block_sparse_attn(_p(Q), _p(K), _p(V), R, N, D, b, C.c_double(scale), _p(kv_idx),
                                   _p(kv_cnt), kv_idx.shape[-1], _p(O), _p(lse))
    return (O, lse) if want_lse else O


def dense_attn(Q, K, V, scale=0.0):
    Q, K, V = _u16(Q), _u16(K), _u16(V)
    R, N, D = Q.shape
    O = np.empty((R, N, D), np.float64)
    lib().oracle_dense_attn(_p(Q), _p(K), _p(V), R, N, D, C.c_double(scale), _p(O))
    return O


def step(Q, K, V, delta, tau, st: State, scale=0.0, gate_lo=0.0, gate_hi=1.0, flags=0,
         want_O=True, want_lse=False):
    """O8.  Returns (O or None, lse or None, drift[R], refresh[R]); st is updated in place."""
    Q, K, V = _u16(Q), _u16(K), _u16(V)
    R, N, D = Q.shape
    assert R == st.R
    delta = np.ascontiguousarray(delta, np.float64)
    tau = np.ascontiguousarray(tau, np.float64)
    O = np.empty((R, N, D), np.float64) if want_O else None
    lse = np.empty((R, N), np.float64) if (want_O and want_lse) else None
    drift = np.empty(R, np.float64)
    refresh = np.empty(R, np.uint8)
    lib().oracle_step(_p(Q), _p(K), _p(V), st.B, st.H, N, D, st.block, C.c_double(scale),
                      C.c_double(gate_lo), C.c_double(gate_hi), C.c_uint32(flags), _p(delta), _p(tau),
                      _p(st.anchor_q), _p(st.anchor_k), _p(st.has_anchor), _p(st.mask_bits),
                      _p(st.kv_idx), _p(st.kv_cnt), st.idx_stride, _p(O), _p(lse), _p(drift),
                      _p(refresh))
    return O, lse, drift, refresh


def mask_iou(mask_a, mask_b, nb):
    """Block-mask IoU per head between two [R, nb, W] bit masks -> (iou[R], counts[R, 2])."""
    mask_a = np.ascontiguousarray(mask_a, np.uint32)
    mask_b = np.ascontiguousarray(mask_b, np.uint32)
    R = mask_a.shape[0]
    iou = np.empty(R, np.float64)
    counts = np.empty((R, 2), np.int64)
    lib().oracle_mask_iou(_p(mask_a), _p(mask_b), R, int(nb), _p(iou), _p(counts))
    return iou, counts


def assign_thresholds(E, S, S_min):
    """One-choice-per-head assignment under a sparsity budget by exhaustive enumeration.
    E, S: [M, K].  Returns (choice[M] int32, objective, mean sparsity) or None when infeasible."""
    E = np.ascontiguousarray(E, np.float64)
    S = np.ascontiguousarray(S, np.float64)
    M, K = E.shape
    assert S.shape == (M, K) and K ** M <= 20_000_000, "exhaustive: keep K^M small"
    choice = np.empty(M, np.int32)
    obj, ms = C.c_double(0), C.c_double(0)
    lib().oracle_assign_thresholds.restype = C.c_int
    ok = lib().oracle_assign_thresholds(_p(E), _p(S), M, K, C.c_double(S_min), _p(choice), C.byref(obj), C.byref(ms))
    return (choice, obj.value, ms.value) if ok else None


# ---------------------------------------------------------------------------
# Frequency-aware velocity error of the offline calibration (Eq. calibration error; appendix
# "Frequency-aware velocity error"): 3-D DFT over (t, y, x) of every channel, fftshift, a frequency
# is low along an axis of length n when it lies within floor(n/4) of the zero-frequency centre;
# LL = low t, low y and low x; LH = low t, high on at least one spatial axis; HL = high t, low on
# both spatial axes; HH = the rest.  Written straight from that definition with numpy's FFT.
# ---------------------------------------------------------------------------
BAND_WEIGHTS = (1.0, 0.5, 0.01, 0.01)  # (LL, LH, HL, HH)
BAND_EPS = 1e-10


def low_frequency_mask(n):
    """Boolean mask over the fftshift-ed frequency index of an axis of length n."""
    idx = np.arange(n)
    return np.abs(idx - n // 2) <= n // 4


def band_error(y_sparse, y_dense, weights=BAND_WEIGHTS, eps=BAND_EPS):
    """y_*: [C, T, H, W].  Returns (e, band energies [LL, LH, HL, HH], denominator)."""
    ys = np.asarray(y_sparse, np.float64)
    yd = np.asarray(y_dense, np.float64)
    err = ys - yd
    E = np.fft.fftshift(np.fft.fftn(err, axes=(1, 2, 3)), axes=(1, 2, 3))
    Y = np.fft.fftn(yd, axes=(1, 2, 3))
    _, T, H, W = err.shape
    lt = low_frequency_mask(T)[:, None, None]
    ls = low_frequency_mask(H)[None, :, None] & low_frequency_mask(W)[None, None, :]
    p = (E.real ** 2 + E.imag ** 2).sum(axis=0)
    bands = np.array([p[lt & ls].sum(), p[lt & ~ls].sum(), p[~lt & ls].sum(), p[~lt & ~ls].sum()])
    denom = float((Y.real ** 2 + Y.imag ** 2).sum() + eps)
    return float(np.dot(np.asarray(weights, np.float64), bands) / denom), bands, denom
