"""Thin Python binding of the C ABI in include/heart.h (argument marshalling only).

Every step of the hot path runs in the CUDA kernels of libheart.so; torch is used
for device memory and streams.  Importing this module loads the library and
fails loudly if it has not been built -- there is no CPU or eager fallback.
"""
from __future__ import annotations

import ctypes as C
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.environ.get("HEART_LIB") or os.path.join(_HERE, "libheart.so")

OK, ERR_INVALID, ERR_UNSUPPORTED, ERR_CUDA, ERR_DEVICE_CHECK, ERR_TOO_LARGE, ERR_INFEASIBLE = 0, 1, 2, 3, 4, 5, 6
STATIC_SCRATCH_BYTES = 16 << 20
FORCE_REFRESH, FORCE_DENSE, BLOCK_MEANS_VALID, ESTIMATOR_ANTIDIAG = 1, 2, 4, 8
MAX_BLOCKS = 1024

# Every symbol include/heart.h declares.
SYMBOLS = (
    "heart_workspace_bytes", "heart_state_reset", "heart_drift", "heart_predict_mask",
    "heart_block_sparse_attn", "heart_step", "heart_step_host", "heart_get_status", "heart_strerror",
    "heart_last_launch_count", "heart_drift_static", "heart_full_token_drift", "heart_mask_iou",
    "heart_band_error_workspace_bytes", "heart_band_error", "heart_drift_workspace_bytes",
    "heart_assign_thresholds",
)


class Config(C.Structure):
    _fields_ = [("B", C.c_int32), ("H", C.c_int32), ("N", C.c_int32), ("D", C.c_int32),
                ("block", C.c_int32),
                ("stride_b", C.c_int64), ("stride_h", C.c_int64), ("stride_n", C.c_int64),
                ("scale", C.c_double), ("gate_lo", C.c_double), ("gate_hi", C.c_double),
                ("idx_stride", C.c_int32), ("flags", C.c_uint32)]


class StateStruct(C.Structure):
    _fields_ = [("anchor_q", C.c_void_p), ("anchor_k", C.c_void_p), ("has_anchor", C.c_void_p),
                ("mask_bits", C.c_void_p), ("kv_idx", C.c_void_p), ("kv_cnt", C.c_void_p)]


class HeartError(RuntimeError):
    def __init__(self, code):
        self.code = code
        super().__init__(f"heart error {code}: {lib().heart_strerror(code).decode()}")


_lib = None


def lib():
    """The loaded libheart.so (raises if it is missing: build it with build.py)."""
    global _lib
    if _lib is None:
        _lib = load(_LIB_PATH)
    return _lib


def load(path):
    """Loads a build of the library and declares its signatures (the tests use this for the
    test-hook build; everything else goes through lib())."""
    if True:
        if not os.path.exists(path):
            raise ImportError(f"{path} not found: run `python -m paper_2605_14513_b200.build` "
                              "(or __graft_entry__.build()) -- there is no fallback path")
        l = C.CDLL(path)
        l.heart_workspace_bytes.restype = C.c_size_t
        l.heart_workspace_bytes.argtypes = [C.POINTER(Config)]
        l.heart_drift_workspace_bytes.restype = C.c_size_t
        l.heart_drift_workspace_bytes.argtypes = [C.POINTER(Config)]
        l.heart_strerror.restype = C.c_char_p
        l.heart_strerror.argtypes = [C.c_int]
        l.heart_last_launch_count.restype = C.c_int
        vp = C.c_void_p
        l.heart_state_reset.argtypes = [C.POINTER(Config), C.POINTER(StateStruct), vp]
        l.heart_drift.argtypes = [C.POINTER(Config), vp, vp, vp, C.POINTER(StateStruct), vp, vp, vp, vp]
        l.heart_predict_mask.argtypes = [C.POINTER(Config), vp, vp, vp, vp, C.POINTER(StateStruct), vp, vp]
        l.heart_block_sparse_attn.argtypes = [C.POINTER(Config), vp, vp, vp, vp, vp, vp, vp, vp, vp]
        l.heart_step.argtypes = [C.POINTER(Config), vp, vp, vp, vp, vp, C.POINTER(StateStruct), vp, vp, vp, vp, vp, vp]
        l.heart_step_host.argtypes = [C.POINTER(Config), vp, vp, vp, vp, vp, C.POINTER(StateStruct)] + [vp] * 9
        l.heart_get_status.argtypes = [vp, vp, C.POINTER(C.c_int32)]
        l.heart_drift_static.argtypes = [C.POINTER(Config), vp, vp, vp, C.POINTER(StateStruct), vp, vp, vp]
        l.heart_drift_static.restype = C.c_int
        l.heart_full_token_drift.argtypes = [C.POINTER(Config)] + [vp] * 7
        l.heart_full_token_drift.restype = C.c_int
        l.heart_mask_iou.argtypes = [C.POINTER(Config)] + [vp] * 5
        l.heart_mask_iou.restype = C.c_int
        l.heart_band_error_workspace_bytes.argtypes = [C.c_int32] * 4
        l.heart_band_error_workspace_bytes.restype = C.c_size_t
        l.heart_band_error.argtypes = [vp, vp] + [C.c_int32] * 4 + [C.POINTER(C.c_double), C.c_double, vp, vp, vp]
        l.heart_band_error.restype = C.c_int
        l.heart_assign_thresholds.argtypes = [vp, vp, C.c_int32, C.c_int32, C.c_double, vp, C.POINTER(C.c_double),
                                              C.POINTER(C.c_double), C.POINTER(C.c_int32)]
        l.heart_assign_thresholds.restype = C.c_int
        for fn in ("heart_state_reset", "heart_drift", "heart_predict_mask", "heart_block_sparse_attn",
                   "heart_step", "heart_step_host", "heart_get_status"):
            getattr(l, fn).restype = C.c_int
    return l


def _ptr(t):
    return None if t is None else C.c_void_p(t.data_ptr())


def _stream():
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


def _check(rc):
    if rc != OK:
        raise HeartError(rc)


def _with_flags(cfg, flags):
    c = Config.from_buffer_copy(cfg)
    c.flags = flags
    return c


def n_blocks(N, block):
    return (N + block - 1) // block


def make_config(B, H, N, block, D=128, scale=0.0, gate_lo=0.0, gate_hi=1.0, idx_stride=None, flags=0,
                strides=(0, 0, 0)) -> Config:
    nb = n_blocks(N, block)
    return Config(B, H, N, D, block, strides[0], strides[1], strides[2], scale, gate_lo, gate_hi,
                  idx_stride if idx_stride is not None else nb, flags)


def config_for(x: torch.Tensor, block, **kw) -> Config:
    """Config for a [B, H, N, D] bf16 tensor (strides taken from the tensor)."""
    assert x.dim() == 4 and x.dtype == torch.bfloat16 and x.stride(3) == 1
    B, H, N, D = x.shape
    return make_config(B, H, N, block, D=D, strides=(x.stride(0), x.stride(1), x.stride(2)), **kw)


class State:
    """Caller-owned TMR state of one layer (device tensors + the C struct that points at them)."""

    def __init__(self, cfg: Config, device="cuda"):
        R, nb = cfg.B * cfg.H, n_blocks(cfg.N, cfg.block)
        self.R, self.nb, self.W = R, nb, (nb + 31) // 32
        self.anchor_q = torch.zeros((R, cfg.D), dtype=torch.float64, device=device)
        self.anchor_k = torch.zeros((R, cfg.D), dtype=torch.float64, device=device)
        self.has_anchor = torch.zeros(R, dtype=torch.uint8, device=device)
        self.mask_bits = torch.zeros((R, nb, self.W), dtype=torch.int32, device=device)
        self.kv_idx = torch.full((R, nb, cfg.idx_stride), -1, dtype=torch.int32, device=device)
        self.kv_cnt = torch.zeros((R, nb), dtype=torch.int32, device=device)
        self.struct = StateStruct(*(t.data_ptr() for t in self.tensors()))

    def tensors(self):
        return (self.anchor_q, self.anchor_k, self.has_anchor, self.mask_bits, self.kv_idx, self.kv_cnt)

    def state_dict(self):
        return {k: getattr(self, k).clone() for k in ("anchor_q", "anchor_k", "has_anchor", "mask_bits", "kv_idx", "kv_cnt")}

    def load_state_dict(self, d):
        for k, v in d.items():
            getattr(self, k).copy_(v)


def workspace_bytes(cfg: Config) -> int:
    return int(lib().heart_workspace_bytes(C.byref(cfg)))


def drift_workspace_bytes(cfg: Config) -> int:
    """The leading part of the workspace that heart_drift alone touches."""
    return int(lib().heart_drift_workspace_bytes(C.byref(cfg)))


def new_workspace(cfg: Config, device="cuda") -> torch.Tensor:
    n = workspace_bytes(cfg)
    if n == 0:
        raise HeartError(ERR_UNSUPPORTED)
    return torch.zeros(n, dtype=torch.uint8, device=device)


def heart_state_reset(cfg, st: State):
    _check(lib().heart_state_reset(C.byref(cfg), C.byref(st.struct), _stream()))


def heart_drift(cfg, Q, K, delta, st: State, ws, drift_out=None, refresh_out=None):
    _check(lib().heart_drift(C.byref(cfg), _ptr(Q), _ptr(K), _ptr(delta), C.byref(st.struct), _ptr(drift_out),
                             _ptr(refresh_out), _ptr(ws), _stream()))


def heart_predict_mask(cfg, Q, K, tau, st: State, ws, refresh=None, means_valid=False):
    """means_valid: pass HEART_BLOCK_MEANS_VALID for this call (heart_drift has just run on the same
    Q, K and workspace), so the pass over Q and K is not repeated."""
    if means_valid:
        cfg = _with_flags(cfg, cfg.flags | BLOCK_MEANS_VALID)
    _check(lib().heart_predict_mask(C.byref(cfg), _ptr(Q), _ptr(K), _ptr(tau), _ptr(refresh), C.byref(st.struct),
                                    _ptr(ws), _stream()))


def heart_block_sparse_attn(cfg, Q, K, V, kv_idx, kv_cnt, O, ws, lse=None):
    _check(lib().heart_block_sparse_attn(C.byref(cfg), _ptr(Q), _ptr(K), _ptr(V), _ptr(kv_idx), _ptr(kv_cnt),
                                         _ptr(O), _ptr(lse), _ptr(ws), _stream()))


def heart_step(cfg, Q, K, V, delta, tau, st: State, O, ws, lse=None, drift_out=None, refresh_out=None):
    _check(lib().heart_step(C.byref(cfg), _ptr(Q), _ptr(K), _ptr(V), _ptr(delta), _ptr(tau), C.byref(st.struct),
                            _ptr(O), _ptr(lse), _ptr(drift_out), _ptr(refresh_out), _ptr(ws), _stream()))


def heart_step_host(cfg, Qh, Kh, Vh, delta, tau, st: State, Oh, staging, ws, drift_host=None, refresh_host=None):
    """Host-buffer step: Qh/Kh/Vh/Oh (and the optional drift/refresh) are CPU tensors, ideally pinned;
    `staging` = (Q_dev, K_dev, V_dev, O_dev) device tensors.  Asynchronous on the current stream."""
    for t in (Qh, Kh, Vh, Oh):
        assert t.device.type == "cpu" and t.is_contiguous()
    _check(lib().heart_step_host(C.byref(cfg), _ptr(Qh), _ptr(Kh), _ptr(Vh), _ptr(delta), _ptr(tau),
                                 C.byref(st.struct), _ptr(Oh), _ptr(drift_host), _ptr(refresh_host),
                                 _ptr(staging[0]), _ptr(staging[1]), _ptr(staging[2]), _ptr(staging[3]), _ptr(ws),
                                 _stream()))


def heart_drift_static(cfg, Q, K, delta, st: State, drift_out=None, refresh_out=None):
    """heart_drift for callers that cannot allocate: scratch comes from the library's built-in
    16 MiB array (shapes that need more raise ERR_TOO_LARGE).  Calls on one device must not overlap."""
    _check(lib().heart_drift_static(C.byref(cfg), _ptr(Q), _ptr(K), _ptr(delta), C.byref(st.struct),
                                    _ptr(drift_out), _ptr(refresh_out), _stream()))


def heart_full_token_drift(cfg, Qa, Ka, Qb, Kb, drift_out, ws):
    """Full-token drift (Eq. full-token drift) between a cached step (Qa, Ka) and the current one
    (Qb, Kb) into drift_out [R] fp64."""
    _check(lib().heart_full_token_drift(C.byref(cfg), _ptr(Qa), _ptr(Ka), _ptr(Qb), _ptr(Kb), _ptr(drift_out),
                                        _ptr(ws), _stream()))


def heart_mask_iou(cfg, mask_a, mask_b, iou_out, counts_out=None):
    """Block-mask IoU per head between two [R, n_b, W] bit masks (Observation I) into iou_out [R] fp64;
    counts_out: optional int64 [R, 2] = (intersection, union)."""
    _check(lib().heart_mask_iou(C.byref(cfg), _ptr(mask_a), _ptr(mask_b), _ptr(iou_out), _ptr(counts_out),
                                _stream()))


def heart_band_error(y_sparse, y_dense, weights=(1.0, 0.5, 0.01, 0.01), eps=1e-10):
    """Four-band 3-D DFT calibration error of y_sparse against y_dense (fp32 [C, T, H, W] on the GPU).
    Returns a device tensor of 6 doubles: (e, E_LL, E_LH, E_HL, E_HH, denominator)."""
    assert y_sparse.dtype == torch.float32 and y_dense.dtype == torch.float32
    assert y_sparse.is_contiguous() and y_dense.is_contiguous() and y_sparse.shape == y_dense.shape
    Cc, T, H, W = y_sparse.shape
    nbytes = lib().heart_band_error_workspace_bytes(Cc, T, H, W)
    if nbytes == 0:
        raise HeartError(ERR_INVALID)
    ws = torch.empty(nbytes, dtype=torch.uint8, device=y_sparse.device)
    out = torch.empty(6, dtype=torch.float64, device=y_sparse.device)
    w = (C.c_double * 4)(*weights)
    _check(lib().heart_band_error(_ptr(y_sparse), _ptr(y_dense), Cc, T, H, W, w, float(eps), _ptr(out), _ptr(ws),
                                  _stream()))
    return out


def heart_assign_thresholds(E, S, S_min):
    """One threshold candidate per head under a mean-sparsity budget (host-side, exact).
    E, S: [n_heads, n_candidates] float64 numpy arrays.  Returns (choice int32 [n_heads], objective,
    mean sparsity, proved_optimal) or None when no assignment meets the budget."""
    import numpy as np

    E = np.ascontiguousarray(E, np.float64)
    S = np.ascontiguousarray(S, np.float64)
    M, K = E.shape
    assert S.shape == (M, K)
    choice = np.empty(M, np.int32)
    obj, ms, proved = C.c_double(0), C.c_double(0), C.c_int32(0)
    rc = lib().heart_assign_thresholds(E.ctypes.data_as(C.c_void_p), S.ctypes.data_as(C.c_void_p), M, K,
                                       float(S_min), choice.ctypes.data_as(C.c_void_p), C.byref(obj), C.byref(ms),
                                       C.byref(proved))
    if rc == ERR_INFEASIBLE:
        return None
    _check(rc)
    return choice, obj.value, ms.value, bool(proved.value)


def heart_get_status(ws) -> int:
    code = C.c_int32(0)
    _check(lib().heart_get_status(_ptr(ws), _stream(), C.byref(code)))
    return code.value


def heart_last_launch_count() -> int:
    return int(lib().heart_last_launch_count())
