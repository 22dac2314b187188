"""Host-side checks of the C-ABI library that need no GPU: it loads, exports every symbol the
header declares, sizes its workspace, and rejects bad arguments before touching the device."""
import ctypes as C
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def heart():
    from paper_2605_14513_b200 import build, heart as h

    build.build()
    return h


def test_every_declared_symbol_is_exported(heart):
    text = open(os.path.join(ROOT, "include", "heart.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    declared = set(re.findall(r"\b(heart_[a-z_]+)\s*\(", text))
    assert declared == set(heart.SYMBOLS)
    lib = heart.lib()
    for name in declared:
        assert hasattr(lib, name), name


def test_struct_layout_matches_header(heart):
    # int32 x5, pad, int64 x3, double x3, int32, uint32
    assert C.sizeof(heart.Config) == 80
    assert heart.Config.stride_b.offset == 24 and heart.Config.scale.offset == 48
    assert heart.Config.idx_stride.offset == 72 and heart.Config.flags.offset == 76
    assert C.sizeof(heart.StateStruct) == 48


def test_workspace_size_and_shape_validation(heart):
    cfg = heart.make_config(1, 12, 32760, 64)
    n = heart.workspace_bytes(cfg)
    nb = 512
    assert n >= 2 * 12 * nb * 128 * 8 and n % 256 == 0
    assert heart.workspace_bytes(heart.make_config(1, 12, 32760, 64, D=64)) == 0      # head_dim
    assert heart.workspace_bytes(heart.make_config(1, 12, 32760, 32)) == 0            # block size
    assert heart.workspace_bytes(heart.make_config(1, 1, 64 * 1025, 64)) == 0         # too many blocks
    assert heart.workspace_bytes(heart.make_config(1, 1, 64 * 1024, 64)) > 0
    assert heart.workspace_bytes(heart.make_config(1, 0, 128, 64)) == 0
    # the drift-only prefix: block means, token means, flags -- without the pooled scores of the mask
    # predictor (8 bytes per (head, query block, key block) with the key blocks padded to 32)
    d = heart.drift_workspace_bytes(cfg)
    assert 2 * 12 * nb * 128 * 8 <= d < n and d % 256 == 0
    assert n - d == 12 * nb * nb * 8
    assert d <= 16 << 20                                                               # fits the built-in scratch
    assert heart.drift_workspace_bytes(heart.make_config(1, 12, 32760, 32)) == 0


def test_bad_arguments_are_rejected_on_the_host(heart):
    lib = heart.lib()
    cfg = heart.make_config(1, 2, 2048, 64)
    st = heart.StateStruct(0, 0, 0, 0, 0, 0)
    null = C.c_void_p(0)
    fake = C.c_void_p(256)  # never dereferenced: validation fails first
    assert lib.heart_drift(C.byref(cfg), null, fake, fake, C.byref(st), null, null, fake, null) == heart.ERR_INVALID
    assert lib.heart_drift(C.byref(cfg), fake, fake, fake, C.byref(st), null, null, fake, null) == heart.ERR_INVALID  # null state
    st2 = heart.StateStruct(256, 256, 256, 256, 256, 256)
    misaligned = C.c_void_p(264)
    assert lib.heart_drift(C.byref(cfg), misaligned, fake, fake, C.byref(st2), null, null, fake, null) == heart.ERR_INVALID
    assert lib.heart_step(C.byref(cfg), fake, fake, fake, fake, fake, C.byref(st2), null, null, null, null, fake, null) == heart.ERR_INVALID
    bad = heart.make_config(1, 2, 2048, 64, idx_stride=3)
    assert lib.heart_block_sparse_attn(C.byref(bad), fake, fake, fake, fake, fake, fake, null, fake, null) == heart.ERR_INVALID
    bad = heart.make_config(1, 2, 2048, 96)
    assert lib.heart_block_sparse_attn(C.byref(bad), fake, fake, fake, fake, fake, fake, null, fake, null) == heart.ERR_UNSUPPORTED
    bad = heart.make_config(1, 2, 2048, 64, strides=(2048 * 128 * 2, 2048 * 128, 100))
    assert lib.heart_predict_mask(C.byref(bad), fake, fake, fake, null, C.byref(st2), fake, null) == heart.ERR_INVALID
    assert b"invalid" in lib.heart_strerror(heart.ERR_INVALID)
    assert b"unsupported" in lib.heart_strerror(heart.ERR_UNSUPPORTED)
