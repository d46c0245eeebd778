"""Host-side checks that need no GPU: the shared library loads, exports every symbol the
header declares, and rejects bad arguments before touching the device."""
import ctypes as C
import os
import re

import pytest

from paper_2502_00425_b200 import binding as B
from paper_2502_00425_b200 import build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build_library()
    return B.load()


def test_header_symbols_are_exported(lib):
    hdr = open(os.path.join(ROOT, "include", "mq.h")).read()
    declared = set(re.findall(r"\b(mq_[a-z0-9_]+)\s*\(", hdr))
    assert {"mq_calibrate_static_scales", "mq_pack_w4", "mq_aifs_reorder", "mq_fwht_quant_i8",
            "mq_w4a8_msq_linear", "mq_attn_mask_remap"} <= declared
    for name in declared:
        assert hasattr(lib, name), name
    assert declared == set(B.EXPORTED)
    assert lib.mq_version() == 1


def test_status_strings(lib):
    assert B.status_string(0) == "MQ_OK"
    assert B.status_string(B.MQ_ERR_ALIGNMENT) == "MQ_ERR_ALIGNMENT"
    assert B.status_string(-99) == "MQ_ERR_UNKNOWN"


def test_size_queries(lib):
    assert B.mq_w4_layout_bytes(128, 128) == 8192
    assert B.mq_w4_layout_bytes(3584, 18944) == 28 * 148 * 8192
    assert B.mq_w4_layout_bytes(16, 32) == 8192                     # padded to one tile
    assert B.mq_w4_layout_bytes(0, 32) == 0
    big = B.mq_workspace_bytes(1088, 18944, 3584, 128)
    assert big >= 256 + 1088 * 18944
    assert B.mq_workspace_bytes(1088, 18944, 3584, 0, B.MQ_FLAG_X_IS_INT8) == 256
    assert B.mq_workspace_bytes(8, 4096, 256) >= 256 + 8 * 4096 + 2 * 8 * 256 * 4   # split-K slices
    assert (B.mq_workspace_bytes(8, 4096, 256) - 256 - 8 * 4096) % (8 * 256 * 4) == 0  # whole [T,N] slices
    assert B.mq_workspace_bytes(8, 100, 256) == 0                   # K % 32
    assert B.mq_workspace_bytes(8, 128, 100) == 0                   # N % 16
    assert B.mq_workspace_bytes(8, 128, 128, 48) == 0               # rotation block not a power of two


def _desc(T=8, K=128, N=128, rot=0, group=0, flags=0):
    return B.mq_linear_desc(T, K, N, rot, group, flags)


def test_linear_argument_validation(lib):
    A = 0x10000  # fake, aligned "device" address: validation must fail before it is used
    seg = B.mq_segments(0, None, None)

    def call(d, x=A, ldx=128, s_v=1.0, s_t=1.0, w=A, s_w=A, y=A, ldy=128, ws=A, ws_bytes=1 << 30):
        return lib.mq_w4a8_msq_linear(C.byref(d), x, ldx, C.byref(seg), s_v, s_t, w, s_w, None, y, ldy, None, ws,
                                      ws_bytes, None)

    assert lib.mq_w4a8_msq_linear(None, A, 128, None, 1.0, 1.0, A, A, None, A, 128, None, A, 1 << 30, None) \
        == B.MQ_ERR_INVALID_ARG
    assert call(_desc(K=100)) == B.MQ_ERR_INVALID_ARG
    assert call(_desc(N=100)) == B.MQ_ERR_INVALID_ARG
    assert call(_desc(T=-1)) == B.MQ_ERR_INVALID_ARG
    assert call(_desc(group=64)) == B.MQ_ERR_UNSUPPORTED                      # a weight group is one K block of 128
    assert call(_desc(group=-128)) == B.MQ_ERR_INVALID_ARG
    assert call(_desc(K=160, group=128), ldx=160) == B.MQ_ERR_INVALID_ARG     # K must be whole groups
    assert call(_desc(group=128, flags=B.MQ_FLAG_W8)) == B.MQ_ERR_UNSUPPORTED
    assert call(_desc(rot=16)) == B.MQ_ERR_UNSUPPORTED
    assert call(_desc(rot=96)) == B.MQ_ERR_INVALID_ARG
    assert call(_desc(K=384, rot=256), ldx=384) == B.MQ_ERR_INVALID_ARG      # rotation block must divide K
    assert call(_desc(flags=16)) == B.MQ_ERR_INVALID_ARG
    assert call(_desc(rot=128, flags=B.MQ_FLAG_X_IS_INT8)) == B.MQ_ERR_INVALID_ARG
    assert call(_desc(K=1 << 20), ldx=1 << 20) == B.MQ_ERR_UNSUPPORTED
    assert call(_desc(), s_v=0.0) == B.MQ_ERR_INVALID_ARG
    assert call(_desc(), s_t=float("inf")) == B.MQ_ERR_INVALID_ARG
    assert call(_desc(), s_t=float("nan")) == B.MQ_ERR_INVALID_ARG
    assert call(_desc(), x=None) == B.MQ_ERR_INVALID_ARG
    assert call(_desc(), ldx=64) == B.MQ_ERR_INVALID_ARG
    assert call(_desc(), x=A + 2) == B.MQ_ERR_ALIGNMENT
    assert call(_desc(), ldx=132) == B.MQ_ERR_ALIGNMENT
    assert call(_desc(), w=A + 64) == B.MQ_ERR_ALIGNMENT
    assert call(_desc(), ws=None) == B.MQ_ERR_WORKSPACE
    assert call(_desc(), ws=A + 16) == B.MQ_ERR_ALIGNMENT
    assert call(_desc(), ws_bytes=100) == B.MQ_ERR_WORKSPACE
    assert call(_desc(T=0)) == B.MQ_OK                                        # empty input: no-op
    bad_seg = B.mq_segments(-1, None, None)
    assert lib.mq_w4a8_msq_linear(C.byref(_desc()), A, 128, C.byref(bad_seg), 1.0, 1.0, A, A, None, A, 128, None, A,
                                  1 << 30, None) == B.MQ_ERR_INVALID_ARG
    bad_seg = B.mq_segments(2, None, None)
    assert lib.mq_w4a8_msq_linear(C.byref(_desc()), A, 128, C.byref(bad_seg), 1.0, 1.0, A, A, None, A, 128, None, A,
                                  1 << 30, None) == B.MQ_ERR_INVALID_ARG


def test_other_entry_points_validate(lib):
    A = 0x10000
    seg = B.mq_segments(0, None, None)
    f = lib.mq_fwht_quant_i8
    assert f(A, 4, 100, 100, C.byref(seg), 1.0, 1.0, 0, A, 112, None, None) == B.MQ_ERR_INVALID_ARG
    assert f(A, 4, 128, 128, C.byref(seg), -1.0, 1.0, 0, A, 128, None, None) == B.MQ_ERR_INVALID_ARG
    assert f(A, 4, 128, 128, C.byref(seg), 1.0, 1.0, 2048, A, 128, None, None) == B.MQ_ERR_UNSUPPORTED
    assert f(A, 4, 128, 128, C.byref(seg), 1.0, 1.0, 0, A + 1, 128, None, None) == B.MQ_ERR_ALIGNMENT
    assert f(A, 4, 128, 128, C.byref(seg), 1.0, 1.0, 0, A, 136, None, None) == B.MQ_ERR_ALIGNMENT
    assert f(None, 4, 128, 128, C.byref(seg), 1.0, 1.0, 0, A, 128, None, None) == B.MQ_ERR_INVALID_ARG
    c = lib.mq_calibrate_static_scales
    assert c(A, 4, 128, 128, C.byref(seg), 0, 0, None, A, A, None) == B.MQ_ERR_INVALID_ARG
    assert c(A, 4, 128, 128, C.byref(seg), 24, 0, A, A, A, None) == B.MQ_ERR_INVALID_ARG
    p = lib.mq_pack_w4
    assert p(A, 128, 128, 128, 64, None, A, None, None) == B.MQ_ERR_UNSUPPORTED
    assert p(A, 128, 160, 160, 128, None, A, None, None) == B.MQ_ERR_INVALID_ARG
    p8 = lib.mq_pack_w8
    assert p8(A, 128, 128, 128, None, 0, A, None, None) == B.MQ_ERR_INVALID_ARG       # neither codes nor layout wanted
    assert p8(A, 128, 128, 128, A, 64, A, None, None) == B.MQ_ERR_INVALID_ARG         # ldq < K
    assert p8(A, 128, 128, 128, None, 0, A, A + 16, None) == B.MQ_ERR_ALIGNMENT
    assert B.mq_w8_layout_bytes(3584, 18944) == 2 * B.mq_w4_layout_bytes(3584, 18944)
    qb = lib.mq_fwht_quant_bits
    assert qb(A, 4, 128, 128, C.byref(seg), 1.0, 1.0, 0, 5, A, 128, None) == B.MQ_ERR_UNSUPPORTED
    assert qb(A, 4, 128, 128, C.byref(seg), 1.0, 0.0, 0, 4, A, 128, None) == B.MQ_ERR_INVALID_ARG
    kq = lib.mq_kron_quant_i8
    assert kq(A, 4, 14336, 14336, C.byref(seg), 1.0, 1.0, 24, A, A, 14336, None, None) == B.MQ_ERR_INVALID_ARG      # 24 does not divide K
    assert kq(A, 4, 96, 96, C.byref(seg), 1.0, 1.0, 1, A, A, 96, None, None) == B.MQ_ERR_INVALID_ARG               # K / m = 96 is not a power of two
    assert kq(A, 4, 448, 448, C.byref(seg), 1.0, 1.0, 28, A, A, 448, None, None) == B.MQ_ERR_UNSUPPORTED       # K / m = 16 is below 32
    assert kq(A, 4, 3584, 3584, C.byref(seg), 1.0, 1.0, 28, None, A, 3584, None, None) == B.MQ_ERR_INVALID_ARG  # no sign table
    assert kq(A, 4, 3584, 3584, C.byref(seg), 1.0, -1.0, 28, A, A, 3584, None, None) == B.MQ_ERR_INVALID_ARG
    cb = lib.mq_calibrate_static_scales_bits
    assert cb(A, 4, 128, 128, C.byref(seg), 0, 3, 0, A, A, A, None) == B.MQ_ERR_UNSUPPORTED
    assert cb(A, 4, 128, 128, C.byref(seg), 0, 4, 0, None, A, A, None) == B.MQ_ERR_INVALID_ARG
    assert p(A, 128, 100, 100, 0, None, A, None, None) == B.MQ_ERR_INVALID_ARG
    assert p(A, 128, 128, 128, 0, None, None, None, None) == B.MQ_ERR_INVALID_ARG
    assert p(A, 128, 128, 128, 0, None, A, A + 16, None) == B.MQ_ERR_ALIGNMENT
    r = lib.mq_aifs_reorder
    assert r(A, A, 4, 8, 8, 8, A, None, A, A, A, 0, None) == B.MQ_ERR_INVALID_ARG      # in place
    assert r(A, None, 4, 8, 8, 8, A, None, A, A, A, 0, None) == B.MQ_ERR_INVALID_ARG
    assert r(A, A + 64, 4, 12, 12, 12, A, None, A, A, A, 0, None) == B.MQ_ERR_ALIGNMENT
    assert r(A, A + 64, 4, 8, 8, 8, A, None, A, A, A, 2, None) == B.MQ_ERR_INVALID_ARG
    assert r(A, A + 64, 4, 8, 8, 8, None, None, A, A, A, 0, None) == B.MQ_ERR_INVALID_ARG
    m = lib.mq_attn_mask_remap
    assert m(A, None, None, None, 4, A, A, A, None, None) == B.MQ_ERR_INVALID_ARG       # seg out needs n_first
    assert m(A, None, None, A, 20000, A, None, None, A, None) == B.MQ_ERR_UNSUPPORTED
    assert m(None, None, None, A, 4, A, None, None, None, None) == B.MQ_ERR_INVALID_ARG
    assert lib.mq_last_device_status(None, None, None) == B.MQ_ERR_INVALID_ARG


def test_rms_entry_points_validate(lib):
    A = 0x10000
    seg = B.mq_segments(0, None, None)
    assert B.mq_rms_side_ld(18944, 128) == 160                     # 148 blocks, padded to a multiple of 32
    assert B.mq_rms_side_ld(1152, 128) == 32
    assert B.mq_rms_side_ld(1152, 0) == 0 and B.mq_rms_side_ld(1152, 48) == 0
    base = B.mq_workspace_bytes(1088, 18944, 3584, 128)
    assert B.mq_rms_workspace_bytes(1088, 18944, 3584, 128) == base + 1088 * 160    # + the gathered split codes
    small_t = B.mq_workspace_bytes(8, 4096, 256, 128)
    assert B.mq_rms_workspace_bytes(8, 4096, 256, 128) == small_t + 256 + 8 * 256 * 4   # + codes, + one more slice
    assert B.mq_rms_workspace_bytes(1088, 18944, 3584, 0) == 0      # no rotation, no split columns
    assert B.mq_rms_workspace_bytes(8, 128, 128, 0, B.MQ_FLAG_X_IS_INT8) == 0
    det = lib.mq_rms_detect
    assert det(A, 128, 256, 256, 0, A, A, None) == B.MQ_ERR_INVALID_ARG
    assert det(A, 128, 256, 256, 128, None, None, None) == B.MQ_ERR_INVALID_ARG
    assert det(A, 128, 256, 256, 16, A, A, None) == B.MQ_ERR_UNSUPPORTED
    assert det(A, 128, 256, 200, 128, A, A, None) == B.MQ_ERR_INVALID_ARG      # ldw < K
    pk = lib.mq_pack_w4_rms
    assert pk(A, 128, 256, 256, 128, None, A, None, None, A, None, None) == B.MQ_ERR_INVALID_ARG   # q_side missing
    assert pk(A, 128, 256, 256, 128, None, A, None, A, A, A + 16, None) == B.MQ_ERR_ALIGNMENT
    assert pk(A, 128, 256, 256, 96, None, A, None, A, A, None, None) == B.MQ_ERR_INVALID_ARG
    f = lib.mq_w4a8_msq_linear_rms
    d = _desc(8, 256, 128, rot=0)
    assert f(C.byref(d), A, 256, C.byref(seg), 1.0, 1.0, A, A, A, A, None, A, 128, None, None, A, 1 << 30,
             None) == B.MQ_ERR_INVALID_ARG
    d = _desc(8, 256, 128, rot=128)
    assert f(C.byref(d), A, 256, C.byref(seg), 1.0, 1.0, A, A, None, A, None, A, 128, None, None, A, 1 << 30,
             None) == B.MQ_ERR_INVALID_ARG
    assert f(C.byref(d), A, 256, C.byref(seg), 1.0, 1.0, A, A, A, A, None, A, 128, None, None, None, 0,
             None) == B.MQ_ERR_WORKSPACE
    small = B.mq_workspace_bytes(8, 256, 128, 128)                  # enough for the plain linear only
    assert f(C.byref(d), A, 256, C.byref(seg), 1.0, 1.0, A, A, A, A, None, A, 128, None, None, A, small,
             None) == B.MQ_ERR_WORKSPACE


def test_dynamic_entry_points_validate(lib):
    A = 0x10000
    base = B.mq_workspace_bytes(1088, 18944, 3584, 128)
    d = _desc(1088, 18944, 3584, rot=128)
    assert lib.mq_dynamic_workspace_bytes(C.byref(d)) == base + 4352       # + 1088 floats
    assert lib.mq_dynamic_workspace_bytes(C.byref(_desc(8, 65536, 128))) == 0   # rows longer than 32768
    q = lib.mq_dynamic_quant_i8
    assert q(A, 4, 100, 100, 0, A, 112, A, None) == B.MQ_ERR_INVALID_ARG
    assert q(A, 4, 128, 128, 0, A, 128, None, None) == B.MQ_ERR_INVALID_ARG
    assert q(A, 4, 128, 128, 0, A + 1, 128, A, None) == B.MQ_ERR_ALIGNMENT
    assert q(A, 4, 65536, 65536, 0, A, 65536, A, None) == B.MQ_ERR_UNSUPPORTED
    assert q(A, 4, 128, 128, 48, A, 128, A, None) == B.MQ_ERR_INVALID_ARG
    f = lib.mq_w4a8_dynamic_linear
    d = _desc(8, 256, 128, flags=B.MQ_FLAG_X_IS_INT8)
    assert f(C.byref(d), A, 256, A, A, None, A, 128, None, None, A, 1 << 30, None) == B.MQ_ERR_INVALID_ARG
    d = _desc(8, 256, 128)
    assert f(C.byref(d), A, 256, A, A, None, A, 128, None, None, None, 0, None) == B.MQ_ERR_WORKSPACE
    assert f(C.byref(d), A, 256, A, A, None, A, 128, None, None, A, B.mq_workspace_bytes(8, 256, 128), None) == B.MQ_ERR_WORKSPACE
    assert f(C.byref(d), A, 200, A, A, None, A, 128, None, None, A, 1 << 30, None) == B.MQ_ERR_INVALID_ARG


def test_binding_refuses_cpu_tensors():
    import torch
    with pytest.raises(ValueError):
        B._ptr(torch.zeros(4))


def test_attention_entry_point_validates(lib):
    A = 0x10000
    at = lib.mq_aifs_attention
    ws_bytes = B.mq_aifs_attention_workspace_bytes(3360, 4)
    # V transposed (4 heads x 128 channels x 27 tiles of 128 keys, bf16) + four index bounds per tile
    assert ws_bytes == 4 * 128 * 27 * 128 * 2 + 512
    assert B.mq_aifs_attention_workspace_bytes(3360, 4, 64) == 0
    assert B.mq_aifs_attention_workspace_bytes(0, 4) == 0

    def call(L=256, hq=4, hkv=2, d=128, q=A, ldq=512, ldk=256, ldv=256, ldo=512, perm=A, ws=A, wsb=1 << 30, status=A):
        return at(q, ldq, A, ldk, A, ldv, perm, None, L, hq, hkv, d, A, ldo, ws, wsb, status, None)

    assert call(L=-1) == B.MQ_ERR_INVALID_ARG
    assert call(hq=3) == B.MQ_ERR_INVALID_ARG                      # query heads not a multiple of key/value heads
    assert call(d=64) == B.MQ_ERR_UNSUPPORTED
    assert call(L=131072 + 1) == B.MQ_ERR_UNSUPPORTED
    assert call(ldq=256) == B.MQ_ERR_INVALID_ARG                   # pitch shorter than the heads
    assert call(L=0) == B.MQ_OK                                    # nothing to do
    assert call(perm=None) == B.MQ_ERR_INVALID_ARG
    assert call(status=None) == B.MQ_ERR_INVALID_ARG
    assert call(q=A + 2) == B.MQ_ERR_ALIGNMENT
    assert call(ldq=516) == B.MQ_ERR_ALIGNMENT
    assert call(wsb=1024) == B.MQ_ERR_WORKSPACE
