"""Thin ctypes binding over the C ABI in include/mq.h.

Argument marshalling only: every step of the path runs in the CUDA kernels of
libmq.so.  torch supplies device memory and the current stream; nothing here
computes on tensors.  There is no CPU fallback: if the library is missing or a
tensor is not on a CUDA device the call raises.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional

import torch

MQ_OK = 0
MQ_ERR_INVALID_ARG = -1
MQ_ERR_UNSUPPORTED = -2
MQ_ERR_ALIGNMENT = -3
MQ_ERR_CUDA = -4
MQ_ERR_TIMEOUT = -5
MQ_ERR_WORKSPACE = -6
MQ_FLAG_X_IS_INT8 = 1
MQ_FLAG_Y_IS_F32 = 2
MQ_FLAG_A4 = 4
MQ_FLAG_W8 = 8
MQ_NOALLOC_WS_BYTES = 4 << 20
MQ_W_TILE_N, MQ_W_TILE_K = 128, 128
TEXT, VISUAL = 0, 1

_LIB_NAME = "libmq.so"
_lib = None


class MqError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {status_string(status)} ({status})")


class mq_segments(C.Structure):
    _fields_ = [("n_seg", C.c_int32), ("seg_end", C.c_void_p), ("seg_mod", C.c_void_p)]


class mq_linear_desc(C.Structure):
    _fields_ = [("T", C.c_int32), ("K", C.c_int32), ("N", C.c_int32), ("rot_block", C.c_int32),
                ("group_size", C.c_int32), ("flags", C.c_uint32)]


def lib_path() -> str:
    return os.path.join(os.path.dirname(os.path.abspath(__file__)), _LIB_NAME)


def load(build_if_missing: bool = False):
    """Loads libmq.so (raises if it is absent: the product has no other path)."""
    global _lib
    if _lib is not None:
        return _lib
    path = lib_path()
    if not os.path.exists(path):
        if not build_if_missing:
            raise RuntimeError(f"{path} not found: run `python -m paper_2502_00425_b200.build` "
                               "(or __graft_entry__.build()) first; there is no fallback path")
        from . import build as _build
        _build.build_library()
    lib = C.CDLL(path)
    vp, i32, i64, f32, sz = C.c_void_p, C.c_int32, C.c_int64, C.c_float, C.c_size_t
    segp, descp = C.POINTER(mq_segments), C.POINTER(mq_linear_desc)
    sigs = {
        "mq_version": (C.c_int, []),
        "mq_status_string": (C.c_char_p, [C.c_int]),
        "mq_workspace_bytes": (sz, [descp]),
        "mq_w4_layout_bytes": (sz, [i32, i32]),
        "mq_calibrate_static_scales": (C.c_int, [vp, i32, i32, i64, segp, i32, i32, vp, vp, vp, vp]),
        "mq_pack_w4": (C.c_int, [vp, i32, i32, i64, i32, vp, vp, vp, vp]),
        "mq_calibrate_static_scales_bits": (C.c_int, [vp, i32, i32, i64, segp, i32, i32, i32, vp, vp, vp, vp]),
        "mq_w8_layout_bytes": (sz, [i32, i32]),
        "mq_pack_w8": (C.c_int, [vp, i32, i32, i64, vp, i64, vp, vp, vp]),
        "mq_fwht_quant_bits": (C.c_int, [vp, i32, i32, i64, segp, f32, f32, i32, i32, vp, i64, vp]),
        "mq_kron_quant_i8": (C.c_int, [vp, i32, i32, i64, segp, f32, f32, i32, vp, vp, i64, vp, vp]),
        "mq_glue_rmsnorm": (C.c_int, [vp, i32, i32, i64, vp, f32, vp, i64, vp]),
        "mq_glue_rope": (C.c_int, [vp, i32, i32, i32, i64, vp, f32, vp, i64, vp]),
        "mq_glue_swiglu": (C.c_int, [vp, i64, vp, i64, i32, i32, vp, i64, vp]),
        "mq_glue_residual_add": (C.c_int, [vp, i64, vp, i64, i32, i32, vp, i64, vp]),
        "mq_aifs_attention_workspace_bytes": (sz, [i32, i32, i32]),
        "mq_aifs_attention": (C.c_int, [vp, i64, vp, i64, vp, i64, vp, vp, i32, i32, i32, i32, vp, i64, vp, sz, vp, vp]),
        "mq_repack_w4": (C.c_int, [vp, i32, i32, vp, vp]),
        "mq_unpack_w4": (C.c_int, [vp, vp, i32, i32, vp, i64, vp]),
        "mq_aifs_reorder": (C.c_int, [vp, vp, i32, i32, i64, i64, vp, vp, vp, vp, vp, i32, vp]),
        "mq_attn_mask_remap": (C.c_int, [vp, vp, vp, vp, i32, vp, vp, vp, vp, vp]),
        "mq_fwht_quant_i8": (C.c_int, [vp, i32, i32, i64, segp, f32, f32, i32, vp, i64, vp, vp]),
        "mq_w4a8_msq_linear": (C.c_int, [descp, vp, i64, segp, f32, f32, vp, vp, vp, vp, i64, vp, vp, sz, vp]),
        "mq_w4a8_msq_linear_noalloc": (C.c_int, [descp, vp, i64, segp, f32, f32, vp, vp, vp, vp, i64, vp, vp, vp]),
        "mq_rms_side_ld": (sz, [i32, i32]),
        "mq_rms_detect": (C.c_int, [vp, i32, i32, i64, i32, vp, vp, vp]),
        "mq_pack_w4_rms": (C.c_int, [vp, i32, i32, i64, i32, vp, vp, vp, vp, vp, vp, vp]),
        "mq_rms_workspace_bytes": (sz, [descp]),
        "mq_w4a8_msq_linear_rms": (C.c_int, [descp, vp, i64, segp, f32, f32, vp, vp, vp, vp, vp, vp, i64, vp, vp,
                                             vp, sz, vp]),
        "mq_dynamic_quant_i8": (C.c_int, [vp, i32, i32, i64, i32, vp, i64, vp, vp]),
        "mq_dynamic_workspace_bytes": (sz, [descp]),
        "mq_w4a8_dynamic_linear": (C.c_int, [descp, vp, i64, vp, vp, vp, vp, i64, vp, vp, vp, sz, vp]),
        "mq_ubench_mma_i8": (C.c_int, [i32, i32, i32, i32, i32, i32, vp, vp, vp]),
        "mq_selftest_bounded_wait": (C.c_int, [C.c_uint64, i32, vp, vp, vp]),
        "mq_ubench_expand": (C.c_int, [i32, i32, i32, vp, vp]),
        "mq_last_device_status": (C.c_int, [vp, vp, C.POINTER(C.c_int32)]),
        "mq_reset_device_status": (C.c_int, [vp, vp]),
    }
    for name, (res, args) in sigs.items():
        fn = getattr(lib, name)
        fn.restype = res
        fn.argtypes = args
    _lib = lib
    return lib


EXPORTED = ["mq_version", "mq_status_string", "mq_workspace_bytes", "mq_w4_layout_bytes",
            "mq_calibrate_static_scales", "mq_pack_w4", "mq_repack_w4", "mq_unpack_w4", "mq_aifs_reorder",
            "mq_attn_mask_remap", "mq_fwht_quant_i8", "mq_w4a8_msq_linear", "mq_w4a8_msq_linear_noalloc", "mq_last_device_status",
            "mq_reset_device_status", "mq_rms_side_ld", "mq_rms_detect", "mq_pack_w4_rms", "mq_rms_workspace_bytes",
            "mq_w4a8_msq_linear_rms", "mq_dynamic_quant_i8", "mq_dynamic_workspace_bytes", "mq_w4a8_dynamic_linear",
            "mq_ubench_mma_i8", "mq_selftest_bounded_wait", "mq_ubench_expand", "mq_calibrate_static_scales_bits",
            "mq_w8_layout_bytes", "mq_pack_w8", "mq_fwht_quant_bits", "mq_kron_quant_i8", "mq_glue_rmsnorm", "mq_glue_rope",
            "mq_glue_swiglu", "mq_glue_residual_add", "mq_aifs_attention_workspace_bytes", "mq_aifs_attention"]


def status_string(status: int) -> str:
    return load().mq_status_string(int(status)).decode()


def _check(status: int, where: str):
    if status != MQ_OK:
        raise MqError(status, where)


def _ptr(t: Optional[torch.Tensor]):
    if t is None:
        return None
    if not t.is_cuda:
        raise ValueError("tensor must live on a CUDA device (the library has no CPU path)")
    return C.c_void_p(t.data_ptr())


def _stream():
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


class Segments:
    """Device-resident segment table (Eq. 3: spans of one modality share a static scale)."""

    def __init__(self, seg_end: torch.Tensor, seg_mod: torch.Tensor):
        assert seg_end.dtype == torch.int32 and seg_mod.dtype == torch.uint8
        assert seg_end.numel() == seg_mod.numel()
        self.seg_end, self.seg_mod = seg_end.contiguous(), seg_mod.contiguous()
        self.c = mq_segments(self.seg_end.numel(), self.seg_end.data_ptr() if self.seg_end.numel() else None,
                             self.seg_mod.data_ptr() if self.seg_mod.numel() else None)

    @classmethod
    def from_host(cls, seg_end, seg_mod, device="cuda"):
        return cls(torch.as_tensor(seg_end, dtype=torch.int32).to(device),
                   torch.as_tensor(seg_mod, dtype=torch.uint8).to(device))

    def ref(self):
        return C.byref(self.c)


def _ld(t: torch.Tensor) -> int:
    assert t.dim() == 2 and t.stride(1) == 1
    return t.stride(0)


# ----------------------------------------------------------------------------- calls (same names as the C ABI)
def mq_workspace_bytes(T, K, N, rot_block=0, flags=0, group_size=0) -> int:
    d = mq_linear_desc(T, K, N, rot_block, group_size, flags)
    return int(load().mq_workspace_bytes(C.byref(d)))


def mq_w4_layout_bytes(N, K) -> int:
    return int(load().mq_w4_layout_bytes(N, K))


def new_workspace(T, K, N, rot_block=0, flags=0, device="cuda", group_size=0) -> torch.Tensor:
    """Allocates (with torch) and clears a workspace for mq_w4a8_msq_linear."""
    n = mq_workspace_bytes(T, K, N, rot_block, flags, group_size)
    if n == 0:
        raise MqError(MQ_ERR_INVALID_ARG, "mq_workspace_bytes")
    ws = torch.empty(n, dtype=torch.uint8, device=device)
    _check(load().mq_reset_device_status(_ptr(ws), _stream()), "mq_reset_device_status")
    return ws


def mq_calibrate_static_scales(x, seg: Segments, rot_block, amax_state, s_vis_out, s_txt_out, accumulate=False,
                               act_bits=8):
    assert x.dtype == torch.bfloat16
    T, K = x.shape
    if act_bits != 8:
        _check(load().mq_calibrate_static_scales_bits(_ptr(x), T, K, _ld(x), seg.ref(), rot_block, act_bits,
                                                      int(accumulate), _ptr(amax_state), _ptr(s_vis_out),
                                                      _ptr(s_txt_out), _stream()), "mq_calibrate_static_scales_bits")
        return
    _check(load().mq_calibrate_static_scales(_ptr(x), T, K, _ld(x), seg.ref(), rot_block, int(accumulate),
                                            _ptr(amax_state), _ptr(s_vis_out), _ptr(s_txt_out), _stream()),
           "mq_calibrate_static_scales")


def mq_pack_w4(w, packed=None, s_w=None, gemm_layout=None, group_size=0):
    assert w.dtype == torch.float32
    N, K = w.shape
    _check(load().mq_pack_w4(_ptr(w), N, K, _ld(w), group_size, _ptr(packed), _ptr(s_w), _ptr(gemm_layout),
                             _stream()), "mq_pack_w4")


def mq_w8_layout_bytes(N, K) -> int:
    return int(load().mq_w8_layout_bytes(N, K))


def mq_pack_w8(w, q_out=None, s_w=None, gemm_layout=None):
    """8-bit per-channel weight quantizer (W8A8): codes int8 [N,K], scales max/127, GEMM layout."""
    assert w.dtype == torch.float32
    N, K = w.shape
    _check(load().mq_pack_w8(_ptr(w), N, K, _ld(w), _ptr(q_out), _ld(q_out) if q_out is not None else 0, _ptr(s_w),
                             _ptr(gemm_layout), _stream()), "mq_pack_w8")


def mq_fwht_quant_bits(x, seg: Segments, s_vis, s_txt, rot_block, act_bits, q_out):
    assert x.dtype == torch.bfloat16 and q_out.dtype == torch.int8
    T, K = x.shape
    _check(load().mq_fwht_quant_bits(_ptr(x), T, K, _ld(x), seg.ref(), float(s_vis), float(s_txt), rot_block,
                                     act_bits, _ptr(q_out), _ld(q_out), _stream()), "mq_fwht_quant_bits")


def mq_kron_quant_i8(x, seg: Segments, s_vis, s_txt, h_neg, q_out, rotated_out=None):
    """Full-width rotation H_m (x) H_(K/m) + MSQ quantizer; h_neg: uint8 [m, m], 1 where H_m is -1."""
    assert x.dtype == torch.bfloat16 and q_out.dtype == torch.int8 and h_neg.dtype == torch.uint8
    T, K = x.shape
    m = h_neg.shape[0]
    _check(load().mq_kron_quant_i8(_ptr(x), T, K, _ld(x), seg.ref(), float(s_vis), float(s_txt), m, _ptr(h_neg),
                                   _ptr(q_out), _ld(q_out), _ptr(rotated_out), _stream()), "mq_kron_quant_i8")


def mq_repack_w4(packed, N, K, gemm_layout):
    _check(load().mq_repack_w4(_ptr(packed), N, K, _ptr(gemm_layout), _stream()), "mq_repack_w4")


def mq_unpack_w4(N, K, q_out, packed=None, gemm_layout=None):
    _check(load().mq_unpack_w4(_ptr(packed), _ptr(gemm_layout), N, K, _ptr(q_out), _ld(q_out), _stream()),
           "mq_unpack_w4")


def mq_aifs_reorder(x, x_out, is_visual, is_pad, perm, inv_perm, n_first_out, direction=0, L=None):
    if x is not None:
        assert x.dtype == torch.bfloat16 and x_out.dtype == torch.bfloat16
        L, D = x.shape
        ldx, ldo = _ld(x), _ld(x_out)
    else:
        D, ldx, ldo = 0, 0, 0
        L = perm.numel() if L is None else L
    _check(load().mq_aifs_reorder(_ptr(x), _ptr(x_out), L, D, ldx, ldo, _ptr(is_visual), _ptr(is_pad), _ptr(perm),
                                  _ptr(inv_perm), _ptr(n_first_out), direction, _stream()), "mq_aifs_reorder")


def mq_attn_mask_remap(perm, pos_ids, is_pad, n_first, pos_ids_out, seg_end_out=None, seg_mod_out=None,
                       dense_mask_out=None):
    L = perm.numel()
    _check(load().mq_attn_mask_remap(_ptr(perm), _ptr(pos_ids), _ptr(is_pad), _ptr(n_first), L, _ptr(pos_ids_out),
                                     _ptr(seg_end_out), _ptr(seg_mod_out), _ptr(dense_mask_out), _stream()),
           "mq_attn_mask_remap")


def mq_fwht_quant_i8(x, seg: Segments, s_vis, s_txt, rot_block, q_out, rotated_out=None):
    assert x.dtype == torch.bfloat16 and q_out.dtype == torch.int8
    T, K = x.shape
    _check(load().mq_fwht_quant_i8(_ptr(x), T, K, _ld(x), seg.ref(), float(s_vis), float(s_txt), rot_block,
                                   _ptr(q_out), _ld(q_out), _ptr(rotated_out), _stream()), "mq_fwht_quant_i8")


def mq_w4a8_msq_linear(x, seg: Segments, s_vis, s_txt, w_layout, s_w, y, ws, N, rot_block=0, bias=None,
                       acc_out=None, group_size=0, extra_flags=0):
    """x: bf16 [T,K] (rotated + quantized inside) or int8 [T,K] codes; y: bf16 or float32 [T,N].
    extra_flags: MQ_FLAG_A4 / MQ_FLAG_W8; group_size: 0 or 128 (see include/mq.h)."""
    T, K = x.shape
    flags = extra_flags
    if x.dtype == torch.int8:
        flags |= MQ_FLAG_X_IS_INT8
    else:
        assert x.dtype == torch.bfloat16
    if y.dtype == torch.float32:
        flags |= MQ_FLAG_Y_IS_F32
    else:
        assert y.dtype == torch.bfloat16
    d = mq_linear_desc(T, K, N, rot_block, group_size, flags)
    _check(load().mq_w4a8_msq_linear(C.byref(d), _ptr(x), _ld(x), seg.ref(), float(s_vis), float(s_txt),
                                     _ptr(w_layout), _ptr(s_w), _ptr(bias), _ptr(y), _ld(y), _ptr(acc_out),
                                     _ptr(ws), ws.numel(), _stream()), "mq_w4a8_msq_linear")


def mq_w4a8_msq_linear_noalloc(x, seg: Segments, s_vis, s_txt, w_layout, s_w, y, N, rot_block=0, bias=None,
                               acc_out=None, status_out=None):
    """mq_w4a8_msq_linear without a workspace argument: the scratch is a fixed 4 MiB array
    inside the library, for callers that are not in a position to allocate one (see
    include/mq.h).  Problems whose workspace would exceed MQ_NOALLOC_WS_BYTES raise
    MqError(MQ_ERR_WORKSPACE).  status_out: optional device int32[2] for {status, site}."""
    T, K = x.shape
    flags = 0
    if x.dtype == torch.int8:
        flags |= MQ_FLAG_X_IS_INT8
    else:
        assert x.dtype == torch.bfloat16
    if y.dtype == torch.float32:
        flags |= MQ_FLAG_Y_IS_F32
    else:
        assert y.dtype == torch.bfloat16
    d = mq_linear_desc(T, K, N, rot_block, 0, flags)
    _check(load().mq_w4a8_msq_linear_noalloc(C.byref(d), _ptr(x), _ld(x), seg.ref(), float(s_vis), float(s_txt),
                                             _ptr(w_layout), _ptr(s_w), _ptr(bias), _ptr(y), _ld(y),
                                             _ptr(acc_out), _ptr(status_out), _stream()),
           "mq_w4a8_msq_linear_noalloc")


def mq_rms_side_ld(K, rot_block) -> int:
    return int(load().mq_rms_side_ld(K, rot_block))


def mq_rms_detect(w, rot_block, flags=None, count_out=None):
    """Eq. 9 on the unrotated weight [N, K]: flags uint8 [N, K / rot_block], count int32[1]."""
    assert w.dtype == torch.float32
    N, K = w.shape
    _check(load().mq_rms_detect(_ptr(w), N, K, _ld(w), rot_block, _ptr(flags), _ptr(count_out), _stream()),
           "mq_rms_detect")


def mq_pack_w4_rms(w_rot, rot_block, s_w, q_side, s_w_side, packed=None, gemm_layout=None, side_layout=None):
    assert w_rot.dtype == torch.float32 and q_side.dtype == torch.int8
    N, K = w_rot.shape
    _check(load().mq_pack_w4_rms(_ptr(w_rot), N, K, _ld(w_rot), rot_block, _ptr(packed), _ptr(s_w),
                                 _ptr(gemm_layout), _ptr(q_side), _ptr(s_w_side), _ptr(side_layout), _stream()),
           "mq_pack_w4_rms")


def mq_rms_workspace_bytes(T, K, N, rot_block, flags=0) -> int:
    d = mq_linear_desc(T, K, N, rot_block, 0, flags)
    return int(load().mq_rms_workspace_bytes(C.byref(d)))


def new_rms_workspace(T, K, N, rot_block, flags=0, device="cuda") -> torch.Tensor:
    n = mq_rms_workspace_bytes(T, K, N, rot_block, flags)
    if n == 0:
        raise MqError(MQ_ERR_INVALID_ARG, "mq_rms_workspace_bytes")
    ws = torch.empty(n, dtype=torch.uint8, device=device)
    _check(load().mq_reset_device_status(_ptr(ws), _stream()), "mq_reset_device_status")
    return ws


def mq_w4a8_msq_linear_rms(x, seg: Segments, s_vis, s_txt, w_layout, s_w, side_layout, s_w_side, y, N, rot_block, ws,
                           bias=None, acc_out=None, acc_side_out=None):
    """The rotated linear with rotation magnitude suppression (Sec. 3.2): main GEMM plus the
    split first-channel-of-each-block product, added before the bias."""
    assert x.dtype == torch.bfloat16
    T, K = x.shape
    flags = 0
    if y.dtype == torch.float32:
        flags |= MQ_FLAG_Y_IS_F32
    else:
        assert y.dtype == torch.bfloat16
    d = mq_linear_desc(T, K, N, rot_block, 0, flags)
    _check(load().mq_w4a8_msq_linear_rms(C.byref(d), _ptr(x), _ld(x), seg.ref(), float(s_vis), float(s_txt),
                                         _ptr(w_layout), _ptr(s_w), _ptr(side_layout), _ptr(s_w_side), _ptr(bias),
                                         _ptr(y), _ld(y), _ptr(acc_out), _ptr(acc_side_out), _ptr(ws), ws.numel(),
                                         _stream()), "mq_w4a8_msq_linear_rms")


def mq_dynamic_quant_i8(x, rot_block, q, s_rows):
    """Rotation + per-token dynamic int8 quantizer (the comparison scheme): codes and one scale per row."""
    assert x.dtype == torch.bfloat16 and q.dtype == torch.int8 and s_rows.dtype == torch.float32
    T, K = x.shape
    _check(load().mq_dynamic_quant_i8(_ptr(x), T, K, _ld(x), rot_block, _ptr(q), _ld(q), _ptr(s_rows), _stream()),
           "mq_dynamic_quant_i8")


def new_dynamic_workspace(T, K, N, rot_block=0, device="cuda") -> torch.Tensor:
    d = mq_linear_desc(T, K, N, rot_block, 0, 0)
    n = int(load().mq_dynamic_workspace_bytes(C.byref(d)))
    if n == 0:
        raise MqError(MQ_ERR_INVALID_ARG, "mq_dynamic_workspace_bytes")
    ws = torch.empty(n, dtype=torch.uint8, device=device)
    _check(load().mq_reset_device_status(_ptr(ws), _stream()), "mq_reset_device_status")
    return ws


def mq_w4a8_dynamic_linear(x, w_layout, s_w, y, ws, N, rot_block=0, bias=None, acc_out=None, s_rows_out=None):
    """The W4A8 linear with per-token dynamic activation scales (comparison scheme, Sec. 1 / Sec. 4.3)."""
    assert x.dtype == torch.bfloat16
    T, K = x.shape
    flags = MQ_FLAG_Y_IS_F32 if y.dtype == torch.float32 else 0
    d = mq_linear_desc(T, K, N, rot_block, 0, flags)
    _check(load().mq_w4a8_dynamic_linear(C.byref(d), _ptr(x), _ld(x), _ptr(w_layout), _ptr(s_w), _ptr(bias), _ptr(y),
                                         _ld(y), _ptr(acc_out), _ptr(s_rows_out), _ptr(ws), ws.numel(), _stream()),
           "mq_w4a8_dynamic_linear")


def mq_ubench_mma_i8(n_tok, n_mma, n_acc, a_from_smem, ctas, cycles_out, status, commit_every=0):
    """Issue-rate microbenchmark of tcgen05.mma kind::i8; cycles_out int64 [ctas], status int32 [2] (zeroed)."""
    assert cycles_out.dtype == torch.int64 and cycles_out.numel() >= ctas and status.dtype == torch.int32
    _check(load().mq_ubench_mma_i8(n_tok, n_mma, n_acc, int(a_from_smem), int(commit_every), ctas, _ptr(cycles_out), _ptr(status),
                                   _stream()), "mq_ubench_mma_i8")


def mq_ubench_expand(n_iter, warps, mode, cycles_out):
    """Cycles of the weight expander's inner step (see include/mq.h); cycles_out int64 [warps]."""
    assert cycles_out.dtype == torch.int64 and cycles_out.numel() >= warps
    _check(load().mq_ubench_expand(n_iter, warps, mode, _ptr(cycles_out), _stream()), "mq_ubench_expand")


def mq_selftest_bounded_wait(limit_ns, site, status, waited_ns_out):
    """Bounded mbarrier wait on a barrier nobody arrives at; status int32 [2] (zeroed), waited_ns_out int64 [4]."""
    assert status.dtype == torch.int32 and waited_ns_out.dtype == torch.int64 and waited_ns_out.numel() >= 4
    _check(load().mq_selftest_bounded_wait(int(limit_ns), int(site), _ptr(status), _ptr(waited_ns_out), _stream()),
           "mq_selftest_bounded_wait")


def mq_glue_rmsnorm(x, gain, y, eps=1e-6):
    assert x.dtype == torch.bfloat16 and y.dtype == torch.bfloat16 and gain.dtype == torch.float32
    T, D = x.shape
    _check(load().mq_glue_rmsnorm(_ptr(x), T, D, _ld(x), _ptr(gain), float(eps), _ptr(y), _ld(y), _stream()),
           "mq_glue_rmsnorm")


def mq_glue_rope(x, pos, n_heads, y, base=10000.0):
    assert x.dtype == torch.bfloat16 and y.dtype == torch.bfloat16 and pos.dtype == torch.int32
    L, width = x.shape
    _check(load().mq_glue_rope(_ptr(x), L, n_heads, width // n_heads, _ld(x), _ptr(pos), float(base), _ptr(y), _ld(y),
                               _stream()), "mq_glue_rope")


def mq_glue_swiglu(gate, up, y):
    assert gate.dtype == torch.bfloat16 and up.dtype == torch.bfloat16 and y.dtype == torch.bfloat16
    T, M = gate.shape
    _check(load().mq_glue_swiglu(_ptr(gate), _ld(gate), _ptr(up), _ld(up), T, M, _ptr(y), _ld(y), _stream()),
           "mq_glue_swiglu")


def mq_glue_residual_add(a, b, y):
    assert a.dtype == torch.bfloat16 and b.dtype == torch.bfloat16 and y.dtype == torch.bfloat16
    T, D = a.shape
    _check(load().mq_glue_residual_add(_ptr(a), _ld(a), _ptr(b), _ld(b), T, D, _ptr(y), _ld(y), _stream()),
           "mq_glue_residual_add")


def mq_aifs_attention_workspace_bytes(L, n_kv_heads, head_dim=128) -> int:
    return int(load().mq_aifs_attention_workspace_bytes(L, n_kv_heads, head_dim))


def mq_aifs_attention(q, k, v, perm, pad_u, n_q_heads, n_kv_heads, o, ws, status):
    """Attention under the unified mask (Eq. 5) of one sequence in AIFS order; see include/mq.h.
    ws: uint8 tensor of mq_aifs_attention_workspace_bytes(); status: zeroed int32[2]."""
    for t in (q, k, v, o):
        assert t.dtype == torch.bfloat16
    assert perm.dtype == torch.int32 and status.dtype == torch.int32 and status.numel() >= 2
    assert pad_u is None or pad_u.dtype == torch.uint8
    L = q.shape[0]
    head_dim = q.shape[1] // n_q_heads
    _check(load().mq_aifs_attention(_ptr(q), _ld(q), _ptr(k), _ld(k), _ptr(v), _ld(v), _ptr(perm), _ptr(pad_u), L,
                                    n_q_heads, n_kv_heads, head_dim, _ptr(o), _ld(o), _ptr(ws), ws.numel(), _ptr(status),
                                    _stream()), "mq_aifs_attention")


def mq_last_device_status(ws):
    site = C.c_int32(0)
    st = load().mq_last_device_status(_ptr(ws), _stream(), C.byref(site))
    return st, site.value


def mq_reset_device_status(ws):
    _check(load().mq_reset_device_status(_ptr(ws), _stream()), "mq_reset_device_status")
