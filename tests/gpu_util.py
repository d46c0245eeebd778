"""Helpers shared by the GPU parity tests: host <-> device marshalling around the C ABI."""
import numpy as np
import torch

from paper_2502_00425_b200 import binding as B
from paper_2502_00425_b200 import synth

DEV = "cuda"


def bf16_to_dev(x_f32: np.ndarray) -> torch.Tensor:
    """float32 array of bf16-representable values -> device bf16 tensor (exact)."""
    bits = synth.to_bf16_bits(x_f32).astype(np.int16)
    return torch.from_numpy(bits).to(DEV).view(torch.bfloat16)


def bf16_from_dev(t: torch.Tensor) -> np.ndarray:
    bits = t.contiguous().view(torch.int16).cpu().numpy().view(np.uint16)
    return synth.bf16_bits_to_f32(bits)


def dev_segments(seg) -> B.Segments:
    return B.Segments.from_host(seg.seg_end, seg.seg_mod, DEV)


def gpu_calibrate(x_calib, seg_calib, rot_block):
    xc = bf16_to_dev(x_calib)
    state = torch.zeros(2, dtype=torch.int32, device=DEV)
    sv = torch.zeros(1, dtype=torch.float32, device=DEV)
    stx = torch.zeros(1, dtype=torch.float32, device=DEV)
    B.mq_calibrate_static_scales(xc, dev_segments(seg_calib), rot_block, state, sv, stx)
    return np.float32(sv.item()), np.float32(stx.item())


def gpu_pack(w: np.ndarray):
    N, K = w.shape
    wd = torch.from_numpy(np.ascontiguousarray(w)).to(DEV)
    packed = torch.empty((N, K // 2), dtype=torch.uint8, device=DEV)
    s_w = torch.empty(N, dtype=torch.float32, device=DEV)
    layout = torch.empty(B.mq_w4_layout_bytes(N, K), dtype=torch.uint8, device=DEV)
    B.mq_pack_w4(wd, packed, s_w, layout)
    return packed, s_w, layout


def gpu_linear(case, s_vis, s_txt, layout, s_w, bias=None, y_dtype=torch.bfloat16, x_codes=None, want_acc=True,
               y_pad=0):
    """Runs mq_w4a8_msq_linear on a synth.LinearCase; returns (y, acc, status).  y_pad > 0 makes Y a
    view of a wider array (row pitch N + y_pad elements); the padding must come back untouched."""
    T, K, N = case.T, case.K, case.N
    x = x_codes if x_codes is not None else bf16_to_dev(case.x)
    flags = B.MQ_FLAG_X_IS_INT8 if x_codes is not None else 0
    rot = 0 if x_codes is not None else case.rot_block
    ws = B.new_workspace(T, K, N, rot, flags)
    y_full = torch.full((T, N + y_pad), float("nan"), dtype=y_dtype, device=DEV)
    y = y_full[:, :N] if y_pad else y_full
    acc = torch.full((T, N), -(2 ** 31), dtype=torch.int32, device=DEV) if want_acc else None
    bias_d = None if bias is None else torch.from_numpy(bias).to(DEV)
    B.mq_w4a8_msq_linear(x, dev_segments(case.seg), s_vis, s_txt, layout, s_w, y, ws, N, rot_block=rot,
                         bias=bias_d, acc_out=acc)
    st = B.mq_last_device_status(ws)
    if y_pad:
        assert bool(torch.isnan(y_full[:, N:]).all())
    return y, acc, st
