"""The neighbouring settings of the W4A8 MSQ linear, through the same C-ABI call, against the oracle:
group-wise W4 scales (g = 128, App. A.12), 8-bit weights (W8A8) and 4-bit activations (W4A4) of the main
results table (Sec. 4.1).  Integers bit for bit; float32 output equal to the oracle's float32 twin and
within 1e-5 of float64 (relative to the size of the terms), bf16 equal to the oracle's and within 1e-2."""
import numpy as np
import pytest
import torch

from oracle import mq_oracle as O
from paper_2502_00425_b200 import binding as B
from paper_2502_00425_b200 import synth

from gpu_util import DEV, bf16_from_dev, bf16_to_dev, dev_segments

pytestmark = pytest.mark.gpu


def _calibrate(c, act_bits):
    xc = bf16_to_dev(c.x_calib)
    state = torch.zeros(2, dtype=torch.int32, device=DEV)
    sv, st = torch.zeros(1, device=DEV), torch.zeros(1, device=DEV)
    B.mq_calibrate_static_scales(xc, dev_segments(c.seg_calib), c.rot_block, state, sv, st, act_bits=act_bits)
    got = (np.float32(sv.item()), np.float32(st.item()))
    want = O.calibrate_static_scales_bits(c.x_calib, c.seg_calib.seg_end, c.seg_calib.seg_mod, c.rot_block, act_bits)
    assert got == want
    return got


def _run(c, s_v, s_t, layout, s_w, y_dtype, bias, group=0, flags=0, acc=None, rows=None):
    x = bf16_to_dev(c.x)
    ws = B.new_workspace(c.T, c.K, c.N, c.rot_block, flags, group_size=group)
    y = torch.full((c.T, c.N), float("nan"), dtype=y_dtype, device=DEV)
    b = None if bias is None else torch.from_numpy(bias).to(DEV)
    B.mq_w4a8_msq_linear(x, dev_segments(c.seg), s_v, s_t, layout, s_w, y, ws, c.N, rot_block=c.rot_block, bias=b,
                         acc_out=acc, group_size=group, extra_flags=flags)
    assert B.mq_last_device_status(ws) == (B.MQ_OK, 0)
    return y


def _check_float_outputs(y32, yb, ref, mag):
    assert np.array_equal(y32, ref["y32"])
    nz = mag > 0
    assert (np.abs(y32 - ref["y64"])[nz] / mag[nz]).max() <= 1e-5
    assert np.array_equal(yb, ref["y_bf16"])
    assert (np.abs(yb - ref["y64"])[nz] / mag[nz]).max() <= 1e-2


# ----------------------------------------------------------------------------- group-wise W4 (g = 128)
def _grouped_case(seed, T_vis, T_txt, K, N, rot):
    c = synth.small_linear(seed, T_vis, T_txt, K, N, rot, calib_vis=16, calib_txt=8)
    # give the groups of every output channel their own range, the structure group scales exist for
    rng = np.random.default_rng(seed + 1)
    c.w = (c.w * np.repeat(rng.uniform(0.05, 4.0, (N, K // 128)), 128, axis=1)).astype(np.float32)
    return c


@pytest.mark.parametrize("T_vis,T_txt,K,N,rot", [
    (40, 24, 512, 256, 128),     # one 64-token tile, four groups
    (100, 37, 1152, 272, 128),   # ragged token tiles (three of 48), ragged channel tile, nine groups
    (3, 2, 256, 128, 0),         # five tokens: the few-token kernel does not apply to group scales
    (0, 70, 128, 16, 0),         # a single group
    (300, 20, 384, 2048, 128),   # more tiles than SMs' worth: several tiles per CTA, accumulator hand-over across tiles
])
def test_grouped_linear_matches_oracle(T_vis, T_txt, K, N, rot):
    c = _grouped_case(700 + K + N, T_vis, T_txt, K, N, rot)
    s_v, s_t = _calibrate(c, 8)
    wd = torch.from_numpy(c.w).to(DEV)
    G = K // 128
    packed = torch.empty((N, K // 2), dtype=torch.uint8, device=DEV)
    s_wg = torch.empty((G, N), dtype=torch.float32, device=DEV)
    layout = torch.empty(B.mq_w4_layout_bytes(N, K), dtype=torch.uint8, device=DEV)
    B.mq_pack_w4(wd, packed, s_wg, layout, group_size=128)
    qw, s_ref = O.quantize_weight_sym(c.w, 4, 128)
    assert np.array_equal(s_wg.cpu().numpy(), s_ref.T)              # the library keeps the scales group-major
    assert np.array_equal(packed.cpu().numpy(), O.pack_w4(qw))
    q2 = torch.empty((N, K), dtype=torch.int8, device=DEV)
    B.mq_unpack_w4(N, K, q2, gemm_layout=layout)
    assert np.array_equal(q2.cpu().numpy(), qw)
    bias = np.random.default_rng(3).standard_normal(N).astype(np.float32)
    for b in (None, bias):
        ref = O.linear_wa_sym(c.x, c.seg.seg_end, c.seg.seg_mod, s_v, s_t, rot, qw, s_ref, 8, 128, b)
        acc = torch.full((G, c.T, N), -(2 ** 31), dtype=torch.int32, device=DEV)
        y32 = _run(c, s_v, s_t, layout, s_wg, torch.float32, b, group=128, acc=acc).cpu().numpy()
        assert np.array_equal(acc.cpu().numpy(), np.transpose(ref["acc_g"], (2, 0, 1)))   # every group's accumulator
        yb = bf16_from_dev(_run(c, s_v, s_t, layout, s_wg, torch.bfloat16, b, group=128))
        mag = np.abs(ref["acc_g"].astype(np.float64) * ref["s_rows"].astype(np.float64)[:, None, None]
                     * s_ref.astype(np.float64)[None, :, :]).sum(axis=2) + (0 if b is None else np.abs(b)[None, :])
        _check_float_outputs(y32, yb, ref, mag)


def test_grouped_linear_config2_shape_sampled():
    """Group-wise scales at the size of config 2 (T = 1088, K = 18944 = 148 groups, N = 3584): sampled rows."""
    c = synth.config2()
    s_v, s_t = _calibrate(c, 8)
    wd = torch.from_numpy(c.w).to(DEV)
    G = c.K // 128
    s_wg = torch.empty((G, c.N), dtype=torch.float32, device=DEV)
    layout = torch.empty(B.mq_w4_layout_bytes(c.N, c.K), dtype=torch.uint8, device=DEV)
    B.mq_pack_w4(wd, None, s_wg, layout, group_size=128)
    qw, s_ref = O.quantize_weight_sym(c.w, 4, 128)
    assert np.array_equal(s_wg.cpu().numpy(), s_ref.T)
    rows = np.array(sorted({0, 63, 64, 1023, 1024, 1087} | set(c.meta["massive_rows"]) | set(range(5, c.T, 97))))
    sub = synth.segments_from_row_modality(c.seg.row_modality(c.T)[rows])
    ref = O.linear_wa_sym(c.x[rows], sub.seg_end, sub.seg_mod, s_v, s_t, c.rot_block, qw, s_ref, 8, 128)
    y32 = _run(c, s_v, s_t, layout, s_wg, torch.float32, None, group=128).cpu().numpy()
    assert np.array_equal(y32[rows], ref["y32"])
    yb = bf16_from_dev(_run(c, s_v, s_t, layout, s_wg, torch.bfloat16, None, group=128))
    assert np.array_equal(yb[rows], ref["y_bf16"])


# ----------------------------------------------------------------------------- W8A8 and W4A4
@pytest.mark.parametrize("T_vis,T_txt,K,N,rot", [
    (200, 100, 1152, 272, 128),   # prefill-sized: ragged tiles
    (3, 5, 4096, 256, 128),       # decode-sized: K splits and the finalize kernel
    (0, 2, 512, 48, 64),          # two tokens
    (250, 263, 160, 144, 32),     # K not a multiple of the K block
])
def test_w8a8_linear_matches_oracle(T_vis, T_txt, K, N, rot):
    c = synth.small_linear(800 + K + N, T_vis, T_txt, K, N, rot, calib_vis=16, calib_txt=8)
    s_v, s_t = _calibrate(c, 8)
    wd = torch.from_numpy(c.w).to(DEV)
    q8 = torch.empty((N, K), dtype=torch.int8, device=DEV)
    s_w = torch.empty(N, dtype=torch.float32, device=DEV)
    layout = torch.empty(B.mq_w8_layout_bytes(N, K), dtype=torch.uint8, device=DEV)
    B.mq_pack_w8(wd, q8, s_w, layout)
    qw, s_ref = O.quantize_weight_sym(c.w, 8, 0)
    assert np.array_equal(s_w.cpu().numpy(), s_ref) and np.array_equal(q8.cpu().numpy(), qw)
    bias = np.random.default_rng(4).standard_normal(N).astype(np.float32)
    for b in (None, bias):
        ref = O.linear_wa_sym(c.x, c.seg.seg_end, c.seg.seg_mod, s_v, s_t, rot, qw, s_ref, 8, 0, b)
        acc = torch.full((c.T, N), -(2 ** 31), dtype=torch.int32, device=DEV)
        y32 = _run(c, s_v, s_t, layout, s_w, torch.float32, b, flags=B.MQ_FLAG_W8, acc=acc).cpu().numpy()
        assert np.array_equal(acc.cpu().numpy(), ref["acc"])
        yb = bf16_from_dev(_run(c, s_v, s_t, layout, s_w, torch.bfloat16, b, flags=B.MQ_FLAG_W8))
        mag = np.abs(O.dequant(ref["acc"], ref["s_rows"], s_ref)) + (0 if b is None else np.abs(b)[None, :])
        _check_float_outputs(y32, yb, ref, mag)


@pytest.mark.parametrize("T_vis,T_txt,K,N,rot", [
    (200, 100, 1152, 272, 128),
    (3, 5, 4096, 256, 128),
    (1, 1, 2048, 96, 1024),       # two tokens: quantizer kernel + few-token product on 4-bit codes
])
def test_w4a4_linear_matches_oracle(T_vis, T_txt, K, N, rot):
    c = synth.small_linear(900 + K + N, T_vis, T_txt, K, N, rot, calib_vis=16, calib_txt=8)
    s_v, s_t = _calibrate(c, 4)
    wd = torch.from_numpy(c.w).to(DEV)
    s_w = torch.empty(N, dtype=torch.float32, device=DEV)
    layout = torch.empty(B.mq_w4_layout_bytes(N, K), dtype=torch.uint8, device=DEV)
    B.mq_pack_w4(wd, None, s_w, layout)
    qw, s_ref = O.quantize_weight_int4(c.w)
    ref = O.linear_wa_sym(c.x, c.seg.seg_end, c.seg.seg_mod, s_v, s_t, rot, qw, s_ref, 4, 0)
    assert ref["qx"].min() >= -8 and ref["qx"].max() <= 7 and (np.abs(ref["qx"]) == 7).any()
    q = torch.empty((c.T, K), dtype=torch.int8, device=DEV)
    B.mq_fwht_quant_bits(bf16_to_dev(c.x), dev_segments(c.seg), s_v, s_t, rot, 4, q)
    assert np.array_equal(q.cpu().numpy(), ref["qx"])
    acc = torch.full((c.T, N), -(2 ** 31), dtype=torch.int32, device=DEV)
    y32 = _run(c, s_v, s_t, layout, s_w, torch.float32, None, flags=B.MQ_FLAG_A4, acc=acc).cpu().numpy()
    assert np.array_equal(acc.cpu().numpy(), ref["acc"])
    yb = bf16_from_dev(_run(c, s_v, s_t, layout, s_w, torch.bfloat16, None, flags=B.MQ_FLAG_A4))
    _check_float_outputs(y32, yb, ref, np.abs(O.dequant(ref["acc"], ref["s_rows"], s_ref)))
