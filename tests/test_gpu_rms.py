"""GPU parity of rotation magnitude suppression (Sec. 3.2, Eq. 9) against the CPU oracle."""
import numpy as np
import pytest
import torch

from oracle import mq_oracle as O
from paper_2502_00425_b200 import binding as B
from paper_2502_00425_b200 import synth
from tests.gpu_util import DEV, bf16_from_dev, bf16_to_dev, dev_segments, gpu_calibrate

pytestmark = pytest.mark.gpu


def _rms_case(seed, T_vis, T_txt, K, N, rot):
    c = synth.small_linear(seed, T_vis, T_txt, K, N, rot, calib_vis=24, calib_txt=8)
    w = synth.mean_shifted_weight(seed + 1, N, K, rot)
    w_rot = O.rotate_weight_input_dim(w, rot).astype(np.float32)
    return c, w, w_rot


def _gpu_pack_rms(w_rot, rot):
    N, K = w_rot.shape
    side_ld = B.mq_rms_side_ld(K, rot)
    wd = torch.from_numpy(np.ascontiguousarray(w_rot)).to(DEV)
    packed = torch.empty((N, K // 2), dtype=torch.uint8, device=DEV)
    s_w = torch.empty(N, dtype=torch.float32, device=DEV)
    layout = torch.empty(B.mq_w4_layout_bytes(N, K), dtype=torch.uint8, device=DEV)
    q_side = torch.full((N, side_ld), 99, dtype=torch.int8, device=DEV)
    s_side = torch.empty(N, dtype=torch.float32, device=DEV)
    side_layout = torch.empty(B.mq_w4_layout_bytes(N, side_ld), dtype=torch.uint8, device=DEV)
    B.mq_pack_w4_rms(wd, rot, s_w, q_side, s_side, packed, layout, side_layout)
    return packed, s_w, layout, q_side, s_side, side_layout


@pytest.mark.parametrize("N,K,rot", [(64, 512, 128), (272, 1152, 128), (48, 160, 32), (16, 2048, 1024)])
def test_rms_detect_matches_oracle(N, K, rot):
    w = synth.mean_shifted_weight(7 + N, N, K, rot)
    ref = O.rms_detect(w, rot)
    assert 0 < ref.sum() < ref.size          # the case has both outcomes
    flags = torch.full((N, K // rot), 7, dtype=torch.uint8, device=DEV)
    count = torch.full((1,), -5, dtype=torch.int32, device=DEV)
    B.mq_rms_detect(torch.from_numpy(w).to(DEV), rot, flags, count)
    assert np.array_equal(flags.cpu().numpy().astype(bool), ref)
    assert int(count.item()) == int(ref.sum())
    # count only
    count.fill_(123)
    B.mq_rms_detect(torch.from_numpy(w).to(DEV), rot, None, count)
    assert int(count.item()) == int(ref.sum())


@pytest.mark.parametrize("N,K,rot", [(272, 1152, 128), (48, 160, 32), (128, 768, 256)])
def test_rms_pack_matches_oracle(N, K, rot):
    w = synth.mean_shifted_weight(11 + N, N, K, rot)
    w_rot = O.rotate_weight_input_dim(w, rot).astype(np.float32)
    w_main, w_side = O.rms_split(w_rot, rot)
    q_main, s_main = O.quantize_weight_int4(w_main)
    q_sd, s_sd = O.quantize_weight_int4(w_side)
    packed, s_w, layout, q_side, s_side, side_layout = _gpu_pack_rms(w_rot, rot)
    assert np.array_equal(s_w.cpu().numpy(), s_main)
    assert np.array_equal(s_side.cpu().numpy(), s_sd)
    nb = K // rot
    qs = q_side.cpu().numpy()
    assert np.array_equal(qs[:, :nb], q_sd)
    assert not qs[:, nb:].any()               # padding codes
    side = torch.empty((N, qs.shape[1]), dtype=torch.int8, device=DEV)
    B.mq_unpack_w4(N, qs.shape[1], side, gemm_layout=side_layout)
    assert np.array_equal(side.cpu().numpy(), qs)
    for src in ("packed", "layout"):
        out = torch.empty((N, K), dtype=torch.int8, device=DEV)
        B.mq_unpack_w4(N, K, out, packed=packed if src == "packed" else None,
                       gemm_layout=layout if src == "layout" else None)
        got = out.cpu().numpy()
        assert np.array_equal(got, q_main), src
        assert not got[:, ::rot].any()


@pytest.mark.parametrize("T_vis,T_txt,K,N,rot,with_bias", [
    (40, 27, 1152, 272, 128, False),   # ragged token group, ragged channel tile, 9 blocks (side row padded to 32)
    (3, 5, 4096, 256, 128, True),      # T = 8: the small-T GEMM path underneath, 32 blocks
    (150, 60, 160, 144, 32, True),     # five blocks of 32, two token tiles of the main GEMM
    (0, 9, 2048, 64, 1024, False),     # two blocks of 1024
    (0, 1, 1152, 272, 128, True),      # one token: the split path keeps the tensor-core kernel (no GEMV variant)
    (1, 2, 13696, 144, 128, False),    # three tokens at the decode row length, split-K with the split accumulator's slice
    (300, 33, 2304, 528, 128, True),   # 18 blocks, five channel tiles, two token tiles
])
def test_rms_linear_matches_oracle(T_vis, T_txt, K, N, rot, with_bias):
    c, w, w_rot = _rms_case(300 + K + N, T_vis, T_txt, K, N, rot)
    s_v, s_t = gpu_calibrate(c.x_calib, c.seg_calib, rot)
    w_main, w_side = O.rms_split(w_rot, rot)
    q_main, s_main = O.quantize_weight_int4(w_main)
    q_sd, s_sd = O.quantize_weight_int4(w_side)
    bias = None
    if with_bias:
        bias = (np.random.default_rng(5).standard_normal(N) * 0.5).astype(np.float32)
    ref = O.linear_w4a8_msq_rms(c.x, c.seg.seg_end, c.seg.seg_mod, s_v, s_t, rot, q_main, s_main, q_sd, s_sd, bias)
    assert np.abs(ref["acc_side"]).max() > 0
    packed, s_w, layout, q_side, s_side, side_layout = _gpu_pack_rms(w_rot, rot)
    T = c.T
    x = bf16_to_dev(c.x)
    seg = dev_segments(c.seg)
    bias_d = None if bias is None else torch.from_numpy(bias).to(DEV)
    for dt in (torch.float32, torch.bfloat16):
        ws = B.new_rms_workspace(T, K, N, rot)
        y = torch.full((T, N), float("nan"), dtype=dt, device=DEV)
        acc = torch.full((T, N), -(2 ** 31), dtype=torch.int32, device=DEV)
        acc_s = torch.full((T, N), -(2 ** 31), dtype=torch.int32, device=DEV)
        B.mq_w4a8_msq_linear_rms(x, seg, s_v, s_t, layout, s_w, side_layout, s_side, y, N, rot, ws, bias=bias_d,
                                 acc_out=acc, acc_side_out=acc_s)
        assert B.mq_last_device_status(ws) == (B.MQ_OK, 0)
        assert np.array_equal(acc.cpu().numpy(), ref["acc_main"])
        assert np.array_equal(acc_s.cpu().numpy(), ref["acc_side"])
        if dt == torch.float32:
            y32 = y.cpu().numpy()
            assert np.array_equal(y32, ref["y32"])
            mag = (np.abs(O.dequant(ref["acc_main"], ref["s_rows"], s_main))
                   + np.abs(O.dequant(ref["acc_side"], ref["s_rows"], s_sd))
                   + (0 if bias is None else np.abs(bias)[None, :]))
            nz = mag > 0
            assert (np.abs(y32 - ref["y64"])[nz] / mag[nz]).max() <= 1e-5
        else:
            assert np.array_equal(bf16_from_dev(y), ref["y_bf16"])
    # without the optional accumulator outputs
    ws = B.new_rms_workspace(T, K, N, rot)
    y2 = torch.empty((T, N), dtype=torch.bfloat16, device=DEV)
    B.mq_w4a8_msq_linear_rms(x, seg, s_v, s_t, layout, s_w, side_layout, s_side, y2, N, rot, ws, bias=bias_d)
    assert np.array_equal(bf16_from_dev(y2), ref["y_bf16"])


def test_rms_recovers_what_plain_w4_loses():
    """The point of the remedy: on a weight with block-mean outliers, the split linear is
    closer to the unquantized product than the plain W4A8 linear on the same rotated weight."""
    rot, K, N = 128, 1152, 272
    c, w, w_rot = _rms_case(900, 64, 32, K, N, rot)
    s_v, s_t = gpu_calibrate(c.x_calib, c.seg_calib, rot)
    exact = c.x.astype(np.float64) @ w.astype(np.float64).T
    packed, s_w, layout, q_side, s_side, side_layout = _gpu_pack_rms(w_rot, rot)
    x, seg = bf16_to_dev(c.x), dev_segments(c.seg)
    ws = B.new_rms_workspace(c.T, K, N, rot)
    y_rms = torch.empty((c.T, N), dtype=torch.float32, device=DEV)
    B.mq_w4a8_msq_linear_rms(x, seg, s_v, s_t, layout, s_w, side_layout, s_side, y_rms, N, rot, ws)
    # plain: same rotated weight, one scale per channel over all input channels
    wd = torch.from_numpy(w_rot).to(DEV)
    s_plain = torch.empty(N, dtype=torch.float32, device=DEV)
    lay_plain = torch.empty(B.mq_w4_layout_bytes(N, K), dtype=torch.uint8, device=DEV)
    B.mq_pack_w4(wd, None, s_plain, lay_plain)
    ws2 = B.new_workspace(c.T, K, N, rot)
    y_plain = torch.empty((c.T, N), dtype=torch.float32, device=DEV)
    B.mq_w4a8_msq_linear(x, seg, s_v, s_t, lay_plain, s_plain, y_plain, ws2, N, rot_block=rot)
    err_rms = np.linalg.norm(y_rms.cpu().numpy() - exact)
    err_plain = np.linalg.norm(y_plain.cpu().numpy() - exact)
    assert err_rms < err_plain
