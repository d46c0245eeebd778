"""GPU parity of the per-token dynamic A8 comparison path (Sec. 1, Sec. 4.3) against the CPU oracle."""
import numpy as np
import pytest
import torch

from oracle import mq_oracle as O
from paper_2502_00425_b200 import binding as B
from paper_2502_00425_b200 import synth
from tests.gpu_util import DEV, bf16_from_dev, bf16_to_dev, gpu_pack

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("T_vis,T_txt,K,N,rot,with_bias", [
    (40, 27, 1152, 272, 128, True),    # two warp passes per row (the second one ragged), ragged channel tile
    (3, 5, 4096, 256, 128, False),     # T = 8: split-K slices underneath
    (1, 2, 160, 144, 32, True),        # T = 3: the few-token GEMV with per-token scales
    (150, 60, 2368, 144, 0, False),    # no rotation, 2.3 warp passes
    (0, 9, 2048, 64, 1024, True),      # the largest rotation block
    (20, 13, 18944, 128, 128, False),  # the config-2 row length: 19 warps per row
])
def test_dynamic_linear_matches_oracle(T_vis, T_txt, K, N, rot, with_bias):
    c = synth.small_linear(700 + K + N, T_vis, T_txt, K, N, rot, calib_vis=8, calib_txt=8)
    T = c.T
    qw, s_w_ref = O.quantize_weight_int4(c.w)
    packed, s_w, layout = gpu_pack(c.w)
    bias = (np.random.default_rng(6).standard_normal(N) * 0.5).astype(np.float32) if with_bias else None
    ref = O.linear_w4a8_dynamic(c.x, rot, qw, s_w_ref, bias)
    x = bf16_to_dev(c.x)
    # the quantizer entry point alone
    q = torch.full((T, K), 99, dtype=torch.int8, device=DEV)
    s_rows = torch.full((T,), -1.0, dtype=torch.float32, device=DEV)
    B.mq_dynamic_quant_i8(x, rot, q, s_rows)
    assert np.array_equal(s_rows.cpu().numpy(), ref["s_rows"])
    assert np.array_equal(q.cpu().numpy(), ref["qx"])
    # the linear
    bias_d = None if bias is None else torch.from_numpy(bias).to(DEV)
    for dt in (torch.float32, torch.bfloat16):
        ws = B.new_dynamic_workspace(T, K, N, rot)
        y = torch.full((T, N), float("nan"), dtype=dt, device=DEV)
        acc = torch.full((T, N), -(2 ** 31), dtype=torch.int32, device=DEV)
        s_out = torch.zeros(T, dtype=torch.float32, device=DEV)
        B.mq_w4a8_dynamic_linear(x, layout, s_w, y, ws, N, rot_block=rot, bias=bias_d, acc_out=acc, s_rows_out=s_out)
        assert B.mq_last_device_status(ws) == (B.MQ_OK, 0)
        assert np.array_equal(s_out.cpu().numpy(), ref["s_rows"])
        assert np.array_equal(acc.cpu().numpy(), ref["acc"])
        if dt == torch.float32:
            assert np.array_equal(y.cpu().numpy(), ref["y32"])
        else:
            assert np.array_equal(bf16_from_dev(y), ref["y_bf16"])
    # product configuration: no dumps, scales kept in the workspace
    ws = B.new_dynamic_workspace(T, K, N, rot)
    y2 = torch.empty((T, N), dtype=torch.bfloat16, device=DEV)
    B.mq_w4a8_dynamic_linear(x, layout, s_w, y2, ws, N, rot_block=rot, bias=bias_d)
    assert np.array_equal(bf16_from_dev(y2), ref["y_bf16"])


def test_dynamic_quant_zero_row_and_strided_rows():
    T, K = 5, 256
    rng = np.random.default_rng(8)
    xf = synth.round_to_bf16(rng.standard_normal((T, K)).astype(np.float32))
    xf[2] = 0.0
    ref_q, ref_s = O.quantize_act_int8_dynamic(O.fwht_blocks(xf, 64, np.float32))
    wide = torch.zeros((T, K + 64), dtype=torch.bfloat16, device=DEV)
    wide[:, :K] = bf16_to_dev(xf)
    q = torch.zeros((T, K + 32), dtype=torch.int8, device=DEV)
    s = torch.zeros(T, dtype=torch.float32, device=DEV)
    B.mq_dynamic_quant_i8(wide[:, :K], 64, q[:, :K], s)
    assert np.array_equal(s.cpu().numpy(), ref_s) and ref_s[2] == 1.0
    assert np.array_equal(q[:, :K].cpu().numpy(), ref_q)
    assert not q[:, K:].any()
