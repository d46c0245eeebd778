"""Full-width Kronecker rotation H_m (x) H_(K/m) + MSQ quantizer (mq_kron_quant_i8) against the oracle: the
float32 rotated values bit for bit (same order of additions), the codes bit for bit, and the linear that
consumes them (int8 entry of mq_w4a8_msq_linear) against the oracle's integer product; the rotation's
invariance (x H)(W H)^T = x W^T holds up to the quantization error."""
import numpy as np
import pytest
import torch

from oracle import mq_oracle as O
from paper_2502_00425_b200 import binding as B
from paper_2502_00425_b200 import synth

from gpu_util import DEV, bf16_from_dev, bf16_to_dev, dev_segments, gpu_pack

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("m,n2,T", [(12, 32, 7), (1, 64, 3), (20, 1024, 4), (28, 512, 9), (148, 128, 6)])
def test_kron_quant_matches_oracle(m, n2, T):
    K = m * n2
    rng = np.random.default_rng(m * 1000 + n2)
    Hm = O.paley_hadamard(m) if m > 1 else np.array([[1]])
    row_mod = (rng.random(T) < 0.5).astype(np.uint8)
    seg = synth.segments_from_row_modality(row_mod)
    x = rng.standard_t(3.0, size=(T, K)).astype(np.float32)
    x[row_mod == 1] *= 2
    x = synth.round_to_bf16(x)
    r_ref = O.kron_rotate_f32(x, Hm, n2)
    s_vis = O.static_scale(r_ref[row_mod == 1]) if row_mod.any() else np.float32(1.0)
    s_txt = O.static_scale(r_ref[row_mod == 0]) if (row_mod == 0).any() else np.float32(1.0)
    h_neg = torch.from_numpy((Hm < 0).astype(np.uint8)).to(DEV)
    q = torch.empty((T, K), dtype=torch.int8, device=DEV)
    dump = torch.empty((T, K), dtype=torch.float32, device=DEV)
    B.mq_kron_quant_i8(bf16_to_dev(x), dev_segments(seg), s_vis, s_txt, h_neg, q, dump)
    q2 = torch.empty((T, K), dtype=torch.int8, device=DEV)
    B.mq_kron_quant_i8(bf16_to_dev(x), dev_segments(seg), s_vis, s_txt, h_neg, q2, None)
    torch.cuda.synchronize()
    r_gpu = dump.cpu().numpy()
    assert np.array_equal(r_gpu, r_ref)                                       # same order of float32 additions
    assert np.max(np.abs(r_gpu - O.kron_rotate_dense(x, Hm, n2))) <= 1e-5 * np.abs(x).max() * np.sqrt(K)
    s_rows = O.row_scales(T, seg.seg_end, seg.seg_mod, s_vis, s_txt)
    q_ref = O.quantize_act_int8(r_gpu, s_rows)
    assert np.array_equal(q.cpu().numpy(), q_ref) and torch.equal(q, q2)
    assert np.abs(q_ref.astype(np.int32)).max() == 127                        # the scales came from these very rows


def test_kron_rotated_linear_reproduces_the_unrotated_product():
    # K = 14336 = 28 * 512 (the 8B-shaped down-projection): rotate the weight offline with the same matrix, run
    # the online rotation + quantizer, then the W4A8 product on the codes
    m, n2, T, N = 28, 512, 24, 128
    K = m * n2
    rng = np.random.default_rng(77)
    Hm = O.paley_hadamard(m)
    row_mod = np.concatenate([np.ones(16), np.zeros(8)]).astype(np.uint8)
    seg = synth.segments_from_row_modality(row_mod)
    x = synth.round_to_bf16((rng.standard_t(3.0, size=(T, K)) * np.where(row_mod[:, None] == 1, 2.0, 1.0)).astype(np.float32))
    x[3, 100] = 300.0                                                         # an outlier the rotation spreads out
    x = synth.round_to_bf16(x)
    w = (rng.standard_normal((N, K)) * 0.02).astype(np.float32)
    w_rot = O.kron_rotate_dense(w, Hm, n2).astype(np.float32)                  # offline: W H
    r = O.kron_rotate_f32(x, Hm, n2)
    s_vis, s_txt = O.static_scale(r[row_mod == 1]), O.static_scale(r[row_mod == 0])
    h_neg = torch.from_numpy((Hm < 0).astype(np.uint8)).to(DEV)
    q = torch.empty((T, K), dtype=torch.int8, device=DEV)
    B.mq_kron_quant_i8(bf16_to_dev(x), dev_segments(seg), s_vis, s_txt, h_neg, q, None)
    packed, s_w, layout = gpu_pack(w_rot)
    qw, s_ref = O.quantize_weight_int4(w_rot)
    ws = B.new_workspace(T, K, N, 0, B.MQ_FLAG_X_IS_INT8)
    y = torch.empty((T, N), dtype=torch.float32, device=DEV)
    acc = torch.empty((T, N), dtype=torch.int32, device=DEV)
    B.mq_w4a8_msq_linear(q, dev_segments(seg), s_vis, s_txt, layout, s_w, y, ws, N, acc_out=acc)
    assert B.mq_last_device_status(ws) == (B.MQ_OK, 0)
    s_rows = O.row_scales(T, seg.seg_end, seg.seg_mod, s_vis, s_txt)
    qx_ref = O.quantize_act_int8(r, s_rows)
    assert np.array_equal(q.cpu().numpy(), qx_ref)
    assert np.array_equal(acc.cpu().numpy(), O.int_gemm(qx_ref, qw))
    assert np.array_equal(y.cpu().numpy(), O.dequant(O.int_gemm(qx_ref, qw), s_rows, s_ref, None, np.float32))
    # invariance: close to the product of the unrotated operands, and closer than quantizing without rotation
    exact = x.astype(np.float64) @ w.astype(np.float64).T
    err_rot = np.abs(y.cpu().numpy() - exact).mean()
    plain = O.linear_w4a8_msq(x, seg.seg_end, seg.seg_mod, *O.calibrate_static_scales(x, seg.seg_end, seg.seg_mod, 0), 0,
                              *O.quantize_weight_int4(w))
    err_plain = np.abs(plain["y64"] - exact).mean()
    # (the 4-bit weight error dominates what is left: random weights have no structure for a rotation to help)
    assert err_rot < err_plain and err_rot <= 0.25 * np.abs(exact).mean()
