"""GPU parity: every CUDA entry point, called through the C ABI, against the CPU oracle on
the same seeded inputs.  Integer results (codes, accumulators, indices, masks) must match
bit for bit; float results within the stated tolerances (float32 dequant 1e-5 relative,
bf16 output 1e-2 relative)."""
import numpy as np
import pytest
import torch

from oracle import mq_oracle as O
from paper_2502_00425_b200 import binding as B
from paper_2502_00425_b200 import synth

from gpu_util import DEV, bf16_from_dev, bf16_to_dev, dev_segments, gpu_calibrate, gpu_linear, gpu_pack

pytestmark = pytest.mark.gpu


def _rel(a, ref, floor=2.0 ** -126):
    return np.abs(a.astype(np.float64) - ref) / np.maximum(np.abs(ref), floor)


# ----------------------------------------------------------------------------- K1: rotation + quantizer
@pytest.mark.parametrize("rot,K,T", [(0, 256, 5), (0, 1056, 19), (32, 96, 7), (64, 1088, 9), (128, 1152, 33),
                                     (128, 18944, 6), (256, 2304, 10), (512, 2560, 11), (1024, 3072, 4)])
def test_fwht_quant_matches_oracle(rot, K, T):
    rng = np.random.default_rng(1000 + rot + K)
    row_mod = (rng.random(T) < 0.6).astype(np.uint8)
    seg = synth.segments_from_row_modality(row_mod)
    x = rng.standard_t(3.0, size=(T, K)).astype(np.float32)
    x[row_mod == 1] *= 2
    x[0, :8] = [np.inf, -np.inf, np.nan, 0.0, -0.0, 3e38, -3e38, 1e-40]
    x = synth.round_to_bf16(x)
    s_vis, s_txt = np.float32(0.0731), np.float32(0.0217)
    xd = bf16_to_dev(x)
    q = torch.empty((T, K), dtype=torch.int8, device=DEV)
    rdump = torch.empty((T, K), dtype=torch.float32, device=DEV)
    B.mq_fwht_quant_i8(xd, dev_segments(seg), s_vis, s_txt, rot, q, rdump)
    q2 = torch.empty((T, K), dtype=torch.int8, device=DEV)
    B.mq_fwht_quant_i8(xd, dev_segments(seg), s_vis, s_txt, rot, q2, None)
    torch.cuda.synchronize()
    r_gpu = rdump.cpu().numpy()
    with np.errstate(invalid="ignore", over="ignore"):
        r_ref = O.fwht_blocks(x, rot, np.float32)
    finite = np.isfinite(r_ref)
    # the kernel keeps the canonical butterfly order, so the float32 rotation is bit-identical
    assert np.array_equal(r_gpu[finite], r_ref[finite])
    assert np.array_equal(np.isnan(r_gpu), np.isnan(r_ref))
    r64 = O.rotate_dense(np.where(np.isfinite(x), x, 0.0), rot)
    ok_rows = np.isfinite(x).all(axis=1)
    tol = 1e-5 * np.abs(x[ok_rows]).max(axis=1, keepdims=True) * max(1.0, np.sqrt(rot))
    assert np.all(np.abs(r_gpu[ok_rows] - r64[ok_rows]) <= tol)
    # codes: bit-exact given the GPU's own rotated float32 values, and equal with/without the dump
    s_rows = O.row_scales(T, seg.seg_end, seg.seg_mod, s_vis, s_txt)
    q_ref = O.quantize_act_int8(r_gpu, s_rows)
    assert np.array_equal(q.cpu().numpy(), q_ref)
    assert torch.equal(q, q2)


def test_fwht_quant_strided_rows_and_saturation():
    rng = np.random.default_rng(5)
    T, K, ld = 6, 256, 384
    big = synth.round_to_bf16(rng.standard_normal((T, ld)).astype(np.float32) * 100)
    xd_full = bf16_to_dev(big)
    xd = xd_full[:, :K]
    q_full = torch.zeros((T, 512), dtype=torch.int8, device=DEV)
    q = q_full[:, :K]
    seg = synth.Segments(np.array([T], np.int32), np.array([1], np.uint8))
    B.mq_fwht_quant_i8(xd, dev_segments(seg), 0.5, 0.5, 128, q, None)
    want = O.quantize_act_int8(O.fwht_blocks(big[:, :K], 128), np.full(T, 0.5, np.float32))
    assert np.array_equal(q.cpu().numpy(), want)
    assert want.min() == -128 and want.max() == 127          # both clamp branches were taken
    assert int(q_full[:, K:].abs().sum()) == 0                # nothing written outside [T,K]


@pytest.mark.parametrize("rot", [0, 128])
def test_calibration_matches_oracle(rot):
    c = synth.small_linear(21, 40, 9, 1152, 16, rot)
    s_v, s_t = gpu_calibrate(c.x_calib, c.seg_calib, rot)
    o_v, o_t = O.calibrate_static_scales(c.x_calib, c.seg_calib.seg_end, c.seg_calib.seg_mod, rot)
    assert s_v == o_v and s_t == o_t
    # two batches folded into one maximum == one batch holding both
    xa, xb = bf16_to_dev(c.x_calib[:100]), bf16_to_dev(c.x_calib[100:])
    ra, rb = c.seg_calib.row_modality(c.x_calib.shape[0])[:100], c.seg_calib.row_modality(c.x_calib.shape[0])[100:]
    state = torch.zeros(2, dtype=torch.int32, device=DEV)
    sv, st = torch.zeros(1, device=DEV), torch.zeros(1, device=DEV)
    B.mq_calibrate_static_scales(xa, dev_segments(synth.segments_from_row_modality(ra)), rot, state, sv, st)
    B.mq_calibrate_static_scales(xb, dev_segments(synth.segments_from_row_modality(rb)), rot, state, sv, st,
                                 accumulate=True)
    assert np.float32(sv.item()) == o_v and np.float32(st.item()) == o_t
    # a modality without rows gets 1.0
    only_txt = synth.Segments(np.array([100], np.int32), np.array([0], np.uint8))
    B.mq_calibrate_static_scales(xa, dev_segments(only_txt), rot, state, sv, st)
    assert sv.item() == 1.0


# ----------------------------------------------------------------------------- K0b: weight quantizer + layouts
@pytest.mark.parametrize("N,K", [(16, 32), (256, 256), (272, 1152), (128, 160)])
def test_pack_w4_matches_oracle(N, K):
    rng = np.random.default_rng(N + K)
    w = (rng.standard_normal((N, K)) * 0.02).astype(np.float32)
    w[3] = 0.0
    w[5, :4] = [0.5, -0.5, 0.25, 1.0]
    packed, s_w, layout = gpu_pack(w)
    q_ref, s_ref = O.quantize_weight_int4(w)
    assert np.array_equal(s_w.cpu().numpy(), s_ref)
    assert np.array_equal(packed.cpu().numpy(), O.pack_w4(q_ref))
    q1 = torch.empty((N, K), dtype=torch.int8, device=DEV)
    q2 = torch.empty((N, K), dtype=torch.int8, device=DEV)
    B.mq_unpack_w4(N, K, q1, packed=packed)
    B.mq_unpack_w4(N, K, q2, gemm_layout=layout)
    assert np.array_equal(q1.cpu().numpy(), q_ref)
    assert np.array_equal(q2.cpu().numpy(), q_ref)
    layout2 = torch.full_like(layout, 0x5A)
    B.mq_repack_w4(packed, N, K, layout2)
    assert torch.equal(layout, layout2)
    # the layout is a permutation of the canonical nibbles plus zero padding
    lay = layout.cpu().numpy()
    hist = lambda a: np.bincount(np.concatenate([a & 15, a >> 4]).ravel(), minlength=16)
    hl, hc = hist(lay), hist(packed.cpu().numpy())
    assert np.array_equal(hl[1:], hc[1:]) and hl[0] >= hc[0]


# ----------------------------------------------------------------------------- K3: AIFS
def _aifs_case(is_vis, is_pad, D, seed):
    L = len(is_vis)
    x = synth.embedding_rows(seed, L, D, is_vis)
    xd = bf16_to_dev(x)
    xo = torch.zeros_like(xd)
    vis_d = torch.from_numpy(is_vis).to(DEV)
    pad_d = None if is_pad is None else torch.from_numpy(is_pad).to(DEV)
    perm = torch.full((L,), -1, dtype=torch.int32, device=DEV)
    inv = torch.full((L,), -1, dtype=torch.int32, device=DEV)
    n_first = torch.full((1,), -1, dtype=torch.int32, device=DEV)
    B.mq_aifs_reorder(xd, xo, vis_d, pad_d, perm, inv, n_first, direction=0)
    p_ref = O.aifs_perm(is_vis, is_pad)
    assert np.array_equal(perm.cpu().numpy(), p_ref)
    assert np.array_equal(inv.cpu().numpy(), O.inverse_perm(p_ref))
    first = is_vis.astype(bool) if is_pad is None else (is_vis.astype(bool) | is_pad.astype(bool))
    assert n_first.item() == int(first.sum())
    assert np.array_equal(bf16_from_dev(xo), O.aifs_gather(x, p_ref))
    back = torch.zeros_like(xd)
    B.mq_aifs_reorder(xo, back, None, None, perm, None, None, direction=1)
    assert torch.equal(back, xd)
    return perm, n_first, pad_d, p_ref


@pytest.mark.parametrize("name", ["c3", "c4", "tiny", "all_text", "all_visual", "long", "very_long"])
def test_aifs_reorder_and_remap(name):
    rng = np.random.default_rng(7)
    is_pad = None
    if name == "c3":
        is_vis, D = synth.config3_sequence(), 64
    elif name == "c4":
        is_vis, D = synth.config4_sequence(), 32
    elif name == "tiny":
        is_vis, D = np.array([0, 1, 1, 0, 0, 1, 0], np.uint8), 8
        is_pad = np.array([1, 0, 0, 0, 0, 0, 0], np.uint8)
    elif name == "all_text":
        is_vis, D = np.zeros(37, np.uint8), 8
    elif name == "all_visual":
        is_vis, D = np.ones(1025, np.uint8), 8
    elif name == "very_long":      # beyond the single-launch limit: separate index-scan and row-move kernels
        is_vis, D = (rng.random(20000) < 0.4).astype(np.uint8), 8
    else:
        is_vis, D = (rng.random(5000) < 0.7).astype(np.uint8), 16
        is_pad = np.zeros(5000, np.uint8)
        is_pad[:13] = 1
        is_vis[:13] = 0
    perm, n_first, pad_d, p_ref = _aifs_case(is_vis, is_pad, D, 3)
    L = len(is_vis)
    pos = torch.arange(100, 100 + L, dtype=torch.int32, device=DEV)
    pos_out = torch.empty(L, dtype=torch.int32, device=DEV)
    seg_end = torch.empty(2, dtype=torch.int32, device=DEV)
    seg_mod = torch.empty(2, dtype=torch.uint8, device=DEV)
    dense = torch.full((L, L), 7, dtype=torch.uint8, device=DEV) if L <= 4096 else None
    B.mq_attn_mask_remap(perm, pos, pad_d, n_first, pos_out, seg_end, seg_mod, dense)
    assert np.array_equal(pos_out.cpu().numpy(), O.remap_positions(p_ref, np.arange(100, 100 + L)))
    se, sm = O.segments_after_aifs(p_ref, is_vis, is_pad)
    assert np.array_equal(seg_end.cpu().numpy(), se) and np.array_equal(seg_mod.cpu().numpy(), sm)
    if dense is not None:
        assert np.array_equal(dense.cpu().numpy().astype(bool), O.unified_mask(p_ref, is_pad))
    pos_iota = torch.empty(L, dtype=torch.int32, device=DEV)
    B.mq_attn_mask_remap(perm, None, pad_d, n_first, pos_iota)
    assert np.array_equal(pos_iota.cpu().numpy(), p_ref)


def test_aifs_index_only_call():
    is_vis = synth.config3_sequence()
    L = len(is_vis)
    perm = torch.full((L,), -1, dtype=torch.int32, device=DEV)
    inv = torch.full((L,), -1, dtype=torch.int32, device=DEV)
    n_first = torch.full((1,), -1, dtype=torch.int32, device=DEV)
    B.mq_aifs_reorder(None, None, torch.from_numpy(is_vis).to(DEV), None, perm, inv, n_first, direction=0, L=L)
    p_ref = O.aifs_perm(is_vis)
    assert np.array_equal(perm.cpu().numpy(), p_ref) and n_first.item() == int(is_vis.sum())
    assert np.array_equal(inv.cpu().numpy(), O.inverse_perm(p_ref))


# ----------------------------------------------------------------------------- the linear
def _check_linear(case, bias=None, clipping_expected=None):
    """Full protocol on one case; returns the oracle bundle."""
    s_v, s_t = gpu_calibrate(case.x_calib, case.seg_calib, case.rot_block)
    o_v, o_t = O.calibrate_static_scales(case.x_calib, case.seg_calib.seg_end, case.seg_calib.seg_mod,
                                         case.rot_block)
    assert (s_v, s_t) == (o_v, o_t)
    packed, s_w, layout = gpu_pack(case.w)
    qw, sw_ref = O.quantize_weight_int4(case.w)
    assert np.array_equal(s_w.cpu().numpy(), sw_ref)
    ref = O.linear_w4a8_msq(case.x, case.seg.seg_end, case.seg.seg_mod, s_v, s_t, case.rot_block, qw, sw_ref, bias)
    # activation codes through the public quantizer entry point
    q = torch.empty((case.T, case.K), dtype=torch.int8, device=DEV)
    B.mq_fwht_quant_i8(bf16_to_dev(case.x), dev_segments(case.seg), s_v, s_t, case.rot_block, q, None)
    assert np.array_equal(q.cpu().numpy(), ref["qx"])
    if clipping_expected is not None:
        assert (np.abs(ref["qx"].astype(np.int32)).max() >= 127) and \
               ((ref["qx"] == -128).any() or (ref["qx"] == 127).any()) == clipping_expected
    # whole call, bf16 in -> float32 out: accumulators bit-exact, dequant == float32 oracle
    y32, acc, st = gpu_linear(case, s_v, s_t, layout, s_w, bias, torch.float32)
    assert st == (B.MQ_OK, 0)
    assert np.array_equal(acc.cpu().numpy(), ref["acc"])
    y32 = y32.cpu().numpy()
    assert np.array_equal(y32, ref["y32"])
    # relative to the size of the terms (product and bias), so that cancellation between
    # them does not inflate the figure
    mag = np.abs(O.dequant(ref["acc"], ref["s_rows"], sw_ref)) + (0 if bias is None else np.abs(bias)[None, :])
    nz = mag > 0
    assert (np.abs(y32 - ref["y64"])[nz] / mag[nz]).max() <= 1e-5
    # bf16 out with the accumulator dump: within 1e-2 of float64, and equal to the oracle's bf16
    yb, acc2, st = gpu_linear(case, s_v, s_t, layout, s_w, bias, torch.bfloat16)
    assert st == (B.MQ_OK, 0)
    yb = bf16_from_dev(yb)
    assert np.array_equal(yb, ref["y_bf16"])
    assert (np.abs(yb - ref["y64"])[nz] / mag[nz]).max() <= 1e-2
    # the product configuration (bf16 out, no dump: the epilogue with 16-byte stores), and the same
    # with a row pitch that is not a multiple of 16 bytes (falls back to per-element stores)
    for y_pad in (0, 4):
        yp, _, st = gpu_linear(case, s_v, s_t, layout, s_w, bias, torch.bfloat16, want_acc=False, y_pad=y_pad)
        assert st == (B.MQ_OK, 0)
        assert np.array_equal(bf16_from_dev(yp), ref["y_bf16"]), y_pad
    # pre-quantized entry (X already int8) gives the same accumulators
    y3, acc3, st = gpu_linear(case, s_v, s_t, layout, s_w, bias, torch.bfloat16, x_codes=q)
    assert st == (B.MQ_OK, 0) and torch.equal(acc3, acc2)
    return ref


def test_config1_full():
    c = synth.config1()
    ref = _check_linear(c)
    # brute force (nested loops over Python integers) on a corner of the problem
    qw = O.quantize_weight_int4(c.w)[0]
    assert np.array_equal(ref["acc"][:3, :5], O.int_gemm_loops(ref["qx"][:3], qw[:5]))


@pytest.mark.parametrize("T_vis,T_txt,K,N,rot", [
    (200, 100, 1152, 272, 128),    # ragged token tile, ragged channel tile, 9 K blocks
    (0, 70, 256, 128, 0),          # no visual rows
    (70, 0, 256, 128, 64),         # no text rows
    (1, 0, 32, 16, 32),            # the smallest legal problem
    (250, 263, 160, 144, 32),      # K not a multiple of the K block; two token tiles
    (3, 5, 4096, 256, 128),        # T = 8: one 16-token tile, split-K slices + finalize kernel
    (5, 8, 160, 144, 32),          # T = 13: ragged K block, second channel tile mostly empty
    (0, 27, 1152, 272, 128),       # T = 27: three channel tiles, the last one ragged
    (20, 13, 2048, 128, 0),        # T = 33: a 48-token tile, three 16-column epilogue chunks
    (100, 28, 4096, 512, 1024),    # T = 128: the largest decode-shaped problem, split-K
    (100, 29, 1024, 384, 0),       # T = 129: just past the decode-shaped range
])
def test_linear_edge_shapes(T_vis, T_txt, K, N, rot):
    c = synth.small_linear(100 + K + N, T_vis, T_txt, K, N, rot, calib_vis=24, calib_txt=8)
    bias = (np.random.default_rng(1).standard_normal(N)).astype(np.float32)
    _check_linear(c, bias=bias)


@pytest.mark.parametrize("T_vis,T_txt,K,N,rot", [
    (0, 1, 4096, 272, 128),    # one token, ragged last channel quarter (N % 32 = 16), 32 K blocks
    (1, 1, 160, 144, 32),      # two tokens of different modality, K not a multiple of the K block
    (1, 2, 1152, 528, 128),    # three tokens, nine K blocks
    (2, 2, 13696, 64, 128),    # four tokens: the first count that takes the tensor-core path (split K, 107 K blocks)
    (1, 2, 13696, 64, 128),    # three tokens, 107 K blocks over 32 warps, 14 warp passes per row
    (0, 1, 32, 16, 0),         # one K piece, half a channel quarter
    (1, 1, 2048, 96, 1024),    # the largest rotation block (a whole warp pass)
    (0, 2, 512, 48, 64),       # rotation 64
])
def test_linear_gemv_shapes(T_vis, T_txt, K, N, rot):
    # T <= 3 runs the CUDA-core GEMV (mq_gemv.cu): with bf16 input it rotates and quantizes in the
    # same kernel, with int8 input it only multiplies; _check_linear exercises both
    c = synth.small_linear(500 + K + N + T_vis, T_vis, T_txt, K, N, rot, calib_vis=24, calib_txt=8)
    bias = (np.random.default_rng(2).standard_normal(N)).astype(np.float32)
    _check_linear(c, bias=bias)
    _check_linear(c)


@pytest.mark.parametrize("T_vis,T_txt,K,N,rot", [
    (0, 1, 131040, 16, 32),    # the largest K the 16x accumulators allow, one token: GEMV with 1024 K blocks
    (2, 2, 131040, 16, 0),     # four tokens: too long for the GEMV's shared memory, quantizer + split-K GEMM instead
    (5, 4, 131040, 32, 32),    # nine tokens at the largest K
])
def test_linear_maximum_k(T_vis, T_txt, K, N, rot):
    c = synth.small_linear(900 + T_vis + T_txt, T_vis, T_txt, K, N, rot, calib_vis=4, calib_txt=4)
    _check_linear(c)


def test_linear_sixty_four_segments():
    # a batch of 32 short sequences after per-sequence AIFS: 64 alternating segments in one call
    row_mod = synth.interleaved_modality([(1, 5), (0, 3)] * 32)
    c = synth.heavy_tail_linear("many_segments", 78, 0, 0, 256, 64, 64, calib_vis=8, calib_txt=8, row_mod=row_mod)
    assert c.seg.n_seg == 64
    _check_linear(c)


def test_linear_many_segments_without_aifs():
    # MSQ without AIFS: interleaved spans, one segment per span, boundary inside a token tile
    row_mod = synth.interleaved_modality([(0, 5), (1, 130), (0, 17), (1, 64), (0, 40), (1, 33), (0, 11)])
    c = synth.heavy_tail_linear("interleaved", 77, 0, 0, 384, 128, 128, calib_vis=16, calib_txt=16, row_mod=row_mod)
    assert c.seg.n_seg == 7
    _check_linear(c)


def test_linear_many_tiles_per_cta():
    # more tiles than SMs: exercises the persistent loop, both accumulator buffers and stage wrap-around
    c = synth.small_linear(9, 2000, 48, 256, 2560, 0, calib_vis=16, calib_txt=16)
    _check_linear(c)


def test_linear_clipping_variant():
    # calibration without the massive tokens: the quantizer must saturate on them
    c = synth.config2(seed=1, T_vis=96, T_txt=32, K=1024, N=128, clipping_variant=True)
    _check_linear(c, clipping_expected=True)


def test_config2_clipping_variant_full_size_sampled():
    """The clipping variant at the size of config 2: the calibration draw has no massive-activation
    token, so the quantizer saturates; codes of the whole batch against the oracle, the product on
    the sampled rows (which include both massive rows)."""
    c = synth.config2(clipping_variant=True)
    s_v, s_t = gpu_calibrate(c.x_calib, c.seg_calib, c.rot_block)
    o_v, o_t = O.calibrate_static_scales(c.x_calib, c.seg_calib.seg_end, c.seg_calib.seg_mod, c.rot_block)
    assert (s_v, s_t) == (o_v, o_t)
    q = torch.empty((c.T, c.K), dtype=torch.int8, device=DEV)
    B.mq_fwht_quant_i8(bf16_to_dev(c.x), dev_segments(c.seg), s_v, s_t, c.rot_block, q, None)
    q_ref = O.quantize_act_int8(O.fwht_blocks(c.x, c.rot_block, np.float32),
                                O.row_scales(c.T, c.seg.seg_end, c.seg.seg_mod, s_v, s_t))
    assert np.array_equal(q.cpu().numpy(), q_ref)
    # with the massive tokens left out of the calibration draw both clamp branches are taken (the rotation
    # spreads a massive channel over its block, so it is not necessarily the massive rows that saturate)
    assert (q_ref == -128).any() and (q_ref == 127).any()
    _check_full_size_sampled(c, tile_rows=224)


@pytest.mark.parametrize("T,K,N", [(128, 13696, 512), (8, 4096, 1024), (600, 2048, 640), (3, 13696, 4096),
                                   # the decode shapes of config 5 (gate / up and down) over the decode range of T
                                   (5, 4096, 13696), (16, 4096, 13696), (64, 4096, 13696), (128, 4096, 13696),
                                   (5, 13696, 4096), (16, 13696, 4096), (64, 13696, 4096), (128, 13696, 4096),
                                   (8, 4096, 27392),      # gate and up as one weight: more channel tiles than SMs
                                   (24, 96, 4096),        # one K block per channel tile
                                   (16, 13696, 256)])     # two channel tiles, 107 K blocks: many K splits
def test_repeated_launches_give_identical_accumulators(T, K, N):
    """A race in the producer / expander / MMA pipeline shows as a result that changes from launch
    to launch.  Exact integer reference (int8 x int4 codes, float64 matmul is exact here), the
    first launch cold, then back-to-back launches without host synchronisation in between."""
    g = torch.Generator().manual_seed(T + K + N)
    x = torch.randint(-127, 128, (T, K), dtype=torch.int8, generator=g)
    qw = torch.randint(-8, 8, (N, K), dtype=torch.int8, generator=g)
    packed = ((qw[:, 0::2] & 15) | ((qw[:, 1::2] & 15) << 4)).to(torch.uint8)
    layout = torch.empty(B.mq_w4_layout_bytes(N, K), dtype=torch.uint8, device=DEV)
    B.mq_repack_w4(packed.to(DEV), N, K, layout)
    ref = (x.to(torch.float64) @ qw.to(torch.float64).T).to(torch.int32)
    xd, ones = x.to(DEV), torch.ones(N, device=DEV)
    seg = B.Segments.from_host([T // 2, T], [1, 0], DEV)
    ws = B.new_workspace(T, K, N, 0, B.MQ_FLAG_X_IS_INT8)
    y = torch.empty((T, N), dtype=torch.float32, device=DEV)
    accs = [torch.full((T, N), -7, dtype=torch.int32, device=DEV) for _ in range(12)]
    for a in accs:
        B.mq_w4a8_msq_linear(xd, seg, 1.0, 1.0, layout, ones, y, ws, N, acc_out=a)
    assert B.mq_last_device_status(ws) == (B.MQ_OK, 0)
    for a in accs:
        assert torch.equal(a.cpu(), ref)


def test_zero_rows_is_a_noop():
    c = synth.small_linear(3, 4, 4, 128, 128, 0, calib_vis=4, calib_txt=4)
    packed, s_w, layout = gpu_pack(c.w)
    ws = B.new_workspace(8, 128, 128)
    x = torch.empty((0, 128), dtype=torch.bfloat16, device=DEV)
    y = torch.empty((0, 128), dtype=torch.bfloat16, device=DEV)
    B.mq_w4a8_msq_linear(x, dev_segments(c.seg), 1.0, 1.0, layout, s_w, y, ws, 128)
    assert B.mq_last_device_status(ws) == (B.MQ_OK, 0)


def test_config5_decode_shapes():
    for which in ("gate_proj", "down_proj"):
        for T in (1, 8, 32, 128):
            c = synth.config5_linear(which, T)
            _check_linear(c)


def test_config2_full_size_sampled():
    """Config 2 at full size in the launch configuration the benchmark times; the oracle
    checks every column of a deterministic row sample (every 16th row, rows within 2 of the
    modality boundary, first/last rows of each 224-token tile)."""
    c = synth.config2()
    s_v, s_t = gpu_calibrate(c.x_calib, c.seg_calib, c.rot_block)
    o_v, o_t = O.calibrate_static_scales(c.x_calib, c.seg_calib.seg_end, c.seg_calib.seg_mod, c.rot_block)
    assert (s_v, s_t) == (o_v, o_t)
    packed, s_w, layout = gpu_pack(c.w)
    qw, sw_ref = O.quantize_weight_int4(c.w)
    assert np.array_equal(s_w.cpu().numpy(), sw_ref)
    assert np.array_equal(packed.cpu().numpy(), O.pack_w4(qw))
    rows = set(range(0, c.T, 16)) | set(range(1022, 1027)) | {c.T - 1}
    for t0 in range(0, c.T, 224):
        rows |= {t0, min(c.T - 1, t0 + 223)}
    rows |= set(c.meta["massive_rows"])
    rows = np.array(sorted(rows))
    yb, acc, st = gpu_linear(c, s_v, s_t, layout, s_w, None, torch.bfloat16)
    assert st == (B.MQ_OK, 0)
    sub_mod = c.seg.row_modality(c.T)[rows]
    ref = O.linear_w4a8_msq(c.x[rows], *_seg_arrays(sub_mod), s_v, s_t, c.rot_block, qw, sw_ref)
    assert np.array_equal(acc.cpu().numpy()[rows], ref["acc"])
    assert np.array_equal(bf16_from_dev(yb)[rows], ref["y_bf16"])
    nz = np.abs(ref["y64"]) > 0
    assert _rel(bf16_from_dev(yb)[rows], ref["y64"])[nz].max() <= 1e-2
    # property that holds at any size: every accumulator obeys |acc| <= 128 * 8 * K
    assert int(acc.abs().max()) <= 128 * 8 * c.K
    # the launch the benchmark times (no accumulator dump: 16-byte stores) writes the same bits everywhere
    yp, _, st = gpu_linear(c, s_v, s_t, layout, s_w, None, torch.bfloat16, want_acc=False)
    assert st == (B.MQ_OK, 0) and torch.equal(yp.view(torch.int16), yb.view(torch.int16))


def _check_full_size_sampled(c, tile_rows, n_sample=24):
    """Full-size linear in the launch configuration a layer would use; the oracle checks every
    column of a deterministic row sample: rows around every segment boundary, first / last rows
    of token tiles, the massive-activation rows and an even spread."""
    s_v, s_t = gpu_calibrate(c.x_calib, c.seg_calib, c.rot_block)
    o_v, o_t = O.calibrate_static_scales(c.x_calib, c.seg_calib.seg_end, c.seg_calib.seg_mod, c.rot_block)
    assert (s_v, s_t) == (o_v, o_t)
    packed, s_w, layout = gpu_pack(c.w)
    qw, sw_ref = O.quantize_weight_int4(c.w)
    assert np.array_equal(s_w.cpu().numpy(), sw_ref)
    rows = {0, c.T - 1} | set(c.meta["massive_rows"])
    for e in np.asarray(c.seg.seg_end)[:-1].tolist():
        rows |= {e - 1, e}
    for t0 in range(0, c.T, tile_rows):
        rows |= {t0, min(c.T - 1, t0 + tile_rows - 1)}
    rows = sorted(rows)
    if len(rows) > n_sample:                     # thin the tile-edge rows, keep boundaries and massive rows
        keep = set(c.meta["massive_rows"]) | {0, c.T - 1}
        for e in np.asarray(c.seg.seg_end)[:-1].tolist():
            keep |= {e - 1, e}
        rest = [r for r in rows if r not in keep]
        step = max(1, len(rest) // max(1, n_sample - len(keep)))
        rows = sorted(keep | set(rest[::step]))
    rows = np.array(rows)
    yb, acc, st = gpu_linear(c, s_v, s_t, layout, s_w, None, torch.bfloat16)
    assert st == (B.MQ_OK, 0)
    sub_mod = c.seg.row_modality(c.T)[rows]
    ref = O.linear_w4a8_msq(c.x[rows], *_seg_arrays(sub_mod), s_v, s_t, c.rot_block, qw, sw_ref)
    assert np.array_equal(acc.cpu().numpy()[rows], ref["acc"])
    assert np.array_equal(bf16_from_dev(yb)[rows], ref["y_bf16"])
    nz = np.abs(ref["y64"]) > 0
    assert _rel(bf16_from_dev(yb)[rows], ref["y64"])[nz].max() <= 1e-2
    assert int(acc.abs().max()) <= 128 * 8 * c.K
    # the launch the benchmark times (no accumulator dump: 16-byte stores) writes the same bits everywhere
    yp, _, st = gpu_linear(c, s_v, s_t, layout, s_w, None, torch.bfloat16, want_acc=False)
    assert st == (B.MQ_OK, 0) and torch.equal(yp.view(torch.int16), yb.view(torch.int16))


@pytest.mark.parametrize("which", ["k_proj", "down_proj"])
def test_config3_linears_full_size_sampled(which):
    """Qwen2-7B-shaped block at T = 3360 in AIFS order (3072 visual, 288 text): the narrow
    k-projection (N = 512) and the rotated down-projection (K = 18944)."""
    _check_full_size_sampled(synth.config3_linear(which), tile_rows=192)


@pytest.mark.parametrize("which", ["q_proj", "k_proj", "v_proj", "o_proj", "gate_proj", "up_proj", "down_proj"])
def test_config4_linears_full_size_sampled(which):
    """8B-shaped block, batch of 4 sequences flattened to 9728 rows with 8 segments: all seven linears
    (gate / up are the deepest persistent loop: 112 channel tiles x 51 token tiles)."""
    c = synth.config4_linear(which)
    assert c.seg.n_seg == 8 and c.T == 9728
    _check_full_size_sampled(c, tile_rows=192)


def _seg_arrays(row_mod):
    s = synth.segments_from_row_modality(row_mod)
    return s.seg_end, s.seg_mod
