"""Pins for the CPU oracle: each function is tied to something other than itself
(integer identities, closed forms, hand-worked cases, brute force, the paper's
printed maps), chosen so that a dropped term, a wrong sign or index or a
transposed operand fails at least one of them.  CPU only."""
import itertools
import os

import numpy as np
import pytest

from oracle import mq_oracle as O

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _read_ints(name):
    rows = []
    with open(os.path.join(GOLD, name)) as f:
        for line in f:
            line = line.strip()
            if line and not line.startswith("#"):
                rows.append([int(v) for v in line.split()])
    return rows


# ----------------------------------------------------------------------------- Hadamard / FWHT (App. A.3, Sec. 3.2)
def test_hadamard_h4_matches_hand_written_fixture():
    assert np.array_equal(O.hadamard_matrix(4), np.array(_read_ints("hadamard_h4.txt")))


@pytest.mark.parametrize("n", [1, 2, 4, 8, 16, 32, 64])
def test_hadamard_gram_is_n_identity_in_integers(n):
    H = O.hadamard_matrix(n)
    assert set(np.unique(H).tolist()) <= {-1, 1}
    assert np.array_equal(H @ H.T, n * np.eye(n, dtype=np.int64))
    assert np.array_equal(H, H.T)
    # Sylvester closed form: H[i,j] = (-1)^popcount(i & j)
    i, j = np.meshgrid(np.arange(n), np.arange(n), indexing="ij")
    pc = np.vectorize(lambda v: bin(v).count("1"))(i & j)
    assert np.array_equal(H, np.where(pc % 2 == 0, 1, -1))


@pytest.mark.parametrize("n", [2, 4, 8, 16, 32, 64, 128])
@pytest.mark.parametrize("dtype", [np.float32, np.float64])
def test_fwht_equals_dense_hadamard_product(n, dtype):
    rng = np.random.default_rng(n)
    x = rng.standard_normal((5, 3 * n)).astype(np.float32)
    fast = O.fwht_blocks(x, n, dtype).astype(np.float64)
    dense = O.rotate_dense(x, n)
    tol = (1e-6 if dtype == np.float32 else 1e-13) * np.abs(x).max() * np.sqrt(n)
    assert np.max(np.abs(fast - dense)) <= tol


def test_fwht_unit_impulse_gives_hadamard_columns():
    n = 16
    H = O.hadamard_matrix(n) / np.sqrt(n)
    for j in range(n):
        e = np.zeros((1, n), np.float32)
        e[0, j] = 1.0
        assert np.allclose(O.fwht_blocks(e, n, np.float64)[0], H[j], atol=1e-15)


def test_fwht_first_coefficient_is_sqrt_n_times_mean():
    # Sec. 3.2: (H W)_{0j} = sqrt(n) * mean(w_{:,j}) for the normalised transform,
    # = sum_r w_{rj} without the normalisation (App. A.3).
    rng = np.random.default_rng(7)
    n = 128
    x = rng.standard_normal((4, 2 * n))
    y = O.fwht_blocks(x, n, np.float64)
    for b in range(2):
        blk = x[:, b * n:(b + 1) * n]
        assert np.allclose(y[:, b * n], np.sqrt(n) * blk.mean(axis=1), rtol=1e-12)
        assert np.allclose(y[:, b * n] * np.sqrt(n), blk.sum(axis=1), rtol=1e-12)


def test_fwht_preserves_norm_and_is_an_involution():
    rng = np.random.default_rng(8)
    x = rng.standard_normal((6, 256))
    y = O.fwht_blocks(x, 64, np.float64)
    assert np.allclose(np.linalg.norm(y, axis=1), np.linalg.norm(x, axis=1), rtol=1e-12)
    assert np.allclose(O.fwht_blocks(y, 64, np.float64), x, atol=1e-12)
    y32 = O.fwht_blocks(x.astype(np.float32), 64, np.float32)
    assert np.allclose(np.linalg.norm(y32, axis=1), np.linalg.norm(x, axis=1), rtol=1e-5)


def test_fwht_blocks_are_independent_and_ordered():
    # a value in block 1 must not leak into block 0, and block b lands at columns b*n..
    n = 8
    x = np.zeros((1, 3 * n), np.float32)
    x[0, n + 2] = 1.0
    y = O.fwht_blocks(x, n, np.float64)
    assert np.all(y[0, :n] == 0) and np.all(y[0, 2 * n:] == 0)
    assert np.allclose(y[0, n:2 * n], O.hadamard_matrix(n)[2] / np.sqrt(n))


def test_fwht_float32_exact_on_small_integers():
    # sums of small integers are exact in float32, so with n a power of four the
    # float32 transform equals the integer transform divided by sqrt(n) exactly.
    n = 64
    rng = np.random.default_rng(3)
    x = rng.integers(-8, 9, size=(3, n)).astype(np.float32)
    want = (x.astype(np.int64) @ O.hadamard_matrix(n)) / 8.0
    assert np.array_equal(O.fwht_blocks(x, n, np.float32).astype(np.float64), want)


def test_rotation_off_is_identity():
    x = np.arange(12, dtype=np.float32).reshape(3, 4)
    assert np.array_equal(O.fwht_blocks(x, 0), x)
    assert np.array_equal(O.rotate_dense(x, 0), x)


# ----------------------------------------------------------------------------- scales (Eq. 2, Eq. 3)
def test_static_scale_closed_form():
    x = np.array([[0.5, -3.0, 2.0], [1.0, 254.0, -7.0]], np.float32)
    assert O.static_scale(x) == np.float32(2.0)            # 254 / 127
    assert O.static_scale(np.array([-63.5], np.float32)) == np.float32(0.5)
    assert O.static_scale(np.zeros(4, np.float32)) == np.float32(1.0)
    assert O.static_scale(np.zeros(0, np.float32)) == np.float32(1.0)
    assert O.static_scale(np.array([7.0, -3.5], np.float32), qmax=7) == np.float32(1.0)


def test_calibration_is_per_modality_and_after_rotation():
    # rows 0..1 visual, row 2 text; rotation block 4 turns [a,a,a,a] into [2a,0,0,0]
    x = np.array([[1, 1, 1, 1], [-3, -3, -3, -3], [0.25, 0.25, 0.25, 0.25]], np.float32)
    s_v, s_t = O.calibrate_static_scales(x, [2, 3], [1, 0], 4)
    assert s_v == np.float32(6.0 / 127.0) and s_t == np.float32(0.5 / 127.0)
    s_v0, s_t0 = O.calibrate_static_scales(x, [2, 3], [1, 0], 0)
    assert s_v0 == np.float32(3.0 / 127.0) and s_t0 == np.float32(0.25 / 127.0)
    # the element that sets the scale quantizes to +-127 exactly
    r = O.fwht_blocks(x, 4)
    q = O.quantize_act_int8(r, O.row_scales(3, [2, 3], [1, 0], s_v, s_t))
    assert q[1, 0] == -127 and q[2, 0] == 127 and q[0, 0] == 42  # 2/6*127 = 42.33


def test_calibration_missing_modality_gives_one():
    x = np.ones((2, 4), np.float32)
    s_v, s_t = O.calibrate_static_scales(x, [2], [0], 0)
    assert s_v == np.float32(1.0) and s_t == np.float32(1.0 / 127.0)


def test_row_modality_lookup():
    assert O.row_modality(6, [2, 5], [1, 0]).tolist() == [1, 1, 0, 0, 0, 0]
    assert O.row_modality(5, [1, 3, 5], [0, 1, 0]).tolist() == [0, 1, 1, 0, 0]
    assert O.row_modality(3, [], []).tolist() == [0, 0, 0]


# ----------------------------------------------------------------------------- activation quantizer (Eq. 2)
def test_act_quantizer_hand_cases():
    s = np.float32(0.5)  # a power of two: r/s is exact
    r = np.array([[0.0, 0.5, -0.5, 1.0, 63.5, -64.0, 100.0, -100.0,
                   0.25, 0.75, 1.25, -0.25, -0.75, 0.26, np.inf, -np.inf, np.nan]], np.float32)
    q = O.quantize_act_int8(r, [s])
    #   ties go to the even code: 0.5->0, 1.5->2, 2.5->2, -0.5->-0, -1.5->-2
    assert q.tolist() == [[0, 1, -1, 2, 127, -128, 127, -128, 0, 2, 2, 0, -2, 1, 127, -128, 0]]
    assert np.array_equal(O.quantize_act_int8_divide(r, [s]), q)


def test_act_quantizer_exact_multiples_error_bound_and_idempotence():
    rng = np.random.default_rng(5)
    s = np.float32(0.037)
    k = np.arange(-128, 128, dtype=np.float32)
    assert np.array_equal(O.quantize_act_int8((k * s).reshape(1, -1), [s])[0], k.astype(np.int8))
    r = rng.uniform(-127 * s, 127 * s, size=(4, 500)).astype(np.float32)
    q = O.quantize_act_int8(r, np.full(4, s))
    assert np.max(np.abs(q.astype(np.float64) * s - r)) <= 0.5 * s * (1 + 1e-5)
    rq = (q.astype(np.float32) * s).astype(np.float32)
    assert np.array_equal(O.quantize_act_int8(rq, np.full(4, s)), q)


def test_act_quantizer_uses_the_row_scale():
    r = np.array([[10.0, -10.0], [10.0, -10.0]], np.float32)
    q = O.quantize_act_int8(r, O.row_scales(2, [1, 2], [1, 0], 1.0, 0.25))
    assert q.tolist() == [[10, -10], [40, -40]]


# ----------------------------------------------------------------------------- weight quantizer and packing
def test_weight_quantizer_hand_cases():
    w = np.array([[7.0, -3.5, 0.49, 0.51, -7.0, 1.5, 2.5, 0.0],
                  [0, 0, 0, 0, 0, 0, 0, 0],
                  [-14.0, 14.0, 1.0, 3.0, -1.0, 5.0, -15.9, 16.0]], np.float32)
    q, s = O.quantize_weight_int4(w)
    assert s.tolist() == [1.0, 1.0, np.float32(16.0 / 7.0)]
    assert q[0].tolist() == [7, -4, 0, 1, -7, 2, 2, 0]     # -3.5 -> -4 and 2.5 -> 2: ties to even
    assert q[1].tolist() == [0] * 8
    assert q[2].tolist() == [-6, 6, 0, 1, 0, 2, -7, 7]
    assert q.min() >= -8 and q.max() <= 7


def test_weight_error_bound():
    rng = np.random.default_rng(9)
    w = rng.standard_normal((16, 64)).astype(np.float32)
    q, s = O.quantize_weight_int4(w)
    assert np.max(np.abs(q * s[:, None].astype(np.float64) - w) / s[:, None]) <= 0.5 + 1e-5


def test_pack_layout_and_roundtrip_over_all_byte_values():
    q = np.array([[-8, 7, 1, -1]], np.int8)
    p = O.pack_w4(q)
    assert p.tolist() == [[0x78, 0xF1]]                    # low nibble = even k
    allb = np.arange(256, dtype=np.uint8).reshape(1, 256)
    codes = O.unpack_w4(allb)
    assert codes.min() == -8 and codes.max() == 7
    assert np.array_equal(O.pack_w4(codes), allb)
    # byte 0xF8 = low nibble 8 (-8), high nibble 15 (-1)
    assert O.unpack_w4(np.array([[0xF8]], np.uint8)).tolist() == [[-8, -1]]


# ----------------------------------------------------------------------------- integer GEMM
def test_int_gemm_against_python_loops_and_structure():
    rng = np.random.default_rng(11)
    qx = rng.integers(-128, 128, size=(5, 24)).astype(np.int8)
    qw = rng.integers(-8, 8, size=(7, 24)).astype(np.int8)
    acc = O.int_gemm(qx, qw)
    assert acc.dtype == np.int32 and acc.shape == (5, 7)
    assert np.array_equal(acc, O.int_gemm_loops(qx, qw))
    # an all-ones activation row returns the weight row sums (catches a transposed operand)
    ones = np.ones((1, 24), np.int8)
    assert np.array_equal(O.int_gemm(ones, qw)[0], qw.astype(np.int64).sum(axis=1))
    assert np.max(np.abs(acc)) <= 128 * 8 * 24


def test_int_gemm_extreme_values_exact():
    K = 4096
    qx = np.full((2, K), -128, np.int8)
    qw = np.full((3, K), -8, np.int8)
    assert np.all(O.int_gemm(qx, qw) == 128 * 8 * K)


# ----------------------------------------------------------------------------- dequant
def test_dequant_exact_with_power_of_two_scales():
    acc = np.array([[3, -5], [1 << 20, 7]], np.int32)
    y = O.dequant(acc, [0.5, 0.25], [2.0, 0.125], bias=[1.0, -1.0], dtype=np.float32)
    assert y.tolist() == [[4.0, -1.3125], [524289.0, -0.78125]]
    assert np.array_equal(O.dequant(acc, [0.5, 0.25], [2.0, 0.125], bias=[1.0, -1.0]), y.astype(np.float64))


def test_bf16_rne_hand_cases():
    f = lambda bits: np.array([bits], np.uint32).view(np.float32)
    assert O.bf16_rne(f(0x3F808000)).view(np.uint32)[0] == 0x3F800000   # tie -> even (down)
    assert O.bf16_rne(f(0x3F818000)).view(np.uint32)[0] == 0x3F820000   # tie -> even (up)
    assert O.bf16_rne(f(0x3F808001)).view(np.uint32)[0] == 0x3F810000   # above the tie
    assert O.bf16_rne(f(0x3F807FFF)).view(np.uint32)[0] == 0x3F800000
    assert O.bf16_rne(np.array([1.0, -2.5, 0.0], np.float32)).tolist() == [1.0, -2.5, 0.0]


# ----------------------------------------------------------------------------- whole linear
def test_rotation_invariance_without_quantization():
    # App. A.14 (computational invariance): (x H)(W H)^T = x W^T for orthogonal H
    rng = np.random.default_rng(13)
    x = rng.standard_normal((6, 256))
    w = rng.standard_normal((5, 256))
    lhs = O.rotate_dense(x, 128) @ O.rotate_weight_input_dim(w, 128).T
    assert np.allclose(lhs, x @ w.T, rtol=1e-11, atol=1e-11)


def test_linear_quantization_error_bound_and_msq_benefit():
    from paper_2502_00425_b200 import synth
    c = synth.config1()
    qw, s_w = O.quantize_weight_int4(c.w)
    s_v, s_t = O.calibrate_static_scales(c.x_calib, c.seg_calib.seg_end, c.seg_calib.seg_mod, 0)
    out = O.linear_w4a8_msq(c.x, c.seg.seg_end, c.seg.seg_mod, s_v, s_t, 0, qw, s_w)
    exact = c.x.astype(np.float64) @ c.w.astype(np.float64).T
    # |y - xW^T| <= sum_k (|x| s_w/2 + |w| s_a/2 + s_a s_w/4): half a step on each operand
    s_a = out["s_rows"].astype(np.float64)[:, None]
    bound = (np.abs(c.x).astype(np.float64) @ (np.ones_like(c.w, dtype=np.float64) * (s_w[:, None] / 2)).T
             + s_a / 2 * np.abs(c.w).astype(np.float64).sum(axis=1)[None, :]
             + c.K * s_a * s_w[None, :] / 4)
    assert np.all(np.abs(out["y64"] - exact) <= bound * (1 + 1e-6))
    assert np.abs(out["qx"]).max() == 127                  # scales came from these rows: no clipping
    # Sec. 3.1 advantage (3): with one shared scale the text rows lose resolution
    s_one = max(s_v, s_t)
    shared = O.linear_w4a8_msq(c.x, c.seg.seg_end, c.seg.seg_mod, s_one, s_one, 0, qw, s_w)
    txt = slice(48, 64)
    err_msq = np.linalg.norm(out["y64"][txt] - exact[txt])
    err_one = np.linalg.norm(shared["y64"][txt] - exact[txt])
    assert err_msq < err_one
    # float32 dequant and bf16 output stay within the stated tolerances of float64
    assert np.max(np.abs(out["y32"] - out["y64"]) / np.maximum(np.abs(out["y64"]), 1e-30)) <= 1e-5
    rel = np.abs(out["y_bf16"].astype(np.float64) - out["y64"]) / np.maximum(np.abs(out["y64"]), 2.0 ** -126)
    assert rel.max() <= 2.0 ** -8


# ----------------------------------------------------------------------------- AIFS (Sec. 3.1, App. A.2, A.4)
def test_aifs_perm_matches_printed_index_map():
    (m, n, L), order = _read_ints("aifs_index_map.txt")
    is_vis = np.zeros(L, np.uint8)
    is_vis[m - 1:n] = 1
    perm = O.aifs_perm(is_vis)
    assert (perm + 1).tolist() == order
    assert (perm + 1).tolist() == list(range(m, n + 1)) + list(range(1, m)) + list(range(n + 1, L + 1))
    inv = O.inverse_perm(perm)
    assert np.array_equal(perm[inv], np.arange(L)) and np.array_equal(inv[perm], np.arange(L))


def test_aifs_perm_is_a_stable_partition_for_many_spans():
    is_vis = np.array([0, 1, 1, 0, 0, 1, 0, 1, 1, 0], np.uint8)
    perm = O.aifs_perm(is_vis)
    assert perm.tolist() == [1, 2, 5, 7, 8, 0, 3, 4, 6, 9]
    x = np.arange(20).reshape(10, 2)
    xu = O.aifs_gather(x, perm)
    assert np.array_equal(xu[:, 0] // 2, perm)
    assert np.array_equal(O.aifs_scatter(xu, perm), x)
    assert np.array_equal(O.remap_positions(perm), perm)
    assert np.array_equal(O.remap_positions(perm, np.arange(10) + 100), perm + 100)
    se, sm = O.segments_after_aifs(perm, is_vis)
    assert se.tolist() == [5, 10] and sm.tolist() == [1, 0]


@pytest.mark.parametrize("m,n,L", [(3, 5, 8), (1, 4, 6), (4, 7, 7), (2, 2, 5), (1, 5, 5)])
def test_unified_mask_reduces_to_eq5_cases_for_one_span(m, n, L):
    is_vis = np.zeros(L, np.uint8)
    is_vis[m - 1:n] = 1
    perm = O.aifs_perm(is_vis)
    assert np.array_equal(O.unified_mask(perm), O.unified_mask_single_span(m, n, L))
    # and it is the original causal mask seen through the permutation
    assert np.array_equal(O.unified_mask(perm), O.causal_mask(L)[np.ix_(perm, perm)])


def test_causal_mask_is_lower_triangular():
    assert np.array_equal(O.causal_mask(4), np.tril(np.ones((4, 4), bool)))


def _attn_case(rng, is_vis, is_pad=None, D=8):
    L = len(is_vis)
    q, k, v = (rng.standard_normal((L, D)) for _ in range(3))
    pos = np.arange(L)
    allowed = O.causal_mask(L)
    if is_pad is not None:
        padb = np.asarray(is_pad).astype(bool)
        allowed = (allowed & ~padb[None, :]) | (np.eye(L, dtype=bool) & padb[:, None])
    ref = O.attention(O.rope(q, pos), O.rope(k, pos), v, allowed)
    perm = O.aifs_perm(is_vis, is_pad)
    pos_u = O.remap_positions(perm, pos)
    out_u = O.attention(O.rope(q[perm], pos_u), O.rope(k[perm], pos_u), v[perm], O.unified_mask(perm, is_pad))
    return ref, out_u, perm


def test_attention_hand_worked_three_tokens():
    # Eq. 4: softmax(Q K^T / sqrt(D) + M) V written out by hand for D = 4 (1/sqrt(D) = 1/2).
    # Scores before the scale are 2 ln(w), so the softmax weights are the integers w over their sum:
    #   row 0 sees column 0 only                      -> v0
    #   row 1: weights (3, 1)      over 4             -> 3/4 v0 + 1/4 v1
    #   row 2: weights (2, 1, 5)   over 8             -> (2 v0 + v1 + 5 v2) / 8
    # A missing 1/sqrt(D) would give (9, 1)/10 and (4, 1, 25)/30; a missing normalisation the bare sums.
    ln = np.log
    k = np.array([[1.0, 0, 0, 0], [0, 0, 0, 0], [0, 1.0, 0, 0]])
    q = np.array([[7.0, -3.0, 0, 0], [2 * ln(3.0), 0, 0, 0], [2 * ln(2.0), 2 * ln(5.0), 0, 0]])
    v = np.array([[8.0, 0.0], [0.0, 8.0], [16.0, 16.0]])
    out = O.attention(q, k, v, O.causal_mask(3))
    want = np.array([[8.0, 0.0], [6.0, 2.0], [12.0, 11.0]])
    assert np.max(np.abs(out - want)) <= 1e-12
    # Eq. 5 as a mask: forbid column 1 for row 2 -> weights (2, 5) over 7; an allowed future column counts
    allowed = O.causal_mask(3)
    allowed[2, 1] = False
    out = O.attention(q, k, v, allowed)
    assert np.max(np.abs(out[2] - np.array([(2 * 8 + 5 * 16) / 7.0, 5 * 16 / 7.0]))) <= 1e-12
    everyone = np.ones((3, 3), bool)
    out = O.attention(q, k, v, everyone)
    # row 1 now also sees k2: score 0 -> weights (3, 1, 1) over 5
    assert np.max(np.abs(out[1] - np.array([(3 * 8 + 16) / 5.0, (8 + 16) / 5.0]))) <= 1e-12
    # the scale follows the head dimension: the same vectors zero-padded to D = 16 use 1/4
    pad = lambda a: np.concatenate([a, np.zeros((3, 12))], axis=1)
    out16 = O.attention(pad(q) * 2.0, pad(k), v, O.causal_mask(3))
    assert np.max(np.abs(out16 - want)) <= 1e-12
    # grouped-query form: two query heads share one key/value head; head 0 is the case above, head 1 has
    # q = 0, i.e. uniform weights over the allowed columns
    v4 = np.concatenate([v, np.zeros((3, 2))], axis=1)
    g = O.gqa_attention(np.concatenate([q, np.zeros((3, 4))], axis=1), k, v4, O.causal_mask(3), 2, 1)
    assert np.max(np.abs(g[:, 0:2] - want)) <= 1e-12 and not g[:, 2:4].any() and not g[:, 6:8].any()
    uniform = np.array([[8.0, 0.0], [4.0, 4.0], [8.0, 8.0]])
    assert np.max(np.abs(g[:, 4:6] - uniform)) <= 1e-12


@pytest.mark.parametrize("pattern", ["tvt", "vt", "tv", "tvtvtvt", "t", "v"])
def test_aifs_attention_is_invariant(pattern):
    # Sec. 3.1: with the unified mask and the original position ids, attention on the
    # reordered sequence equals attention on the original one (here: 1e-5 in float64).
    rng = np.random.default_rng(len(pattern))
    is_vis = np.concatenate([np.full(rng.integers(1, 6), 1 if ch == "v" else 0) for ch in pattern]).astype(np.uint8)
    ref, out_u, perm = _attn_case(rng, is_vis)
    assert np.max(np.abs(out_u - ref[perm])) <= 1e-5
    assert np.max(np.abs(O.aifs_scatter(out_u, perm) - ref)) <= 1e-5


def test_aifs_attention_with_left_pads():
    # App. A.4: left pads travel with the visual block and nobody attends to them
    rng = np.random.default_rng(42)
    is_pad = np.array([1, 1, 1, 0, 0, 0, 0, 0, 0, 0], np.uint8)
    is_vis = np.array([0, 0, 0, 0, 0, 1, 1, 1, 0, 0], np.uint8)
    ref, out_u, perm = _attn_case(rng, is_vis, is_pad)
    assert perm.tolist() == [0, 1, 2, 5, 6, 7, 3, 4, 8, 9]
    real = ~is_pad.astype(bool)[perm]
    assert np.max(np.abs(out_u[real] - ref[perm][real])) <= 1e-5
    m = O.unified_mask(perm, is_pad)
    assert not m[real][:, ~real].any()


def test_wrong_positions_break_the_invariance():
    # planting the mistake "positions follow the new order" must be visible
    rng = np.random.default_rng(1)
    is_vis = np.array([0, 0, 1, 1, 1, 0, 0], np.uint8)
    L, D = 7, 8
    q, k, v = (rng.standard_normal((L, D)) for _ in range(3))
    pos = np.arange(L)
    ref = O.attention(O.rope(q, pos), O.rope(k, pos), v, O.causal_mask(L))
    perm = O.aifs_perm(is_vis)
    bad = O.attention(O.rope(q[perm], pos), O.rope(k[perm], pos), v[perm], O.unified_mask(perm))
    assert np.max(np.abs(bad - ref[perm])) > 1e-3
    bad2 = O.attention(O.rope(q[perm], pos[perm]), O.rope(k[perm], pos[perm]), v[perm], O.causal_mask(L))
    assert np.max(np.abs(bad2 - ref[perm])) > 1e-3


def test_rope_is_a_rotation_depending_on_relative_position():
    rng = np.random.default_rng(2)
    x = rng.standard_normal((3, 8))
    assert np.allclose(O.rope(x, [0, 0, 0]), x)
    assert np.allclose(np.linalg.norm(O.rope(x, [5, 9, 2]), axis=1), np.linalg.norm(x, axis=1))
    a, b = rng.standard_normal((1, 8)), rng.standard_normal((1, 8))
    d1 = O.rope(a, [7]) @ O.rope(b, [3]).T
    d2 = O.rope(a, [14]) @ O.rope(b, [10]).T
    assert np.allclose(d1, d2)
    # first pair rotates by pos * theta_0 = pos (theta_0 = base^0 = 1)
    e = np.zeros((1, 8)); e[0, 0] = 1.0
    assert np.allclose(O.rope(e, [0.5])[0, :2], [np.cos(0.5), np.sin(0.5)])


def test_rms_split_cost_fixture():
    # Sec. 4.3: one input row split off a K-row GEMM costs 1/K of it
    for K, N, denom in _read_ints("rms_cost.txt"):
        assert (2 * 1 * N) * denom == 2 * K * N


def test_rms_detect_is_the_first_row_criterion():
    # Eq. 9 on hand-made rows (n = 4): sqrt(4) * mean > max  <=>  2 * mean > max
    w = np.array([[1.0, 1.0, 1.0, 1.0,   3.0, -1.0, -1.0, -1.0],     # block 0: 2*1 > 1 yes; block 1: 2*0 > 3 no
                  [0.5, 0.6, 0.7, 0.4,  -1.0, -1.0, -1.0, -1.0]])    # block 0: 1.1 > 0.7 yes; block 1: -2 > -1 no
    assert O.rms_detect(w, 4).tolist() == [[True, False], [True, False]]
    # the criterion compares the first row of the rotated weight with the original maximum (Sec. 3.2)
    rng = np.random.default_rng(3)
    w = rng.standard_normal((6, 64)) + rng.standard_normal((6, 1)) * 0.5
    first_row = O.rotate_dense(w, 32)[:, ::32]
    assert np.array_equal(O.rms_detect(w, 32), first_row > w.reshape(6, 2, 32).max(axis=2))


def test_rms_split_is_exact_without_quantization_and_costs_one_row_per_block():
    rng = np.random.default_rng(5)
    n, K, N, T = 32, 128, 10, 7
    w_rot = O.rotate_dense(rng.standard_normal((N, K)) + 0.8, n)
    x_rot = rng.standard_normal((T, K))
    w_main, w_side = O.rms_split(w_rot, n)
    assert np.all(w_main[:, ::n] == 0) and np.array_equal(w_side, w_rot[:, ::n])
    # step 3: the GEMV term added back restores the unsplit product exactly (up to float64 rounding)
    assert np.allclose(x_rot @ w_main.T + x_rot[:, ::n] @ w_side.T, x_rot @ w_rot.T, rtol=0, atol=1e-12)
    # the split takes the large first-row entries out of the main matrix ...
    assert np.abs(w_main).max() < np.abs(w_rot).max()
    # ... at a cost of one input row per rotation block: 1/n of the GEMM (1/K when one block spans K)
    assert w_side.size * n == w_rot.size
    assert O.rms_split(w_rot, K)[1].shape == (N, 1)


def test_rms_linear_reduces_to_the_plain_linear_when_the_split_rows_are_zero():
    rng = np.random.default_rng(9)
    T, K, N, n = 9, 64, 6, 32
    x = O.bf16_rne(rng.standard_normal((T, K)).astype(np.float32))
    w = rng.standard_normal((N, K)).astype(np.float32) * 0.02
    w[:, ::n] = 0                                            # nothing to split off
    seg_end, seg_mod = np.array([5, 9]), np.array([1, 0])
    qw, s_w = O.quantize_weight_int4(w)
    plain = O.linear_w4a8_msq(x, seg_end, seg_mod, 0.05, 0.03, n, qw, s_w)
    rms = O.linear_w4a8_msq_rms(x, seg_end, seg_mod, 0.05, 0.03, n, qw, s_w, np.zeros((N, K // n), np.int8),
                                np.ones(N, np.float32))
    assert np.array_equal(rms["acc_main"], plain["acc"]) and not rms["acc_side"].any()
    assert np.array_equal(rms["y32"], plain["y32"])
    # and with a real split the quantized result stays within the quantization error bound of the exact product
    w2 = (rng.standard_normal((N, K)) * 0.02 + 0.05).astype(np.float32)
    w2_rot = O.rotate_dense(w2, n).astype(np.float32)
    w_main, w_side = O.rms_split(w2_rot, n)
    qm, sm = O.quantize_weight_int4(w_main)
    qs, ss = O.quantize_weight_int4(w_side)
    out = O.linear_w4a8_msq_rms(x, seg_end, seg_mod, 0.05, 0.03, n, qm, sm, qs, ss)
    exact = O.rotate_dense(x, n) @ w2_rot.astype(np.float64).T
    plain2 = O.linear_w4a8_msq(x, seg_end, seg_mod, 0.05, 0.03, n, *O.quantize_weight_int4(w2_rot))
    assert np.abs(out["y64"] - exact).mean() < np.abs(plain2["y64"] - exact).mean()   # the point of RMS


def test_dynamic_quantizer_uses_row_absmax():
    r = np.array([[1.0, -2.0], [0.5, 0.25]], np.float32)
    q, s = O.quantize_act_int8_dynamic(r)
    assert s.tolist() == [np.float32(2 / 127), np.float32(0.5 / 127)]
    assert q.tolist() == [[64, -127], [127, 64]]


def test_dynamic_linear_is_scale_invariant_per_row_and_matches_msq_on_equal_scales():
    rng = np.random.default_rng(21)
    T, K, N, n = 6, 64, 5, 32
    x = O.bf16_rne(rng.standard_normal((T, K)).astype(np.float32))
    qw, s_w = O.quantize_weight_int4(rng.standard_normal((N, K)).astype(np.float32) * 0.02)
    d = O.linear_w4a8_dynamic(x, n, qw, s_w)
    # every row uses the whole code range: its largest code is +-127
    assert (np.abs(d["qx"].astype(np.int32)).max(axis=1) == 127).all()
    # scaling a row by a power of two changes its scale, not its codes, and scales its output exactly
    x2 = x.copy()
    x2[1] *= 4.0
    x2[3] *= 0.125
    d2 = O.linear_w4a8_dynamic(x2, n, qw, s_w)
    assert np.array_equal(d2["qx"], d["qx"]) and np.array_equal(d2["acc"], d["acc"])
    assert d2["s_rows"][1] == d["s_rows"][1] * 4 and d2["s_rows"][3] == d["s_rows"][3] * 0.125
    assert np.array_equal(d2["y32"][1], d["y32"][1] * 4) and np.array_equal(d2["y32"][0], d["y32"][0])
    # with a static scale equal to a row's own dynamic scale, MSQ gives that row the same result
    for t in (0, 4):
        m = O.linear_w4a8_msq(x[t:t + 1], np.array([1]), np.array([0]), 1.0, d["s_rows"][t], n, qw, s_w)
        assert np.array_equal(m["qx"][0], d["qx"][t]) and np.array_equal(m["y32"][0], d["y32"][t])
    # the error bound of Eq. 2 per row: |q s - r| <= s / 2
    assert (np.abs(d["qx"] * d["s_rows"][:, None].astype(np.float64) - d["rotated"]) <=
            d["s_rows"][:, None] * 0.5 * (1 + 1e-6)).all()
    # an all-zero row stays defined
    z = O.linear_w4a8_dynamic(np.zeros((1, K), np.float32), n, qw, s_w)
    assert z["s_rows"][0] == 1.0 and not z["qx"].any() and not z["y32"].any()


def test_block_glue_against_hand_values():
    # RMSNorm: unit gain gives unit mean square; a constant row maps to +-1 (up to eps)
    x = np.array([[3.0, -3.0, 3.0, -3.0], [1.0, 2.0, 3.0, 4.0]])
    y = O.rmsnorm(x, np.ones(4), eps=0.0)
    assert np.allclose(y[0], [1, -1, 1, -1]) and np.allclose((y * y).mean(axis=1), 1.0)
    assert np.allclose(O.rmsnorm(x, [2, 2, 2, 2], eps=0.0), 2 * y)
    assert np.allclose(y[1], x[1] / np.sqrt(7.5))
    # SwiGLU: silu(0) = 0, silu(x) -> x for large x, silu(-x) = x sigmoid(-x)
    assert O.swiglu([0.0], [5.0])[0] == 0.0
    assert np.isclose(O.swiglu([30.0], [2.0])[0], 60.0)
    assert np.isclose(O.swiglu([1.0], [1.0])[0], 1.0 / (1.0 + np.exp(-1.0)))
    # grouped-query attention: with one kv head per query head it is per-head attention;
    # with a shared kv head, two query heads given the same q produce the same output
    rng = np.random.default_rng(4)
    L, D = 5, 4
    q, k, v = rng.standard_normal((L, 2 * D)), rng.standard_normal((L, 2 * D)), rng.standard_normal((L, 2 * D))
    allowed = O.causal_mask(L)
    full = O.gqa_attention(q, k, v, allowed, 2, 2)
    assert np.allclose(full[:, D:], O.attention(q[:, D:], k[:, D:], v[:, D:], allowed))
    q2 = np.concatenate([q[:, :D], q[:, :D]], axis=1)
    shared = O.gqa_attention(q2, k[:, :D], v[:, :D], allowed, 2, 1)
    assert np.allclose(shared[:, :D], shared[:, D:]) and np.allclose(shared[:, :D], full[:, :D])
    # first row attends only to itself
    assert np.allclose(full[0, :D], v[0, :D])


# ----------------------------------------------------------------------------- reading of x / s (Eq. 2)
def a4_report():
    """Per config: how many activation codes differ between the reading used everywhere
    (multiply by the float32 reciprocal of the static scale) and Eq. 2 taken literally (x / s).
    The rotated down-projection input of each config (config 1: its only linear): configs 1, 2 and 5
    at full size; configs 3 and 4 with their recipe, K and calibration draw but 256 rows
    (visual : text in the configs' own 12 : 1 and 18 : 1 proportions)."""
    from paper_2502_00425_b200 import synth
    c3 = synth.heavy_tail_linear("c3.down_proj.rows256", 206, 236, 20, 18944, 16, 128)
    c4_mod = np.tile(np.concatenate([np.full(121, 1), np.full(7, 0)]), 2).astype(np.uint8)
    c4 = synth.heavy_tail_linear("c4.down_proj.rows256", 306, 0, 0, 14336, 16, 128, row_mod=c4_mod)
    cases = [("config1", synth.config1()), ("config2", synth.config2()), ("config3.down_proj", c3),
             ("config4.down_proj", c4), ("config5.down_proj.T128", synth.config5_linear("down_proj", 128))]
    out = []
    for name, c in cases:
        s_v, s_t = O.calibrate_static_scales(c.x_calib, c.seg_calib.seg_end, c.seg_calib.seg_mod, c.rot_block)
        r = O.fwht_blocks(c.x, c.rot_block, np.float32)
        s_rows = O.row_scales(c.T, c.seg.seg_end, c.seg.seg_mod, s_v, s_t)
        a = O.quantize_act_int8(r, s_rows).astype(np.int16)
        b = O.quantize_act_int8_divide(r, s_rows).astype(np.int16)
        out.append({"config": name, "rows": int(c.T), "codes": int(a.size), "differ": int((a != b).sum()),
                    "max_abs_code_diff": int(np.abs(a - b).max())})
    return out


def test_reciprocal_and_literal_division_report():
    # informational (the two readings are both self-consistent); what is asserted is only that they
    # can differ by at most one code step, at a rounding tie, and on a vanishing share of the codes
    report = a4_report()
    for row in report:
        print("A4 %(config)s: %(differ)d of %(codes)d codes differ (rows checked: %(rows)d)" % row)
        assert row["max_abs_code_diff"] <= 1
        assert row["differ"] <= 1e-4 * row["codes"]


# ----------------------------------------------------------------------------- other bit widths, weight groups
def test_weight_quantizer_general_reduces_to_the_int4_per_channel_one():
    rng = np.random.default_rng(21)
    w = (rng.standard_normal((24, 256)) * 0.03).astype(np.float32)
    w[5] = 0.0
    q4, s4 = O.quantize_weight_int4(w)
    q, s = O.quantize_weight_sym(w, 4, 0)
    assert np.array_equal(q, q4) and np.array_equal(s, s4)
    # one group spanning all of K is the per-channel quantizer
    qg, sg = O.quantize_weight_sym(w, 4, 256)
    assert np.array_equal(qg, q4) and np.array_equal(sg[:, 0], s4) and sg.shape == (24, 1)


def test_grouped_weight_quantizer_hand_rows():
    # two groups of four with very different ranges: Eq. 2 per group, b = 4 (qmax 7)
    w = np.array([[7.0, -3.5, 1.0, 0.0, 0.07, -0.035, 0.01, 0.0],
                  [0.0, 0.0, 0.0, 0.0, -14.0, 14.0, 2.0, 1.0]], np.float32)
    q, s = O.quantize_weight_sym(w, 4, 4)
    assert np.array_equal(s, np.array([[1.0, np.float32(0.07) / np.float32(7)], [1.0, 2.0]], np.float32))
    #  -3.5 / 1 -> tie -> -4 (even);  -0.035 / 0.01 = -3.5 up to rounding of the scale: checked by value below
    assert q[0, :4].tolist() == [7, -4, 1, 0]
    assert q[1].tolist() == [0, 0, 0, 0, -7, 7, 1, 0]            # 1 / 2 = 0.5 -> tie -> 0 (even)
    assert q[0, 4] == 7 and q[0, 6] == 1 and q[0, 7] == 0 and q[0, 5] in (-3, -4)
    # with one scale per channel the small group collapses to zero codes: the case group scales exist for
    qc, sc = O.quantize_weight_sym(w, 4, 0)
    assert qc[0, 4:].tolist() == [0, 0, 0, 0] and sc[0] == 1.0
    # error bound per group: |q s - w| <= s / 2 wherever the code is not clamped
    rng = np.random.default_rng(22)
    w = (rng.standard_normal((16, 512)) * np.repeat(rng.uniform(0.01, 2.0, (16, 4)), 128, axis=1)).astype(np.float32)
    q, s = O.quantize_weight_sym(w, 4, 128)
    err = np.abs(q.astype(np.float64) * np.repeat(s, 128, axis=1) - w)
    assert np.all(err <= np.repeat(s, 128, axis=1) / 2 * (1 + 1e-6))
    assert np.abs(q).max() <= 7 and (np.abs(q).reshape(16, 4, 128).max(axis=2) == 7).all()


def test_w8_and_a4_quantizers_hand_cases():
    w = np.array([[127.0, -63.5, 0.5, -128.0]], np.float32)   # max 128 -> s = 128 / 127
    q, s = O.quantize_weight_sym(w, 8, 0)
    assert s[0] == np.float32(128.0) / np.float32(127.0)
    assert q[0].tolist() == [126, -63, 0, -127]                 # 127 / s = 126.0078, -63.5 / s = -63.004, 0.5 / s = 0.496
    # 4-bit activations: clamp to [-8, 7], ties to even, same reciprocal multiply as the 8-bit path
    r = np.array([[0.0, 0.5, 1.0, 1.5, 2.5, 7.0, 7.6, 100.0, -8.4, -9.0, -100.0, np.nan, np.inf, -np.inf]], np.float32)
    q = O.quantize_act_sym(r, [1.0], 4)
    assert q[0].tolist() == [0, 0, 1, 2, 2, 7, 7, 7, -8, -8, -8, 0, 7, -8]
    rng = np.random.default_rng(23)
    r = (rng.standard_normal((7, 96)) * 30).astype(np.float32)
    s_rows = rng.uniform(0.1, 3.0, 7).astype(np.float32)
    assert np.array_equal(O.quantize_act_sym(r, s_rows, 8), O.quantize_act_int8(r, s_rows))
    # Eq. 2's scale with b = 4: max / 7; the arg-max element then takes code +-7
    x = np.array([[0.5, -3.5, 1.0], [2.0, 0.25, -0.9]], np.float32)
    s_v, s_t = O.calibrate_static_scales_bits(x, [1, 2], [1, 0], 0, 4)
    assert s_v == np.float32(3.5) / np.float32(7) and s_t == np.float32(2.0) / np.float32(7)
    assert O.quantize_act_sym(x, [s_v, s_t], 4).tolist() == [[1, -7, 2], [7, 1, -3]]    # 0.25 / (2/7) = 0.875 -> 1; -0.9 -> -3.15 -> -3
    assert O.calibrate_static_scales_bits(x, [1, 2], [1, 0], 0, 8) == O.calibrate_static_scales(x, [1, 2], [1, 0], 0)


def test_grouped_linear_against_plain_definitions():
    rng = np.random.default_rng(24)
    T, K, N, g = 9, 512, 20, 128
    x = np.asarray(rng.standard_t(3.0, (T, K)), np.float32)
    w = (rng.standard_normal((N, K)) * np.repeat(rng.uniform(0.005, 0.2, (N, K // g)), g, axis=1)).astype(np.float32)
    seg_end, seg_mod = [5, T], [1, 0]
    s_v, s_t = O.calibrate_static_scales(x, seg_end, seg_mod, 128)
    qw, s_wg = O.quantize_weight_sym(w, 4, g)
    bias = rng.standard_normal(N).astype(np.float32)
    ref = O.linear_wa_sym(x, seg_end, seg_mod, s_v, s_t, 128, qw, s_wg, 8, g, bias)
    # the per-group partial sums add up to the ungrouped integer product, and match nested Python loops
    assert np.array_equal(ref["acc_g"].sum(axis=2), O.int_gemm(ref["qx"], qw))
    assert np.array_equal(ref["acc_g"][:2, :3, 1], O.int_gemm_loops(ref["qx"][:2, g:2 * g], qw[:3, g:2 * g]))
    # the plain definition: dequantized activations times dequantized weights, in float64
    x_hat = ref["qx"].astype(np.float64) * ref["s_rows"].astype(np.float64)[:, None]
    w_hat = qw.astype(np.float64) * np.repeat(s_wg.astype(np.float64), g, axis=1)
    want = x_hat @ w_hat.T + bias.astype(np.float64)[None, :]
    assert np.max(np.abs(ref["y64"] - want)) <= 1e-10 * np.abs(want).max()
    assert np.max(np.abs(ref["y32"] - want) / (np.abs(x_hat) @ np.abs(w_hat).T + np.abs(bias))) <= 1e-5
    # one group: bit for bit the per-channel linear
    q1, s1 = O.quantize_weight_sym(w, 4, K)
    a = O.linear_wa_sym(x, seg_end, seg_mod, s_v, s_t, 128, q1, s1, 8, K, bias)
    b = O.linear_w4a8_msq(x, seg_end, seg_mod, s_v, s_t, 128, *O.quantize_weight_int4(w), bias)
    assert np.array_equal(a["y32"], b["y32"]) and np.array_equal(a["y_bf16"], b["y_bf16"])
    assert np.array_equal(a["acc_g"][:, :, 0], b["acc"])
    # on a weight whose groups differ in range, group scales reconstruct the exact product better
    exact = O.fwht_blocks(x, 128, np.float64) @ w.astype(np.float64).T + bias
    err_g = np.abs(ref["y64"] - exact).mean()
    err_c = np.abs(O.linear_w4a8_msq(x, seg_end, seg_mod, s_v, s_t, 128, *O.quantize_weight_int4(w), bias)["y64"] - exact).mean()
    assert err_g < err_c


def test_w8a8_and_w4a4_linears_order_their_errors():
    # Sec. 4.1 main table: W8A8 is closest to the exact product, W4A8 next, W4A4 last
    rng = np.random.default_rng(25)
    T, K, N = 12, 256, 16
    x = rng.standard_normal((T, K)).astype(np.float32)
    w = (rng.standard_normal((N, K)) * 0.05).astype(np.float32)
    seg_end, seg_mod = [T], [0]
    exact = x.astype(np.float64) @ w.astype(np.float64).T
    errs = {}
    for name, wb, ab in (("w8a8", 8, 8), ("w4a8", 4, 8), ("w4a4", 4, 4)):
        s_v, s_t = O.calibrate_static_scales_bits(x, seg_end, seg_mod, 0, ab)
        qw, s_w = O.quantize_weight_sym(w, wb, 0)
        out = O.linear_wa_sym(x, seg_end, seg_mod, s_v, s_t, 0, qw, s_w, ab, 0)
        assert np.abs(out["qx"]).max() <= 2 ** (ab - 1) and np.abs(qw).max() <= 2 ** (wb - 1)
        errs[name] = np.abs(out["y64"] - exact).mean()
    assert errs["w8a8"] < errs["w4a8"] < errs["w4a4"]
    # W4A8 through the general path is the hot path itself
    s_v, s_t = O.calibrate_static_scales(x, seg_end, seg_mod, 0)
    a = O.linear_wa_sym(x, seg_end, seg_mod, s_v, s_t, 0, *O.quantize_weight_int4(w))
    b = O.linear_w4a8_msq(x, seg_end, seg_mod, s_v, s_t, 0, *O.quantize_weight_int4(w))
    assert np.array_equal(a["acc"], b["acc"]) and np.array_equal(a["y_bf16"], b["y_bf16"])


# ----------------------------------------------------------------------------- full-width rotation, K = m * 2^k
@pytest.mark.parametrize("m", [4, 8, 12, 20, 28, 36, 44, 148])
def test_paley_hadamard_gram_is_m_identity_in_integers(m):
    H = O.paley_hadamard(m)
    assert H.shape == (m, m) and set(np.unique(H).tolist()) == {-1, 1}
    assert np.array_equal(H @ H.T, m * np.eye(m, dtype=np.int64))
    assert np.array_equal(H.T @ H, m * np.eye(m, dtype=np.int64))


def test_paley_hadamard_refuses_orders_it_cannot_build():
    for m in (107, 428, 16 * 107):            # K = 13696 = 107 * 128: no order-m matrix from these constructions
        with pytest.raises((ValueError, AssertionError)):
            O.paley_hadamard(m)


def test_gf27_is_a_field():
    from oracle.mq_oracle import _gf27_tables
    mul, sub = _gf27_tables()
    for a in range(1, 27):
        assert sorted(mul(a, b) for b in range(27)) == list(range(27))      # multiplication by a != 0 permutes the field
        assert sub(a, a) == 0 and mul(a, 1) == a
    assert all(mul(a, mul(b, c)) == mul(mul(a, b), c) for a in (2, 5, 11, 26) for b in (3, 7, 13) for c in (4, 9, 20))


def test_kronecker_rotation_against_the_dense_kronecker_product():
    rng = np.random.default_rng(31)
    m, n2, T = 12, 8, 5
    K = m * n2
    Hm = O.paley_hadamard(m)
    full = np.kron(Hm, O.hadamard_matrix(n2)).astype(np.float64)              # (A (x) B)[i n2 + j, a n2 + b] = A[i,a] B[j,b]
    assert np.array_equal(full @ full.T, K * np.eye(K))
    x = rng.standard_normal((T, K))
    want = x @ full / np.sqrt(K)
    got = O.kron_rotate_dense(x, Hm, n2)
    assert np.max(np.abs(got - want)) <= 1e-12
    # orthonormal: norms are kept and the product with an equally rotated weight is unchanged
    assert np.allclose(np.linalg.norm(got, axis=1), np.linalg.norm(x, axis=1))
    w = rng.standard_normal((7, K))
    assert np.max(np.abs(got @ O.kron_rotate_dense(w, Hm, n2).T - x @ w.T)) <= 1e-10
    # a transposed H_m or swapped factors would fail the dense comparison (H_12 here is not symmetric)
    assert not np.array_equal(Hm, Hm.T)
    # float32 twin: same values within float32 accuracy, exact on small integers
    x32 = rng.standard_normal((T, K)).astype(np.float32)
    y32 = O.kron_rotate_f32(x32, Hm, n2)
    assert np.max(np.abs(y32 - O.kron_rotate_dense(x32, Hm, n2))) <= 1e-5 * np.abs(x32).max() * np.sqrt(K)
    xi = rng.integers(-8, 9, (T, K)).astype(np.float32)
    c = np.float32(1.0 / np.sqrt(np.float64(K)))
    assert np.array_equal(O.kron_rotate_f32(xi, Hm, n2), ((xi.astype(np.float64) @ full).astype(np.float32) * c))
    # m = 1 is the plain block transform
    assert np.array_equal(O.kron_rotate_f32(x32[:, :8], np.array([[1]]), 8),
                          (O.fwht_blocks(x32[:, :8], 8, np.float32, normalise=False) * np.float32(1.0 / np.sqrt(8.0))).astype(np.float32))
