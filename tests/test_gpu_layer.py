"""Layer mode: a whole decoder block over the library's linears, checked step by step against the
oracle with "teacher forcing" -- every step is recomputed on the CPU from the tensor the GPU
actually fed it, so the integer paths stay bit-exact per linear and the float glue (plain torch)
is compared at 2e-2 relative to the row maximum."""
import numpy as np
import pytest
import torch

from oracle import mq_oracle as O
from paper_2502_00425_b200 import binding as B
from paper_2502_00425_b200 import layer as LY
from paper_2502_00425_b200 import synth
from tests.gpu_util import DEV, bf16_from_dev, bf16_to_dev, gpu_pack

pytestmark = pytest.mark.gpu

GLUE_TOL = 2e-2


def _close_rowmax(got, ref, tol=GLUE_TOL):
    ref = np.asarray(ref, dtype=np.float64)
    scale = np.abs(ref).max(axis=-1, keepdims=True)
    scale = np.where(scale > 0, scale, 1.0)
    return (np.abs(np.asarray(got, dtype=np.float64) - ref) / scale).max() <= tol


def _make_block(shape, seed):
    rng = np.random.default_rng(seed)
    weights, ref_w = {}, {}
    for name, K, N, rot in shape.linears():
        w = (rng.standard_normal((N, K)) * (1.0 / np.sqrt(K))).astype(np.float32)
        if rot:
            w = O.rotate_weight_input_dim(w, rot).astype(np.float32)   # offline counterpart of the online rotation
        packed, s_w, layout = gpu_pack(w)
        weights[name] = LY.LinearWeights(layout, s_w, K, N, rot)
        ref_w[name] = O.quantize_weight_int4(w)
    g1 = (1.0 + 0.1 * rng.standard_normal(shape.hidden)).astype(np.float32)
    g2 = (1.0 + 0.1 * rng.standard_normal(shape.hidden)).astype(np.float32)
    blk = LY.W4A8DecoderBlock(shape, weights, torch.from_numpy(g1).to(DEV), torch.from_numpy(g2).to(DEV), DEV)
    return blk, ref_w, g1, g2


def _check_block(shape, is_visual, seed, rows=None):
    L = is_visual.shape[0]
    blk, ref_w, g1, g2 = _make_block(shape, seed)
    emb = synth.embedding_rows(seed + 1, L, shape.hidden, is_visual)
    out, tr = blk.forward(bf16_to_dev(emb), torch.from_numpy(is_visual).to(DEV), calibrate=True)
    assert blk.device_status_ok()
    t = {k: bf16_from_dev(v) for k, v in tr.tensors.items()}
    # AIFS, positions, mask
    perm = O.aifs_perm(is_visual)
    assert np.array_equal(tr.perm.cpu().numpy(), perm)
    assert np.array_equal(tr.pos_u.cpu().numpy(), O.remap_positions(perm))
    allowed = O.unified_mask(perm)
    assert np.array_equal(tr.mask.cpu().numpy(), allowed)
    assert np.array_equal(t["emb_u"], O.aifs_gather(emb, perm))
    seg_end, seg_mod = O.segments_after_aifs(perm, is_visual)
    assert np.array_equal(tr.seg.seg_end.cpu().numpy(), seg_end)
    # every linear from the GPU's own input: scales, then the bf16 output, bit-exact
    sel = np.arange(L) if rows is None else rows
    for name, K, N, rot in shape.linears():
        x_in = t[name + ".in"]
        s_v, s_t = O.calibrate_static_scales(x_in, seg_end, seg_mod, rot)
        lw = blk.w[name]
        assert (np.float32(lw.s_vis), np.float32(lw.s_txt)) == (s_v, s_t), name
        qw, s_w = ref_w[name]
        sub_end = np.searchsorted(sel, seg_end).astype(np.int32)      # segment table of the sampled rows
        ref = O.linear_w4a8_msq(x_in[sel], sub_end, seg_mod, s_v, s_t, rot, qw, s_w)
        assert np.array_equal(t[name + ".out"][sel], ref["y_bf16"]), name
    # glue, each from the GPU's inputs
    assert _close_rowmax(t["attn_norm"], O.rmsnorm(t["emb_u"], g1))
    pos = O.remap_positions(perm)
    D = shape.head_dim
    for nm, src, heads in (("q_rope", "q_proj.out", shape.n_q_heads), ("k_rope", "k_proj.out", shape.n_kv_heads)):
        ref = np.concatenate([O.rope(t[src][:, h * D:(h + 1) * D], pos) for h in range(heads)], axis=1)
        assert _close_rowmax(t[nm], ref), nm
    ref_attn = O.gqa_attention(t["q_rope"], t["k_rope"], t["v_proj.out"], allowed, shape.n_q_heads, shape.n_kv_heads)
    assert _close_rowmax(t["attn"], ref_attn)
    assert _close_rowmax(t["resid1"], t["emb_u"].astype(np.float64) + t["o_proj.out"])
    assert _close_rowmax(t["mlp_norm"], O.rmsnorm(t["resid1"], g2))
    assert _close_rowmax(t["act"], O.swiglu(t["gate_proj.out"], t["up_proj.out"]))
    assert _close_rowmax(t["resid2"], t["resid1"].astype(np.float64) + t["down_proj.out"])
    # back to the original order, exactly
    assert np.array_equal(bf16_from_dev(out), O.aifs_scatter(t["resid2"], perm))
    # a second pass with the stored scales reproduces the first one bit for bit
    out2, _ = blk.forward(bf16_to_dev(emb), torch.from_numpy(is_visual).to(DEV))
    assert torch.equal(out2, out)
    return blk


def test_small_block_interleaved_modalities():
    shape = synth.LayerShape(hidden=256, n_q_heads=4, n_kv_heads=2, head_dim=64, mlp=512)
    is_visual = synth.interleaved_modality([(0, 7), (1, 90), (0, 20), (1, 50), (0, 33)])
    _check_block(shape, is_visual, seed=31)


def test_small_block_text_only_and_visual_only():
    shape = synth.LayerShape(hidden=128, n_q_heads=2, n_kv_heads=1, head_dim=64, mlp=256)
    _check_block(shape, np.zeros(37, np.uint8), seed=32)
    _check_block(shape, np.ones(45, np.uint8), seed=33)


def test_config3_block_full_size_sampled():
    """The Qwen2-7B-shaped block of config 3 at full size (L = 3360); the linears are checked on
    every 64th row and the rows next to the modality boundary, attention on two heads' worth of
    the glue tolerance like everything else."""
    shape = synth.QWEN2_7B
    is_visual = synth.config3_sequence()
    L = is_visual.shape[0]
    n_vis = int(is_visual.sum())
    rows = np.unique(np.concatenate([np.arange(0, L, 64), np.arange(n_vis - 2, n_vis + 2), [L - 1]]))
    _check_block(shape, is_visual, seed=34, rows=rows)


def _check_batched_block(shape, seqs, seed, rows=None):
    """A batch of sequences reordered one by one, their rows stacked for the linears (two segments per
    sequence), attention per sequence.  `rows` (indices into the stacked rows) limits the oracle's
    work on the linears and the attention to a sample; None checks every row."""
    blk, ref_w, g1, g2 = _make_block(shape, seed)
    embs = [synth.embedding_rows(seed + 9 + i, s_.shape[0], shape.hidden, s_) for i, s_ in enumerate(seqs)]
    outs, tr = blk.forward_batch([bf16_to_dev(e) for e in embs], [torch.from_numpy(s_).to(DEV) for s_ in seqs],
                                 calibrate=True)
    assert blk.device_status_ok()
    t = {k: bf16_from_dev(v) for k, v in tr.tensors.items()}
    perms = [O.aifs_perm(s_) for s_ in seqs]
    seg_end, seg_mod, off = [], [], 0
    for s_, p_ in zip(seqs, perms):
        e, m = O.segments_after_aifs(p_, s_)
        seg_end += list(e + off)
        seg_mod += list(m)
        off += s_.shape[0]
    seg_end, seg_mod = np.array(seg_end, np.int32), np.array(seg_mod, np.uint8)
    total = off
    assert np.array_equal(tr.seg.seg_end.cpu().numpy(), seg_end) and np.array_equal(tr.seg.seg_mod.cpu().numpy(), seg_mod)
    assert np.array_equal(t["emb_u"], np.concatenate([O.aifs_gather(e, p_) for e, p_ in zip(embs, perms)]))
    sel = np.arange(total) if rows is None else np.asarray(rows)
    sub_end = np.searchsorted(sel, seg_end).astype(np.int32)
    for name, K, N, rot in shape.linears():
        x_in = t[name + ".in"]
        s_v, s_t = O.calibrate_static_scales(x_in, seg_end, seg_mod, rot)
        assert (np.float32(blk.w[name].s_vis), np.float32(blk.w[name].s_txt)) == (s_v, s_t), name
        qw, s_w = ref_w[name]
        ref = O.linear_w4a8_msq(x_in[sel], sub_end, seg_mod, s_v, s_t, rot, qw, s_w)
        assert np.array_equal(t[name + ".out"][sel], ref["y_bf16"]), name
    bd = tr.bounds
    D = shape.head_dim
    assert _close_rowmax(t["attn_norm"], O.rmsnorm(t["emb_u"], g1))
    for b, (s_, p_) in enumerate(zip(seqs, perms)):
        sl = slice(bd[b], bd[b + 1])
        assert np.array_equal(tr.perms[b].cpu().numpy(), p_)
        pos = O.remap_positions(p_)
        assert np.array_equal(tr.pos_us[b].cpu().numpy(), pos)
        allowed = O.unified_mask(p_)
        assert np.array_equal(tr.masks[b].cpu().numpy(), allowed)
        for nm, src, heads in (("q_rope", "q_proj.out", shape.n_q_heads), ("k_rope", "k_proj.out", shape.n_kv_heads)):
            ref = np.concatenate([O.rope(t[src][sl][:, h * D:(h + 1) * D], pos) for h in range(heads)], axis=1)
            assert _close_rowmax(t[nm][sl], ref), nm
        local = sel[(sel >= bd[b]) & (sel < bd[b + 1])] - bd[b]      # sampled query rows of this sequence
        ref_attn = O.gqa_attention(t["q_rope"][sl][local], t["k_rope"][sl], t["v_proj.out"][sl], allowed[local],
                                   shape.n_q_heads, shape.n_kv_heads)
        assert _close_rowmax(t["attn"][sl][local], ref_attn)
        assert np.array_equal(bf16_from_dev(outs[b]), O.aifs_scatter(t["resid2"][sl], p_))
    assert _close_rowmax(t["resid1"], t["emb_u"].astype(np.float64) + t["o_proj.out"])
    assert _close_rowmax(t["mlp_norm"], O.rmsnorm(t["resid1"], g2))
    assert _close_rowmax(t["act"], O.swiglu(t["gate_proj.out"], t["up_proj.out"]))
    assert _close_rowmax(t["resid2"], t["resid1"].astype(np.float64) + t["down_proj.out"])
    return blk, embs, outs


def test_batched_block_with_eight_segments():
    """Config-4 style batch at a reduced size: four sequences reordered one by one, their rows
    stacked for the linears (eight segments), attention per sequence."""
    shape = synth.LayerShape(hidden=256, n_q_heads=4, n_kv_heads=2, head_dim=64, mlp=512)
    seqs = [synth.interleaved_modality(sp) for sp in ([(0, 5), (1, 60), (0, 12)], [(1, 40), (0, 9)],
                                                      [(0, 3), (1, 30), (0, 4), (1, 20), (0, 6)], [(0, 25)])]
    blk, embs, outs = _check_batched_block(shape, seqs, 41)
    # a sequence run alone with the same scales gives what it gave inside the batch (the glue may pick
    # another attention kernel for another shape, hence a tolerance rather than equality)
    out_single, _ = blk.forward(bf16_to_dev(embs[1]), torch.from_numpy(seqs[1]).to(DEV))
    assert _close_rowmax(bf16_from_dev(out_single), bf16_from_dev(outs[1]))


def test_config4_block_full_size_sampled():
    """The 8B-shaped block of config 4 at full size: four sequences of [32 text][2304 visual][96 text],
    9728 stacked rows with eight segments.  The linears and the attention are checked on the rows next
    to every segment boundary, the first and last rows of the 192-token tiles around them and an even
    spread (every 512th row); the element-wise glue on every row."""
    shape = synth.LLAMA_8B
    seqs = [synth.config4_sequence()] * 4
    L = seqs[0].shape[0]
    rows = set(range(0, 4 * L, 512)) | {4 * L - 1}
    for b in range(4):
        for e in (b * L, b * L + 2304, (b + 1) * L):
            rows |= {r for r in (e - 2, e - 1, e, e + 1) if 0 <= r < 4 * L}
    for t0 in range(0, 4 * L, 192 * 8):
        rows |= {t0, min(4 * L - 1, t0 + 191)}
    _check_batched_block(shape, seqs, 71, rows=np.array(sorted(rows)))


def test_causal_glue_matches_the_unified_mask():
    """Attention invariance (Eq. 5) at the level of the block: running the glue attention in the
    original order with a plain causal mask gives the same block output as the dense unified mask."""
    shape = synth.LayerShape(hidden=256, n_q_heads=4, n_kv_heads=2, head_dim=64, mlp=512)
    is_visual = synth.interleaved_modality([(0, 9), (1, 70), (0, 15), (1, 40), (0, 21)])
    blk, _, _, _ = _make_block(shape, 61)
    emb = bf16_to_dev(synth.embedding_rows(62, is_visual.shape[0], shape.hidden, is_visual))
    vis = torch.from_numpy(is_visual).to(DEV)
    out_mask, tr_mask = blk.forward(emb, vis, calibrate=True)
    blk.causal_glue = True
    out_causal, tr_causal = blk.forward(emb, vis)
    assert _close_rowmax(bf16_from_dev(tr_causal.tensors["attn"]), bf16_from_dev(tr_mask.tensors["attn"]))
    assert _close_rowmax(bf16_from_dev(out_causal), bf16_from_dev(out_mask))


def test_fused_groups_match_separate_linears():
    """q/k/v and gate/up stored as one stacked weight each (one launch per group) give the block the very
    same bits as separate linears on shared codes: every output channel only sees its own weight row."""
    shape = synth.LayerShape(hidden=256, n_q_heads=4, n_kv_heads=2, head_dim=128, mlp=512)
    blk, _, _, _ = _make_block(shape, 81)
    for T_spans in ([(0, 9), (1, 70), (0, 15), (1, 40), (0, 21)], [(0, 3)]):      # a prefill block and a 3-token step
        is_visual = synth.interleaved_modality(T_spans)
        emb = bf16_to_dev(synth.embedding_rows(82, is_visual.shape[0], shape.hidden, is_visual))
        vis = torch.from_numpy(is_visual).to(DEV)
        blk.fuse_groups = False
        out_sep, tr_sep = blk.forward(emb, vis, calibrate=True)
        blk.fuse_groups = True
        out_fused, tr_fused = blk.forward(emb, vis)
        assert blk.fused_group(["q_proj", "k_proj", "v_proj"]) is not None
        assert blk.fused_group(["gate_proj", "up_proj"]) is not None
        for name in ("q_proj", "k_proj", "v_proj", "gate_proj", "up_proj", "down_proj"):
            assert torch.equal(tr_fused.tensors[name + ".out"].contiguous().view(torch.int16),
                               tr_sep.tensors[name + ".out"].contiguous().view(torch.int16)), name
        assert torch.equal(out_fused.view(torch.int16), out_sep.view(torch.int16))
    assert blk.device_status_ok()
