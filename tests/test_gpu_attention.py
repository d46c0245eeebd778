"""mq_aifs_attention against the oracle's masked attention (Eq. 4 - Eq. 5), head by head."""
import numpy as np
import pytest
import torch

from oracle import mq_oracle as O
from paper_2502_00425_b200 import binding as B

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _layout(spans, rng, pad_left=0):
    """is_visual / is_pad of a sequence made of (modality, length) spans, with optional left pads."""
    vis = [0] * pad_left
    for mod, n in spans:
        vis += [1 if mod == "v" else 0] * n
    is_visual = np.array(vis, dtype=np.uint8)
    is_pad = np.zeros_like(is_visual)
    is_pad[:pad_left] = 1
    return is_visual, is_pad


def _run(q, k, v, perm, pad_u, hq, hkv):
    L = q.shape[0]
    dq, dk, dv = (torch.from_numpy(a).to(torch.bfloat16).to(DEV) for a in (q, k, v))
    o = torch.full((L, q.shape[1]), float("nan"), dtype=torch.bfloat16, device=DEV)
    ws = torch.empty(B.mq_aifs_attention_workspace_bytes(L, hkv), dtype=torch.uint8, device=DEV)
    status = torch.zeros(2, dtype=torch.int32, device=DEV)
    dperm = torch.from_numpy(perm.astype(np.int32)).to(DEV)
    dpad = None if pad_u is None else torch.from_numpy(pad_u.astype(np.uint8)).to(DEV)
    B.mq_aifs_attention(dq, dk, dv, dperm, dpad, hq, hkv, o, ws, status)
    torch.cuda.synchronize()
    assert status.tolist() == [B.MQ_OK, 0]
    back = lambda t: t.float().cpu().numpy().astype(np.float64)
    return back(o), back(dq), back(dk), back(dv)


def _check(o, ref, rows=None, tol=2e-2):
    if rows is not None:
        o, ref = o[rows], ref[rows]
    assert np.isfinite(o).all()
    err = np.abs(o - ref).max(axis=1)
    scale = np.abs(ref).max(axis=1) + 1e-6
    assert float((err / scale).max()) < tol, float((err / scale).max())


@pytest.mark.parametrize("spans,pad_left,hq,hkv", [
    ([("t", 5), ("v", 40), ("t", 19)], 0, 2, 1),                    # one tile, one visual span (Eq. 5's cases)
    ([("t", 30), ("v", 150), ("t", 40), ("v", 130), ("t", 37)], 0, 4, 2),   # several tiles, ragged last tile
    ([("v", 128), ("t", 128)], 0, 2, 2),                            # tile-aligned blocks: full and skipped tiles only
    ([("t", 10), ("v", 200), ("t", 70)], 23, 2, 1),                 # left pads sort with the visual block
    ([("t", 300)], 0, 1, 1),                                        # all text: plain causal attention
    ([("v", 260)], 0, 1, 1),                                        # all visual
    ([("t", 1)], 0, 2, 1),                                          # a single token
    ([("v", 100), ("t", 29)], 0, 1, 1),                             # 129 rows: one row in the second tile
])
def test_attention_matches_oracle(spans, pad_left, hq, hkv):
    rng = np.random.default_rng(11)
    is_visual, is_pad = _layout(spans, rng, pad_left)
    L, D = is_visual.shape[0], 128
    perm = O.aifs_perm(is_visual, is_pad if pad_left else None)
    q = rng.standard_normal((L, hq * D)) * 1.5
    k = rng.standard_normal((L, hkv * D)) * 1.5
    v = rng.standard_normal((L, hkv * D))
    pad_u = is_pad[perm] if pad_left else None
    o, qb, kb, vb = _run(q[perm], k[perm], v[perm], perm, pad_u, hq, hkv)
    allowed = O.unified_mask(perm, is_pad if pad_left else None)
    ref = O.gqa_attention(qb, kb, vb, allowed, hq, hkv)
    keep = np.ones(L, dtype=bool) if pad_u is None else ~pad_u.astype(bool)
    _check(o, ref, rows=keep)
    # and the point of the unified mask: it is causal attention of the original order, row for row
    inv = np.argsort(perm)
    causal = np.tril(np.ones((L, L), dtype=bool))
    if pad_left:
        causal &= ~is_pad.astype(bool)[None, :]
        causal |= np.eye(L, dtype=bool)
    ref_orig = O.gqa_attention(qb[inv], kb[inv], vb[inv], causal, hq, hkv)
    _check(o[inv], ref_orig, rows=~is_pad.astype(bool))


def test_attention_config3_shape_sampled_rows():
    """Qwen2-7B-shaped heads (28 query / 4 key-value heads x 128) on the three-image sequence of 3360 tokens:
    sampled rows of sampled heads against the oracle."""
    rng = np.random.default_rng(12)
    spans = [("v", 1024), ("t", 96)] * 3
    is_visual, _ = _layout(spans, rng)
    L, D, hq, hkv = is_visual.shape[0], 128, 28, 4
    perm = O.aifs_perm(is_visual, None)
    q = rng.standard_normal((L, hq * D)).astype(np.float32)
    k = rng.standard_normal((L, hkv * D)).astype(np.float32)
    v = rng.standard_normal((L, hkv * D)).astype(np.float32)
    o, qb, kb, vb = _run(q[perm], k[perm], v[perm], perm, None, hq, hkv)
    rows = np.unique(np.concatenate([np.arange(0, L, 97), [0, 1, 127, 128, 3071, 3072, 3073, L - 1]]))
    for h in (0, 6, 7, 13, 27):
        g = h // (hq // hkv)
        for i in rows:
            allowed = (perm <= perm[i])[None, :]
            ref = O.attention(qb[i:i + 1, h * D:(h + 1) * D], kb[:, g * D:(g + 1) * D], vb[:, g * D:(g + 1) * D], allowed)
            _check(o[i:i + 1, h * D:(h + 1) * D], ref)


def test_attention_config4_shape_sampled_rows():
    """8B-shaped heads (32 query / 8 key-value heads x 128) on one config-4 sequence, [32 text][2304 visual][96 text]:
    leading text rows sit behind the visual block after AIFS and see only themselves and earlier text."""
    rng = np.random.default_rng(13)
    is_visual, _ = _layout([("t", 32), ("v", 2304), ("t", 96)], rng)
    L, D, hq, hkv = is_visual.shape[0], 128, 32, 8
    perm = O.aifs_perm(is_visual, None)
    q = rng.standard_normal((L, hq * D)).astype(np.float32)
    k = rng.standard_normal((L, hkv * D)).astype(np.float32)
    v = rng.standard_normal((L, hkv * D)).astype(np.float32)
    o, qb, kb, vb = _run(q[perm], k[perm], v[perm], perm, None, hq, hkv)
    rows = np.unique(np.concatenate([np.arange(0, L, 131), [0, 127, 128, 2303, 2304, 2305, 2335, 2336, L - 1]]))
    for h in (0, 3, 4, 31):
        g = h // (hq // hkv)
        for i in rows:
            allowed = (perm <= perm[i])[None, :]
            ref = O.attention(qb[i:i + 1, h * D:(h + 1) * D], kb[:, g * D:(g + 1) * D], vb[:, g * D:(g + 1) * D], allowed)
            _check(o[i:i + 1, h * D:(h + 1) * D], ref)
