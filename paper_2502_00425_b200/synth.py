"""Seeded synthetic inputs shaped like the paper's MLLM prefill / decode workloads.

This module holds NO arithmetic of the method (no rotation, no quantizer, no
GEMM): it only draws random tensors with the shapes, value distributions and
modality structure the paper describes (Sec. 1 Fig. 1(b): visual activations
span roughly -20..10 while text stays near 0; Sec. 4: 256 calibration samples;
Sec. 4.3: down-projection 18944x3584 of a Qwen2-7B-shaped block; interleaved
text-image-text-image-text-image-text prompts).  Both the CPU oracle's tests and
the CUDA path's tests/bench draw their inputs from here, so that the two sides
see bit-identical data without sharing any code of the method itself.

Activations are returned as float32 arrays whose values are exactly
representable in bfloat16 (rounded here, to nearest even), together with the
raw 16-bit patterns, because the boundary takes bf16 activations.
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np

TEXT, VISUAL = 0, 1


# --------------------------------------------------------------------------- bf16 helpers
def to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """float32 -> bfloat16 bit patterns (uint16), round-to-nearest-even."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    u = x.view(np.uint32).astype(np.uint64)
    nan = np.isnan(x)
    r = (u + 0x7FFF + ((u >> 16) & 1)) >> 16
    r = r.astype(np.uint16)
    if nan.any():
        r[nan] = 0x7FC0
    return r


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    """bfloat16 bit patterns (uint16) -> float32 (exact)."""
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << 16).view(np.float32)


def round_to_bf16(x: np.ndarray) -> np.ndarray:
    return bf16_bits_to_f32(to_bf16_bits(x))


# --------------------------------------------------------------------------- containers
@dataclass
class Segments:
    """Row -> modality table: `seg_end` are exclusive cumulative row ends."""
    seg_end: np.ndarray  # int32 [n_seg]
    seg_mod: np.ndarray  # uint8 [n_seg], 0 = text, 1 = visual

    @property
    def n_seg(self) -> int:
        return int(self.seg_end.shape[0])

    def row_modality(self, T: int) -> np.ndarray:
        out = np.zeros(T, dtype=np.uint8)
        start = 0
        for e, m in zip(self.seg_end.tolist(), self.seg_mod.tolist()):
            out[start:min(e, T)] = m
            start = e
        return out


def segments_from_row_modality(row_mod: np.ndarray) -> Segments:
    row_mod = np.asarray(row_mod, dtype=np.uint8)
    T = row_mod.shape[0]
    if T == 0:
        return Segments(np.zeros(0, np.int32), np.zeros(0, np.uint8))
    change = np.flatnonzero(np.diff(row_mod.astype(np.int16)) != 0) + 1
    ends = np.concatenate([change, [T]]).astype(np.int32)
    starts = np.concatenate([[0], change]).astype(np.int64)
    return Segments(ends, row_mod[starts].astype(np.uint8))


@dataclass
class LinearCase:
    """One W4A8 MSQ linear call: activations, weights, calibration draw."""
    name: str
    T: int
    K: int
    N: int
    rot_block: int
    x: np.ndarray            # float32 [T,K], bf16-representable
    w: np.ndarray            # float32 [N,K]
    seg: Segments
    x_calib: np.ndarray      # float32 [Tc,K], bf16-representable
    seg_calib: Segments
    bias: np.ndarray | None = None
    meta: dict = field(default_factory=dict)

    @property
    def x_bits(self) -> np.ndarray:
        return to_bf16_bits(self.x)


# --------------------------------------------------------------------------- distributions
def _student_t_rows(rng, rows, K, row_mod, vis_gain=2.0):
    x = rng.standard_t(3.0, size=(rows, K)).astype(np.float32)
    x[row_mod == VISUAL] *= np.float32(vis_gain)
    return x


def _plant_massive_rows(rng, x, row_mod, n_channels=8, magnitude=500.0, per_modality=1):
    """Massive-activation tokens: a few rows with |x| ~ magnitude on a few channels."""
    rows_used = []
    K = x.shape[1]
    for mod in (VISUAL, TEXT):
        cand = np.flatnonzero(row_mod == mod)
        if cand.size == 0:
            continue
        pick = rng.choice(cand, size=min(per_modality, cand.size), replace=False)
        for r in pick.tolist():
            ch = rng.choice(K, size=min(n_channels, K), replace=False)
            sign = rng.choice(np.array([-1.0, 1.0], dtype=np.float32), size=ch.size)
            x[r, ch] = (magnitude * (1.0 + 0.05 * rng.standard_normal(ch.size))).astype(np.float32) * sign
            rows_used.append(r)
    return rows_used


def _outlier_weights(rng, N, K, sigma=0.015, frac=0.001, gain=20.0):
    w = (rng.standard_normal((N, K)) * sigma).astype(np.float32)
    n_out = int(round(frac * N * K))
    if n_out:
        idx = rng.choice(N * K, size=n_out, replace=False)
        w.reshape(-1)[idx] *= np.float32(gain)
    return w


def heavy_tail_linear(name, seed, T_vis, T_txt, K, N, rot_block, calib_vis=224, calib_txt=32,
                      massive=True, calib_massive=True, vis_gain=2.0, order="vis_first",
                      row_mod=None):
    """Config-2-style linear: Student-t(3) activations (visual rows x2), massive
    tokens, outlier weights, separate calibration draw of the same recipe."""
    rng = np.random.default_rng(seed)
    if row_mod is None:
        if order == "vis_first":
            row_mod = np.concatenate([np.full(T_vis, VISUAL), np.full(T_txt, TEXT)]).astype(np.uint8)
        else:
            row_mod = np.concatenate([np.full(T_txt, TEXT), np.full(T_vis, VISUAL)]).astype(np.uint8)
    row_mod = np.asarray(row_mod, dtype=np.uint8)
    T = row_mod.shape[0]
    x = _student_t_rows(rng, T, K, row_mod, vis_gain)
    massive_rows = _plant_massive_rows(rng, x, row_mod) if massive else []
    w = _outlier_weights(rng, N, K)
    cal_mod = np.concatenate([np.full(calib_vis, VISUAL), np.full(calib_txt, TEXT)]).astype(np.uint8)
    xc = _student_t_rows(rng, cal_mod.shape[0], K, cal_mod, vis_gain)
    if calib_massive:
        _plant_massive_rows(rng, xc, cal_mod)
    return LinearCase(name=name, T=T, K=K, N=N, rot_block=rot_block,
                      x=round_to_bf16(x), w=w, seg=segments_from_row_modality(row_mod),
                      x_calib=round_to_bf16(xc), seg_calib=segments_from_row_modality(cal_mod),
                      meta={"seed": seed, "massive_rows": massive_rows})


# --------------------------------------------------------------------------- the five configs
def config1(seed: int = 0) -> LinearCase:
    """T=64 (48 visual then 16 text), K=N=256, rotation off; scales from the same rows."""
    rng = np.random.default_rng(seed)
    T, K, N = 64, 256, 256
    row_mod = np.concatenate([np.full(48, VISUAL), np.full(16, TEXT)]).astype(np.uint8)
    x = rng.standard_normal((T, K)).astype(np.float32)
    x[:48] *= np.float32(4.0)
    x[:, [3, 77, 130, 201]] *= np.float32(50.0)
    w = (rng.standard_normal((N, K)) * 0.02).astype(np.float32)
    xb = round_to_bf16(x)
    seg = segments_from_row_modality(row_mod)
    return LinearCase("c1", T, K, N, 0, xb, w, seg, xb.copy(), seg, meta={"seed": seed})


def config2(seed: int = 1, T_vis=1024, T_txt=64, K=18944, N=3584, rot_block=128,
            clipping_variant=False) -> LinearCase:
    """Qwen2-7B-shaped down-projection with online rotation.  The clipping
    variant leaves the massive tokens out of the calibration draw so that the
    saturating branch of the quantizer is exercised."""
    return heavy_tail_linear("c2" + ("_clip" if clipping_variant else ""), seed, T_vis, T_txt, K, N,
                             rot_block, calib_massive=not clipping_variant)


@dataclass
class LayerShape:
    hidden: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    mlp: int

    def linears(self):
        """(name, K, N, rot_block) for the 7 linears of one decoder block."""
        q = self.n_q_heads * self.head_dim
        kv = self.n_kv_heads * self.head_dim
        return [("q_proj", self.hidden, q, 0), ("k_proj", self.hidden, kv, 0),
                ("v_proj", self.hidden, kv, 0), ("o_proj", q, self.hidden, 0),
                ("gate_proj", self.hidden, self.mlp, 0), ("up_proj", self.hidden, self.mlp, 0),
                ("down_proj", self.mlp, self.hidden, 128)]


QWEN2_7B = LayerShape(hidden=3584, n_q_heads=28, n_kv_heads=4, head_dim=128, mlp=18944)
LLAMA_8B = LayerShape(hidden=4096, n_q_heads=32, n_kv_heads=8, head_dim=128, mlp=14336)
GLM_9B_MLP = (4096, 13696)


def interleaved_modality(spans) -> np.ndarray:
    """spans = [(modality, length), ...] in original token order -> is_visual[L]."""
    return np.concatenate([np.full(n, m, dtype=np.uint8) for m, n in spans]) if spans else np.zeros(0, np.uint8)


def config3_sequence() -> np.ndarray:
    """3 images x 1024 visual tokens interleaved with 3 text spans of 96 tokens."""
    return interleaved_modality([(VISUAL, 1024), (TEXT, 96)] * 3)


def config4_sequence() -> np.ndarray:
    """[32 text][4 tiles x 576 visual][96 text] = 2432 tokens per sequence."""
    return interleaved_modality([(TEXT, 32), (VISUAL, 4 * 576), (TEXT, 96)])


def config3_linear(which: str, seed: int = 2, scale_down: int = 1) -> LinearCase:
    """Linear-suite mode of config 3: the named linear of the Qwen2-7B-shaped
    block at T=3360 in AIFS order (3072 visual then 288 text)."""
    for i, (name, K, N, rot) in enumerate(QWEN2_7B.linears()):
        if name == which:
            return heavy_tail_linear(f"c3.{name}", seed * 100 + i, 3072 // scale_down, 288 // scale_down,
                                     K // scale_down if scale_down > 1 else K,
                                     N // scale_down if scale_down > 1 else N, rot)
    raise KeyError(which)


def config4_linear(which: str, seed: int = 3, batch: int = 4) -> LinearCase:
    """Linear-suite mode of config 4: batch of 4 sequences, each [2304 visual][128 text]
    after per-sequence AIFS, rows flattened -> 8 segments."""
    row_mod = np.tile(np.concatenate([np.full(2304, VISUAL), np.full(128, TEXT)]), batch).astype(np.uint8)
    for i, (name, K, N, rot) in enumerate(LLAMA_8B.linears()):
        if name == which:
            return heavy_tail_linear(f"c4.{name}", seed * 100 + i, 0, 0, K, N, rot, row_mod=row_mod)
    raise KeyError(which)


def config5_linear(which: str, T: int, seed: int = 4) -> LinearCase:
    """Decode-shaped MLP of a 9B-shaped model: gate/up 4096->13696, down 13696->4096
    (rotation 128 on the down-projection input); T text tokens, text scale only."""
    hidden, mlp = GLM_9B_MLP
    shapes = {"gate_proj": (hidden, mlp, 0, 0), "up_proj": (hidden, mlp, 0, 1),
              "down_proj": (mlp, hidden, 128, 2)}
    K, N, rot, i = shapes[which]
    return heavy_tail_linear(f"c5.{which}.T{T}", seed * 100 + i, 0, T, K, N, rot,
                             calib_vis=0, calib_txt=256, massive=False, calib_massive=False, vis_gain=1.0)


def small_linear(seed, T_vis, T_txt, K, N, rot_block, **kw) -> LinearCase:
    """Scaled-down config-2 recipe for parity tests the oracle finishes in seconds."""
    return heavy_tail_linear(f"small_s{seed}", seed, T_vis, T_txt, K, N, rot_block, **kw)


def embedding_rows(seed: int, L: int, D: int, is_visual: np.ndarray) -> np.ndarray:
    """bf16-representable [L,D] token embeddings with the visual/text magnitude gap."""
    rng = np.random.default_rng(seed)
    x = rng.standard_normal((L, D)).astype(np.float32)
    x[np.asarray(is_visual) == VISUAL] *= np.float32(4.0)
    return round_to_bf16(x)


def mean_shifted_weight(seed: int, N: int, K: int, block: int, shifted_fraction: float = 0.3,
                        sigma: float = 0.02, shift: float = 0.01) -> np.ndarray:
    """float32 [N, K] weight in which a fraction of the (output channel, block) pairs has a
    non-zero mean over the block's input channels -- the structure that an online block
    rotation turns into one large entry per block (the case a down-projection shows)."""
    rng = np.random.default_rng(seed)
    w = (rng.standard_normal((N, K)) * sigma).astype(np.float32)
    nb = K // block
    shifted = rng.random((N, nb)) < shifted_fraction
    sign = np.where(rng.random((N, nb)) < 0.5, -1.0, 1.0)
    offs = (shifted * sign * shift * (0.5 + rng.random((N, nb)))).astype(np.float32)
    return (w.reshape(N, nb, block) + offs[:, :, None]).reshape(N, K).astype(np.float32)
