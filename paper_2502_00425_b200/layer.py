"""Layer mode: one decoder block whose seven linears are the W4A8 MSQ linear of this library.

The linears, the AIFS reorder and the mask / position remap run through the C ABI (the
product).  Everything between them -- RMSNorm, rotary embedding, masked grouped-query
attention, SwiGLU, the residual adds -- runs as the library's glue kernels (mq_glue_*,
mq_aifs_attention) or, with those switched off, as plain torch on the same device: glue that lets a
sequence flow through a whole block (Sec. 3.1: AIFS once at the input, the unified mask and the
remapped positions in attention, MSQ in front of every linear, the online Hadamard in front of
the down-projection, Fig. 4(a)).

A block takes one sequence, or a batch of sequences, in the original token order and returns
the outputs in that order.  Every sequence is reordered on its own; the linears then see the
rows of all sequences stacked (two segments per sequence in the segment table), attention
runs per sequence.  `forward` keeps every linear's input and output so that a checker can
recompute each step from the tensor the GPU actually fed it.
"""
from dataclasses import dataclass, field
from typing import Dict, List, Optional, Tuple

import torch

from . import binding as B
from .synth import LayerShape


@dataclass
class LinearWeights:
    layout: torch.Tensor          # GEMM weight layout (uint8)
    s_w: torch.Tensor             # float32 [N]
    K: int
    N: int
    rot_block: int = 0
    bias: Optional[torch.Tensor] = None
    s_vis: float = 1.0            # static activation scales of this linear's input (Eq. 3)
    s_txt: float = 1.0


@dataclass
class BlockTrace:
    """What one forward pass saw: tensors in AIFS order unless the name says otherwise."""
    perm: torch.Tensor = None      # of the first (or only) sequence; all of them in `perms`
    pos_u: torch.Tensor = None
    seg: B.Segments = None         # over the stacked rows
    mask: torch.Tensor = None
    perms: List[torch.Tensor] = field(default_factory=list)
    pos_us: List[torch.Tensor] = field(default_factory=list)
    masks: List[torch.Tensor] = field(default_factory=list)
    bounds: List[int] = field(default_factory=list)   # row offsets of the sequences in the stacked tensors
    tensors: Dict[str, torch.Tensor] = field(default_factory=dict)


def rmsnorm(x: torch.Tensor, gain: torch.Tensor, eps: float = 1e-6) -> torch.Tensor:
    xf = x.float()
    return (xf * torch.rsqrt(xf.pow(2).mean(-1, keepdim=True) + eps) * gain.float()).to(torch.bfloat16)


def rope(x: torch.Tensor, pos: torch.Tensor, n_heads: int, base: float = 10000.0) -> torch.Tensor:
    """Rotary embedding on consecutive channel pairs of every head (App. A.2), positions `pos`."""
    L, width = x.shape
    D = width // n_heads
    xf = x.float().view(L, n_heads, D // 2, 2)
    # float32 angles: positions are exact, the product is off by ~1e-4 rad at a few thousand tokens
    theta = (base ** (-2.0 * torch.arange(D // 2, device=x.device, dtype=torch.float64) / D)).float()
    ang = pos.to(torch.float32)[:, None] * theta[None, :]
    c, s = torch.cos(ang)[:, None, :], torch.sin(ang)[:, None, :]
    out = torch.stack((xf[..., 0] * c - xf[..., 1] * s, xf[..., 0] * s + xf[..., 1] * c), dim=-1)
    return out.view(L, width).to(torch.bfloat16)


def gqa_attention_unpermuted(q, k, v, perm, n_q_heads: int, n_kv_heads: int) -> torch.Tensor:
    """The same attention without a dense mask, for sequences without pads: the unified mask is the
    causal mask of the ORIGINAL order (Eq. 5), so the rows are put back in that order, a plain
    causal attention runs (which the library's fused kernels support), and the result returns to
    AIFS order.  Mathematically identical to gqa_attention with the unified mask."""
    L = q.shape[0]
    D = q.shape[1] // n_q_heads
    group = n_q_heads // n_kv_heads
    idx = perm.long()

    def to_orig(x, heads):
        out = torch.empty_like(x)
        out[idx] = x
        return out.view(L, heads, D).transpose(0, 1)

    qh = to_orig(q, n_q_heads)
    kh = to_orig(k, n_kv_heads).repeat_interleave(group, dim=0)
    vh = to_orig(v, n_kv_heads).repeat_interleave(group, dim=0)
    o = torch.nn.functional.scaled_dot_product_attention(qh[None], kh[None], vh[None], is_causal=True)
    return o[0].transpose(0, 1).reshape(L, n_q_heads * D)[idx].contiguous()


def gqa_attention(q, k, v, mask, n_q_heads: int, n_kv_heads: int) -> torch.Tensor:
    L = q.shape[0]
    D = q.shape[1] // n_q_heads
    group = n_q_heads // n_kv_heads
    qh = q.view(L, n_q_heads, D).transpose(0, 1)
    kh = k.view(L, n_kv_heads, D).transpose(0, 1).repeat_interleave(group, dim=0)
    vh = v.view(L, n_kv_heads, D).transpose(0, 1).repeat_interleave(group, dim=0)
    o = torch.nn.functional.scaled_dot_product_attention(qh[None], kh[None], vh[None], attn_mask=mask[None, None])
    return o[0].transpose(0, 1).reshape(L, n_q_heads * D).contiguous()


class W4A8DecoderBlock:
    """One decoder block over the library's linears.  `weights` maps the seven linear names of
    LayerShape.linears() to LinearWeights; `g_attn`, `g_mlp` are the RMSNorm gains."""

    def __init__(self, shape: LayerShape, weights: Dict[str, LinearWeights], g_attn: torch.Tensor,
                 g_mlp: torch.Tensor, device="cuda"):
        self.shape, self.w, self.g_attn, self.g_mlp, self.device = shape, weights, g_attn, g_mlp, device
        self._ws: Dict[Tuple[str, int], torch.Tensor] = {}
        self._fused: Dict[str, Optional[LinearWeights]] = {}
        self._attn_ws: Dict[int, Tuple[torch.Tensor, torch.Tensor]] = {}   # per sequence length: (scratch, status word)
        # True: q/k/v and gate/up each run as one linear over the stacked weight (same results)
        self.fuse_groups = False
        # True: RMSNorm, rotary embedding, SwiGLU and the residual adds run as the library's single-pass
        # kernels (mq_glue_*); False: the plain torch expressions above (float32 temporaries in HBM)
        self.cuda_glue = True
        # True: attention in the original order with a plain causal mask instead of the dense unified
        # mask (same result, much faster glue); the dense mask is still produced and kept in the trace
        self.causal_glue = False
        # True: attention under the unified mask runs as the library's tensor-core kernel (mq_aifs_attention),
        # in AIFS order, straight from the permutation -- no dense mask, no reordering; head_dim must be 128
        self.cuda_attention = shape.head_dim == 128

    # ---- pieces ------------------------------------------------------------------------
    def aifs(self, embs, is_visuals, tr: BlockTrace) -> torch.Tensor:
        """AIFS reorder of every sequence plus its remapped positions and mask; returns the stacked
        rows and leaves the segment table over them in the trace."""
        dev = embs[0].device
        parts, ends, mods, off = [], [], [], 0
        tr.bounds = [0]
        for emb, is_visual in zip(embs, is_visuals):
            L = emb.shape[0]
            emb_u = torch.empty_like(emb)
            perm = torch.empty(L, dtype=torch.int32, device=dev)
            inv = torch.empty(L, dtype=torch.int32, device=dev)
            n_first = torch.zeros(1, dtype=torch.int32, device=dev)
            B.mq_aifs_reorder(emb, emb_u, is_visual, None, perm, inv, n_first, direction=0)
            pos_u = torch.empty(L, dtype=torch.int32, device=dev)
            seg_end = torch.empty(2, dtype=torch.int32, device=dev)
            seg_mod = torch.empty(2, dtype=torch.uint8, device=dev)
            mask = torch.empty((L, L), dtype=torch.uint8, device=dev)
            B.mq_attn_mask_remap(perm, None, None, n_first, pos_u, seg_end, seg_mod, mask)
            parts.append(emb_u)
            ends.append(seg_end + off)
            mods.append(seg_mod)
            tr.perms.append(perm)
            tr.pos_us.append(pos_u)
            tr.masks.append(mask.bool())
            off += L
            tr.bounds.append(off)
        tr.perm, tr.pos_u, tr.mask = tr.perms[0], tr.pos_us[0], tr.masks[0]
        tr.seg = B.Segments(torch.cat(ends), torch.cat(mods))
        return parts[0] if len(parts) == 1 else torch.cat(parts, dim=0)

    def linear(self, name: str, x: torch.Tensor, tr: BlockTrace, calibrate: bool) -> torch.Tensor:
        lw = self.w[name]
        T = x.shape[0]
        if calibrate:
            state = torch.zeros(2, dtype=torch.int32, device=x.device)
            sv = torch.zeros(1, dtype=torch.float32, device=x.device)
            st = torch.zeros(1, dtype=torch.float32, device=x.device)
            B.mq_calibrate_static_scales(x, tr.seg, lw.rot_block, state, sv, st)
            lw.s_vis, lw.s_txt = float(sv.item()), float(st.item())
        key = (name, T)
        if key not in self._ws:
            self._ws[key] = B.new_workspace(T, lw.K, lw.N, lw.rot_block)
        y = torch.empty((T, lw.N), dtype=torch.bfloat16, device=x.device)
        B.mq_w4a8_msq_linear(x, tr.seg, lw.s_vis, lw.s_txt, lw.layout, lw.s_w, y, self._ws[key], lw.N,
                             rot_block=lw.rot_block, bias=lw.bias)
        tr.tensors[name + ".in"], tr.tensors[name + ".out"] = x, y
        return y

    def fused_group(self, names) -> Optional[LinearWeights]:
        """The linears of a group stored as ONE weight [sum N, K] (q/k/v as N = q + 2 kv, gate/up as
        N = 2 mlp): the GEMM layout is contiguous per 128-channel tile, so when every member's N is a
        multiple of 128 the concatenation of the members' layouts IS the layout of the stacked weight.
        One launch then serves the whole group (fewer kernel boundaries, fuller waves).  None when a
        member's N is not tile-aligned or has a bias layout that cannot be stacked."""
        key = "+".join(names)
        if key in self._fused:
            return self._fused[key]
        ws = [self.w[n] for n in names]
        ok = all(w.N % B.MQ_W_TILE_N == 0 and w.rot_block == 0 and w.K == ws[0].K for w in ws) and \
            (all(w.bias is None for w in ws) or all(w.bias is not None for w in ws))
        fused = None
        if ok:
            bias = None if ws[0].bias is None else torch.cat([w.bias for w in ws])
            fused = LinearWeights(torch.cat([w.layout for w in ws]), torch.cat([w.s_w for w in ws]), ws[0].K,
                                  sum(w.N for w in ws), 0, bias)
        self._fused[key] = fused
        return fused

    def linear_group(self, names, x: torch.Tensor, tr: BlockTrace, calibrate: bool):
        """Linears that read the same input (q/k/v, gate/up; no rotation).  With `fuse_groups` they run
        as one linear over the stacked weight (see fused_group) and the outputs are column slices of
        its result; otherwise the input is quantized once with mq_fwht_quant_i8 and every linear of
        the group multiplies the same int8 codes."""
        first = self.w[names[0]]
        assert all(self.w[n].rot_block == 0 and self.w[n].K == first.K for n in names)
        T = x.shape[0]
        fused = self.fused_group(names) if self.fuse_groups else None
        if fused is not None and not calibrate:
            fused.s_vis, fused.s_txt = first.s_vis, first.s_txt
            key = ("+".join(names), T)
            if key not in self._ws:
                self._ws[key] = B.new_workspace(T, fused.K, fused.N, 0)
            y = torch.empty((T, fused.N), dtype=torch.bfloat16, device=x.device)
            B.mq_w4a8_msq_linear(x, tr.seg, fused.s_vis, fused.s_txt, fused.layout, fused.s_w, y, self._ws[key],
                                 fused.N, bias=fused.bias)
            outs, off = [], 0
            for n in names:
                yn = y[:, off:off + self.w[n].N]
                off += self.w[n].N
                tr.tensors[n + ".in"], tr.tensors[n + ".out"] = x, yn
                outs.append(yn)
            return outs
        if calibrate:
            state = torch.zeros(2, dtype=torch.int32, device=x.device)
            sv = torch.zeros(1, dtype=torch.float32, device=x.device)
            st = torch.zeros(1, dtype=torch.float32, device=x.device)
            B.mq_calibrate_static_scales(x, tr.seg, 0, state, sv, st)
            for n in names:
                self.w[n].s_vis, self.w[n].s_txt = float(sv.item()), float(st.item())
        if T <= 3:  # the few-token kernel quantizes inside: nothing to share
            return [self.linear(n, x, tr, False) for n in names]
        codes = torch.empty((T, first.K), dtype=torch.int8, device=x.device)
        B.mq_fwht_quant_i8(x, tr.seg, first.s_vis, first.s_txt, 0, codes, None)
        outs = []
        for n in names:
            lw = self.w[n]
            key = (n + ".i8", T)
            if key not in self._ws:
                self._ws[key] = B.new_workspace(T, lw.K, lw.N, 0, B.MQ_FLAG_X_IS_INT8)
            y = torch.empty((T, lw.N), dtype=torch.bfloat16, device=x.device)
            B.mq_w4a8_msq_linear(codes, tr.seg, lw.s_vis, lw.s_txt, lw.layout, lw.s_w, y, self._ws[key], lw.N,
                                 bias=lw.bias)
            tr.tensors[n + ".in"], tr.tensors[n + ".out"] = x, y
            outs.append(y)
        return outs

    # ---- the block ---------------------------------------------------------------------
    def forward(self, emb: torch.Tensor, is_visual: torch.Tensor, calibrate: bool = False):
        """emb: bf16 [L, hidden] in the original token order; is_visual: uint8 [L].
        calibrate=True first sets every linear's static scales from this very input (single-shot
        calibration, Algorithm 1) and then runs with them.  Returns (output in the original
        order, BlockTrace)."""
        outs, tr = self.forward_batch([emb], [is_visual], calibrate)
        return outs[0], tr

    def forward_batch(self, embs, is_visuals, calibrate: bool = False):
        """Several sequences at once: lists of bf16 [L_b, hidden] and uint8 [L_b]."""
        sh, tr = self.shape, BlockTrace()
        x0 = self.aifs(embs, is_visuals, tr)
        t, bd = tr.tensors, tr.bounds
        n_seq = len(embs)
        t["emb_u"] = x0
        h = self._rmsnorm(x0, self.g_attn)
        t["attn_norm"] = h
        q, k, v = self.linear_group(["q_proj", "k_proj", "v_proj"], h, tr, calibrate)
        qr = self._rope(q, tr, sh.n_q_heads)
        kr = self._rope(k, tr, sh.n_kv_heads)
        t["q_rope"], t["k_rope"] = qr, kr
        if self.cuda_attention:
            a = torch.empty((qr.shape[0], qr.shape[1]), dtype=torch.bfloat16, device=qr.device)
            for b in range(n_seq):
                L_b = bd[b + 1] - bd[b]
                if L_b not in self._attn_ws:
                    self._attn_ws[L_b] = (torch.empty(B.mq_aifs_attention_workspace_bytes(L_b, sh.n_kv_heads), dtype=torch.uint8,
                                                 device=qr.device), torch.zeros(2, dtype=torch.int32, device=qr.device))
                ws, status = self._attn_ws[L_b]
                B.mq_aifs_attention(qr[bd[b]:bd[b + 1]], kr[bd[b]:bd[b + 1]], v[bd[b]:bd[b + 1]], tr.perms[b], None,
                                    sh.n_q_heads, sh.n_kv_heads, a[bd[b]:bd[b + 1]], ws, status)
        elif self.causal_glue:
            a = torch.cat([gqa_attention_unpermuted(qr[bd[b]:bd[b + 1]], kr[bd[b]:bd[b + 1]], v[bd[b]:bd[b + 1]],
                                                    tr.perms[b], sh.n_q_heads, sh.n_kv_heads) for b in range(n_seq)])
        else:
            a = torch.cat([gqa_attention(qr[bd[b]:bd[b + 1]], kr[bd[b]:bd[b + 1]], v[bd[b]:bd[b + 1]], tr.masks[b],
                                         sh.n_q_heads, sh.n_kv_heads) for b in range(n_seq)])
        t["attn"] = a
        o = self.linear("o_proj", a, tr, calibrate)
        x1 = self._add(x0, o)
        t["resid1"] = x1
        h2 = self._rmsnorm(x1, self.g_mlp)
        t["mlp_norm"] = h2
        gate, up = self.linear_group(["gate_proj", "up_proj"], h2, tr, calibrate)
        if self.cuda_glue:
            act = torch.empty((gate.shape[0], gate.shape[1]), dtype=torch.bfloat16, device=gate.device)
            B.mq_glue_swiglu(gate, up, act)
        else:
            act = (torch.nn.functional.silu(gate.float()) * up.float()).to(torch.bfloat16)
        t["act"] = act
        down = self.linear("down_proj", act, tr, calibrate)
        x2 = self._add(x1, down)
        t["resid2"] = x2
        outs = []
        for b in range(n_seq):
            out = torch.empty((bd[b + 1] - bd[b], x2.shape[1]), dtype=torch.bfloat16, device=x2.device)
            B.mq_aifs_reorder(x2[bd[b]:bd[b + 1]], out, None, None, tr.perms[b], None, None, direction=1)
            outs.append(out)
        return outs, tr

    # ---- glue: the library's single-pass kernels, or the torch expressions -------------------------
    def _rmsnorm(self, x, gain):
        if not self.cuda_glue:
            return rmsnorm(x, gain)
        y = torch.empty_like(x)
        B.mq_glue_rmsnorm(x, gain, y)
        return y

    def _rope(self, x, tr: BlockTrace, n_heads: int):
        bd = tr.bounds
        if not self.cuda_glue:
            return torch.cat([rope(x[bd[b]:bd[b + 1]], tr.pos_us[b], n_heads) for b in range(len(bd) - 1)])
        y = torch.empty((x.shape[0], x.shape[1]), dtype=torch.bfloat16, device=x.device)
        for b in range(len(bd) - 1):
            B.mq_glue_rope(x[bd[b]:bd[b + 1]], tr.pos_us[b], n_heads, y[bd[b]:bd[b + 1]])
        return y

    def _add(self, a, b):
        if not self.cuda_glue:
            return (a.float() + b.float()).to(torch.bfloat16)
        y = torch.empty_like(a)
        B.mq_glue_residual_add(a, b, y)
        return y

    def device_status_ok(self) -> bool:
        return (all(B.mq_last_device_status(ws)[0] == B.MQ_OK for ws in self._ws.values())
                and all(int(status[0]) == B.MQ_OK for _, status in self._attn_ws.values()))


def random_block(shape: LayerShape, seed: int, device="cuda") -> W4A8DecoderBlock:
    """A block with random valid weight bytes and scales: for timing only (no float weights exist)."""
    g = torch.Generator(device="cpu").manual_seed(seed)
    w = {}
    for name, K, N, rot in shape.linears():
        lay = torch.randint(0, 256, (B.mq_w4_layout_bytes(N, K),), dtype=torch.uint8, generator=g).to(device)
        s_w = (torch.rand(N, generator=g) * 0.002 + 0.0005).to(device)
        w[name] = LinearWeights(lay, s_w, K, N, rot)
    ones = torch.ones(shape.hidden, device=device)
    return W4A8DecoderBlock(shape, w, ones, ones.clone(), device)
