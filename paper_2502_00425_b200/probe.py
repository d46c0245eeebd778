"""Prints the library's tensor-pipe measurements on the current GPU:

    python -m paper_2502_00425_b200.probe [--ctas N]
    python -m paper_2502_00425_b200.probe --attention [--reps R]

1. cycles per tcgen05.mma kind::i8 (128 x N x 32) for several token-tile widths N, accumulator counts and both
   sources of the A operand (mq_ubench_mma_i8), and the int8 operations per clock and SM they amount to;
2. cycles of the weight expander's inner step (mq_ubench_expand).
--attention instead times mq_aifs_attention on the 3360-token, three-image sequence with 28 / 4 heads of 128
(the run that the attention kernel's profile is captured from).
Timing only: it needs a CUDA device and the built library, computes nothing with the results."""
from __future__ import annotations

import argparse

import torch

from . import binding as B


def mma_table(ctas: int, n_mma: int = 4096):
    rows = []
    for a_smem in (0, 1):
        for n_tok in (16, 32, 64, 96, 128, 160, 192, 224, 256):
            for n_acc in (1, 2, 4):
                if n_acc * n_tok > 480:
                    continue
                cyc = torch.zeros(ctas, dtype=torch.int64, device="cuda")
                st = torch.zeros(2, dtype=torch.int32, device="cuda")
                for _ in range(2):
                    B.mq_ubench_mma_i8(n_tok, n_mma, n_acc, a_smem, ctas, cyc, st)
                torch.cuda.synchronize()
                per = float(cyc.cpu().double().mean()) / n_mma
                rows.append({"a_from_smem": a_smem, "n_tok": n_tok, "n_acc": n_acc, "cycles_per_mma": per,
                             "ops_per_clk_sm": 2.0 * 128 * n_tok * 32 / per, "status": st.cpu().tolist()})
    return rows


def expand_table(n_iter: int = 2000):
    rows = []
    for warps in (4, 8):
        for mode in (0, 1, 2):
            cyc = torch.zeros(warps, dtype=torch.int64, device="cuda")
            for _ in range(2):
                B.mq_ubench_expand(n_iter, warps, mode, cyc)
            torch.cuda.synchronize()
            rows.append({"warps": warps, "mode": mode, "cycles_per_round": float(cyc.cpu().double().mean()) / n_iter})
    return rows


def attention_run(reps: int):
    from . import synth
    is_visual = synth.config3_sequence()
    L, D, hq, hkv = int(is_visual.shape[0]), 128, 28, 4
    g = torch.Generator(device="cpu").manual_seed(5)
    q = torch.randn((L, hq * D), generator=g).to(torch.bfloat16).cuda()
    k = torch.randn((L, hkv * D), generator=g).to(torch.bfloat16).cuda()
    v = torch.randn((L, hkv * D), generator=g).to(torch.bfloat16).cuda()
    o = torch.empty_like(q)
    perm = torch.empty(L, dtype=torch.int32, device="cuda")
    dummy = torch.zeros((L, 64), dtype=torch.bfloat16, device="cuda")
    B.mq_aifs_reorder(dummy, torch.empty_like(dummy), torch.from_numpy(is_visual).cuda(), None, perm,
                      torch.empty(L, dtype=torch.int32, device="cuda"), torch.zeros(1, dtype=torch.int32, device="cuda"),
                      direction=0)
    ws = torch.empty(B.mq_aifs_attention_workspace_bytes(L, hkv), dtype=torch.uint8, device="cuda")
    status = torch.zeros(2, dtype=torch.int32, device="cuda")
    run = lambda: B.mq_aifs_attention(q, k, v, perm, None, hq, hkv, o, ws, status)
    run()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(reps):
        run()
    e1.record()
    torch.cuda.synchronize()
    us = e0.elapsed_time(e1) * 1e3 / reps
    flops = 4.0 * D * hq * (L * (L + 1) / 2)
    print("mq_aifs_attention, L = %d, %d / %d heads x %d: %.1f us per call, %.0f TFLOP/s over the allowed pairs, status %s"
          % (L, hq, hkv, D, us, flops / us / 1e6, status.cpu().tolist()))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--ctas", type=int, default=0, help="CTAs of the MMA microbenchmark (default: one per SM)")
    ap.add_argument("--attention", action="store_true", help="time the attention kernel instead")
    ap.add_argument("--reps", type=int, default=5)
    args = ap.parse_args()
    B.load(build_if_missing=True)
    if args.attention:
        attention_run(args.reps)
        return
    ctas = args.ctas or torch.cuda.get_device_properties(0).multi_processor_count
    print("tcgen05.mma kind::i8, 128 x N x 32, %d CTAs" % ctas)
    for r in mma_table(ctas):
        print("  A from %-6s N %3d  accumulators %d : %6.1f cycles per MMA, %6.0f int8 op / clk / SM  %s" % (
            "smem" if r["a_from_smem"] else "tmem", r["n_tok"], r["n_acc"], r["cycles_per_mma"], r["ops_per_clk_sm"],
            "" if r["status"] == [0, 0] else "status %s" % r["status"]))
    print("weight expander step (mode 0: tensor-memory store + wait; 1: loads + expansion + store + wait; "
          "2: as 1, one wait at the end)")
    for r in expand_table():
        print("  %d warps, mode %d : %6.1f cycles per round and warp" % (r["warps"], r["mode"], r["cycles_per_round"]))


if __name__ == "__main__":
    main()
