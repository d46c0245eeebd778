"""The block-glue kernels (RMSNorm, rotary embedding, SwiGLU, residual add) against the oracle's float64
versions: bf16 outputs within one bf16 rounding step of the float64 value (relative 2^-8, plus a small
absolute term for the rotary embedding's float32 angle)."""
import numpy as np
import pytest
import torch

from oracle import mq_oracle as O
from paper_2502_00425_b200 import binding as B
from paper_2502_00425_b200 import synth

from gpu_util import DEV, bf16_from_dev, bf16_to_dev

pytestmark = pytest.mark.gpu
BF16_STEP = 2.0 ** -8


def _close(got, ref, atol=0.0):
    ref = np.asarray(ref, np.float64)
    return np.all(np.abs(got.astype(np.float64) - ref) <= BF16_STEP * np.abs(ref) + atol)


@pytest.mark.parametrize("T,D", [(5, 256), (33, 3584), (7, 4096), (3, 8200)])
def test_rmsnorm(T, D):
    rng = np.random.default_rng(D)
    x = synth.round_to_bf16((rng.standard_normal((T, D)) * 3).astype(np.float32))
    x[0] = 0.0
    gain = (1.0 + 0.1 * rng.standard_normal(D)).astype(np.float32)
    y = torch.full((T, D), float("nan"), dtype=torch.bfloat16, device=DEV)
    B.mq_glue_rmsnorm(bf16_to_dev(x), torch.from_numpy(gain).to(DEV), y)
    assert _close(bf16_from_dev(y), O.rmsnorm(x, gain), atol=1e-30)


def test_rope_with_permuted_positions_and_row_slices():
    rng = np.random.default_rng(3)
    L, H, D = 37, 3, 64
    x = synth.round_to_bf16(rng.standard_normal((L, H * D)).astype(np.float32))
    pos = rng.permutation(4000)[:L].astype(np.int32)          # AIFS hands over the original indices, in any order
    xd = bf16_to_dev(x)
    y = torch.zeros((L, H * D), dtype=torch.bfloat16, device=DEV)
    B.mq_glue_rope(xd[:20], torch.from_numpy(pos[:20]).to(DEV), H, y[:20])
    B.mq_glue_rope(xd[20:], torch.from_numpy(pos[20:]).to(DEV), H, y[20:])
    ref = np.concatenate([O.rope(x[:, h * D:(h + 1) * D], pos) for h in range(H)], axis=1)
    # float32 angles of a few thousand radians are off by ~1e-4 rad: an absolute term on top of the bf16 step
    assert _close(bf16_from_dev(y), ref, atol=2e-3 * np.abs(x).max())
    z = xd.clone()                                            # in place
    B.mq_glue_rope(z, torch.from_numpy(pos).to(DEV), H, z)
    assert torch.equal(z, y)


def test_swiglu_on_column_slices_and_residual_add():
    rng = np.random.default_rng(4)
    T, M = 19, 1024
    both = synth.round_to_bf16((rng.standard_normal((T, 2 * M)) * 4).astype(np.float32))
    both[0, :4] = [0.0, 30.0, -30.0, -100.0]
    bd = bf16_to_dev(both)
    y = torch.empty((T, M), dtype=torch.bfloat16, device=DEV)
    B.mq_glue_swiglu(bd[:, :M], bd[:, M:], y)                 # gate and up as halves of one stacked output
    assert _close(bf16_from_dev(y), O.swiglu(both[:, :M], both[:, M:]), atol=1e-30)
    a, b = both[:, :M], both[:, M:]
    s = torch.empty((T, M), dtype=torch.bfloat16, device=DEV)
    B.mq_glue_residual_add(bf16_to_dev(a), bf16_to_dev(b), s)
    # one rounding to float32 (as the kernel adds), then one to bf16
    assert np.array_equal(bf16_from_dev(s), O.bf16_rne(a.astype(np.float32) + b.astype(np.float32)))
