"""mq_w4a8_msq_linear_noalloc: the linear for callers that cannot bring a workspace.

Some users of the library are handed nothing but their input and output tensors -- a plugin
inside another runtime's decode loop, or a process whose device memory already belongs to
another pool -- and may not call cudaMalloc or a framework allocator.  For them the scratch
is a fixed 4 MiB array inside the library.  These tests call that entry point through the C
ABI and require exactly what the workspace-taking entry point produces (the other GPU tests
compare that one with the CPU oracle bit for bit, so equality is the tolerance), on two
calls in a row that share the array.  The file sorts last so that a run stopping at the
first failure has already been through every other test.
"""
import ctypes as C

import numpy as np
import pytest

from paper_2502_00425_b200 import binding as B
from paper_2502_00425_b200 import build


def test_noalloc_rejects_oversized_problems_on_the_host():
    """Needs no GPU: the size check comes before any CUDA call."""
    build.build_library()
    lib = B.load()
    assert B.mq_workspace_bytes(1088, 18944, 3584, 128) > B.MQ_NOALLOC_WS_BYTES
    d = B.mq_linear_desc(1088, 18944, 3584, 128, 0, 0)
    rc = lib.mq_w4a8_msq_linear_noalloc(C.byref(d), None, 18944, None, 1.0, 1.0, None, None, None, None, 3584,
                                        None, None, None)
    assert rc == B.MQ_ERR_WORKSPACE
    assert B.status_string(rc) == "MQ_ERR_WORKSPACE"
    # the limits the header documents for the decode shapes of a 4096 / 13696 MLP
    assert B.mq_workspace_bytes(256, 4096, 13696, 0) <= B.MQ_NOALLOC_WS_BYTES
    assert B.mq_workspace_bytes(48, 13696, 4096, 128) <= B.MQ_NOALLOC_WS_BYTES
    assert B.mq_workspace_bytes(64, 13696, 4096, 128) == 5071104 > B.MQ_NOALLOC_WS_BYTES
    d = B.mq_linear_desc(64, 13696, 4096, 128, 0, 0)
    assert lib.mq_w4a8_msq_linear_noalloc(C.byref(d), None, 13696, None, 1.0, 1.0, None, None, None, None, 4096,
                                          None, None, None) == B.MQ_ERR_WORKSPACE
    bad = B.mq_linear_desc(8, 100, 128, 0, 0, 0)     # K % 32 != 0: same verdict as the main entry point
    rc = lib.mq_w4a8_msq_linear_noalloc(C.byref(bad), None, 100, None, 1.0, 1.0, None, None, None, None, 128,
                                        None, None, None)
    assert rc == B.MQ_ERR_INVALID_ARG


@pytest.mark.gpu
def test_noalloc_matches_workspace_entry_point_twice_in_a_row():
    import torch
    from paper_2502_00425_b200 import synth
    from gpu_util import DEV, bf16_to_dev, dev_segments, gpu_calibrate, gpu_linear, gpu_pack

    # two different small problems -- the first large enough to take the split-K path of the
    # GEMM, the second GEMV-shaped -- so that each call finds the other's codes and partial sums
    # in the shared array
    cases = [synth.small_linear(41, 3, 45, 4096, 512, 128, calib_vis=8, calib_txt=24),
             synth.small_linear(42, 0, 8, 2048, 256, 0, calib_vis=8, calib_txt=8)]
    bias = [np.random.default_rng(5).standard_normal(512).astype(np.float32), None]
    prepared = []
    for c, b in zip(cases, bias):
        assert 256 < B.mq_workspace_bytes(c.T, c.K, c.N, c.rot_block) <= B.MQ_NOALLOC_WS_BYTES
        s_v, s_t = gpu_calibrate(c.x_calib, c.seg_calib, c.rot_block)
        packed, s_w, layout = gpu_pack(c.w)
        y_ref, acc_ref, st = gpu_linear(c, s_v, s_t, layout, s_w, b, torch.bfloat16)
        assert st == (B.MQ_OK, 0)
        prepared.append((c, b, s_v, s_t, s_w, layout, y_ref, acc_ref))

    for rep in range(2):                      # A, B, A, B: every call follows a different one
        for c, b, s_v, s_t, s_w, layout, y_ref, acc_ref in prepared:
            y = torch.full((c.T, c.N), float("nan"), dtype=torch.bfloat16, device=DEV)
            acc = torch.full((c.T, c.N), -(2 ** 31), dtype=torch.int32, device=DEV)
            status = torch.full((2,), 77, dtype=torch.int32, device=DEV)
            b_d = None if b is None else torch.from_numpy(b).to(DEV)
            B.mq_w4a8_msq_linear_noalloc(bf16_to_dev(c.x), dev_segments(c.seg), s_v, s_t, layout, s_w, y, c.N,
                                         rot_block=c.rot_block, bias=b_d, acc_out=acc, status_out=status)
            torch.cuda.synchronize()
            assert status.tolist() == [B.MQ_OK, 0]
            assert torch.equal(acc, acc_ref)
            assert torch.equal(y.view(torch.int16), y_ref.view(torch.int16))

    # a problem too large for the array is refused, and nothing is written
    big = synth.small_linear(43, 0, 4, 128, 128, 0, calib_vis=4, calib_txt=4)
    y = torch.zeros((40000, 128), dtype=torch.bfloat16, device=DEV)
    x = torch.zeros((40000, 128), dtype=torch.bfloat16, device=DEV)
    packed, s_w, layout = gpu_pack(big.w)
    with pytest.raises(B.MqError) as err:
        B.mq_w4a8_msq_linear_noalloc(x, dev_segments(big.seg), 1.0, 1.0, layout, s_w, y, 128)
    assert err.value.status == B.MQ_ERR_WORKSPACE
