"""The measurement and self-test entry points: the bounded wait's give-up path (no barrier inside a
real kernel is starved for it) and the tensor-core issue-rate microbenchmark."""
import pytest
import torch

from paper_2502_00425_b200 import binding as B

pytestmark = pytest.mark.gpu
DEV = "cuda"


def test_bounded_wait_gives_up_and_reports():
    status = torch.zeros(2, dtype=torch.int32, device=DEV)
    waited = torch.full((4,), -1, dtype=torch.int64, device=DEV)
    limit_ns = 2_000_000                                     # 2 ms
    B.mq_selftest_bounded_wait(limit_ns, 41, status, waited)
    torch.cuda.synchronize()                                 # the kernel returned: the context is intact
    assert status.tolist() == [B.MQ_ERR_TIMEOUT, 41]
    first_ns, first_ok, second_ns, second_ok = waited.tolist()
    assert first_ok == 0 and second_ok == 0
    assert limit_ns <= first_ns <= 50 * limit_ns             # waited out its limit, then stopped
    assert 0 <= second_ns < limit_ns                         # the abort flag ends other waits at once
    # the first reporter wins: a later expiry does not overwrite status / site
    B.mq_selftest_bounded_wait(limit_ns, 55, status, waited)
    torch.cuda.synchronize()
    assert status.tolist() == [B.MQ_ERR_TIMEOUT, 41]
    # and the device still works
    assert int((torch.arange(10, device=DEV) * 2).sum()) == 90


@pytest.mark.parametrize("n_tok,n_acc,a_from_smem", [(256, 1, 0), (128, 2, 0), (64, 4, 1), (16, 1, 0)])
def test_mma_issue_microbenchmark_runs(n_tok, n_acc, a_from_smem):
    ctas, n_mma = 8, 512
    cycles = torch.zeros(ctas, dtype=torch.int64, device=DEV)
    status = torch.zeros(2, dtype=torch.int32, device=DEV)
    B.mq_ubench_mma_i8(n_tok, n_mma, n_acc, a_from_smem, ctas, cycles, status)
    torch.cuda.synchronize()
    assert status.tolist() == [B.MQ_OK, 0]
    per_mma = cycles.double() / n_mma
    # an MMA of 128 x n_tok x 32 cannot beat 16384 int8 operations per clock and SM, and anything above a
    # few hundred cycles per instruction would mean the measurement is broken
    assert float(per_mma.min()) >= 2 * 128 * n_tok * 32 / 16384 / 1.05
    assert float(per_mma.max()) < 600
