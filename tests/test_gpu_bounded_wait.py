"""The give-up path of the bounded device-side waits.

Every wait of the GEMM kernels on a shared-memory barrier polls a limited number of times.  The
self-test entry point runs that path on its own: CTAs with the GEMM kernel's roles allocate tensor
memory and wait on barriers nothing arrives at, with a short limit and no copy in flight.  The waits
must run out (none may report success), the status word must read SX_ERR_TIMEOUT, every CTA must
return through the common tear-down, and the device must go on working: a parity case runs right after.
"""
import pytest
import torch

from paper_2509_24248_b200 import binding
from tests import harness, parity

pytestmark = pytest.mark.gpu

SX_ERR_TIMEOUT = -6


@pytest.mark.parametrize("ctas,limit", [(1, 500), (8, 2000), (300, 1000)])
def test_a_wait_that_runs_out_reports_a_timeout_and_returns(ctas, limit):
    lib = binding.load_library()
    dev = torch.device("cuda:0")
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    reached = torch.zeros(2, dtype=torch.int32, device=dev)
    code = lib.sx_selftest_bounded_wait(limit, ctas, status.data_ptr(), reached.data_ptr(),
                                        torch.cuda.current_stream().cuda_stream)
    assert code == 0
    torch.cuda.synchronize()
    assert int(status.item()) == SX_ERR_TIMEOUT
    assert b"wait" in lib.sx_strerror(SX_ERR_TIMEOUT)
    assert reached.cpu().tolist() == [0, ctas]
    # tensor memory was freed and the context is intact: the GEMM kernels run a whole iteration
    rep = parity.run_chain(harness.build_case(harness.tiny_workload(B=2, K=3, len_lo=5, len_hi=40)))
    assert all(0 <= l <= 3 for l in rep.accept_len)


def test_selftest_rejects_unbounded_requests():
    lib = binding.load_library()
    buf = torch.zeros(4, dtype=torch.int32, device="cuda:0")
    p = buf.data_ptr()
    assert lib.sx_selftest_bounded_wait(0, 1, p, p + 8, 0) == -1
    assert lib.sx_selftest_bounded_wait(1 << 21, 1, p, p + 8, 0) == -1
    assert lib.sx_selftest_bounded_wait(100, 0, p, p + 8, 0) == -1
    assert lib.sx_selftest_bounded_wait(100, 5000, p, p + 8, 0) == -1
    torch.cuda.synchronize()
    assert buf.cpu().tolist() == [0, 0, 0, 0]
