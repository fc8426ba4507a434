"""The bounded wait of the ring kernels, driven into its limit on purpose by the library's own
self-test kernel (one warp waiting on a barrier that nothing completes).  The product kernels are
not touched: no copy is withheld and nothing is broken to provoke an expiry there."""
import pytest
import torch

from gpu_utils import DeviceBatch, assert_parity
from paper_2411_00853_b200 import binding
from paper_2411_00853_b200 import workloads as W

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("limit", [200_000, 2_000_000])
def test_an_expired_wait_reports_itself_and_the_kernel_ends(limit):
    err, first, second, reached_end = binding.selftest_bounded_wait(limit)
    assert reached_end == 1                     # the kernel returned normally
    assert err == 77                            # the wait that gave up names itself
    assert limit < first < limit + 20_000_000   # it lasted the limit (a single look at the barrier may doze a little)
    assert second < 20_000                      # a later wait returns at once: the block has failed
    # the context is intact: an ordinary pass right after it is correct
    w = W.make_config(5, B=70, V=8000)
    assert_parity(w, DeviceBatch(w).run())


def test_limits_out_of_range_are_refused():
    out = torch.zeros(4, dtype=torch.int64, device="cuda")
    lib = binding.load()
    assert lib.spec_verify_selftest_bounded_wait(0, out.data_ptr(), None) == 2
    assert lib.spec_verify_selftest_bounded_wait(3_000_000_000, out.data_ptr(), None) == 2
    assert lib.spec_verify_selftest_bounded_wait(1000, None, None) == 1
    torch.cuda.synchronize()
    assert int(out.sum()) == 0
