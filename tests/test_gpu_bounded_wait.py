"""A device wait that runs out: the kernels never spin without bound; a wait that is not
satisfied within its limit reports OMNI_DEV_TIMEOUT and the kernel returns.  The self-test entry
point makes the very helper the product kernels use run out (a barrier nobody arrives on, one
small warp, no copy and no tensor memory in flight) and the test checks the status word, that
the wait ended near its limit, and that the context is as usable afterwards as before."""
import pytest
import torch

from paper_2511_22481_b200 import binding as B
from paper_2511_22481_b200 import workloads as W
from parity import check_workload

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("limit", [20_000, 2_000_000])
def test_a_wait_nobody_satisfies_ends_with_a_timeout_status(limit):
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    waited = torch.zeros(1, dtype=torch.int64, device="cuda")
    B.omni_selftest_bounded_wait(limit, status, waited)
    torch.cuda.synchronize()
    word = int(status.item())
    assert word & B.OMNI_DEV_TIMEOUT and not (word & B.OMNI_DEV_BAD_INDEX)
    cycles = int(waited.item())
    # it gave up after the limit, and soon after it: the clock is read every 64 attempts and one
    # unsuccessful attempt may itself park the thread for a few microseconds
    assert limit <= cycles <= limit + 4_000_000
    # the context is intact: an ordinary decode call right after it matches the oracle
    check_workload(W.config1_tiny("cuda"), what="decode after a timed-out wait")


def test_selftest_argument_checks():
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    for bad in (0, -5, (1 << 31) + 1):
        with pytest.raises(B.OmniError) as info:
            B.omni_selftest_bounded_wait(bad, status)
        assert info.value.code == 2
    with pytest.raises(B.OmniError) as info:
        B.omni_selftest_bounded_wait(1000, None)
    assert info.value.code == 1
