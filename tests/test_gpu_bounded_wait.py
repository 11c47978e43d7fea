"""A bounded wait that runs out ends in REGIONE_DEV_TIMEOUT and leaves the context usable.

The wait is made to expire in the only harmless way: a self-test kernel of the library calls the
wait routine of the attention kernel on a barrier that nothing arrives on, with a limit of about
a tenth of a millisecond and nothing else in flight.  No attention launch is starved.
"""
import numpy as np
import pytest

from paper_2510_25590_b200 import binding

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("limit", [100_000, 2_000_000])
def test_expired_wait_reports_timeout_and_returns(limit):
    import torch
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    out = torch.full((3,), -1, dtype=torch.int64, device="cuda")
    binding.selftest_bounded_wait(limit, st, out)
    torch.cuda.synchronize()                              # the kernel ended by itself
    assert int(st[0]) == binding.DEV_TIMEOUT
    done, spent, aborted = (int(x) for x in out.cpu())
    assert done == 0 and aborted == 1
    assert limit <= spent <= limit + 1_000_000            # gave up at the limit, not before, not much later
    # the first recorded anomaly is kept; a caller that zeroes the word sees later launches succeed
    st.zero_()
    x = torch.arange(1000, device="cuda").sum()
    assert int(x) == 499500 and int(st[0]) == 0


def test_status_word_keeps_the_first_anomaly():
    import torch
    st = torch.full((1,), binding.DEV_BOUNDS, dtype=torch.int32, device="cuda")
    binding.selftest_bounded_wait(50_000, st)
    torch.cuda.synchronize()
    assert int(st[0]) == binding.DEV_BOUNDS
