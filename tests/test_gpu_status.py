"""Failure reporting without a GPU fault: a bounded wait that nothing satisfies runs out, the kernel
exits normally, the host reads the status, and the context keeps working."""
import pytest
import torch

from paper_1810_00952_b200 import binding as B

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def test_expired_wait_is_reported_and_cleared():
    torch.zeros(1, device=DEV)
    B.relay_poll_status()                       # clean before
    B.relay_debug_expire_wait(2000)             # 2 ms limit on a barrier nobody signals
    with pytest.raises(B.RelayError) as e:
        B.relay_poll_status()
    assert e.value.status_name == "ERR_TIMEOUT"
    B.relay_poll_status()                       # the word was cleared by the poll
    # the context is still usable: a normal call runs and checks out
    x = torch.randn(64, 64, device=DEV); w = torch.randn(64, 64, device=DEV); y = torch.empty(64, 64, device=DEV)
    B.relay_fused_dense_act(x, w, None, B.ACT_NONE, y)
    B.relay_poll_status()
    assert torch.allclose(y, x @ w, rtol=1e-4, atol=1e-3)


def test_expire_wait_rejects_bad_limits_without_launching():
    n0 = B.relay_launch_count()
    for bad in (0, -5, 2_000_000):
        with pytest.raises(B.RelayError) as e:
            B.relay_debug_expire_wait(bad)
        assert e.value.status_name == "ERR_ATTR"
    assert B.relay_launch_count() == n0
