"""The bounded device-side wait runs out and returns (it never hangs), and the context stays usable."""
import pytest
import torch

from paper_2504_00030_b200 import binding as sv

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def test_a_wait_nothing_satisfies_expires_with_the_timeout_bit():
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    result = torch.full((1,), 7, dtype=torch.int32, device=DEV)
    sv.sv_selftest_wait_expiry(status, result, 2_000_000)        # about a millisecond
    torch.cuda.synchronize()
    assert status.item() & sv.SV_DEV_TIMEOUT
    assert result.item() == 0
    # the context is intact: ordinary work still runs and a second expiry behaves the same
    x = torch.arange(1024, device=DEV).sum().item()
    assert x == 1023 * 1024 // 2
    status.zero_()
    sv.sv_selftest_wait_expiry(status, result, 50_000)
    torch.cuda.synchronize()
    assert status.item() == sv.SV_DEV_TIMEOUT and result.item() == 0


def test_budget_outside_the_documented_range_is_refused_on_the_host():
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    result = torch.zeros(1, dtype=torch.int32, device=DEV)
    for bad in (0, -5, 3_000_000_000):
        with pytest.raises(sv.SpecVerifyError) as e:
            sv.sv_selftest_wait_expiry(status, result, bad)
        assert e.value.status == sv.SV_EINVAL
