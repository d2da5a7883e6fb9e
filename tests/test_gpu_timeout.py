"""The failure path of the bounded waits.  Every wait on a hardware barrier in the tensor-core
kernels polls a limited number of times; when the limit is reached the kernel raises the
library's timeout flag, drains and returns, and the host reads DSA3D_ERR_DEVICE_TIMEOUT.
Here that path runs for real, without provoking a fault: the test-aid entry point launches
one warp whose wait is on a barrier nothing arrives at, with a limit of a few thousand
polls, so the wait runs out by itself and the kernel returns normally."""
import pytest
import torch

from paper_2607_22696_b200 import binding, inputs

pytestmark = pytest.mark.gpu


def test_a_wait_that_runs_out_is_reported_then_cleared_and_the_library_still_works():
    binding.load()
    binding.dsa3d_clear_device_timeout()
    assert binding.dsa3d_device_timeout_flag() == 0
    binding.dsa3d_check_device_timeout()                         # no error yet

    binding.dsa3d_test_wait_timeout(4096)
    torch.cuda.synchronize()                                     # the kernel came back by itself
    assert binding.dsa3d_device_timeout_flag() == 99
    with pytest.raises(binding.Dsa3dError) as err:
        binding.dsa3d_check_device_timeout()
    assert err.value.status == 7
    assert b"bounded wait" in binding.load().dsa3d_status_string(7)
    # sticky until cleared
    with pytest.raises(binding.Dsa3dError):
        binding.dsa3d_check_device_timeout()

    binding.dsa3d_clear_device_timeout()
    assert binding.dsa3d_device_timeout_flag() == 0
    binding.dsa3d_check_device_timeout()

    # the context is intact: a tensor-core kernel with bounded waits runs and raises nothing
    T, H, W, heads, d, window = 4, 5, 9, 2, 128, (3, 3, 3)
    shape = (T, H, W, heads, d)
    q, k, v = (inputs.normal(shape, 400, i, 1.0, torch.bfloat16).cuda() for i in range(3))
    out = torch.empty_like(q)
    lse = torch.empty((T, H, W, heads), dtype=torch.float32, device="cuda")
    binding.dsa3d_forward_fixed_window(q, k, v, T, H, W, heads, d, window, out, lse)
    torch.cuda.synchronize()
    assert torch.isfinite(out.float()).all()
    binding.dsa3d_check_device_timeout()


def test_the_probe_rejects_limits_outside_its_range():
    lib = binding.load()
    assert lib.dsa3d_test_wait_timeout(0, None) == 2
    assert lib.dsa3d_test_wait_timeout((1 << 20) + 1, None) == 2
