"""The entry point that allocates nothing (stq_grad_stats_static) against the regular statistics path.

Kept in a file that pytest collects last, so that a run stopping at the first failure has already
been through every other test.  Some callers cannot let a library call cudaMalloc (their framework
owns all free device memory, or they run under a fixed budget); for them the library keeps the
scratch of this one kernel in a static device array.  The test calls it through the C ABI twice in
a row, with a smaller second input, so that stale scratch from the first call would show.
"""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu


def _reference(grad: torch.Tensor) -> np.ndarray:
    """The existing entry points: stq_grad_stats + stq_layer_stats through a handle."""
    from paper_2604_06836_b200 import stq
    h = stq.Handle()
    row = stq.CTensor()
    row.grad = grad.data_ptr()
    row.numel = grad.numel()
    row.block = 128
    tbl = stq.table([row])
    h.grad_stats(tbl, stq.GRAD_BF16 if grad.dtype == torch.bfloat16 else stq.GRAD_F32)
    out = h.layer_stats(1)
    h.close()
    return out


def _close(got: np.ndarray, want: np.ndarray):
    # the tolerance the other statistics tests use: sum g cancels, so it is held to the scale of sum |g|
    assert abs(got[0] - want[0]) <= 2e-6 * max(want[1], 1e-300)
    np.testing.assert_allclose(got[1:3], want[1:3], rtol=2e-6)
    assert got[3] == want[3]


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_two_calls_in_a_row_match_the_regular_path(dtype):
    from paper_2604_06836_b200 import stq
    gen = torch.Generator(device="cuda").manual_seed(5)
    out = torch.zeros(4, dtype=torch.float64, device="cuda")
    for n in (5_000_017, 70_001):          # second call is smaller: leftovers of the first must not leak in
        g = (torch.randn(n, generator=gen, device="cuda") * 3e-3).to(dtype)
        assert stq.grad_stats_static(g, out) == 0
        torch.cuda.synchronize()
        _close(out.cpu().numpy(), _reference(g)[0])


def test_calls_leave_device_memory_as_it_was():
    """The point of the entry point: no call allocates.  After a warm-up call (which loads the kernel and
    looks the scratch address up) the free device memory reported by the driver does not move over a
    series of calls of different sizes, and the torch allocator is not involved either."""
    from paper_2604_06836_b200 import stq
    out = torch.zeros(4, dtype=torch.float64, device="cuda")
    grads = [torch.randn(n, device="cuda") for n in (1_000_003, 4096, 9_999_999)]
    grads.append(grads[0].to(torch.bfloat16))
    for g in grads:                                # warm-up: both kernel variants, every size
        assert stq.grad_stats_static(g, out) == 0
    torch.cuda.synchronize()
    free0, _ = torch.cuda.mem_get_info()
    reserved0, alloc0 = torch.cuda.memory_reserved(), torch.cuda.memory_allocated()
    for _ in range(5):
        for g in grads:
            assert stq.grad_stats_static(g, out) == 0
    torch.cuda.synchronize()
    free1, _ = torch.cuda.mem_get_info()
    assert free1 == free0
    assert torch.cuda.memory_reserved() == reserved0 and torch.cuda.memory_allocated() == alloc0


def test_tiny_and_ragged_sizes():
    from paper_2604_06836_b200 import stq
    out = torch.zeros(4, dtype=torch.float64, device="cuda")
    for n in (1, 3, 4095, 4096, 4097, 12_289):
        g = torch.linspace(-1.0, 2.0, n, device="cuda")
        assert stq.grad_stats_static(g, out) == 0
        torch.cuda.synchronize()
        got = out.cpu().numpy()
        g64 = g.double()
        want = np.array([g64.sum().item(), g64.abs().sum().item(), (g64 * g64).sum().item(), n])
        _close(got, want)


def test_rejects_what_it_cannot_hold():
    from paper_2604_06836_b200 import stq
    lib = stq.lib()
    out = torch.full((4,), -1.0, dtype=torch.float64, device="cuda")
    g = torch.zeros(1024, device="cuda")
    too_many = stq.STATIC_STATS_MAX_NUMEL + 1          # only the count is checked: nothing is read or launched
    assert lib.stq_grad_stats_static(0, g.data_ptr(), too_many, stq.GRAD_F32, out.data_ptr(), None) == -12
    assert lib.stq_grad_stats_static(0, g.data_ptr() + 4, 8, stq.GRAD_F32, out.data_ptr(), None) == -4    # misaligned
    assert lib.stq_grad_stats_static(0, None, 8, stq.GRAD_F32, out.data_ptr(), None) == -1
    assert lib.stq_grad_stats_static(0, g.data_ptr(), 0, stq.GRAD_F32, out.data_ptr(), None) == -6
    assert lib.stq_grad_stats_static(0, g.data_ptr(), 8, 7, out.data_ptr(), None) == -9
    torch.cuda.synchronize()
    assert (out.cpu().numpy() == -1.0).all()            # no rejected call touched the output
    assert b"capacity" in lib.stq_strerror(-12)
