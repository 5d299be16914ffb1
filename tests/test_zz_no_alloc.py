"""stand_row_stats_static: the row pass for callers that cannot allocate device memory.

Some users of the library run where cudaMalloc is not an option: a serving loop with a fixed
memory budget, a plugin whose host hands it every buffer, a latency-critical region where an
allocation could stall.  For them the library carries its own scratch buffer.  This test calls
that entry point through the C ABI twice in a row (the buffer is shared and keeps the previous
call's contents, so the second call runs on a dirty buffer) and checks both results against
stand_row_stats, which takes caller-allocated scratch.

The test does not depend on the order of the run: it passes alone in a fresh process and after
the other tests (its file is merely collected last).
"""
import numpy as np
import pytest

from paper_2506_04708_b200 import inputs
from tests import harness

pytestmark = pytest.mark.gpu


def _case(rng, rows, V, dtype):
    x = (rng.standard_normal((rows, V)) * 2.5).astype(np.float32)
    x[np.arange(rows), rng.integers(0, V, rows)] += 8.0
    return inputs.f32_to_bf16_bits(x) if dtype == "bf16" else x


def _same(a, b, tol):
    lse_a, ids_a, val_a, p_a = (t.cpu().numpy() for t in a)
    lse_b, ids_b, val_b, p_b = (t.cpu().numpy() for t in b)
    assert np.array_equal(ids_a, ids_b)          # indices: bit-exact
    assert np.array_equal(val_a, val_b)          # input values: bit-exact
    assert np.allclose(lse_a, lse_b, rtol=1e-5, atol=1e-5)
    assert np.allclose(p_a, p_b, rtol=tol, atol=1e-30)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_static_scratch_matches_caller_scratch_twice_in_a_row(dtype):
    from paper_2506_04708_b200 import binding
    rng = np.random.default_rng(11)
    tol = harness.value_tol(inputs.DTYPE_BF16 if dtype == "bf16" else inputs.DTYPE_F32)
    # two different shapes back to back: the second call finds the first one's leftovers in the buffer
    for rows, V, k, T in [(24, 151936, 10, 0.7), (7, 5000, 8, 1.0)]:
        dl = harness.to_device_logits(_case(rng, rows, V, dtype))
        want = binding.row_stats(dl, T, k)
        got = binding.row_stats_static(dl, T, k)
        _same(got, want, tol)
        again = binding.row_stats_static(dl, T, k)
        _same(again, want, tol)


def test_static_calls_leave_device_memory_as_it_is():
    """With the outputs made beforehand and the buffer's address resolved by a first call, further calls must
    not change the amount of device memory in use: nothing is allocated or freed, by the library or below it."""
    import torch
    from paper_2506_04708_b200 import binding
    rng = np.random.default_rng(12)
    rows, V, k = 16, 40000, 10
    dl = harness.to_device_logits(_case(rng, rows, V, "bf16"))
    out = (torch.empty(rows, dtype=torch.float32, device="cuda:0"), torch.empty((rows, k), dtype=torch.int32, device="cuda:0"),
           torch.empty((rows, k), dtype=torch.float32, device="cuda:0"), torch.empty((rows, k), dtype=torch.float32, device="cuda:0"))
    want = binding.row_stats(dl, 0.9, k)
    binding.row_stats_static(dl, 0.9, k, out=out)  # the first call on this device resolves the buffer's address
    torch.cuda.synchronize()
    free_before, total = torch.cuda.mem_get_info()
    for _ in range(5):
        binding.row_stats_static(dl, 0.9, k, out=out)
    torch.cuda.synchronize()
    free_after, _ = torch.cuda.mem_get_info()
    assert free_after == free_before
    _same(out, want, 4e-3)


def test_static_scratch_refuses_what_does_not_fit():
    import torch
    from paper_2506_04708_b200 import binding
    rows, V, k = 8192, 151936, 10
    assert binding.lib().stand_row_stats_scratch_bytes(rows, V, binding.DTYPE_BF16, k) > binding.STATIC_SCRATCH_BYTES
    # the refusal comes before any launch, so the logits are never read: a small tensor stands in
    dl = torch.zeros((rows, 8), dtype=torch.bfloat16, device="cuda:0")
    out = tuple(torch.zeros(1, device="cuda:0") for _ in range(4))
    rc = binding.lib().stand_row_stats_static(dl.data_ptr(), rows, V, binding.DTYPE_BF16, 1.0, k,
                                              *(t.data_ptr() for t in out), None)
    assert rc == -5
    assert b"built-in scratch" in binding.lib().stand_strerror(rc)
    # an invalid call is reported as such whatever its size: the argument checks come first
    rc = binding.lib().stand_row_stats_static(dl.data_ptr(), rows, V, binding.DTYPE_BF16, 0.0, k,
                                              *(t.data_ptr() for t in out), None)
    assert rc == -1
    rc = binding.lib().stand_row_stats_static(dl.data_ptr(), rows, V, binding.DTYPE_BF16, 1.0, k, None,
                                              *(t.data_ptr() for t in out[1:]), None)
    assert rc == -1
