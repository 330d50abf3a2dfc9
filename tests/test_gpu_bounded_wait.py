"""The bounded device-side wait ends in an error status, not in a stuck launch: a one-warp kernel waits, through the
pipelines' own wait routine, on a barrier that nothing signals, gives up after its cycle limit, ORs its code into the
error word and returns.  Nothing is in flight in that kernel (no copies, no tensor memory, no cluster), and no
production kernel is starved or altered."""
import pytest
import torch

pytestmark = pytest.mark.gpu


def test_expired_wait_sets_the_error_word_and_the_context_stays_usable():
    import paper_2511_20390_b200 as free
    from paper_2511_20390_b200 import binding
    L = binding.lib()
    assert L.free_device_error_code(0) == 0
    for limit in (20_000, 100_000, 2_000_000):
        word, waited, code = free.selftest_bounded_wait(limit)
        assert word != 0 and code == -8                       # FREE_ERR_DEVICE_TIMEOUT
        assert b"timed out" in L.free_strerror(code)
        assert limit < waited < limit + 50_000_000            # gave up past the limit (polls come in groups of 64 suspending waits)
    # the device is still healthy: an ordinary call of the library runs and is correct afterwards
    x = torch.randn(256, 128, device="cuda")
    z = torch.zeros(1, 128, device="cuda")
    y = binding.op_ln_modulate(x, z, z, 256)
    torch.cuda.synchronize()
    assert torch.allclose(y, torch.nn.functional.layer_norm(x, (128,), eps=1e-6), atol=1e-5)


def test_argument_errors():
    from paper_2511_20390_b200 import binding
    L = binding.lib()
    err = torch.zeros(1, dtype=torch.int32, device="cuda")
    assert L.free_selftest_bounded_wait(None, 1000, None, None) == -1
    assert L.free_selftest_bounded_wait(err.data_ptr(), 0, None, None) == -2
    assert L.free_selftest_bounded_wait(err.data_ptr(), 10**9, None, None) == -2       # would spin for about a second
