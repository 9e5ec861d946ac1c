"""The bounded-wait machinery, exercised without hanging or faulting anything: a one-warp kernel
waits on a barrier that nothing completes, its time budget (1 ms here) runs out, it records
BRO_ERR_TIMEOUT with its site in the device status word and returns normally.  The host then reads
the word once (7, site 10), finds it cleared on the next read, and the library still computes
bit-identical results afterwards."""
import time

import pytest
import torch

from paper_2511_04214_b200 import synth

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def bro():
    from paper_2511_04214_b200 import binding
    return binding


def test_expired_wait_is_reported_once_and_leaves_the_context_usable(bro):
    M, K, N = 200, 512, 264
    x = synth.activations(M, K, seed=5).cuda()
    w = synth.weights(N, K, seed=6).cuda()
    wcodes = bro.alloc_codes(N, K)
    wscales = bro.alloc_scales(N, K, bro.LAYOUT_GEMM)
    bro.pack_weights(w, 32, wcodes, wscales)
    ws = bro.alloc_workspace(bro.linear_workspace_bytes(M, N, K))
    before = torch.empty((M, N), dtype=torch.bfloat16, device="cuda")
    bro.linear(x, 32, wcodes, wscales, N, before, ws)
    assert bro.last_device_status_ex() == (0, 0)

    t0 = time.perf_counter()
    bro.selftest_expire_wait(1_000_000)                 # 1 ms budget
    code, site = bro.last_device_status_ex()            # synchronises the stream
    elapsed = time.perf_counter() - t0
    assert (code, site) == (7, 10), (code, site)
    assert bro.status_string(code) == "BRO_ERR_TIMEOUT"
    assert elapsed < 1.0, f"a 1 ms budget took {elapsed:.3f} s to run out"
    assert bro.last_device_status_ex() == (0, 0)        # read-and-clear

    after = torch.full((M, N), float("nan"), dtype=torch.bfloat16, device="cuda")
    bro.linear(x, 32, wcodes, wscales, N, after, ws)
    assert bro.last_device_status() == 0
    assert torch.equal(before.view(torch.int16), after.view(torch.int16))


def test_budget_is_clamped_and_first_report_wins(bro):
    """Two expiries before a read leave the first one's record; a zero budget is raised to 1 us."""
    bro.selftest_expire_wait(0)
    bro.selftest_expire_wait(2_000_000)
    assert bro.last_device_status_ex() == (7, 10)
    assert bro.last_device_status() == 0
