"""The bounded-wait path on the GPU: a wait that nothing satisfies must run out, not hang.

Nothing here breaks a product kernel: a one-warp self-test kernel calls the library's own bounded-wait helper with a
short limit on a barrier nobody arrives at.  The kernel returns, the status word names the wait, the host call maps
it to KSA_ERR_TIMEOUT, and the context keeps working afterwards."""
import pytest
import torch

from oracle import ksa_oracle as orc
from paper_2604_24432_b200 import binding as ksa
from paper_2604_24432_b200 import build as ksa_build
from paper_2604_24432_b200 import synth
from tests import parity

pytestmark = pytest.mark.gpu


def test_wait_runs_out_and_context_stays_usable():
    ksa_build.build()
    ctx = ksa.Context(0)
    dev = torch.device("cuda", 0)
    report = torch.full((5,), -1, dtype=torch.int32, device=dev)
    ctx.clear_device_status()
    assert ctx.device_status_rc() == ksa.KSA_OK
    ctx.selftest_bounded_wait(200_000, report)          # about 0.1 ms
    torch.cuda.synchronize()
    first_ok, second_ok, abort_flag, kc_first, kc_second = report.cpu().tolist()
    assert first_ok == 0 and second_ok == 0 and abort_flag == 1
    assert 190 <= kc_first <= 2000, kc_first             # gave up after the limit, not before and not much later
    assert kc_second <= 2000                             # the second wait only had to see the abort flag
    assert ctx.device_status() == 8                      # kStatusWaitTest: the first wait's code, not the second's
    assert ctx.device_status_rc() == ksa.KSA_ERR_TIMEOUT
    assert "wait" in ksa.strerror(ksa.KSA_ERR_TIMEOUT)
    # the context is still usable: clear and run a forward pass against the oracle
    ctx.clear_device_status()
    wl = synth.Workload("after", 31, [700], 4, 2, 128)
    parity.check_workload(ctx, wl, synth.Layout("after", 8, 1, 4), 0)
    assert ctx.device_status_rc() == ksa.KSA_OK
    ctx.close()
