"""The bounded wait of the attention pipeline, exercised without faulting or hanging the GPU:
a wait that nothing completes gives up after its limit, the CTA reports ADAPSHOT_ETIMEOUT and the
kernel returns; a second waiter leaves as soon as it sees the CTA's abort flag; the context
stays usable afterwards."""
import math

import pytest
import torch

from tests import helpers as hp

pytestmark = pytest.mark.gpu


def test_wait_gives_up_reports_timeout_and_context_survives():
    ab = hp.gpu_binding()
    st = hp.new_status()
    cycles = torch.zeros(2, dtype=torch.int64, device="cuda")
    ab.adapshot_selftest_wait_timeout(st, cycles)
    torch.cuda.synchronize()
    assert st.item() == ab.ETIMEOUT
    c = cycles.tolist()
    assert 2_000_000 < c[0] < 50_000_000           # gave up at its limit (about a millisecond), not later
    assert 0 < c[1] < 50_000_000                   # the other waiter followed the abort flag
    # the context still works: run a real call afterwards
    logits = torch.zeros(2, 4096, device="cuda")
    H, _, st2 = hp.run_entropy(ab, logits, 0.5, 1)
    assert st2 == 0 and abs(H[0].item() - math.log(4096)) < 1e-3
