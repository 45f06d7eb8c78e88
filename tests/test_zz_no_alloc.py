"""adapshot_entropy_static: the entropy entry point for callers that cannot allocate
device memory (its scratch is a fixed array inside the library).  It must give what
adapshot_entropy gives, and what the oracle gives, call after call, although all calls
share that array; and a call must leave the amount of free device memory as it found it."""
import numpy as np
import pytest
import torch

from oracle import adapshot_oracle as orc
from tests import helpers as hp

pytestmark = pytest.mark.gpu
REL_TOL = 1e-4          # the entropy tolerance used throughout the GPU tests


def _static(ab, logits, tau, P):
    R = logits.shape[0]
    H = torch.full((R,), -1.0, dtype=torch.float32, device="cuda")
    fo = torch.full((R // P,), -7, dtype=torch.int32, device="cuda")
    status = hp.new_status()
    ab.adapshot_entropy_static(logits, H, tau, P, fo, status)      # through the C ABI, no workspace
    torch.cuda.synchronize()
    assert status.item() == 0
    return H, fo


def _both(ab, logits, tau, P):
    want_H, want_fo, st = hp.run_entropy(ab, logits, tau, P)
    assert st == 0
    H, fo = _static(ab, logits, tau, P)
    assert torch.all((H - want_H).abs() <= REL_TOL * want_H.abs().clamp_min(1e-3))
    assert torch.equal(fo, want_fo)
    # and against the CPU oracle (Eq. 2 over the whole vocabulary; the threshold rule)
    H_orc = orc.entropy(hp.f64(logits))
    assert np.all(np.abs(H.cpu().numpy() - H_orc) <= REL_TOL * np.maximum(np.abs(H_orc), 1e-3))
    margin = np.abs(H_orc - tau).min()
    if margin > 1e-3:                 # no row sits on the threshold: the rule's result is unique
        assert np.array_equal(fo.cpu().numpy(), orc.first_ok(H_orc, tau, P))


def test_static_entropy_matches_workspace_entropy_on_two_calls_in_a_row():
    ab = hp.gpu_binding()
    g = torch.Generator().manual_seed(77)
    big = (torch.randn(8, 128256, generator=g) * 2.0).to(torch.bfloat16).cuda()
    small = (torch.randn(3, 1000, generator=g) * 4.0).cuda()
    _both(ab, big, 6.0, 4)        # fills much of the shared array
    _both(ab, small, 3.0, 1)      # a smaller call right after: stale states must not leak in
    _both(ab, big, 6.0, 4)


def test_static_entropy_leaves_free_device_memory_unchanged():
    ab = hp.gpu_binding()
    g = torch.Generator().manual_seed(78)
    logits = torch.randn(16, 50000, generator=g).cuda()
    R = logits.shape[0]
    H = torch.empty(R, dtype=torch.float32, device="cuda")
    fo = torch.empty(R // 4, dtype=torch.int32, device="cuda")
    status = hp.new_status()
    ab.adapshot_entropy_static(logits, H, 5.0, 4, fo, status)      # the first call on this device resolves the array
    torch.cuda.synchronize()
    free0, _ = torch.cuda.mem_get_info()
    held0 = torch.cuda.memory_allocated()
    for _ in range(20):
        ab.adapshot_entropy_static(logits, H, 5.0, 4, fo, status)
    torch.cuda.synchronize()
    free1, _ = torch.cuda.mem_get_info()
    assert free1 == free0, "the call changed the amount of free device memory"
    assert torch.cuda.memory_allocated() == held0, "the call went through torch's allocator"
    assert status.item() == 0
    H_orc = orc.entropy(hp.f64(logits))
    assert np.all(np.abs(H.cpu().numpy() - H_orc) <= REL_TOL * np.abs(H_orc))


def test_static_entropy_capacity_boundary():
    ab = hp.gpu_binding()
    # 16384 rows of 8 logits: one state per row, exactly the size of the array
    g = torch.Generator().manual_seed(79)
    logits = (torch.randn(16384, 8, generator=g) * 3.0).cuda()
    H, _ = _static(ab, logits, 0.5, 1)
    H_orc = orc.entropy(hp.f64(logits))
    assert np.all(np.abs(H.cpu().numpy() - H_orc) <= REL_TOL * np.maximum(np.abs(H_orc), 1e-3))
    # one row more does not fit
    logits = torch.zeros(16385, 8, device="cuda")
    H = torch.zeros(16385, device="cuda")
    with pytest.raises(ab.AdapshotError) as e:
        ab.adapshot_entropy_static(logits, H, 0.5, 1, None, hp.new_status())
    assert e.value.code == ab.ECAPACITY
    logits = torch.zeros(20000, 8, device="cuda")
    H = torch.zeros(20000, device="cuda")
    with pytest.raises(ab.AdapshotError) as e:
        ab.adapshot_entropy_static(logits, H, 0.5, 1, None, hp.new_status())
    assert e.value.code == ab.ECAPACITY
