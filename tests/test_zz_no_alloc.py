"""adapshot_entropy_static: the entropy entry point for callers that cannot allocate
device memory (its scratch is a fixed array inside the library).  It must give what
adapshot_entropy gives, call after call, although all calls share that array."""
import ctypes as C

import pytest
import torch

from tests import helpers as hp

pytestmark = pytest.mark.gpu
REL_TOL = 1e-4          # the entropy tolerance used throughout the GPU tests


def _both(ab, logits, tau, P):
    want_H, want_fo, st = hp.run_entropy(ab, logits, tau, P)
    assert st == 0
    R = logits.shape[0]
    H = torch.full((R,), -1.0, dtype=torch.float32, device="cuda")
    fo = torch.full((R // P,), -7, dtype=torch.int32, device="cuda")
    status = hp.new_status()
    ab.adapshot_entropy_static(logits, H, tau, P, fo, status)      # through the C ABI, no workspace
    torch.cuda.synchronize()
    assert status.item() == 0
    assert torch.all((H - want_H).abs() <= REL_TOL * want_H.abs().clamp_min(1e-3))
    assert torch.equal(fo, want_fo)


def test_static_entropy_matches_workspace_entropy_on_two_calls_in_a_row():
    ab = hp.gpu_binding()
    g = torch.Generator().manual_seed(77)
    big = (torch.randn(8, 128256, generator=g) * 2.0).to(torch.bfloat16).cuda()
    small = (torch.randn(3, 1000, generator=g) * 4.0).cuda()
    _both(ab, big, 6.0, 4)        # fills much of the shared array
    _both(ab, small, 3.0, 1)      # a smaller call right after: stale states must not leak in
    _both(ab, big, 6.0, 4)


def test_static_entropy_rejects_sizes_beyond_its_array():
    ab = hp.gpu_binding()
    logits = torch.zeros(20000, 8, device="cuda")                 # 20000 states > 16384
    H = torch.zeros(20000, device="cuda")
    with pytest.raises(ab.AdapshotError) as e:
        ab.adapshot_entropy_static(logits, H, 0.5, 1, None, hp.new_status())
    assert e.value.code == ab.ECAPACITY
