"""adapshot_entropy vs the fp64 oracle: relative error <= 1e-4."""
import math

import numpy as np
import pytest
import torch

from oracle import adapshot_oracle as orc
from paper_2605_03644_b200 import workloads as wl
from tests import helpers as hp

pytestmark = pytest.mark.gpu
REL_TOL = 1e-4


def _check(ab, logits, tau=None, P=1):
    H, fo, st = hp.run_entropy(ab, logits.cuda(), 0.0 if tau is None else tau, P)
    want = orc.entropy(hp.f64(logits))
    got = H.cpu().numpy().astype(np.float64)
    assert st == 0
    rel = np.abs(got - want) / np.maximum(np.abs(want), 1e-3)
    assert rel.max() <= REL_TOL, rel.max()
    if tau is not None:
        # keep the threshold decision away from rounding: every |H - tau| must be clear
        assert np.abs(want - tau).min() > 1e-3 * max(tau, 1.0)
        assert np.array_equal(fo.cpu().numpy(), orc.first_ok(want, tau, P))
    return got


@pytest.mark.parametrize("name", ["cfg1", "cfg2", "cfg3"])
def test_entropy_on_config_logits(name):
    ab = hp.gpu_binding()
    w = wl.CONFIGS[name]
    P = len(w.probes)
    g = torch.Generator().manual_seed(w.seed)
    ldt = torch.float32 if w.logits_dtype == "fp32" else torch.bfloat16
    logits = (torch.randn(w.batch * P, w.vocab, generator=g) * w.logits_std).to(ldt)
    _check(ab, logits)


def test_entropy_cfg5_probe_rows_bf16():
    ab = hp.gpu_binding()
    g = torch.Generator().manual_seed(9)
    # 3 queries x 7 nested probes at the full vocabulary; sharper rows for later probes
    sharp = torch.tensor([0.5, 1.0, 1.5, 2.0, 3.0, 4.0, 6.0]).repeat(3)[:, None]
    logits = (torch.randn(21, 128256, generator=g) * sharp).to(torch.bfloat16)
    want = orc.entropy(hp.f64(logits))
    tau = float((want.reshape(3, 7)[:, 3] + want.reshape(3, 7)[:, 4]).mean() / 2)
    _check(ab, logits, tau=tau, P=7)


@pytest.mark.parametrize("V", [1, 2, 7, 8, 9, 1023, 4097, 50001])
@pytest.mark.parametrize("dt", [torch.float32, torch.bfloat16])
def test_entropy_ragged_vocab(V, dt):
    ab = hp.gpu_binding()
    g = torch.Generator().manual_seed(V)
    stride = (V + 7) // 8 * 8                      # rows must start on 16 bytes
    buf = (torch.randn(5, stride, generator=g) * 3).to(dt).cuda()
    H, _, st = hp.run_entropy(ab, buf[:, :V], 0.0, 1, want_first=False)
    want = orc.entropy(hp.f64(buf[:, :V]))
    assert st == 0
    assert np.all(np.abs(H.cpu().numpy() - want) <= REL_TOL * np.maximum(want, 1e-3) + 1e-7)


def test_entropy_closed_forms_and_threshold():
    ab = hp.gpu_binding()
    V = 32000
    x = torch.zeros(4, V)
    x[1, 5] = 200.0                                # one dominant logit -> 0
    x[2, :10] = 1.5; x[2, 10:] = -0.5              # two-level row
    x[3] = -1e4; x[3, :2] = 0.0                    # two equal survivors -> ln 2
    x[3, 100:200] = float("-inf")
    got = _check(ab, x)
    assert abs(got[0] - math.log(V)) < 1e-4 * math.log(V)
    assert got[1] < 1e-6 and abs(got[3] - math.log(2)) < 1e-5
    H, fo, _ = hp.run_entropy(ab, x.cuda(), 1.0, 2)
    assert fo.tolist() == [1, 1]                   # groups (uniform, peaked) and (two-level, ln 2)
    H, fo, _ = hp.run_entropy(ab, x.cuda(), 1e-9, 4)
    assert fo.tolist() == [1]
    H, fo, _ = hp.run_entropy(ab, x[:1].cuda(), 1.0, 1)
    assert fo.tolist() == [-1]


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("renorm", [False, True])
def test_subset_entropy_two_tokens_and_more(dtype, renorm):
    # the two-token ({Yes, No}) form of Eq. 2 and a larger subset, both readings
    ab = hp.gpu_binding()
    g = torch.Generator().manual_seed(9)
    R, V, P = 8, 32000, 4
    logits = (torch.randn(R, V, generator=g) * 2.0).to(dtype)
    for ids in ([9891, 2822], [5, 31999, 17, 4000, 123]):
        logits[:, ids] += 6.0                       # answer tokens carry visible probability mass
        ids_t = torch.tensor(ids, dtype=torch.int32, device="cuda")
        H = torch.full((R,), -1.0, device="cuda")
        fo = torch.full((R // P,), -7, dtype=torch.int32, device="cuda")
        ws = torch.empty(max(ab.adapshot_entropy_workspace_bytes(R, V), 256), dtype=torch.uint8, device="cuda")
        st = hp.new_status()
        want = orc.entropy_subset(hp.f64(logits), ids, renorm=renorm)
        tau = float(np.sort(want)[R // 2]) + 1e-3
        ab.adapshot_entropy_subset(logits.cuda(), ids_t, H, tau, P, fo, ws, st, renorm=renorm)
        torch.cuda.synchronize()
        assert st.item() == 0
        got = H.cpu().numpy().astype(np.float64)
        assert (np.abs(got - want) <= REL_TOL * np.maximum(np.abs(want), 1e-3)).all(), (got, want)
        if np.abs(want - tau).min() > 1e-4:
            assert np.array_equal(fo.cpu().numpy(), orc.first_ok(want, tau, P))


def test_subset_entropy_reports_a_bad_token_id():
    ab = hp.gpu_binding()
    logits = torch.zeros(2, 1000, device="cuda")
    ids_t = torch.tensor([3, 1000], dtype=torch.int32, device="cuda")
    H = torch.zeros(2, device="cuda")
    ws = torch.empty(max(ab.adapshot_entropy_workspace_bytes(2, 1000), 256), dtype=torch.uint8, device="cuda")
    st = hp.new_status()
    ab.adapshot_entropy_subset(logits, ids_t, H, 0.5, 1, None, ws, st)
    torch.cuda.synchronize()
    assert st.item() == ab.EINDEX
    assert np.allclose(H.cpu().numpy(), math.log(1000) / 1000, rtol=1e-4)      # the valid token alone


@pytest.mark.parametrize("R,V", [(1, 8191), (3, 8192), (3, 8193), (5, 16384), (7, 40001), (300, 24577),
                                 (1000, 16392), (2, 128256)])
@pytest.mark.parametrize("dt", [torch.float32, torch.bfloat16])
def test_entropy_slice_boundaries(R, V, dt):
    # rows are cut into slices of multiples of 8192 entries: lengths around the unit, a last slice
    # of a few entries, many rows with several slices each, a few rows with sixteen
    ab = hp.gpu_binding()
    g = torch.Generator().manual_seed(R * 131 + V)
    stride = (V + 7) // 8 * 8
    scale = torch.linspace(0.5, 5.0, R)[:, None]
    buf = (torch.randn(R, stride, generator=g) * scale).to(dt)
    buf[:, V - 1] += 7.0                            # the row maximum sits in the last (shortest) slice
    H, _, st = hp.run_entropy(ab, buf.cuda()[:, :V], 0.0, 1, want_first=False)
    want = orc.entropy(hp.f64(buf[:, :V]))
    assert st == 0
    assert np.all(np.abs(H.cpu().numpy() - want) <= REL_TOL * np.maximum(want, 1e-3) + 1e-7)


@pytest.mark.parametrize("dt", [torch.float32, torch.bfloat16])
def test_entropy_minus_infinity_conventions(dt):
    # -inf (and anything at or below -2^97) adds nothing wherever it sits: inside a vector, as a whole
    # vector, as a whole slice; a row of nothing else has H = 0 by the stated convention
    ab = hp.gpu_binding()
    V = 20000
    x = torch.zeros(5, V)
    x[0, 3:11] = float("-inf")                      # whole 16-byte vectors and parts of them
    x[1, :8192] = float("-inf")                     # the whole first slice
    x[1, 8192:8194] = 1.0                           # two equal survivors beside 11 806 zeros
    x[2, :] = float("-inf")
    x[3, :] = -3.0e38
    x[4, 8192:] = -1.0e30                           # below the floor: counts as -inf
    got, _, st = hp.run_entropy(ab, x.to(dt).cuda(), 0.0, 1, want_first=False)
    got = got.cpu().numpy()
    assert st == 0
    assert abs(got[0] - math.log(V - 8)) < 1e-4 * math.log(V)
    want1 = orc.entropy(hp.f64(x[1:2].to(dt)))[0]
    assert abs(got[1] - want1) < 1e-4 * want1
    assert got[2] == 0.0 and got[3] == 0.0
    assert abs(got[4] - math.log(8192)) < 1e-4 * math.log(8192)
