"""adapshot_select vs the fp64 oracle: indices bit-exact (ties -> lowest shot id)."""
import numpy as np
import pytest
import torch

from oracle import adapshot_oracle as orc
from paper_2605_03644_b200 import workloads as wl
from tests import helpers as hp

pytestmark = pytest.mark.gpu


def _check(ab, emb, q_emb, k):
    so = torch.arange(emb.shape[0] + 1, dtype=torch.int64, device="cuda")
    pool = ab.Pool(so, None, None, emb.cuda().contiguous())
    sel, score, st = hp.run_select(ab, pool, q_emb, k)
    want, want_sc = orc.select_topk(hp.f64(q_emb), hp.f64(emb), k)
    assert st == 0
    assert np.array_equal(sel.cpu().numpy(), want), "top-k indices must be bit-exact"
    assert np.allclose(score.cpu().numpy(), want_sc, atol=1e-6)


@pytest.mark.parametrize("name", ["cfg1", "cfg2", "cfg3", "cfg5"])
def test_select_matches_oracle_on_the_configs(name):
    ab = hp.gpu_binding()
    w = wl.CONFIGS[name]
    g = torch.Generator().manual_seed(w.seed)
    emb = torch.randn(w.n_shots, w.emb_dim, generator=g)
    emb = emb / emb.norm(dim=1, keepdim=True)
    q = torch.randn(w.batch, w.emb_dim, generator=g)
    q = q / q.norm(dim=1, keepdim=True)
    assert orc.min_adjacent_gap(hp.f64(q), hp.f64(emb), w.k) > 1e-12
    _check(ab, emb, q, w.k)


@pytest.mark.parametrize("N,E,B,k", [(1, 4, 1, 1), (5, 3, 2, 5), (33, 130, 3, 7), (1000, 64, 2, 1000),
                                     (8192, 16, 1, 8192), (8193, 16, 2, 100), (20000, 32, 2, 4096)])
def test_select_edge_shapes(N, E, B, k):
    ab = hp.gpu_binding()
    g = torch.Generator().manual_seed(N + E)
    _check(ab, torch.randn(N, E, generator=g), torch.randn(B, E, generator=g), k)


def test_select_ties_and_zero_norm():
    ab = hp.gpu_binding()
    g = torch.Generator().manual_seed(5)
    emb = torch.randn(300, 64, generator=g)
    emb[200] = emb[7]; emb[100] = emb[7]; emb[250] = emb[7]     # exact duplicates
    emb[13] = 0.0                                              # zero norm -> score 0
    emb[40:60] = emb[40]                                       # a run of equal rows
    q = torch.cat([emb[7:8], emb[40:41], torch.randn(1, 64, generator=g)])
    _check(ab, emb, q, 300)
    _check(ab, emb, q, 5)
    sel, _, _ = hp.run_select(ab, ab.Pool(torch.arange(301, device="cuda"), None, None, emb.cuda()), q, 4)
    assert sel[0].tolist() == [7, 100, 200, 250]
    assert sel[1, :4].tolist() == [40, 41, 42, 43]


def test_nested_probes_are_prefixes():
    ab = hp.gpu_binding()
    g = torch.Generator().manual_seed(6)
    emb, q = torch.randn(500, 32, generator=g), torch.randn(2, 32, generator=g)
    pool = ab.Pool(torch.arange(501, device="cuda"), None, None, emb.cuda())
    full, _, _ = hp.run_select(ab, pool, q, 128)
    for n in (1, 16, 64):
        part, _, _ = hp.run_select(ab, pool, q, n)
        assert torch.equal(part, full[:, :n])
