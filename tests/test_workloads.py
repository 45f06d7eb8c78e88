"""The seeded generators are deterministic and have the stated shapes."""
import numpy as np
import torch

from paper_2605_03644_b200 import workloads as wl


def test_lengths_follow_the_recipes():
    for name, w in wl.CONFIGS.items():
        t = wl.shot_lengths(w)
        assert np.array_equal(t, wl.shot_lengths(w))
        assert t.min() >= w.len_lo and t.max() <= w.len_hi
        if w.n_shots:
            assert len(t) == w.n_shots
        else:
            assert t.sum() >= w.pool_token_target > t[:-1].sum()
    t5 = wl.shot_lengths(wl.CONFIGS["cfg5"])
    assert 110 <= np.median(t5) <= 130


def test_small_pool_and_queries_are_reproducible():
    w = wl.CONFIGS["cfg1"]
    a, b = wl.make_pool(w), wl.make_pool(w)
    assert torch.equal(a["k"], b["k"]) and torch.equal(a["emb"], b["emb"])
    assert a["k"].shape == (1, 64 * 32, 1, 64) and a["k"].dtype == torch.float32
    assert torch.allclose(a["emb"].norm(dim=1), torch.ones(64), atol=1e-6)
    q = wl.make_queries(w)
    assert q["q"].shape == (1, 1, 1, 16, 4, 64) and q["logits"].shape == (1, 1024)
    assert abs(q["logits"].var().item() - 2.0) < 0.3
    w2 = wl.CONFIGS["cfg2"].scaled(n_shots=32)
    p2 = wl.make_pool(w2)
    assert p2["k"].dtype == torch.bfloat16 and p2["pool_tokens"] == int(p2["shot_off"][-1])
    x = wl.to_f64(p2["k"])
    assert x.dtype == np.float64 and np.array_equal(x.astype(np.float32), p2["k"].float().numpy())


def test_layer_chunks_cover_the_layers_in_order():
    from paper_2605_03644_b200.pipeline import layer_chunks
    for n in (1, 2, 3, 7, 8, 32, 80):
        for lpc in (1, 2, 3, 4, 8, 20, 32, 80):
            for ramp in (False, True):
                c = layer_chunks(n, lpc, ramp)
                assert c[0][0] == 0 and c[-1][1] == n
                assert all(a[1] == b[0] for a, b in zip(c, c[1:]))
                assert all(0 < e - b <= lpc for b, e in c)
    assert [e - b for b, e in layer_chunks(32, 4, True)] == [1, 3, 4, 4, 4, 4, 4, 4, 3, 1]
    assert [e - b for b, e in layer_chunks(32, 8, True)] == [2, 6, 8, 8, 6, 2]
    assert [e - b for b, e in layer_chunks(32, 32, True)] == [32]
    assert [e - b for b, e in layer_chunks(32, 8, False)] == [8, 8, 8, 8]
