"""adapshot_query_attn vs the fp64 oracle: bf16 output within max-abs 2e-2 and
mean-abs 2e-3 (the stated tolerance, plus the bf16 result's own rounding where a short
context makes the outputs larger than one; tests.helpers states both bounds and the one
used for the log-sum-exp output)."""
import numpy as np
import pytest
import torch

from oracle import adapshot_oracle as orc
from paper_2605_03644_b200 import workloads as wl
from tests import helpers as hp

pytestmark = pytest.mark.gpu


def _oracle_ctx(w, pool, sel_np, nl):
    """Assembled cache from the oracle, rounded once to the bf16 storage format."""
    kp, vp = hp.f64(pool["k"][:nl]), hp.f64(pool["v"][:nl])
    outs = []
    for b in range(sel_np.shape[0]):
        ok, ov, off = orc.assemble_kv(kp, vp, pool["shot_off"], sel_np[b], w.rope_base)
        outs.append((torch.from_numpy(ok).to(torch.bfloat16), torch.from_numpy(ov).to(torch.bfloat16), off))
    return outs


def _run_case(w, sel_np, probes, nl, cap_extra=37, k_gain=1.0):
    ab = hp.gpu_binding()
    w = w.scaled(probes=tuple(probes))
    pool = wl.make_pool(w, n_layers=nl)
    qs = wl.make_queries(w, n_layers=nl)
    if k_gain != 1.0:            # peaked scores: the running maximum keeps growing along the context
        pool["k"] = (pool["k"].float() * k_gain).to(pool["k"].dtype)
        qs["kq"] = (qs["kq"].float() * k_gain).to(qs["kq"].dtype)
    if w.dtype == "fp32":        # the attention kernel is bf16: round the inputs once, for both sides
        w = w.scaled(dtype="bf16")
        for key in ("k", "v"):
            pool[key] = pool[key].to(torch.bfloat16)
        for key in ("q", "kq", "vq"):
            qs[key] = qs[key].to(torch.bfloat16)
    B, k = sel_np.shape
    ctxs = _oracle_ctx(w, pool, sel_np, nl)
    cap = max(int(c[2][-1]) for c in ctxs) + cap_extra
    kc = torch.zeros((B, nl, cap, w.n_kv_heads, w.head_dim), dtype=torch.bfloat16)
    vc = torch.zeros_like(kc)
    off = torch.zeros((B, k + 1), dtype=torch.int64)
    for b, (ok, ov, o) in enumerate(ctxs):
        L = int(o[-1])
        kc[b, :, :L], vc[b, :, :L] = ok, ov
        off[b] = torch.from_numpy(o)
    model = hp.model_of(ab, w, n_layers=nl)
    q, kq, vq = qs["q"].cuda(), qs["kq"].cuda(), qs["vq"].cuda()
    out = torch.full_like(q, 9.0)
    lse = torch.zeros((B, nl, len(probes), w.n_q_heads, w.t_q), dtype=torch.float32, device="cuda")
    ws = torch.empty(ab.adapshot_attn_workspace_bytes(model, B, len(probes), w.t_q, nl, cap),
                     dtype=torch.uint8, device="cuda")
    st = hp.new_status()
    ab.adapshot_query_attn(model, kc.cuda(), vc.cuda(), cap, off.cuda(), k, list(probes), q, kq, vq, 0, nl,
                           out, lse, ws, st)
    torch.cuda.synchronize()
    assert st.item() == 0
    got_all, want_all = [], []
    for b in range(B):
        L_list = [int(off[b, n_j]) for n_j in probes]
        for l in range(nl):
            want, want_lse = orc.query_attn(hp.f64(qs["q"][b, l]), hp.f64(qs["kq"][b, l]), hp.f64(qs["vq"][b, l]),
                                            hp.f64(kc[b, l]), hp.f64(vc[b, l]), L_list, w.rope_base)
            got_all.append(out[b, l].cpu().double().numpy())
            want_all.append(want)
            assert np.abs(lse[b, l].cpu().double().numpy() - want_lse).max() <= hp.lse_bound(k_gain)
    hp.assert_attn_close(np.stack(got_all), np.stack(want_all))


def test_cfg1_attention():
    w = wl.CONFIGS["cfg1"]
    pool = wl.make_pool(w)
    qs = wl.make_queries(w)
    sel, _ = orc.select_topk(hp.f64(qs["q_emb"]), hp.f64(pool["emb"]), w.k)
    _run_case(w, sel, [8], 1)


def test_8b_shape_ragged_probes_and_cut_units():
    # several 128-key tiles, a ragged last tile, nested probes, two layers, two queries; the few
    # hundred tiles are spread over all CTAs, so most units are cut and merged from partials
    w = wl.CONFIGS["cfg2"].scaled(n_shots=64, len_lo=30, len_hi=90, batch=2, k=40, t_q=40, seed=21)
    rng = np.random.default_rng(1)
    sel = np.stack([rng.permutation(64)[:40], rng.permutation(64)[:40]]).astype(np.int32)
    _run_case(w, sel, [3, 17, 40], 2)


def test_tq_longer_than_a_key_tile_and_g8():
    # T_q = 150 > 128: two own-key tiles with the causal diagonal; G = 8 rows per token
    w = wl.CONFIGS["cfg4"].scaled(n_shots=20, len_lo=40, len_hi=70, batch=1, k=9, t_q=150, n_q_heads=16,
                                  n_kv_heads=2, pool_token_target=0, seed=22)
    sel = np.arange(9, dtype=np.int32)[None, ::-1].copy()
    _run_case(w, sel, [4, 9], 1)


def test_single_token_probe_and_tiny_context():
    # one probe token over 2-6 context tokens
    w = wl.CONFIGS["cfg2"].scaled(n_shots=8, len_lo=1, len_hi=3, batch=1, k=2, t_q=1, seed=23)
    _run_case(w, np.array([[5, 1]], dtype=np.int32), [1, 2], 1)


def test_head_dim_64_bf16_many_tiles():
    w = wl.CONFIGS["cfg2"].scaled(n_shots=32, len_lo=50, len_hi=120, batch=1, k=20, t_q=33, head_dim=64,
                                  n_q_heads=6, n_kv_heads=3, seed=24)
    sel = np.random.default_rng(2).permutation(32)[:20].astype(np.int32)[None]
    _run_case(w, sel, [20], 1)


def test_maximum_number_of_probe_query_pairs():
    # B * P = 256 (the most one call takes): 64 queries x 4 nested probes, short shots, G = 8
    w = wl.CONFIGS["cfg2"].scaled(n_shots=40, len_lo=20, len_hi=60, batch=64, k=6, t_q=5, n_q_heads=8,
                                  n_kv_heads=1, seed=25)
    rng = np.random.default_rng(3)
    sel = np.stack([rng.permutation(40)[:6] for _ in range(64)]).astype(np.int32)
    _run_case(w, sel, [1, 2, 4, 6], 1)


def test_sixteen_nested_probes():
    # P = 16 (the most one call takes), every prefix length from one shot to all sixteen, two layers
    w = wl.CONFIGS["cfg2"].scaled(n_shots=48, len_lo=30, len_hi=200, batch=3, k=16, t_q=24, seed=27)
    rng = np.random.default_rng(5)
    sel = np.stack([rng.permutation(48)[:16] for _ in range(3)]).astype(np.int32)
    _run_case(w, sel, list(range(1, 17)), 2)


def test_peaked_scores_rescale_the_accumulator():
    # keys three times larger: scores of a row spread over tens of log2 units, so the row maximum
    # grows by more than the lazy-rescale threshold several times along the context and the
    # output approaches single value rows.  The factor 3 takes the place of the per-channel scale here
    # (both together would push the keys six times beyond the configurations' magnitude, and the
    # score error of the bf16 query with them).
    w = wl.CONFIGS["cfg2"].scaled(n_shots=48, len_lo=60, len_hi=140, batch=1, k=30, t_q=24, seed=26,
                                  channel_scale=False)
    sel = np.random.default_rng(4).permutation(48)[:30].astype(np.int32)[None]
    _run_case(w, sel, [7, 30], 1, k_gain=3.0)


def test_a_range_that_spans_more_pairs_than_the_schedule_cache_holds():
    # T_q * G = 2048 rows make gangs of eight CTAs, i.e. 18 ranges of equal cost on 148 SMs.  With 64
    # queries and probes (1, 2, 3, k) the 64 long pairs carry 17/18 of the cost, so the last range holds
    # all 192 short pairs: far more than a CTA copies to shared memory, the rest of the schedule is read
    # from the workspace.  Rows of short and long pairs are compared with the oracle.
    ab = hp.gpu_binding()
    B, k, probes, t_q = 64, 720, (1, 2, 3, 720), 128
    w = wl.CONFIGS["cfg2"].scaled(n_shots=1024, len_dist="const", len_lo=64, len_hi=64, batch=B, k=k, probes=probes,
                                  t_q=t_q, n_q_heads=16, n_kv_heads=1, head_dim=64, seed=27)
    pool = wl.make_pool(w, n_layers=1)
    qs = wl.make_queries(w, n_layers=1)
    rng = np.random.default_rng(5)
    sel4 = np.stack([rng.permutation(1024)[:k] for _ in range(4)]).astype(np.int32)   # four selections, dealt out
    ctx4 = _oracle_ctx(w, pool, sel4, 1)
    L = k * 64
    cap = L + 64
    kc = torch.zeros((B, 1, cap, 1, 64), dtype=torch.bfloat16)
    vc = torch.zeros_like(kc)
    off = torch.zeros((B, k + 1), dtype=torch.int64)
    for b in range(B):
        ok, ov, o = ctx4[b % 4]
        kc[b, :, :L], vc[b, :, :L] = ok, ov
        off[b] = torch.from_numpy(o)
    model = hp.model_of(ab, w, n_layers=1)
    out, lse, st = hp.run_attn(ab, model, kc.cuda(), vc.cuda(), cap, off.cuda(), k, list(probes),
                               qs["q"].cuda(), qs["kq"].cuda(), qs["vq"].cuda(), 0, 1)
    assert st == 0
    out, lse = out.cpu(), lse.cpu()
    got, want, rows = [], [], []
    for j in range(len(probes)):
        n_rows = 40 if j < 3 else 8                      # the short pairs are the ones behind the cache
        for _ in range(n_rows):
            rows.append((int(rng.integers(B)), j, int(rng.integers(t_q)), int(rng.integers(16))))
    rows += [(63, 0, 127, 15), (0, 2, 0, 0), (63, 2, 127, 15)]        # the last pair of the call, and corners
    for b, j, t, h in rows:
        o_want, l_want = orc.attn_row(hp.f64(qs["q"][b, 0, j, t, h]), hp.f64(qs["kq"][b, 0, j]),
                                      hp.f64(qs["vq"][b, 0, j]), hp.f64(kc[b, 0]), hp.f64(vc[b, 0]),
                                      int(off[b, probes[j]]), t, 0, w.rope_base)
        got.append(out[b, 0, j, t, h].double().numpy())
        want.append(o_want)
        assert abs(float(lse[b, 0, j, h, t]) - l_want) <= hp.lse_bound()
    hp.assert_attn_close(np.stack(got), np.stack(want))
