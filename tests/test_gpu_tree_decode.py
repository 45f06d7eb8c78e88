"""The literal single-sequence form of the parallel multi-probe pass (Sec. 4.1: interleaved
sequence and tree mask) and the decode step over the chosen prefix, against the oracle."""
import numpy as np
import pytest
import torch

from oracle import adapshot_oracle as orc
from paper_2605_03644_b200 import workloads as wl
from tests import helpers as hp


def test_segment_table_parser_on_the_host():
    from paper_2605_03644_b200 import binding as ab
    S, P = ab.SEG_SHOTS, ab.SEG_PROBE
    # the case study's first round: probes after 4, 8, 12 and 16 shots
    segs = [(S, 4), (P, 7), (S, 4), (P, 7), (S, 4), (P, 7), (S, 4), (P, 7)]
    assert ab.adapshot_tree_layout(segs, 16) == ([4, 8, 12, 16], 7)
    assert ab.adapshot_tree_layout([(S, 1), (S, 2), (P, 3)], 3) == ([3], 3)        # shot runs may be split
    for bad in ([(P, 3)],                                   # a probe before any shot
                [(S, 2), (P, 3), (P, 3)],                   # two probes with the same shot count
                [(S, 2), (P, 3), (S, 1), (P, 4)],           # unequal probe lengths
                [(S, 2), (P, 3), (S, 1)],                   # does not end with a probe
                [(S, 5), (P, 3)],                           # more shots than were selected (k = 4)
                [(S, 0), (P, 3)]):
        with pytest.raises(ab.AdapshotError) as e:
            ab.adapshot_tree_layout(bad, 4)
        assert e.value.code == ab.ESHAPE
    with pytest.raises(ab.AdapshotError) as e:
        ab.adapshot_tree_layout([(7, 1), (P, 3)], 4)
    assert e.value.code == ab.EINVAL


def _setup(w, nl, seed_sel):
    ab = hp.gpu_binding()
    pool, qs = wl.make_pool(w, n_layers=nl), wl.make_queries(w, n_layers=nl)
    rng = np.random.default_rng(seed_sel)
    sel_np = np.stack([rng.permutation(w.n_shots)[:w.k] for _ in range(w.batch)]).astype(np.int32)
    dp = hp.dev_pool(ab, pool)
    model = hp.model_of(ab, w, n_layers=nl)
    off_np = orc.plan_offsets(sel_np, pool["shot_off"])
    cap = int(-(-int(off_np[:, -1].max()) // 8) * 8) + 24
    kc, vc, off, st = hp.run_assemble(ab, model, dp, torch.from_numpy(sel_np).cuda(), cap, 0, nl, torch.bfloat16)
    assert st == 0 and np.array_equal(off.cpu().numpy(), off_np)
    return ab, pool, qs, sel_np, off_np, model, cap, kc, vc, off


@pytest.mark.gpu
def test_tree_sequence_entry_point_against_the_dense_mask_oracle():
    nl, probes, t_q = 2, (2, 5, 9), 6
    w = wl.CONFIGS["cfg2"].scaled(n_shots=24, len_lo=3, len_hi=20, batch=2, k=9, probes=probes, t_q=t_q, seed=71,
                                  n_q_heads=8, n_kv_heads=2)
    ab, pool, qs, sel_np, off_np, model, cap, kc, vc, off = _setup(w, nl, 7)
    S, P = ab.SEG_SHOTS, ab.SEG_PROBE
    segs = [(S, 2), (P, t_q), (S, 3), (P, t_q), (S, 1), (S, 3), (P, t_q)]
    assert ab.adapshot_tree_layout(segs, w.k) == (list(probes), t_q)
    n_new = len(probes) * t_q
    # the probe tokens in sequence order: [B][nl][P * T_q][heads][d]
    q_seq = qs["q"].reshape(w.batch, nl, n_new, w.n_q_heads, w.head_dim).cuda()
    kq_seq = qs["kq"].reshape(w.batch, nl, n_new, w.n_kv_heads, w.head_dim).cuda()
    vq_seq = qs["vq"].reshape(w.batch, nl, n_new, w.n_kv_heads, w.head_dim).cuda()
    out_seq = torch.full_like(q_seq, 9.0)
    pos_seq = torch.full((w.batch, n_new), -1, dtype=torch.int64, device="cuda")
    ws = torch.empty(ab.adapshot_attn_workspace_bytes(model, w.batch, len(probes), t_q, nl, cap), dtype=torch.uint8,
                     device="cuda")
    st = hp.new_status()
    ab.adapshot_tree_attn(model, kc, vc, cap, off, w.k, segs, q_seq, kq_seq, vq_seq, 0, nl, out_seq, None, pos_seq,
                          ws, st)
    torch.cuda.synchronize()
    assert st.item() == 0
    kp, vp = hp.f64(pool["k"][:nl]), hp.f64(pool["v"][:nl])
    for b in range(w.batch):
        k_ctx, v_ctx, _ = orc.assemble_kv(kp, vp, pool["shot_off"], sel_np[b], w.rope_base)
        kind, src, pos, owner, mask = orc.tree_layout(off_np[b], list(probes), t_q)
        assert np.array_equal(pos_seq[b].cpu().numpy(), pos[kind == 1])          # position ids of the probe tokens
        for l in range(nl):
            want = orc.tree_attention(hp.f64(qs["q"][b, l]), hp.f64(qs["kq"][b, l]), hp.f64(qs["vq"][b, l]),
                                      k_ctx[l], v_ctx[l], off_np[b], list(probes), w.rope_base)
            got = out_seq[b, l].cpu().double().numpy().reshape(want.shape)
            hp.assert_attn_close(got, want, what=(b, l))


@pytest.mark.gpu
@pytest.mark.parametrize("t_new,t_own,d", [(1, 1, 128), (1, 37, 128), (1, 200, 64), (5, 140, 128), (33, 33, 64)])
def test_decode_step_over_the_chosen_prefix(t_new, t_own, d):
    # every query continues over its own shot count (as the threshold rule left it): the newest T_new of
    # T_own own tokens attend to that prefix and, causally, to the own tokens
    nl = 2
    w = wl.CONFIGS["cfg2"].scaled(n_shots=40, len_lo=5, len_hi=60, batch=3, k=12, probes=(12,), t_q=t_own, seed=73,
                                  head_dim=d, n_q_heads=8, n_kv_heads=2)
    ab, pool, qs, sel_np, off_np, model, cap, kc, vc, off = _setup(w, nl, 9)
    n_star = np.array([12, 1, 7], dtype=np.int32)
    q_new = qs["q"][:, :, 0, t_own - t_new:].contiguous().cuda()                 # [B][nl][T_new][Hq][d]
    k_own, v_own = qs["kq"][:, :, 0].contiguous().cuda(), qs["vq"][:, :, 0].contiguous().cuda()
    out = torch.full_like(q_new, 9.0)
    lse = torch.zeros((w.batch, nl, w.n_q_heads, t_new), dtype=torch.float32, device="cuda")
    ws = torch.empty(ab.adapshot_decode_workspace_bytes(model, w.batch, t_new, t_own, nl), dtype=torch.uint8,
                     device="cuda")
    st = hp.new_status()
    ab.adapshot_decode_attn(model, kc, vc, cap, off, w.k, torch.from_numpy(n_star).cuda(), q_new, k_own, v_own, 0, nl,
                            out, lse, ws, st)
    torch.cuda.synchronize()
    assert st.item() == 0
    kp, vp = hp.f64(pool["k"][:nl]), hp.f64(pool["v"][:nl])
    G = w.group
    got_all, want_all = [], []
    for b in range(w.batch):
        k_ctx, v_ctx, _ = orc.assemble_kv(kp, vp, pool["shot_off"], sel_np[b], w.rope_base)
        L = int(off_np[b, n_star[b]])
        for l in range(nl):
            ko, vo = hp.f64(qs["kq"][b, l, 0]), hp.f64(qs["vq"][b, l, 0])
            for t in range(t_new):
                u = t_own - t_new + t                                            # own index of the row's token
                for h in range(w.n_q_heads):
                    o_want, l_want = orc.decode_row(hp.f64(q_new[b, l, t, h].cpu()), ko[:u + 1], vo[:u + 1],
                                                    k_ctx[l], v_ctx[l], L, h // G, w.rope_base)
                    got_all.append(out[b, l, t, h].cpu().double().numpy())
                    want_all.append(o_want)
                    assert abs(float(lse[b, l, h, t]) - l_want) <= hp.lse_bound()
    hp.assert_attn_close(np.stack(got_all), np.stack(want_all))


@pytest.mark.gpu
def test_decode_reports_a_shot_count_outside_the_selection():
    nl = 1
    w = wl.CONFIGS["cfg2"].scaled(n_shots=16, len_lo=5, len_hi=20, batch=2, k=6, probes=(6,), t_q=4, seed=75)
    ab, pool, qs, sel_np, off_np, model, cap, kc, vc, off = _setup(w, nl, 11)
    q_new = qs["q"][:, :, 0, 3:].contiguous().cuda()
    k_own, v_own = qs["kq"][:, :, 0].contiguous().cuda(), qs["vq"][:, :, 0].contiguous().cuda()
    out = torch.zeros_like(q_new)
    ws = torch.empty(ab.adapshot_decode_workspace_bytes(model, w.batch, 1, 4, nl), dtype=torch.uint8, device="cuda")
    st = hp.new_status()
    ab.adapshot_decode_attn(model, kc, vc, cap, off, w.k, torch.tensor([3, 9], dtype=torch.int32).cuda(), q_new, k_own,
                            v_own, 0, nl, out, None, ws, st)
    torch.cuda.synchronize()
    assert st.item() == ab.EINDEX
