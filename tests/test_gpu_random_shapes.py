"""The attention variants on seeded random small shapes against the oracle: ragged shot
lengths down to one token, k = 1 and k = N, T_q = 1 and T_q just above a tile, head dims 64 and
128, group sizes 1..8, nested probes, duplicated shot ids, several layers and queries.  Each case
runs the materialised path (assemble + attention), the fused path and the V-from-pool path (K-only
cache) on the same inputs."""
import numpy as np
import pytest
import torch

from oracle import adapshot_oracle as orc
from paper_2605_03644_b200 import workloads as wl
from tests import helpers as hp

pytestmark = pytest.mark.gpu


def _case(seed):
    rng = np.random.default_rng(seed)
    d = int(rng.choice([64, 128]))
    hkv = int(rng.integers(1, 4))
    g = int(rng.choice([1, 2, 4, 8]))
    n_shots = int(rng.integers(2, 24))
    k = int(rng.choice([1, n_shots, int(rng.integers(1, n_shots + 1))]))
    n_probes = int(rng.integers(1, min(3, k) + 1))
    probes = tuple(sorted(rng.choice(np.arange(1, k + 1), size=n_probes, replace=False).tolist()))
    t_q = int(rng.choice([1, 2, 17, 64, 129]))
    w = wl.CONFIGS["cfg2"].scaled(n_layers=int(rng.integers(1, 3)), n_q_heads=hkv * g, n_kv_heads=hkv, head_dim=d,
                                  n_shots=n_shots, len_lo=1, len_hi=int(rng.choice([3, 40, 150])),
                                  batch=int(rng.integers(1, 3)), k=k, probes=probes, t_q=t_q, seed=1000 + seed)
    sel = rng.integers(0, n_shots, size=(w.batch, k)).astype(np.int32)     # any order, duplicates allowed
    return w, sel


@pytest.mark.parametrize("seed", range(12))
def test_random_shape_both_variants(seed):
    ab = hp.gpu_binding()
    w, sel_np = _case(seed)
    nl = w.n_layers
    pool, qs = wl.make_pool(w), wl.make_queries(w)
    dp = hp.dev_pool(ab, pool)
    model = hp.model_of(ab, w)
    off_np = orc.plan_offsets(sel_np, pool["shot_off"])
    cap = int(-(-max(int(off_np[:, -1].max()), 1) // 8) * 8) + 8
    sel = torch.from_numpy(sel_np).cuda()
    q, kq, vq = qs["q"].cuda(), qs["kq"].cuda(), qs["vq"].cuda()
    # materialised
    kc, vc, off, st = hp.run_assemble(ab, model, dp, sel, cap, 0, nl, torch.bfloat16)
    assert st == 0 and np.array_equal(off.cpu().numpy(), off_np)
    out_m, _, st = hp.run_attn(ab, model, kc, vc, cap, off, w.k, list(w.probes), q, kq, vq, 0, nl)
    assert st == 0
    # fused
    out_f = torch.full_like(q, 9.0)
    ws = torch.empty(max(ab.adapshot_attn_fused_workspace_bytes(model, w.batch, len(w.probes), w.t_q, nl, cap), 256),
                     dtype=torch.uint8, device="cuda")
    stf = hp.new_status()
    ab.adapshot_query_attn_fused(model, dp, sel, off, cap, list(w.probes), q, kq, vq, 0, nl, out_f, None, ws, stf)
    torch.cuda.synchronize()
    assert stf.item() == 0
    # K-only cache, V from the pool
    out_v = torch.full_like(q, 9.0)
    ws = torch.empty(max(ab.adapshot_attn_vpool_workspace_bytes(model, w.batch, len(w.probes), w.t_q, nl, cap), 256),
                     dtype=torch.uint8, device="cuda")
    stv = hp.new_status()
    ab.adapshot_query_attn_vpool(model, dp, sel, kc, cap, off, list(w.probes), q, kq, vq, 0, nl, out_v, None, ws, stv)
    torch.cuda.synchronize()
    assert stv.item() == 0
    assert torch.equal(out_v, out_m), "V from the pool must give the full cache's result bit for bit"
    # oracle (K' in fp64, never rounded)
    kp, vp = hp.f64(pool["k"][:nl]), hp.f64(pool["v"][:nl])
    for b in range(w.batch):
        k_ctx, v_ctx, _ = orc.assemble_kv(kp, vp, pool["shot_off"], sel_np[b], w.rope_base)
        L_list = [int(off_np[b, n]) for n in w.probes]
        for l in range(nl):
            want, _ = orc.query_attn(hp.f64(qs["q"][b, l]), hp.f64(qs["kq"][b, l]), hp.f64(qs["vq"][b, l]),
                                     k_ctx[l], v_ctx[l], L_list, w.rope_base)
            for name, got in (("materialised", out_m), ("fused", out_f)):
                hp.assert_attn_close(got[b, l].cpu().double().numpy(), want, what=(seed, name, b, l))
