"""adapshot_select_attn (the paper's attention-based relevance ranking, Sec. 4.2) against the oracle's
relevance_attention: scores within 1e-3 relative (bf16 inputs are shared; the differences are fp32
accumulation and the exponential), indices bit-exact wherever the oracle's scores are further apart
than that, ties by the lower shot id."""
import numpy as np
import pytest
import torch

from oracle import adapshot_oracle as orc
from paper_2605_03644_b200 import workloads as wl
from tests import helpers as hp

pytestmark = pytest.mark.gpu
SCORE_REL = 1e-3


def _run(ab, model, dp, layer, q, k, per_token=False):
    B = q.shape[0]
    sel = torch.full((B, k), -1, dtype=torch.int32, device="cuda")
    score = torch.zeros((B, k), dtype=torch.float32, device="cuda")
    ws = torch.empty(max(256, ab.adapshot_select_attn_workspace_bytes(model, dp, B, q.shape[1], k)), dtype=torch.uint8,
                     device="cuda")
    st = hp.new_status()
    ab.adapshot_select_attn(model, dp, layer, q.cuda(), k, sel, score, ws, st, per_token=per_token)
    torch.cuda.synchronize()
    assert st.item() == 0
    return sel.cpu().numpy(), score.cpu().numpy()


def _check(w, nl, layer, k, per_token=False, q_gain=1.0):
    ab = hp.gpu_binding()
    pool = wl.make_pool(w, n_layers=nl)
    qs = wl.make_queries(w, n_layers=nl, n_probes=1)
    q = (qs["q"][:, layer, 0].float() * q_gain).to(torch.bfloat16).contiguous()      # [B][T_q][Hq][d] as stored
    dp = hp.dev_pool(ab, pool)
    model = hp.model_of(ab, w, n_layers=nl)
    sel, score = _run(ab, model, dp, layer, q, k, per_token)
    k_layer = hp.f64(pool["k"][layer])
    for b in range(w.batch):
        s = orc.relevance_attention(hp.f64(q[b]), k_layer, pool["shot_off"], per_token=per_token)
        # scores of the shots the kernel chose, against the oracle's values for those shots
        assert np.all(np.abs(score[b] - s[sel[b]]) <= SCORE_REL * np.abs(s[sel[b]]) + 1e-30), b
        # the choice itself: the oracle's order, up to pairs the tolerance cannot tell apart
        order = np.argsort(-s, kind="stable")
        assert len(set(sel[b].tolist())) == k
        for r in range(k):
            if sel[b, r] != order[r]:
                assert abs(s[sel[b, r]] - s[order[r]]) <= 2 * SCORE_REL * abs(s[order[r]]), (b, r)
        # nothing better was left out: the weakest chosen shot is within the tolerance of rank k
        assert s[sel[b]].min() >= s[order[k - 1]] * (1 - 2 * SCORE_REL)
    return sel, score


def test_tiny_pool_one_tile():
    w = wl.CONFIGS["cfg1"].scaled(dtype="bf16", n_shots=12, len_lo=5, len_hi=5, t_q=7, seed=81)
    _check(w, 1, 0, 5)


def test_8b_shape_many_tiles_and_splits():
    # 8B head shape, 96 shots of 30-200 tokens (about 11 K pool tokens: 86 key tiles, several ranges per unit),
    # T_q * G = 192 rows: two M tiles, the second half empty; the third of three layers is the representative one
    w = wl.CONFIGS["cfg2"].scaled(n_shots=96, len_lo=30, len_hi=200, batch=2, k=24, t_q=48, seed=82)
    _check(w, 3, 2, 24)
    _check(w, 3, 2, 24, per_token=True)


def test_head_dim_64_group_of_three_and_one_token_shots():
    w = wl.CONFIGS["cfg2"].scaled(n_shots=300, len_lo=1, len_hi=9, batch=3, k=300, t_q=5, head_dim=64, n_q_heads=6,
                                  n_kv_heads=2, seed=83)
    _check(w, 1, 0, 300)


def test_peaked_queries_single_out_their_shot():
    # queries five times larger: the softmax over the pool concentrates on a few keys
    w = wl.CONFIGS["cfg2"].scaled(n_shots=64, len_lo=20, len_hi=90, batch=2, k=8, t_q=16, seed=84)
    sel, score = _check(w, 1, 0, 8, q_gain=5.0)
    assert (score[:, 0] > 1.5 / 64).all()                 # well above the uniform share of 1 / 64


def test_identical_shots_get_equal_masses():
    # a pool made of one shot repeated: every shot gets the same mass (the order among them is decided by the
    # last bits of the fp64 sums, which depend on how the keys fall into warps: only exact ties go by shot id,
    # and that rule is the top-k kernel's, tested with the embedding selector)
    ab = hp.gpu_binding()
    w = wl.CONFIGS["cfg2"].scaled(n_shots=1, len_lo=17, len_hi=17, batch=1, k=1, t_q=8, seed=85)
    pool = wl.make_pool(w, n_layers=1)
    n_rep = 9
    pool["k"] = pool["k"].repeat(1, n_rep, 1, 1).contiguous()
    pool["v"] = pool["v"].repeat(1, n_rep, 1, 1).contiguous()
    pool["shot_off"] = np.arange(n_rep + 1, dtype=np.int64) * 17
    pool["emb"] = pool["emb"].repeat(n_rep, 1).contiguous()
    qs = wl.make_queries(w, n_layers=1, n_probes=1)
    q = qs["q"][:, 0, 0].contiguous()
    dp = hp.dev_pool(ab, pool)
    sel, score = _run(ab, hp.model_of(ab, w, n_layers=1), dp, 0, q, n_rep)
    assert np.allclose(score, 1.0 / n_rep, rtol=1e-4)
    assert sorted(sel[0].tolist()) == list(range(n_rep))
