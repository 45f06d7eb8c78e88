"""Pins of the fp64 oracle against things other than itself (CPU only).

Each test ties one oracle function to a closed form, a differently-written
definition (complex rotation, explicit-mask dense attention, python loops), a
scipy routine, or a value/rule the paper prints.  The last test plants typical
mistakes into the oracle and checks that the pins notice each of them.
"""
import math
import os

import numpy as np
import pytest
import scipy.special
import scipy.stats
import scipy.spatial.distance

from oracle import adapshot_oracle as orc

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _rows(name):
    out = []
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            line = line.strip()
            if line and not line.startswith("#"):
                out.append(line.split())
    return out


# ------------------------------------------------------------------ RoPE
def test_rope_hand_value_quarter_turn():
    # d = 2, theta_0 = 1: a rotation by pi/2 maps (1, 0) to (0, 1)
    y = orc.rope(np.array([1.0, 0.0]), math.pi / 2, base=10000.0)
    assert np.allclose(y, [0.0, 1.0], atol=1e-15)
    y = orc.rope(np.array([0.0, 1.0]), math.pi / 2, base=10000.0)
    assert np.allclose(y, [-1.0, 0.0], atol=1e-15)


def test_rope_theta_values():
    th = orc.rope_theta(8, 10000.0)
    assert np.allclose(th, [1.0, 0.1, 0.01, 0.001], rtol=1e-14)
    th = orc.rope_theta(128, 500000.0)
    assert th[0] == 1.0 and np.isclose(th[32], 500000.0 ** -0.5, rtol=1e-14)


def test_rope_equals_complex_rotation():
    # (x_i + i x_{i+d/2}) * exp(i p theta_i): the same map, written differently
    rng = np.random.default_rng(1)
    d, base = 64, 10000.0
    x = rng.standard_normal((5, 3, d))
    p = rng.integers(0, 5000, size=(5, 3)).astype(np.float64)
    z = x[..., : d // 2] + 1j * x[..., d // 2:]
    th = np.array([base ** (-2.0 * i / d) for i in range(d // 2)])
    zr = z * np.exp(1j * p[..., None] * th)
    want = np.concatenate([zr.real, zr.imag], axis=-1)
    assert np.allclose(orc.rope(x, p, base), want, atol=1e-12)


def test_rope_identity_norm_and_composition():
    rng = np.random.default_rng(2)
    d, base = 128, 500000.0
    x = rng.standard_normal((7, d))
    assert np.array_equal(orc.rope(x, np.zeros(7), base), x)
    y = orc.rope(x, np.arange(7) * 913.0, base)
    pair = lambda v: v[..., : d // 2] ** 2 + v[..., d // 2:] ** 2
    assert np.allclose(pair(y), pair(x), rtol=1e-12)
    # a vector at p1 moves to p2 by one more rotation of p2 - p1 (Sec. 4.3)
    p1, p2 = 37.0, 4242.0
    assert np.allclose(orc.rope(orc.rope(x, p1, base), p2 - p1, base),
                       orc.rope(x, p2, base), atol=1e-11)


def test_rotary_scores_depend_on_relative_position_only():
    rng = np.random.default_rng(3)
    d, base = 64, 10000.0
    q, k = rng.standard_normal(d), rng.standard_normal(d)
    a = orc.rope(q, 100.0, base) @ orc.rope(k, 40.0, base)
    b = orc.rope(q, 1100.0, base) @ orc.rope(k, 1040.0, base)
    c = orc.rope(q, 100.0, base) @ orc.rope(k, 41.0, base)
    assert abs(a - b) < 1e-10 and abs(a - c) > 1e-3


# ------------------------------------------------------- offsets / gather
def test_two_shot_positions_golden():
    for ta, tb, oa, ob, tot in _rows("two_shot_positions.txt"):
        ta, tb, oa, ob, tot = map(int, (ta, tb, oa, ob, tot))
        shot_off = np.array([0, ta, ta + tb])
        off = orc.plan_offsets(np.array([[0, 1]]), shot_off)[0]
        assert off.tolist() == [oa, ob, tot]
        # reversed order: B first, A gets Delta = T_B
        off = orc.plan_offsets(np.array([[1, 0]]), shot_off)[0]
        assert off.tolist() == [0, tb, tot]


def _tiny_pool(rng, n_layers=2, lens=(3, 1, 4, 2), hkv=2, d=8):
    off = np.concatenate([[0], np.cumsum(lens)])
    k = rng.standard_normal((n_layers, off[-1], hkv, d))
    v = rng.standard_normal((n_layers, off[-1], hkv, d))
    return k, v, off


def test_identity_order_reproduces_source_cache():
    rng = np.random.default_rng(4)
    k, v, off = _tiny_pool(rng)
    sel = np.arange(len(off) - 1)
    kc, vc, co = orc.assemble_kv(k, v, off, sel, 10000.0, k_pos_mode=0)
    assert np.array_equal(co, off)
    assert np.array_equal(vc, v)                      # V: exact copy
    pos = np.arange(off[-1], dtype=np.float64)
    assert np.allclose(kc, orc.rope(k, pos[None, :, None], 10000.0), atol=1e-13)
    # stored-rotated pool (mode 1): shot 0 has Delta = 0 and is copied exactly
    kc1, _, _ = orc.assemble_kv(k, v, off, sel, 10000.0, k_pos_mode=1)
    assert np.array_equal(kc1[:, : off[1]], k[:, : off[1]])


def test_reencoded_k_equals_fresh_rotation_bruteforce_loop():
    # python loops over every element; new position = ctx_off[r] + t
    rng = np.random.default_rng(5)
    base = 10000.0
    k, v, off = _tiny_pool(rng)
    sel = np.array([2, 0, 3, 0])                      # reordered, one duplicate
    kc, vc, co = orc.assemble_kv(k, v, off, sel, base, k_pos_mode=0)
    d = k.shape[-1]
    pos = 0
    for s in sel:
        for t in range(off[s + 1] - off[s]):
            for l in range(k.shape[0]):
                for h in range(k.shape[2]):
                    src = k[l, off[s] + t, h]
                    assert np.array_equal(vc[l, pos, h], v[l, off[s] + t, h])
                    for i in range(d // 2):
                        ang = pos * base ** (-2.0 * i / d)
                        lo = src[i] * math.cos(ang) - src[i + d // 2] * math.sin(ang)
                        hi = src[i + d // 2] * math.cos(ang) + src[i] * math.sin(ang)
                        assert abs(kc[l, pos, h, i] - lo) < 1e-12
                        assert abs(kc[l, pos, h, i + d // 2] - hi) < 1e-12
            pos += 1
    assert pos == co[-1]


def test_both_pool_conventions_agree():
    # a pool that stores K rotated at shot-local positions, corrected by the
    # shot offset (Eq. 7), gives the same cache as an un-rotated pool
    rng = np.random.default_rng(6)
    base = 500000.0
    k, v, off = _tiny_pool(rng, lens=(5, 2, 7))
    local = np.concatenate([np.arange(off[i + 1] - off[i]) for i in range(len(off) - 1)])
    k_stored = orc.rope(k, local[None, :, None].astype(np.float64), base)
    sel = np.array([1, 2, 0])
    a, _, _ = orc.assemble_kv(k, v, off, sel, base, k_pos_mode=0)
    b, _, _ = orc.assemble_kv(k_stored, v, off, sel, base, k_pos_mode=1)
    assert np.allclose(a, b, atol=1e-12)


# ------------------------------------------------------------- attention
def _tiny_attn_case(rng, P=2, Tq=3, Hq=4, Hkv=2, d=8, L=9):
    q = rng.standard_normal((P, Tq, Hq, d))
    kq = rng.standard_normal((P, Tq, Hkv, d))
    vq = rng.standard_normal((P, Tq, Hkv, d))
    kraw = rng.standard_normal((L, Hkv, d))
    vctx = rng.standard_normal((L, Hkv, d))
    return q, kq, vq, kraw, vctx


def _dense_masked_attention(q, kq, vq, kraw, vctx, L_list, base, shift=0.0):
    """Explicit-mask softmax(QK^T/sqrt d)V over [all shots ; all probes' tokens],
    python loops, written independently of attn_row."""
    P, Tq, Hq, d = q.shape
    Hkv = kq.shape[2]
    G = Hq // Hkv
    L = kraw.shape[0]
    out = np.zeros_like(q)
    for h in range(Hq):
        g = h // G
        keys, vals, owner, kpos = [], [], [], []
        for p in range(L):
            keys.append(orc.rope(kraw[p, g], p + shift, base)); vals.append(vctx[p, g])
            owner.append((-1, p)); kpos.append(p)
        for j in range(P):
            for t in range(Tq):
                keys.append(orc.rope(kq[j, t, g], L_list[j] + t + shift, base))
                vals.append(vq[j, t, g]); owner.append((j, t))
        keys, vals = np.array(keys), np.array(vals)
        for j in range(P):
            for t in range(Tq):
                qq = orc.rope(q[j, t, h], L_list[j] + t + shift, base)
                mask = np.array([(o[0] == -1 and o[1] < L_list[j]) or
                                 (o[0] == j and o[1] <= t) for o in owner])
                s = keys @ qq / math.sqrt(d)
                s = np.where(mask, s, -np.inf)
                p_ = scipy.special.softmax(s)
                out[j, t, h] = p_ @ vals
    return out


def test_attention_matches_dense_masked_bruteforce():
    rng = np.random.default_rng(7)
    base = 10000.0
    q, kq, vq, kraw, vctx = _tiny_attn_case(rng)
    L_list = [4, 9]
    pos = np.arange(kraw.shape[0], dtype=np.float64)
    kctx = orc.rope(kraw, pos[:, None], base)
    out, lse = orc.query_attn(q, kq, vq, kctx, vctx, L_list, base)
    want = _dense_masked_attention(q, kq, vq, kraw, vctx, L_list, base)
    assert np.allclose(out, want, atol=1e-12)
    # invariance to a uniform shift of every position (relative-position property)
    want_shift = _dense_masked_attention(q, kq, vq, kraw, vctx, L_list, base, shift=777.0)
    assert np.allclose(out, want_shift, atol=1e-9)


def test_attention_probe_equals_standalone_call_and_prefix_only():
    rng = np.random.default_rng(8)
    base = 10000.0
    q, kq, vq, kraw, vctx = _tiny_attn_case(rng)
    kctx = orc.rope(kraw, np.arange(9.0)[:, None], base)
    out, _ = orc.query_attn(q, kq, vq, kctx, vctx, [4, 9], base)
    solo, _ = orc.query_attn(q[:1], kq[:1], vq[:1], kctx[:4], vctx[:4], [4], base)
    assert np.allclose(out[0], solo[0], atol=1e-13)
    # probe 0 must ignore everything after its 4 context tokens
    k2, v2 = kctx.copy(), vctx.copy()
    k2[4:] += 5.0; v2[4:] -= 3.0
    out2, _ = orc.query_attn(q, kq, vq, k2, v2, [4, 9], base)
    assert np.array_equal(out2[0], out[0]) and not np.allclose(out2[1], out[1])


def test_attention_closed_forms():
    rng = np.random.default_rng(9)
    base = 10000.0
    q, kq, vq, kraw, vctx = _tiny_attn_case(rng, P=1)
    kctx = orc.rope(kraw, np.arange(9.0)[:, None], base)
    # constant V everywhere -> output is that constant (weights sum to one)
    out, _ = orc.query_attn(q, kq, np.full_like(vq, 2.5), kctx, np.full_like(vctx, 2.5), [9], base)
    assert np.allclose(out, 2.5, atol=1e-13)
    # all keys zero -> uniform weights -> plain mean over visible values; lse = ln(n)
    out, lse = orc.query_attn(q, kq * 0, vq, kctx * 0, vctx, [9], base)
    for t in range(q.shape[1]):
        for h in range(q.shape[2]):
            g = h // 2
            vis = np.concatenate([vctx[:, g], vq[0, : t + 1, g]])
            assert np.allclose(out[0, t, h], vis.mean(axis=0), atol=1e-13)
            assert abs(lse[0, h, t] - math.log(9 + t + 1)) < 1e-13
    # causal inside the query: row t ignores its later tokens
    kq2, vq2 = kq.copy(), vq.copy()
    kq2[0, 2] += 9.0; vq2[0, 2] += 9.0
    out_a, _ = orc.query_attn(q, kq, vq, kctx, vctx, [9], base)
    out_b, _ = orc.query_attn(q, kq2, vq2, kctx, vctx, [9], base)
    assert np.array_equal(out_a[0, :2], out_b[0, :2]) and not np.allclose(out_a[0, 2], out_b[0, 2])


def test_attention_scale_is_inverse_sqrt_head_dim():
    # one context key, one query token: two keys in all, weights by hand
    d, base = 4, 10000.0
    q = np.zeros((1, 1, 1, d)); q[0, 0, 0, 0] = 2.0
    kctx = np.zeros((1, 1, d)); kctx[0, 0, 0] = 3.0       # position 0: unrotated
    vctx = np.zeros((1, 1, d)); vctx[0, 0, 0] = 1.0
    kq = np.zeros((1, 1, 1, d)); vq = np.zeros((1, 1, 1, d)); vq[0, 0, 0, 1] = 1.0
    out, lse = orc.query_attn(q, kq, vq, kctx, vctx, [1], base)
    # the query sits at position 1: its first pair (2,0 | 0) rotates by theta_0 = 1 rad
    s0 = 2.0 * math.cos(1.0) * 3.0 / math.sqrt(d)
    w0 = math.exp(s0) / (math.exp(s0) + 1.0)
    assert np.allclose(out[0, 0, 0], [w0, 1 - w0, 0, 0], atol=1e-14)
    assert abs(lse[0, 0, 0] - math.log(math.exp(s0) + 1.0)) < 1e-14


def test_skipping_the_reencode_changes_the_output():
    # sensitivity (the paper's ablation without re-encoding degrades results)
    rng = np.random.default_rng(10)
    base = 10000.0
    q, kq, vq, kraw, vctx = _tiny_attn_case(rng, P=1, L=40)
    kctx = orc.rope(kraw, np.arange(40.0)[:, None], base)
    a, _ = orc.query_attn(q, kq, vq, kctx, vctx, [40], base)
    b, _ = orc.query_attn(q, kq, vq, kraw, vctx, [40], base)
    assert np.abs(a - b).max() > 5e-2


def test_gqa_head_mapping():
    rng = np.random.default_rng(11)
    base = 10000.0
    q, kq, vq, kraw, vctx = _tiny_attn_case(rng, P=1, Hq=4, Hkv=2)
    kctx = orc.rope(kraw, np.arange(9.0)[:, None], base)
    out, _ = orc.query_attn(q, kq, vq, kctx, vctx, [9], base)
    # heads 0,1 read kv head 0: expanding the KV heads to 4 gives plain MHA
    rep = lambda x: np.repeat(x, 2, axis=-2)
    out_mha, _ = orc.query_attn(q, rep(kq), rep(vq), rep(kctx), rep(vctx), [9], base)
    assert np.allclose(out, out_mha, atol=1e-13)


# ----------------------------------------------------------------- top-k
def test_cosine_against_scipy_and_python_sort():
    rng = np.random.default_rng(12)
    emb = rng.standard_normal((37, 16))
    qe = rng.standard_normal((3, 16))
    s = orc.cosine_scores(qe, emb)
    for b in range(3):
        for i in range(37):
            assert abs(s[b, i] - (1.0 - scipy.spatial.distance.cosine(qe[b], emb[i]))) < 1e-13
    sel, sc = orc.select_topk(qe, emb, 10)
    for b in range(3):
        want = sorted(range(37), key=lambda i: (-s[b, i], i))[:10]
        assert sel[b].tolist() == want
        assert np.array_equal(sc[b], s[b, want])


def test_topk_ties_self_match_and_prefix_property():
    rng = np.random.default_rng(13)
    emb = rng.standard_normal((20, 8))
    emb[11] = emb[3]; emb[17] = emb[3] * 2.0          # same direction -> same cosine
    emb[5] = 0.0                                       # zero norm -> score 0
    qe = emb[3:4].copy()
    sel, sc = orc.select_topk(qe, emb, 20)
    assert sel[0, :3].tolist() == [3, 11, 17]          # ties broken by lowest id
    assert abs(sc[0, 0] - 1.0) < 1e-15
    assert orc.cosine_scores(qe, emb)[0, 5] == 0.0
    for n in (1, 4, 9):                                # nested probes take prefixes
        assert np.array_equal(orc.select_topk(qe, emb, n)[0][0], sel[0, :n])


def test_min_adjacent_gap_on_hand_made_scores():
    # q = e_x and shot i = (s_i, sqrt(1 - s_i^2)) give cosine s_i: the sorted scores and their gaps are known
    s = np.array([0.10, 0.90, 0.50, 0.50, 0.49, 0.30, -0.20])
    emb = np.stack([s, np.sqrt(1.0 - s * s)], axis=1) * np.array([1.0, 3.0, 0.5, 2.0, 1.0, 7.0, 1.0])[:, None]
    qe = np.array([[2.0, 0.0]])
    # ranks 1..4 are 0.9, 0.5, 0.5, 0.49: the true tie is skipped, the smallest real gap is 0.01
    assert abs(orc.min_adjacent_gap(qe, emb, 3) - 0.01) < 1e-12
    assert abs(orc.min_adjacent_gap(qe, emb, 1) - 0.40) < 1e-12          # 0.9 | 0.5
    # the gap between rank k and rank k+1 counts (it decides who is selected): 0.49 | 0.30 is not reached at k = 3
    assert abs(orc.min_adjacent_gap(qe, emb, 5) - 0.01) < 1e-12
    assert abs(orc.min_adjacent_gap(qe, emb[[1, 5, 0]], 2) - 0.20) < 1e-12   # 0.9, 0.3, 0.1
    # several queries: the smallest over the batch
    q2 = np.array([[2.0, 0.0], [0.0, 1.0]])      # second query: cosines sqrt(1 - s^2)
    c2 = np.sort(np.sqrt(1.0 - emb[[1, 5, 0], 0] ** 2 / (emb[[1, 5, 0]] ** 2).sum(1)))[::-1]
    want = min(0.20, float(np.min(c2[:-1] - c2[1:])))
    assert abs(orc.min_adjacent_gap(q2, emb[[1, 5, 0]], 2) - want) < 1e-12
    # only exact ties (identical rows): nothing to report
    assert orc.min_adjacent_gap(qe, np.array([[1.0, 1.0], [1.0, 1.0], [1.0, 1.0]]), 2) == np.inf


# --------------------------------- literal tree layout (Sec. 4.1 mask equation)
def test_tree_layout_hand_example():
    # shots of 2, 1 and 3 tokens, probes after 1 and 3 shots, two probe tokens each:
    # sequence  s0 s0 | p0 p0 | s1 s2 s2 s2 | p1 p1
    off = np.array([0, 2, 3, 6])
    kind, src, pos, owner, mask = orc.tree_layout(off, [1, 3], 2)
    assert kind.tolist() == [0, 0, 1, 1, 0, 0, 0, 0, 1, 1]
    assert src.tolist() == [0, 1, 0, 1, 2, 3, 4, 5, 2, 3]
    assert pos.tolist() == [0, 1, 2, 3, 2, 3, 4, 5, 6, 7]          # shots keep 0..L-1; probe j sits at L_j + t
    want = np.zeros((10, 10), dtype=int)
    want[2, [0, 1, 2]] = 1                                          # probe 0, token 0: shot 0 and itself
    want[3, [0, 1, 2, 3]] = 1
    want[8, [0, 1, 4, 5, 6, 7, 8]] = 1                              # probe 1 sees all three shots, not probe 0
    want[9, [0, 1, 4, 5, 6, 7, 8, 9]] = 1
    assert np.array_equal(mask.astype(int), want)


def test_tree_attention_equals_per_probe_attention_row_for_row():
    rng = np.random.default_rng(41)
    lens = np.array([3, 5, 2, 4, 1, 6])
    so = np.concatenate([[0], np.cumsum(lens)])
    Hq, Hkv, d, Tq, base = 4, 2, 8, 3, 10000.0
    kp, vp = rng.standard_normal((1, int(so[-1]), Hkv, d)), rng.standard_normal((1, int(so[-1]), Hkv, d))
    sel = np.array([4, 0, 5, 2, 1])
    k_ctx, v_ctx, off = orc.assemble_kv(kp, vp, so, sel, base)
    probes = [1, 2, 5]
    q = rng.standard_normal((3, Tq, Hq, d))
    kq, vq = rng.standard_normal((3, Tq, Hkv, d)), rng.standard_normal((3, Tq, Hkv, d))
    tree = orc.tree_attention(q, kq, vq, k_ctx[0], v_ctx[0], off, probes, base)
    per_probe, _ = orc.query_attn(q, kq, vq, k_ctx[0], v_ctx[0], [int(off[n]) for n in probes], base)
    assert np.allclose(tree, per_probe, atol=1e-13)
    # the mask matters: letting probe 0 see every shot changes its rows
    full, _ = orc.query_attn(q, kq, vq, k_ctx[0], v_ctx[0], [int(off[5])] * 3, base)
    assert np.abs(full[0] - tree[0]).max() > 1e-2


def test_masked_attention_against_scipy():
    rng = np.random.default_rng(42)
    S, d = 7, 5
    qm, km, vm = rng.standard_normal((S, d)), rng.standard_normal((S, d)), rng.standard_normal((S, 3))
    mask = rng.random((S, S)) < 0.5
    mask[2] = False                                                   # a row that sees nothing
    got = orc.masked_attention(qm, km, vm, mask, 0.7)
    for i in range(S):
        if not mask[i].any():
            assert np.all(got[i] == 0.0)
            continue
        logits = np.where(mask[i], (km @ qm[i]) * 0.7, -np.inf)
        assert np.allclose(got[i], scipy.special.softmax(logits) @ vm, atol=1e-14)


def test_decode_row_is_the_last_row_of_a_longer_probe():
    rng = np.random.default_rng(43)
    L, Hkv, d, T_own, base = 11, 2, 8, 5, 10000.0
    k_ctx, v_ctx = rng.standard_normal((L + 4, Hkv, d)), rng.standard_normal((L + 4, Hkv, d))
    k_own, v_own = rng.standard_normal((T_own, Hkv, d)), rng.standard_normal((T_own, Hkv, d))
    qn = rng.standard_normal(d)
    out, lse = orc.decode_row(qn, k_own, v_own, k_ctx, v_ctx, L, 1, base)
    # the same through the dense definition: keys = context 0..L-1 and all own tokens at L..L+T_own-1
    keys = np.concatenate([k_ctx[:L, 1], orc.rope(k_own[:, 1], L + np.arange(T_own, dtype=float), base)])
    vals = np.concatenate([v_ctx[:L, 1], v_own[:, 1]])
    s = keys @ orc.rope(qn, float(L + T_own - 1), base) / math.sqrt(d)
    assert np.allclose(out, scipy.special.softmax(s) @ vals, atol=1e-14)
    assert abs(lse - scipy.special.logsumexp(s)) < 1e-13


# ------------------------------------- attention-based relevance (Eq. 5)
def _tiny_relevance_case(seed=31):
    rng = np.random.default_rng(seed)
    lens = np.array([3, 1, 5, 2, 4])
    so = np.concatenate([[0], np.cumsum(lens)])
    Tq, Hq, Hkv, d = 4, 4, 2, 8
    q = rng.standard_normal((Tq, Hq, d))
    k = rng.standard_normal((int(so[-1]), Hkv, d))
    return q, k, so, lens


def test_relevance_attention_matches_python_loops_and_scipy():
    q, k, so, lens = _tiny_relevance_case()
    Tq, Hq, d = q.shape
    G = Hq // k.shape[1]
    want = np.zeros(len(lens))
    for t in range(Tq):
        for h in range(Hq):
            logit = [sum(q[t, h, c] * k[j, h // G, c] for c in range(d)) / math.sqrt(d) for j in range(k.shape[0])]
            a = scipy.special.softmax(np.array(logit))              # over ALL pool keys
            for i in range(len(lens)):
                want[i] += a[so[i]:so[i + 1]].sum()
    want /= Tq * Hq
    got = orc.relevance_attention(q, k, so)
    assert np.allclose(got, want, atol=1e-14)
    assert abs(got.sum() - 1.0) < 1e-13                             # the masses of all shots add up to one
    assert np.allclose(orc.relevance_attention(q, k, so, per_token=True), want / lens, atol=1e-14)
    # an explicit scale replaces 1 / sqrt(d)
    assert np.allclose(orc.relevance_attention(q * 2.0, k, so, scale=0.5 / math.sqrt(d)), want, atol=1e-14)


def test_relevance_attention_closed_forms():
    q, k, so, lens = _tiny_relevance_case(32)
    # identical keys everywhere: uniform attention, a shot's mass is its share of the pool's tokens
    k_same = np.broadcast_to(k[:1], k.shape).copy()
    assert np.allclose(orc.relevance_attention(q, k_same, so), lens / lens.sum(), atol=1e-14)
    assert np.allclose(orc.relevance_attention(q, k_same, so, per_token=True), 1.0 / lens.sum(), atol=1e-15)
    # zero queries: the same uniform distribution whatever the keys
    assert np.allclose(orc.relevance_attention(q * 0.0, k, so), lens / lens.sum(), atol=1e-14)
    # a shot whose keys point along the queries (large scores) takes nearly all of the mass and ranks first
    qd = np.ones_like(q)
    k2 = k * 0.01
    k2[so[3]:so[4]] = 6.0
    s = orc.relevance_attention(qd, k2, so)
    assert s[3] > 0.999 and int(np.argmax(s)) == 3
    sel, sc = orc.select_topk_attention(qd[None], k2, so, 2)
    assert sel[0, 0] == 3 and sc[0, 0] == s[3]
    # ties go to the lower shot id: shots 0 and 4 made of the same single key repeated, equal lengths
    so_t = np.array([0, 2, 3, 5])
    k_t = np.stack([k[0], k[0], k[1], k[0], k[0]])
    sel, _ = orc.select_topk_attention(q[None], k_t, so_t, 3)
    s_t = orc.relevance_attention(q, k_t, so_t)
    assert s_t[0] == s_t[2] and list(sel[0]).index(0) < list(sel[0]).index(2)
    # GQA: head h reads KV head h // G (expanding the KV heads changes nothing)
    rep = np.repeat(k, q.shape[1] // k.shape[1], axis=1)
    assert np.allclose(orc.relevance_attention(q, rep, so), orc.relevance_attention(q, k, so), atol=1e-15)


def test_eq5_as_printed_is_degenerate():
    # softmax over one shot's own tokens (Eq. 5 as printed): every row sums to one, so the mean over all
    # entries of A^(i) is 1 / T_i for every query.  The reading taken must not behave like that.
    q, k, so, lens = _tiny_relevance_case(33)
    printed = []
    for i in range(len(lens)):
        logits = np.einsum("thd,jhd->htj", q[:, :2], k[so[i]:so[i + 1]]) / math.sqrt(q.shape[-1])
        printed.append(scipy.special.softmax(logits, axis=-1).mean())
    assert np.allclose(printed, 1.0 / lens, atol=1e-15)
    got = orc.relevance_attention(q, k, so, per_token=True)
    assert np.abs(got * lens.sum() - 1.0).max() > 0.05 and np.abs(got - 1.0 / lens).max() > 0.05


# --------------------------------------------------------------- entropy
def test_entropy_closed_forms_and_scipy():
    V = 1024
    assert abs(orc.entropy(np.zeros((1, V)))[0] - math.log(V)) < 1e-12
    assert abs(orc.entropy(np.full((1, V), -7.25))[0] - math.log(V)) < 1e-12
    x = np.zeros((1, V)); x[0, 17] = 200.0
    assert orc.entropy(x)[0] < 1e-60 + 1e-12
    # m entries at a, V - m at b
    m, a, b = 10, 1.5, -0.5
    x = np.full((1, V), b); x[0, :m] = a
    Z = m * math.exp(a) + (V - m) * math.exp(b)
    pa, pb = math.exp(a) / Z, math.exp(b) / Z
    want = -(m * pa * math.log(pa) + (V - m) * pb * math.log(pb))
    assert abs(orc.entropy(x)[0] - want) < 1e-12
    rng = np.random.default_rng(14)
    x = rng.standard_normal((5, 777)) * 3.0
    H = orc.entropy(x)
    want = scipy.stats.entropy(scipy.special.softmax(x, axis=1), axis=1)
    assert np.allclose(H, want, rtol=1e-12)
    assert np.allclose(orc.entropy(x + 123.0), H, rtol=1e-11)
    assert np.all(H >= 0) and np.all(H <= math.log(777))
    # -inf logits carry no mass and add nothing
    x2 = np.concatenate([x, np.full((5, 3), -np.inf)], axis=1)
    assert np.allclose(orc.entropy(x2), H, rtol=1e-12)


def test_threshold_rule_on_the_papers_case_study():
    rows = _rows("paper_case_study_entropies.txt")
    shots = [int(r[0]) for r in rows]
    H = np.array([float(r[1]) for r in rows])
    tau = 0.65
    ok = orc.first_ok(H, tau, 4)                       # two rounds of four probes
    assert ok.tolist() == [-1, 2]                      # round 1: none; round 2: third probe
    assert shots[4 + ok[1]] == 28                      # the count the paper selects
    # a two-way renormalised natural-log entropy cannot exceed ln 2; two printed
    # values do, which is why the hot path's entropy is over the full vocabulary
    assert (H > math.log(2)).sum() == 2


def test_probe_rounds_on_the_papers_case_study():
    rows = _rows("paper_case_study_entropies.txt")
    shots = [int(r[0]) for r in rows]
    H = np.array([float(r[1]) for r in rows])
    schedule = [shots[:4], shots[4:]]
    stops, rounds_run = orc.probe_rounds([H[None, :4], H[None, 4:]], schedule, 0.65)
    assert stops == [(1, 2, 28)] and rounds_run == 2          # the paper: second round, 28 shots
    # a second query that is satisfied by the very first probe does not shorten the batch's
    # rounds, and a query that is never satisfied reports -1
    H2 = np.stack([H, np.concatenate([[0.1], H[1:]]), np.full(8, 0.9)])
    stops, rounds_run = orc.probe_rounds([H2[:, :4], H2[:, 4:]], schedule, 0.65)
    assert stops == [(1, 2, 28), (0, 0, 4), (-1, -1, -1)] and rounds_run == 2
    # with only the satisfied query, one round is enough
    stops, rounds_run = orc.probe_rounds([H2[1:2, :4], H2[1:2, 4:]], schedule, 0.65)
    assert stops == [(0, 0, 4)] and rounds_run == 1
    # the threshold is inclusive
    stops, _ = orc.probe_rounds([np.array([[0.65, 0.2]])], [[3, 6]], 0.65)
    assert stops == [(0, 0, 3)]


def test_subset_entropy_closed_forms_and_bounds():
    rng = np.random.default_rng(5)
    V = 50
    # uniform logits: every p_v = 1/V, so n tokens give n (1/V) ln V; renormalised: ln n
    x = np.full((2, V), 0.3)
    ids = [3, 17, 44]
    assert np.allclose(orc.entropy_subset(x, ids), 3 * math.log(V) / V, rtol=1e-13)
    assert np.allclose(orc.entropy_subset(x, ids, renorm=True), math.log(3), rtol=1e-13)
    # the whole vocabulary as the subset is the full entropy, in either reading
    y = rng.normal(size=(4, V)) * 2.0
    assert np.allclose(orc.entropy_subset(y, np.arange(V)), orc.entropy(y), rtol=1e-12)
    assert np.allclose(orc.entropy_subset(y, np.arange(V), renorm=True), orc.entropy(y), rtol=1e-12)
    # two tokens with known probabilities: logits ln(0.6), ln(0.3), ln(0.1)
    z = np.log(np.array([[0.6, 0.3, 0.1]]))
    want = -(0.6 * math.log(0.6) + 0.3 * math.log(0.3))
    assert np.allclose(orc.entropy_subset(z, [0, 1]), want, rtol=1e-13)
    q = np.array([0.6, 0.3]) / 0.9
    assert np.allclose(orc.entropy_subset(z, [0, 1], renorm=True), -(q * np.log(q)).sum(), rtol=1e-13)
    assert np.allclose(orc.entropy_subset(z, [0, 1], renorm=True),
                       scipy.stats.entropy([0.6, 0.3]), rtol=1e-13)          # scipy renormalises itself
    # bounds: -p ln p <= 1/e per token; renormalised <= ln n; shift invariance
    ids2 = [1, 7]
    h = orc.entropy_subset(y, ids2)
    assert (h >= 0).all() and (h <= 2 / math.e + 1e-15).all()
    assert (orc.entropy_subset(y, ids2, renorm=True) <= math.log(2) + 1e-15).all()
    assert np.allclose(orc.entropy_subset(y + 11.0, ids2), h, rtol=1e-12)
    # the paper's printed two-token values: all within 2/e, two above ln 2 (so not renormalised nats)
    H = np.array([float(r[1]) for r in _rows("paper_case_study_entropies.txt")])
    assert (H <= 2 / math.e).all() and (H > math.log(2)).sum() == 2


# --------------------------------------------- planted mistakes are caught
PIN_TESTS = [
    test_rope_hand_value_quarter_turn, test_rope_equals_complex_rotation,
    test_rope_identity_norm_and_composition, test_two_shot_positions_golden,
    test_identity_order_reproduces_source_cache,
    test_reencoded_k_equals_fresh_rotation_bruteforce_loop,
    test_both_pool_conventions_agree,
    test_attention_matches_dense_masked_bruteforce,
    test_attention_probe_equals_standalone_call_and_prefix_only,
    test_attention_closed_forms, test_attention_scale_is_inverse_sqrt_head_dim,
    test_gqa_head_mapping, test_cosine_against_scipy_and_python_sort,
    test_topk_ties_self_match_and_prefix_property, test_min_adjacent_gap_on_hand_made_scores,
    test_tree_layout_hand_example, test_tree_attention_equals_per_probe_attention_row_for_row,
    test_masked_attention_against_scipy, test_decode_row_is_the_last_row_of_a_longer_probe,
    test_relevance_attention_matches_python_loops_and_scipy, test_relevance_attention_closed_forms,
    test_eq5_as_printed_is_degenerate,
    test_entropy_closed_forms_and_scipy, test_threshold_rule_on_the_papers_case_study,
    test_subset_entropy_closed_forms_and_bounds, test_probe_rounds_on_the_papers_case_study,
]


def _caught():
    for t in PIN_TESTS:
        try:
            t()
        except AssertionError:
            return True
        except Exception:
            return True
    return False


def _mut_rotate_half_sign(x):
    h = x.shape[-1] // 2
    return np.concatenate([x[..., h:], -x[..., :h]], axis=-1)


def _mut_rotate_half_interleaved(x):
    y = np.empty_like(x)
    y[..., 0::2] = -x[..., 1::2]
    y[..., 1::2] = x[..., 0::2]
    return y


def _mut_theta(d, base):
    i = np.arange(d // 2, dtype=np.float64)
    return np.power(np.float64(base), -1.0 * i / d)          # dropped factor 2


def _mut_plan_inclusive(sel_idx, shot_off):
    off = _ORIG["plan_offsets"](sel_idx, shot_off)
    out = off.copy()
    out[:, :-1] = off[:, 1:]                                   # inclusive, not exclusive
    return out


def _mut_entropy_log2(logits):
    return _ORIG["entropy"](logits) / math.log(2.0)


def _mut_entropy_no_max(logits):
    x = np.asarray(logits, dtype=np.float64)
    e = np.exp(x)
    p = e / e.sum(axis=-1, keepdims=True)
    return -(p * np.log(p)).sum(axis=-1)


def _mut_subset_always_renorm(logits, subset_ids, renorm=False):
    return _ORIG["entropy_subset"](logits, subset_ids, renorm=True)


def _mut_subset_local_softmax(logits, subset_ids, renorm=False):
    # softmax over the subset's logits only, never over the vocabulary
    x = np.asarray(logits, dtype=np.float64)[..., np.asarray(subset_ids)]
    e = np.exp(x - x.max(axis=-1, keepdims=True))
    p = e / e.sum(axis=-1, keepdims=True)
    return -(p * np.log(p)).sum(axis=-1)


def _mut_cosine_no_norm(q_emb, emb):
    return np.asarray(q_emb, dtype=np.float64) @ np.asarray(emb, dtype=np.float64).T


def _mut_gap_always_inf(q_emb, emb, k):
    return np.inf


def _mut_gap_counts_ties(q_emb, emb, k):
    s = _ORIG["cosine_scores"](q_emb, emb)
    top = -np.sort(-s, axis=1)[:, : k + 1]
    return float((top[:, :-1] - top[:, 1:]).min())              # a true tie gives 0


def _mut_gap_stops_at_rank_k(q_emb, emb, k):
    return _ORIG["min_adjacent_gap"](q_emb, emb, k - 1) if k > 1 else np.inf


def _mut_relevance_softmax_per_shot(q, k_layer, shot_off, per_token=False, scale=None):
    # Eq. 5 as printed: the softmax normalises over one shot's own tokens
    q = np.asarray(q, dtype=np.float64)
    k = np.asarray(k_layer, dtype=np.float64)
    so = np.asarray(shot_off)
    Tq, Hq, d = q.shape
    G = Hq // k.shape[1]
    sc = 1.0 / math.sqrt(d) if scale is None else scale
    out = np.zeros(len(so) - 1)
    for i in range(len(so) - 1):
        for h in range(Hq):
            a = scipy.special.softmax((q[:, h] @ k[so[i]:so[i + 1], h // G].T) * sc, axis=1)
            out[i] += a.sum()
    out /= Tq * Hq
    return out / (so[1:] - so[:-1]) if per_token else out


def _mut_relevance_no_scale(q, k_layer, shot_off, per_token=False, scale=None):
    return _ORIG["relevance_attention"](q, k_layer, shot_off, per_token, 1.0 if scale is None else scale)


def _mut_relevance_kv_head_zero(q, k_layer, shot_off, per_token=False, scale=None):
    k = np.asarray(k_layer, dtype=np.float64)
    return _ORIG["relevance_attention"](q, np.broadcast_to(k[:, :1], k.shape), shot_off, per_token, scale)


def _mut_relevance_inclusive_segments(q, k_layer, shot_off, per_token=False, scale=None):
    so = np.asarray(shot_off).copy()
    so[1:-1] += 1                                               # shot boundaries off by one token
    s = _ORIG["relevance_attention"](q, k_layer, so, False, scale)
    return s / (np.asarray(shot_off)[1:] - np.asarray(shot_off)[:-1]) if per_token else s


def _mut_tree_layout_probe_sees_earlier_probes(ctx_off_row, probes, t_q):
    kind, src, pos, owner, mask = _ORIG["tree_layout"](ctx_off_row, probes, t_q)
    mask = mask.copy()
    for i in np.nonzero(kind == 1)[0]:
        for c in np.nonzero(kind == 1)[0]:
            if owner[c] < owner[i]:
                mask[i, c] = True                                   # an earlier probe's tokens leak in
    return kind, src, pos, owner, mask


def _mut_tree_layout_positions_follow_the_sequence(ctx_off_row, probes, t_q):
    kind, src, pos, owner, mask = _ORIG["tree_layout"](ctx_off_row, probes, t_q)
    return kind, src, np.arange(kind.shape[0]), owner, mask        # position = index in the interleaved sequence


def _mut_tree_layout_not_causal(ctx_off_row, probes, t_q):
    kind, src, pos, owner, mask = _ORIG["tree_layout"](ctx_off_row, probes, t_q)
    mask = mask.copy()
    for i in np.nonzero(kind == 1)[0]:
        mask[i, (kind == 1) & (owner == owner[i])] = True           # a probe token sees its later tokens
    return kind, src, pos, owner, mask


def _mut_first_ok_strict(H, tau, P):
    Hm = np.asarray(H).reshape(-1, P)
    return np.array([next((j for j in range(P) if Hm[b, j] > tau), -1)
                     for b in range(Hm.shape[0])], dtype=np.int32)


def _mut_probe_rounds_lowest_entropy(H_by_round, schedule, tau):
    # takes the probe with the lowest entropy under the threshold, not the first one
    stops, rounds_run = _ORIG["probe_rounds"](H_by_round, schedule, tau)
    out = []
    for b, (r, j, n) in enumerate(stops):
        if r >= 0:
            Hr = np.asarray(H_by_round[r])[b]
            j = int(np.argmin(Hr))
            n = int(schedule[r][j])
        out.append((r, j, n))
    return out, rounds_run


def _mut_probe_rounds_runs_every_round(H_by_round, schedule, tau):
    stops, _ = _ORIG["probe_rounds"](H_by_round, schedule, tau)
    return stops, len(H_by_round)


def _mut_attn_row_factory(kind):
    def f(q_row, kq, vq, k_ctx, v_ctx, L_j, t, kv_head, base, scale=None):
        d = q_row.shape[-1]
        sc = 1.0 / math.sqrt(d) if scale is None else scale
        if kind == "scale":
            sc = 1.0 / d
        q_pos = L_j + t if kind != "qpos" else t
        q = _ORIG["rope"](np.asarray(q_row, dtype=np.float64), np.float64(q_pos), base)
        last = t + 1 if kind != "causal" else max(t, 1)
        own_pos = L_j + np.arange(last, dtype=np.float64)
        g = kv_head if kind != "gqa" else 0
        k_own = _ORIG["rope"](np.asarray(kq, dtype=np.float64)[:last, g], own_pos, base)
        lim = L_j if kind != "prefix" else k_ctx.shape[0]
        keys = np.concatenate([k_ctx[:lim, g], k_own], axis=0)
        vals = np.concatenate([v_ctx[:lim, g], np.asarray(vq)[:last, g]], axis=0)
        s = (keys @ q) * sc
        m = s.max()
        e = np.exp(s - m)
        return (e / e.sum()) @ vals, float(m + np.log(e.sum()))
    return f


_ORIG = {}


@pytest.mark.parametrize("name,mutant", [
    ("rotate_half", _mut_rotate_half_sign),
    ("rotate_half", _mut_rotate_half_interleaved),
    ("rope_theta", _mut_theta),
    ("plan_offsets", _mut_plan_inclusive),
    ("entropy", _mut_entropy_log2),
    ("entropy", _mut_entropy_no_max),
    ("entropy_subset", _mut_subset_always_renorm),
    ("entropy_subset", _mut_subset_local_softmax),
    ("cosine_scores", _mut_cosine_no_norm),
    ("min_adjacent_gap", _mut_gap_always_inf),
    ("min_adjacent_gap", _mut_gap_counts_ties),
    ("min_adjacent_gap", _mut_gap_stops_at_rank_k),
    ("relevance_attention", _mut_relevance_softmax_per_shot),
    ("relevance_attention", _mut_relevance_no_scale),
    ("relevance_attention", _mut_relevance_kv_head_zero),
    ("relevance_attention", _mut_relevance_inclusive_segments),
    ("tree_layout", _mut_tree_layout_probe_sees_earlier_probes),
    ("tree_layout", _mut_tree_layout_positions_follow_the_sequence),
    ("tree_layout", _mut_tree_layout_not_causal),
    ("first_ok", _mut_first_ok_strict),
    ("probe_rounds", _mut_probe_rounds_lowest_entropy),
    ("probe_rounds", _mut_probe_rounds_runs_every_round),
    ("attn_row", _mut_attn_row_factory("scale")),
    ("attn_row", _mut_attn_row_factory("qpos")),
    ("attn_row", _mut_attn_row_factory("causal")),
    ("attn_row", _mut_attn_row_factory("gqa")),
    ("attn_row", _mut_attn_row_factory("prefix")),
])
def test_planted_mistakes_are_caught(name, mutant, monkeypatch):
    for n in ("rope", "plan_offsets", "entropy", "entropy_subset", "probe_rounds", "cosine_scores",
              "min_adjacent_gap", "relevance_attention", "tree_layout"):
        _ORIG[n] = getattr(orc, n)
    assert not _caught(), "pins must pass on the unmodified oracle"
    monkeypatch.setattr(orc, name, mutant)
    assert _caught(), f"no pin noticed the planted mistake in {name}"
