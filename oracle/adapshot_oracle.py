"""fp64 CPU oracle for the AdapShot KV-reuse hot path.

TEST INFRASTRUCTURE ONLY.  This module is the slow, plain statement of what the
path computes, written from the paper's definitions.  Only the test-suite, the
smoke check and the CPU-baseline / reference legs of the benchmark may import
it.  It shares no code with the CUDA library and never imports the package.

Every function works on numpy float64 arrays that hold the *stored* values of
the inputs (fp32 or bf16 values widen to fp64 exactly) and accumulates in fp64.
A matmul / sort from numpy may serve as one step; nothing is blocked, fused or
reordered beyond what the cited definition states.

Pins (tests/test_oracle_pins.py) tie each function to something other than
itself: closed forms, the complex-number form of the rotation, brute-force
loops, scipy routines, the paper's two-shot position example, and the
relative-position invariance of rotary attention.

Parity status: every function here is pinned against closed forms and library
routines.  entropy_subset (the two-token form of Eq. 2, outside the hot path)
is pinned as arithmetic, but which of its two readings the paper means is not
decidable from the text: for that choice it is "parity unpinned".  The same
holds for relevance_attention (Eq. 5): as printed, the softmax runs over one
shot's own tokens, which makes every shot's mean score 1 / T_i; the function
takes the one softmax over all pool keys instead and is pinned as arithmetic
(brute force, closed forms, the printed form shown to be degenerate), while
the choice of reading is "parity unpinned".

Notation (paper, Sec. 3-4): N shots of lengths T_i, k selected shots, Hq/Hkv
heads, G = Hq/Hkv, d head_dim, T_q query tokens, L_j context length of probe j.
"""
from __future__ import annotations

import numpy as np

F64 = np.float64


# --------------------------------------------------------------------------
# Step 1: semantic relevance ranking (Sec. 4.1 "semantic relevance ranking",
# Sec. 4.2 last paragraph "rank ... in descending order and select the top k";
# the score itself is the cosine of embeddings, as the build's problem
# statement fixes it).
# --------------------------------------------------------------------------
def cosine_scores(q_emb: np.ndarray, emb: np.ndarray) -> np.ndarray:
    """s[b, i] = <q_b, e_i> / (|q_b| |e_i|); 0 where either norm is 0."""
    q = np.asarray(q_emb, dtype=F64)
    e = np.asarray(emb, dtype=F64)
    dots = q @ e.T
    qn = np.sqrt(np.sum(q * q, axis=1))
    en = np.sqrt(np.sum(e * e, axis=1))
    denom = qn[:, None] * en[None, :]
    out = np.zeros_like(dots)
    nz = denom > 0.0
    out[nz] = dots[nz] / denom[nz]
    return out


def select_topk(q_emb: np.ndarray, emb: np.ndarray, k: int):
    """Indices of the k most relevant shots per query, most relevant first.

    Equal scores are ordered by the lower shot id (a stable sort on the
    negated score).  Returns (sel_idx int32 [B, k], sel_score fp64 [B, k]).
    """
    s = cosine_scores(q_emb, emb)
    B, N = s.shape
    if not (1 <= k <= N):
        raise ValueError("k must be in 1..N")
    sel = np.empty((B, k), dtype=np.int32)
    sc = np.empty((B, k), dtype=F64)
    for b in range(B):
        order = np.argsort(-s[b], kind="stable")[:k]
        sel[b] = order
        sc[b] = s[b, order]
    return sel, sc


def min_adjacent_gap(q_emb: np.ndarray, emb: np.ndarray, k: int) -> float:
    """Smallest gap between neighbouring sorted scores among ranks 1..k+1.

    A gap of exactly 0 is a true tie (decided by shot id) and is ignored; a
    tiny non-zero gap marks a seed on which fp64 rounding order could decide.
    """
    s = cosine_scores(q_emb, emb)
    best = np.inf
    for b in range(s.shape[0]):
        top = -np.sort(-s[b])[: k + 1]
        gaps = top[:-1] - top[1:]
        gaps = gaps[gaps > 0.0]
        if gaps.size:
            best = min(best, float(gaps.min()))
    return best


# --------------------------------------------------------------------------
# Step 1, the paper's own selector (Sec. 4.2, Eq. 5 and the ranking sentence
# after it): attention of the query's Q at a representative layer against the
# cached K of every shot.  Eq. 5 as printed normalises over one shot's own
# tokens, so every row of A^(i) sums to 1 and "the average over all tokens" is
# 1 / T_i for every shot, whatever the query.  Reading taken: ONE softmax per
# query token and head over the keys of the whole pool; a shot's relevance is
# the attention mass that falls on its tokens, averaged over query tokens and
# heads (per_token=True divides by T_i as well: the mean score of one of its
# tokens).  Q and K enter as stored: no rotary rotation is applied here.
# --------------------------------------------------------------------------
def relevance_attention(q, k_layer, shot_off, per_token: bool = False, scale: float | None = None):
    """s[i] for one query.  q [T_q, Hq, d]; k_layer [pool_tokens, Hkv, d] (the pool's K at the
    representative layer); shot_off [N+1].  Query head h reads KV head h // G.  Returns fp64 [N];
    without per_token the scores sum to 1."""
    q = np.asarray(q, dtype=F64)
    k = np.asarray(k_layer, dtype=F64)
    so = np.asarray(shot_off, dtype=np.int64)
    Tq, Hq, d = q.shape
    Hkv = k.shape[1]
    G = Hq // Hkv
    sc = (1.0 / np.sqrt(F64(d))) if scale is None else F64(scale)
    N = so.shape[0] - 1
    mass = np.zeros(N, dtype=F64)
    for h in range(Hq):
        logits = (q[:, h, :] @ k[:, h // G, :].T) * sc              # [T_q, pool_tokens]
        m = logits.max(axis=1, keepdims=True)
        e = np.exp(logits - m)
        a = e / e.sum(axis=1, keepdims=True)                        # one softmax over the whole pool
        for i in range(N):
            mass[i] += a[:, so[i]:so[i + 1]].sum()
    s = mass / F64(Tq * Hq)
    if per_token:
        s = s / (so[1:] - so[:-1]).astype(F64)
    return s


def select_topk_attention(q, k_layer, shot_off, k: int, per_token: bool = False, scale: float | None = None):
    """Top-k by relevance_attention for a batch: q [B, T_q, Hq, d].  Ties -> lower shot id.
    Returns (sel_idx int32 [B, k], score fp64 [B, k])."""
    q = np.asarray(q, dtype=F64)
    B = q.shape[0]
    N = np.asarray(shot_off).shape[0] - 1
    if not (1 <= k <= N):
        raise ValueError("k must be in 1..N")
    sel = np.empty((B, k), dtype=np.int32)
    sc = np.empty((B, k), dtype=F64)
    for b in range(B):
        s = relevance_attention(q[b], k_layer, shot_off, per_token, scale)
        order = np.argsort(-s, kind="stable")[:k]
        sel[b] = order
        sc[b] = s[order]
    return sel, sc


# --------------------------------------------------------------------------
# Step 2: destination offsets (Sec. 4.3, two-shot example: shot B placed after
# shot A occupies positions T_A .. T_A+T_B-1, its offset is Delta = T_A).
# --------------------------------------------------------------------------
def plan_offsets(sel_idx: np.ndarray, shot_off: np.ndarray) -> np.ndarray:
    """ctx_off[b, r] = sum of the lengths of the first r selected shots."""
    sel = np.asarray(sel_idx)
    so = np.asarray(shot_off, dtype=np.int64)
    B, k = sel.shape
    ctx_off = np.zeros((B, k + 1), dtype=np.int64)
    for b in range(B):
        for r in range(k):
            s = int(sel[b, r])
            ctx_off[b, r + 1] = ctx_off[b, r] + (so[s + 1] - so[s])
    return ctx_off


# --------------------------------------------------------------------------
# Step 3: rotary encoding and re-encoding (Sec. 4.3, Eq. 6 and Eq. 7).
# --------------------------------------------------------------------------
def rope_theta(d: int, base: float) -> np.ndarray:
    """theta_i = base^(-2i/d), i = 0 .. d/2-1 (text after Eq. 6)."""
    i = np.arange(d // 2, dtype=F64)
    return np.power(F64(base), -2.0 * i / F64(d))


def rotate_half(x: np.ndarray) -> np.ndarray:
    """Half-split convention of the evaluated model families:
    rotate_half(x) = [-x_{d/2..d-1}, x_{0..d/2-1}]."""
    h = x.shape[-1] // 2
    return np.concatenate([-x[..., h:], x[..., :h]], axis=-1)


def rope(x: np.ndarray, p, base: float) -> np.ndarray:
    """Eq. 6: RoPE(x, p) = x * cos(p theta) + rotate_half(x) * sin(p theta).

    x [..., d]; p broadcastable to x.shape[:-1].  The d/2 angles are repeated
    over both halves of the vector.  Eq. 7 is the same map with p = Delta.
    """
    x = np.asarray(x, dtype=F64)
    d = x.shape[-1]
    th = rope_theta(d, base)
    ang = np.asarray(p, dtype=F64)[..., None] * th
    c = np.concatenate([np.cos(ang), np.cos(ang)], axis=-1)
    s = np.concatenate([np.sin(ang), np.sin(ang)], axis=-1)
    return x * c + rotate_half(x) * s


def assemble_kv(k_pool, v_pool, shot_off, sel_row, base: float, k_pos_mode: int = 0):
    """Concatenate the selected shots' cached K/V in selection order and move K
    to its new contiguous positions (Sec. 4.3; Eq. 7).

    k_pool, v_pool : [n_layers, pool_tokens, Hkv, d]
    sel_row        : [k] shot ids of ONE query, most relevant first
    k_pos_mode 0   : pool K carries no position; the rotation angle of the
                     token at new position o+t is (o+t) theta.
    k_pos_mode 1   : pool K was rotated at its shot-local position t when the
                     shot was prefilled alone from position 0, so the
                     correction is Delta = o for the whole shot (Eq. 7).
    V is copied unchanged.  Returns (k_ctx, v_ctx [n_layers, L, Hkv, d], ctx_off [k+1]).
    """
    k_pool = np.asarray(k_pool, dtype=F64)
    v_pool = np.asarray(v_pool, dtype=F64)
    so = np.asarray(shot_off, dtype=np.int64)
    ctx_off = plan_offsets(np.asarray(sel_row)[None, :], so)[0]
    n_layers, _, hkv, d = k_pool.shape
    L = int(ctx_off[-1])
    k_ctx = np.zeros((n_layers, L, hkv, d), dtype=F64)
    v_ctx = np.zeros((n_layers, L, hkv, d), dtype=F64)
    for r, s in enumerate(np.asarray(sel_row)):
        a, b = int(so[s]), int(so[s + 1])
        o = int(ctx_off[r])
        T = b - a
        t = np.arange(T, dtype=F64)
        delta = (o + t) if k_pos_mode == 0 else np.full(T, F64(o))
        # delta is per token; broadcast over layers and heads
        k_ctx[:, o:o + T] = rope(k_pool[:, a:b], delta[None, :, None], base)
        v_ctx[:, o:o + T] = v_pool[:, a:b]
    return k_ctx, v_ctx, ctx_off


# --------------------------------------------------------------------------
# Step 4: probe attention (Eq. 1 context; tree mask of Sec. 4.1: probe j sees
# its first n_j shots and, causally, its own tokens; scale 1/sqrt(d) of Eq. 5).
# --------------------------------------------------------------------------
def attn_row(q_row, kq, vq, k_ctx, v_ctx, L_j: int, t: int, kv_head: int,
             base: float, scale: float | None = None):
    """One output row: probe token t (position L_j + t), one query head.

    q_row [d] un-rotated query vector of that head;  kq, vq [T_q, Hkv, d]
    un-rotated keys / values of the probe's own tokens;  k_ctx, v_ctx
    [L, Hkv, d] assembled cache of one layer (K already at positions 0..L-1).
    Returns (out [d], lse) with lse = log sum exp of the scaled scores.
    """
    d = q_row.shape[-1]
    sc = (1.0 / np.sqrt(F64(d))) if scale is None else F64(scale)
    q = rope(np.asarray(q_row, dtype=F64), F64(L_j + t), base)
    own_pos = L_j + np.arange(t + 1, dtype=F64)
    k_own = rope(np.asarray(kq, dtype=F64)[: t + 1, kv_head], own_pos, base)
    keys = np.concatenate([np.asarray(k_ctx, dtype=F64)[:L_j, kv_head], k_own], axis=0)
    vals = np.concatenate([np.asarray(v_ctx, dtype=F64)[:L_j, kv_head],
                           np.asarray(vq, dtype=F64)[: t + 1, kv_head]], axis=0)
    s = (keys @ q) * sc
    m = s.max()
    e = np.exp(s - m)
    z = e.sum()
    return (e / z) @ vals, float(m + np.log(z))


def query_attn(q, kq, vq, k_ctx, v_ctx, L_list, base: float, scale: float | None = None):
    """All rows of all probes of one query at one layer.

    q [P, T_q, Hq, d];  kq, vq [P, T_q, Hkv, d];  k_ctx, v_ctx [L, Hkv, d];
    L_list[j] = context length of probe j.  Query head h reads KV head h // G.
    Returns (out [P, T_q, Hq, d], lse [P, Hq, T_q]).
    """
    q = np.asarray(q, dtype=F64)
    P, Tq, Hq, d = q.shape
    Hkv = np.asarray(kq).shape[2]
    G = Hq // Hkv
    out = np.zeros((P, Tq, Hq, d), dtype=F64)
    lse = np.zeros((P, Hq, Tq), dtype=F64)
    for j in range(P):
        for h in range(Hq):
            for t in range(Tq):
                o, l = attn_row(q[j, t, h], kq[j], vq[j], k_ctx, v_ctx,
                                int(L_list[j]), t, h // G, base, scale)
                out[j, t, h] = o
                lse[j, h, t] = l
    return out, lse


# --------------------------------------------------------------------------
# Step 4 in the paper's literal form (Sec. 4.1, "tree-structured attention"): ONE
# sequence [shot_1 .. shot_n1, probe_1, shot_n1+1 .. shot_n2, probe_2, ...] and a
# mask M.  The printed mask says which shots a probe sees; causality inside a
# probe and the probe's view of its own tokens are added here as they must be for
# the rows to equal Eq. 1 run alone.  Position ids: a shot keeps the position it
# has in the plain concatenation of the shots (0 .. L-1, whatever probes are
# interleaved), probe j's tokens sit at L_j + t.
# --------------------------------------------------------------------------
def tree_layout(ctx_off_row, probes, t_q: int):
    """Token table of the interleaved sequence of one query.

    ctx_off_row [k+1] offsets of the selected shots; probes ascending shot counts n_1 < ... < n_m.
    Returns (kind [S] 0 = shot token / 1 = probe token, src [S] index into the assembled cache
    (shot tokens) or j * t_q + t (probe tokens), pos [S] position ids, owner [S] shot slot r or
    probe j, mask [S, S] bool: mask[i, c] = token i attends to token c)."""
    off = np.asarray(ctx_off_row, dtype=np.int64)
    kind, src, pos, owner = [], [], [], []
    prev = 0
    for j, n_j in enumerate(probes):
        for r in range(prev, n_j):                      # the shots this probe adds
            for p in range(int(off[r]), int(off[r + 1])):
                kind.append(0); src.append(p); pos.append(p); owner.append(r)
        L_j = int(off[n_j])
        for t in range(t_q):
            kind.append(1); src.append(j * t_q + t); pos.append(L_j + t); owner.append(j)
        prev = n_j
    kind, src, pos, owner = (np.asarray(a, dtype=np.int64) for a in (kind, src, pos, owner))
    S = kind.shape[0]
    mask = np.zeros((S, S), dtype=bool)
    for i in range(S):
        if kind[i] != 1:
            continue                                    # shot tokens were prefilled alone: no row is computed
        n_i = probes[int(owner[i])]
        for c in range(S):
            if kind[c] == 0:
                mask[i, c] = owner[c] < n_i             # M_ij = 1 iff shot j is among the probe's first n_k
            else:
                mask[i, c] = owner[c] == owner[i] and src[c] <= src[i]    # its own tokens, causally
    return kind, src, pos, owner, mask


def masked_attention(q_rows, keys, vals, mask, scale: float):
    """Dense attention with an explicit mask: out[i] = softmax_c(q_i . k_c * scale | mask[i, c]) . v_c.
    q_rows [S, d], keys [S, d], vals [S, dv], mask [S, S]; rows without any visible key give zeros."""
    q = np.asarray(q_rows, dtype=F64)
    k = np.asarray(keys, dtype=F64)
    v = np.asarray(vals, dtype=F64)
    out = np.zeros((q.shape[0], v.shape[1]), dtype=F64)
    for i in range(q.shape[0]):
        vis = np.nonzero(mask[i])[0]
        if vis.size == 0:
            continue
        s = (k[vis] @ q[i]) * scale
        e = np.exp(s - s.max())
        out[i] = (e / e.sum()) @ v[vis]
    return out


def tree_attention(q, kq, vq, k_ctx, v_ctx, ctx_off_row, probes, base: float, scale: float | None = None):
    """All probe rows of one query at one layer through the single interleaved sequence and its
    dense mask.  Arguments as query_attn (q [P, T_q, Hq, d], kq / vq [P, T_q, Hkv, d], k_ctx / v_ctx
    [L, Hkv, d] assembled cache); returns out [P, T_q, Hq, d]."""
    q = np.asarray(q, dtype=F64)
    P, Tq, Hq, d = q.shape
    Hkv = np.asarray(kq).shape[2]
    G = Hq // Hkv
    sc = (1.0 / np.sqrt(F64(d))) if scale is None else F64(scale)
    kind, src, pos, owner, mask = tree_layout(ctx_off_row, probes, Tq)
    is_probe = kind == 1
    out = np.zeros((P, Tq, Hq, d), dtype=F64)
    kq_flat = np.asarray(kq, dtype=F64).reshape(P * Tq, Hkv, d)
    vq_flat = np.asarray(vq, dtype=F64).reshape(P * Tq, Hkv, d)
    q_flat = q.reshape(P * Tq, Hq, d)
    for h in range(Hq):
        g = h // G
        keys = np.zeros((kind.shape[0], d), dtype=F64)
        vals = np.zeros((kind.shape[0], d), dtype=F64)
        keys[~is_probe] = np.asarray(k_ctx, dtype=F64)[src[~is_probe], g]          # already at their positions
        vals[~is_probe] = np.asarray(v_ctx, dtype=F64)[src[~is_probe], g]
        keys[is_probe] = rope(kq_flat[src[is_probe], g], pos[is_probe].astype(F64), base)
        vals[is_probe] = vq_flat[src[is_probe], g]
        qr = np.zeros((kind.shape[0], d), dtype=F64)
        qr[is_probe] = rope(q_flat[src[is_probe], h], pos[is_probe].astype(F64), base)
        o = masked_attention(qr, keys, vals, mask, sc)
        out[:, :, h, :] = o[is_probe].reshape(P, Tq, d)
    return out


def decode_row(q_new, k_own, v_own, k_ctx, v_ctx, L: int, kv_head: int, base: float, scale: float | None = None):
    """One decode step after probing (Sec. 4.1: the chosen shots are "used for subsequent formal
    inference"): the newest of T_own own tokens (query tokens plus what has been generated, at
    positions L .. L+T_own-1) attends to the L context tokens of the chosen prefix and to all own
    tokens.  q_new [d] un-rotated; k_own, v_own [T_own, Hkv, d] un-rotated.  Returns (out [d], lse)."""
    T_own = np.asarray(k_own).shape[0]
    return attn_row(q_new, k_own, v_own, k_ctx, v_ctx, L, T_own - 1, kv_head, base, scale)


# --------------------------------------------------------------------------
# Step 5: confidence probe (Eq. 2, taken over the whole vocabulary; natural
# log; the threshold rule of the paragraph after Eq. 2).
# --------------------------------------------------------------------------
def entropy(logits: np.ndarray) -> np.ndarray:
    """H_r = -sum_v p_v ln p_v with p = softmax(logits_r); p = 0 terms add 0."""
    x = np.asarray(logits, dtype=F64)
    m = x.max(axis=-1, keepdims=True)
    e = np.exp(x - m)
    p = e / e.sum(axis=-1, keepdims=True)
    with np.errstate(divide="ignore", invalid="ignore"):
        terms = np.where(p > 0.0, p * np.log(p), 0.0)
    return -terms.sum(axis=-1)


def entropy_subset(logits: np.ndarray, subset_ids, renorm: bool = False) -> np.ndarray:
    """Eq. 2 as printed: the sum runs over a token subset S (the paper's {Yes, No}).

    renorm False: p = softmax over the whole vocabulary, H = -sum_{v in S} p_v ln p_v.
    renorm True : q = p restricted to S and renormalised, H = -sum q ln q.
    (The paper does not say which; two of its printed case-study values exceed ln 2,
    which a renormalised two-token entropy in nats cannot reach.)
    """
    x = np.asarray(logits, dtype=F64)
    ids = np.asarray(subset_ids, dtype=np.int64)
    m = x.max(axis=-1, keepdims=True)
    e = np.exp(x - m)
    p = e / e.sum(axis=-1, keepdims=True)
    ps = p[..., ids]
    if renorm:
        ps = ps / ps.sum(axis=-1, keepdims=True)
    with np.errstate(divide="ignore", invalid="ignore"):
        t = np.where(ps > 0.0, ps * np.log(ps), 0.0)
    return -t.sum(axis=-1)


def probe_rounds(H_by_round, schedule, tau: float):
    """Multi-round probing (Sec. 4.1; the case study of Sec. 5 runs it with rounds 4..16 and
    20..32 and tau = 0.65): rounds are probed in order, and a query's answer is the first
    shot count, in schedule order, whose entropy is at most tau.
    H_by_round[r] is [B][m] (entropies of round r's m probes), schedule[r] the m shot
    counts.  Returns per query (round, probe index, shot count), (-1, -1, -1) when no probe
    meets the threshold, and the number of rounds that had to be run for the whole batch."""
    B = np.asarray(H_by_round[0], dtype=F64).shape[0]
    stops = [(-1, -1, -1)] * B
    rounds_run = 0
    for r, Hr in enumerate(H_by_round):
        rounds_run = r + 1
        Hr = np.asarray(Hr, dtype=F64)
        for b in range(B):
            if stops[b][0] >= 0:
                continue
            for j in range(Hr.shape[1]):
                if Hr[b, j] <= tau:
                    stops[b] = (r, j, int(schedule[r][j]))
                    break
        if all(s[0] >= 0 for s in stops):
            break
    return stops, rounds_run


def first_ok(H: np.ndarray, tau: float, P: int) -> np.ndarray:
    """Per group of P nested probes: index of the first probe with H <= tau,
    -1 if none (the minimum shot count that satisfies the threshold)."""
    Hm = np.asarray(H, dtype=F64).reshape(-1, P)
    out = np.full(Hm.shape[0], -1, dtype=np.int32)
    for b in range(Hm.shape[0]):
        for j in range(P):
            if Hm[b, j] <= tau:
                out[b] = j
                break
    return out
