"""Test helpers: run the CUDA path through the binding; widen inputs for the oracle."""
from __future__ import annotations

import numpy as np
import torch

from paper_2605_03644_b200 import workloads as wl


def gpu_binding():
    from paper_2605_03644_b200 import binding
    return binding


def dev_pool(ab, pool, device="cuda"):
    so = torch.from_numpy(pool["shot_off"]).to(device)
    return ab.Pool(so, pool["k"].to(device), pool["v"].to(device), pool["emb"].to(device))


def model_of(ab, w: wl.Workload, n_layers=None, k_pos_mode=0):
    return ab.make_model(w.n_layers if n_layers is None else n_layers, w.n_q_heads, w.n_kv_heads,
                         w.head_dim, w.dtype, w.rope_base, k_pos_mode)


def new_status(device="cuda"):
    return torch.zeros(1, dtype=torch.int32, device=device)


def run_select(ab, dpool, q_emb, k):
    B = q_emb.shape[0]
    sel = torch.full((B, k), -1, dtype=torch.int32, device="cuda")
    score = torch.zeros((B, k), dtype=torch.float32, device="cuda")
    ws = torch.empty(max(ab.adapshot_select_workspace_bytes(dpool.c.n_shots, B, k), 256),
                     dtype=torch.uint8, device="cuda")
    st = new_status()
    ab.adapshot_select(dpool, q_emb.cuda(), k, sel, score, ws, st)
    torch.cuda.synchronize()
    return sel, score, int(st.item())


def run_assemble(ab, model, dpool, sel, ctx_cap, layer_begin, layer_end, dtype, canary=True):
    B, k = sel.shape
    nl = layer_end - layer_begin
    hkv, d = model.n_kv_heads, model.head_dim
    kc = torch.full((B, nl, ctx_cap, hkv, d), 7.0, dtype=dtype, device="cuda")
    vc = torch.full((B, nl, ctx_cap, hkv, d), 7.0, dtype=dtype, device="cuda")
    off = torch.full((B, k + 1), -1, dtype=torch.int64, device="cuda")
    st = new_status()
    ab.adapshot_assemble_kv(model, dpool, sel, layer_begin, layer_end, kc, vc, ctx_cap, off, st)
    torch.cuda.synchronize()
    return kc, vc, off, int(st.item())


def run_entropy(ab, logits, tau, rows_per_group, want_first=True):
    R, V = logits.shape
    H = torch.full((R,), -1.0, dtype=torch.float32, device="cuda")
    fo = torch.full((R // rows_per_group,), -7, dtype=torch.int32, device="cuda") if want_first else None
    ws = torch.empty(max(ab.adapshot_entropy_workspace_bytes(R, V), 256), dtype=torch.uint8, device="cuda")
    st = new_status()
    ab.adapshot_entropy(logits, H, tau, rows_per_group, fo, ws, st)
    torch.cuda.synchronize()
    return H, fo, int(st.item())


def run_attn(ab, model, kc, vc, ctx_cap, off, k, probes, q, kq, vq, layer_begin, layer_end, want_lse=True):
    B, nl, P, Tq, Hq, d = q.shape
    out = torch.full_like(q, 9.0)
    lse = torch.zeros((B, nl, P, Hq, Tq), dtype=torch.float32, device="cuda") if want_lse else None
    ws = torch.empty(max(ab.adapshot_attn_workspace_bytes(model, B, P, Tq, nl, ctx_cap), 256),
                     dtype=torch.uint8, device="cuda")
    st = new_status()
    ab.adapshot_query_attn(model, kc, vc, ctx_cap, off, k, probes, q, kq, vq, layer_begin, layer_end,
                           out, lse, ws, st)
    torch.cuda.synchronize()
    return out, lse, int(st.item())


# Tolerances of the bf16 attention output against the fp64 oracle.  The stated bounds (max-abs 2e-2,
# mean-abs 2e-3) are for outputs of order one, which is what contexts of thousands of keys give.
# The result itself is stored as bf16: a value x is rounded by up to half a bf16 step, 2^-8 |x|
# (2^-9 |x| on average), so for |x| > 1 that rounding alone approaches the absolute bound (1.6e-2 at
# |x| = 4, reached when a probe averages only a handful of values).  Tests of short contexts allow
# the result's own rounding on top of the stated bounds, element by element; the tests at the
# benchmark configurations use the stated bounds alone (own_rounding=False).
ATTN_MAX_ABS, ATTN_MEAN_ABS = 2e-2, 2e-3
BF16_HALF_STEP = 2.0 ** -8
# The log-sum-exp output has no stated bound.  It inherits the error of the scores, which comes from
# rounding the rotated q and the probe's own rotated k to bf16 (2^-9 relative per element): a few
# 1e-3 on scores of magnitude 1-4, and proportional to the magnitude of the keys.
LSE_ABS = 1e-2


def attn_errors(got, want, own_rounding=True):
    """(largest excess over the element-wise bound, mean error, mean bound) of an attention output."""
    got = np.asarray(got, dtype=np.float64)
    want = np.asarray(want, dtype=np.float64)
    err = np.abs(got - want)
    mag = np.abs(want) if own_rounding else np.zeros_like(want)
    excess = float((err - (ATTN_MAX_ABS + BF16_HALF_STEP * mag)).max())
    return excess, float(err.mean()), float(ATTN_MEAN_ABS + 0.5 * BF16_HALF_STEP * mag.mean())


def assert_attn_close(got, want, own_rounding=True, what=""):
    excess, mean_err, mean_bound = attn_errors(got, want, own_rounding)
    assert excess <= 0.0, (what, "max-abs bound exceeded by", excess)
    assert mean_err <= mean_bound, (what, "mean-abs", mean_err, ">", mean_bound)


def lse_bound(k_gain: float = 1.0) -> float:
    """Absolute bound of the log-sum-exp output for keys `k_gain` times the configurations' magnitude."""
    return LSE_ABS * k_gain


def bf16_ulp_diff(a: torch.Tensor, b: torch.Tensor) -> torch.Tensor:
    """Distance in bf16 code points between two bf16 tensors (sign-magnitude order)."""
    def key(t):
        i = t.contiguous().view(torch.int16).to(torch.int32)
        return torch.where(i < 0, -(i & 0x7fff), i)
    return (key(a) - key(b)).abs()


f64 = wl.to_f64


def golden(name: str) -> str:
    """Path of a fixture under tests/golden."""
    import os
    return os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden", name)
