#!/usr/bin/env python
"""Benchmark of the AdapShot KV-reuse hot path on B200.

One "step" = one pass of the whole path (select -> plan -> gather + RoPE re-encode ->
probe attention -> entropy, all layers) over one batch of seeded synthetic queries.
Metric: reused-context tokens/s = sum over queries of the assembled context length
of the longest probe, per second of the whole step.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload cfg2] [--impl reference]

N > 1 (launched by torch.distributed.run) runs independent replicas: the path has
no exchange step, so ranks share nothing but the start/stop barrier ("weak" scaling).
`--impl reference` times the CPU oracle on a bounded sample of the same workload.
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np
import torch

from paper_2605_03644_b200 import workloads as wl

METRIC = "reused-context tokens/s (select+re-encode+query attn)"
UNIT = "tokens/s"
L2_FLUSH_BYTES = 512 << 20


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {"hbm_gbs": float(p["hbm_gbs"]), "bf16_tflops": float(p["bf16_tflops"]),
                "bf16_tflops_sustained": float(p.get("bf16_tflops_sustained", p["bf16_tflops"])),
                "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


class ClockSampler:
    """Samples SM clock and throttle reasons through NVML while the timed region runs."""

    def __init__(self, index: int, period_s: float = 0.02):
        self.index, self.period, self.samples, self.reasons = index, period_s, [], set()
        self.max_mhz, self._stop, self._thr, self.nv = None, threading.Event(), None, None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
        except Exception:
            self.nv = None

    def _loop(self):
        nv = self.nv
        names = {
            "hw_slowdown": getattr(nv, "nvmlClocksEventReasonHwSlowdown", 0x8),
            "hw_thermal_slowdown": getattr(nv, "nvmlClocksEventReasonHwThermalSlowdown", 0x40),
            "sw_thermal_slowdown": getattr(nv, "nvmlClocksEventReasonSwThermalSlowdown", 0x20),
            "sw_power_cap": getattr(nv, "nvmlClocksEventReasonSwPowerCap", 0x4),
            "hw_power_brake": getattr(nv, "nvmlClocksEventReasonHwPowerBrakeSlowdown", 0x80),
        }
        while not self._stop.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                try:
                    mask = nv.nvmlDeviceGetCurrentClocksEventReasons(self.h)
                except Exception:
                    mask = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                for n, bit in names.items():
                    if mask & bit:
                        self.reasons.add(n)
            except Exception:
                pass
            self._stop.wait(self.period)

    def __enter__(self):
        if self.nv is not None:
            self._thr = threading.Thread(target=self._loop, daemon=True)
            self._thr.start()
        return self

    def __exit__(self, *a):
        self._stop.set()
        if self._thr is not None:
            self._thr.join()

    def summary(self):
        if not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons), "samples": 0}
        return {"sm_mhz": float(np.median(self.samples)), "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(self.samples)}


HEADLINE = "cfg5"            # the largest 8B-shape configuration that fits one GPU
SUB_WORKLOADS = ("cfg2", "cfg3")   # reported beside it in the default run, each with its own roofline / clocks / e2e

# dram__bytes_read.sum + dram__bytes_write.sum per launch, from the ncu captures summarised under
# profiles/ (file named beside each figure).  A capture of a few layers / queries is scaled to a full
# launch by the units it holds: (query, layer, kv head) units are independent and equally sized on
# average, so the traffic grows in proportion.  None = no capture of the kernel as it stands.
NCU_TRAFFIC = {
    # workload: (attn_main bytes per captured launch, layers x queries in that capture,
    #            gather bytes per captured launch, layers x queries in that capture), for the variant
    #            that `--variant auto` picks for the workload
    "cfg2": (102.0e6, 1, 119.6e6, 1),             # profiles/attn_main_kernel_cfg2.md, profiles/gather_rope_kernel.md
    "cfg3": (2.2323e9, 16, 2.113e9, 16),          # profiles/attn_main_kernel_cfg3_2layers.md (2 layers x 8 queries, K-only cache)
    "cfg5": (2.049e9, 4, 1.0660e9, 4),            # profiles/attn_main_and_gather_cfg5_1layer_4queries.md (K-only cache)
}


def resolve_workload(name: str, n_layers: int = 0, n_queries: int = 0) -> wl.Workload:
    w = wl.CONFIGS[name]
    if n_layers:          # a stated smaller case of the same shape (profiling captures)
        w = w.scaled(n_layers=min(w.n_layers, n_layers))
    if n_queries:
        w = w.scaled(batch=min(w.batch, n_queries))
    return w


def resolve_k_by_budget(ab, dpool, q_emb, w: wl.Workload, lengths: np.ndarray) -> wl.Workload:
    """cfg4 names a token budget, not a shot count: k = the longest similarity-ordered prefix whose
    total length stays within the budget (query 0 decides; fixed at set-up, outside the timed region)."""
    dev = q_emb.device
    n = int(dpool.c.n_shots)
    sel = torch.empty((w.batch, n), dtype=torch.int32, device=dev)
    st = torch.zeros(1, dtype=torch.int32, device=dev)
    ws = torch.empty(max(256, ab.adapshot_select_workspace_bytes(n, w.batch, n)), dtype=torch.uint8, device=dev)
    ab.adapshot_select(dpool, q_emb, n, sel, None, ws, st)
    torch.cuda.synchronize()
    order = sel[0].cpu().numpy()
    k = int(np.searchsorted(np.cumsum(lengths[order]), w.ctx_token_limit, side="right"))
    return w.scaled(k=k, probes=(k,))


def layers_per_call_for(w: wl.Workload, ctx_cap: int, device_bytes: float = 0.0, k_only: bool = False) -> int:
    """Layers assembled and attended per call: as many as fit beside the pool, the query-side
    tensors (three times over: device inputs, their end-to-end copies, outputs) and the workspaces,
    at most 36 GB of assembled K + V (k_only: the cache holds K alone).  device_bytes: the GPU's
    memory (asked of the current device when 0; 184e9 without one)."""
    if device_bytes <= 0:
        device_bytes = (float(torch.cuda.get_device_properties(torch.cuda.current_device()).total_memory)
                        if torch.cuda.is_available() else 184e9)
    n_tok = float(wl.shot_lengths(w).sum())
    pool_bytes = n_tok * w.bytes_per_token_layer * w.n_layers
    q_bytes = (w.batch * w.n_layers * max(1, len(w.probes)) * w.t_q * (w.n_q_heads + 2 * w.n_kv_heads)
               * w.head_dim * w.elem_size)
    per_layer = float(w.batch) * ctx_cap * w.bytes_per_token_layer * (0.5 if k_only else 1.0)
    budget = min(36e9, 0.6 * (device_bytes - pool_bytes - 3.0 * q_bytes))
    # at least four chunks where there are layers for it: a caller whose tensors live in host memory
    # has chunk i + 1 on its way up and chunk i - 1 on its way down while chunk i is computed
    return int(max(1, min(w.n_layers, budget // per_layer, max(1, -(-w.n_layers // 4)))))


def choose_variant(w: wl.Workload, ctx_cap: int, variant: str = "auto", layers_per_call: int = 0):
    """(vpool, layers per call) of a run.  auto (the rule of ReusePath(vpool=None)): the K-only cache, V taken
    from the pool, when the full cache of one call would be larger than L2 and a KV head has at most 1024 query
    rows (with more rows the gather is a small share of the call and the dearer V tiles cost more than half a
    gather saves); the full cache otherwise."""
    vpool = variant == "vpool"
    if variant == "auto":
        lpc_full = layers_per_call or layers_per_call_for(w, ctx_cap)
        vpool = (w.batch * lpc_full * ctx_cap * w.bytes_per_token_layer > (128 << 20)
                 and w.t_q * w.group <= 1024)
    return vpool, (layers_per_call or layers_per_call_for(w, ctx_cap, k_only=vpool))


def planned_ctx_cap(ab, dpool, q_emb, w: wl.Workload) -> int:
    """Capacity of the assembled cache: the longest planned context (selection + plan-only
    call of the library), rounded up to the 128-token tile the attention kernel reads."""
    dev = q_emb.device
    sel = torch.empty((w.batch, w.k), dtype=torch.int32, device=dev)
    off = torch.empty((w.batch, w.k + 1), dtype=torch.int64, device=dev)
    st = torch.zeros(1, dtype=torch.int32, device=dev)
    ws = torch.empty(max(256, ab.adapshot_select_workspace_bytes(dpool.c.n_shots, w.batch, w.k)),
                     dtype=torch.uint8, device=dev)
    model = ab.make_model(w.n_layers, w.n_q_heads, w.n_kv_heads, w.head_dim, w.dtype, w.rope_base)
    ab.adapshot_select(dpool, q_emb, w.k, sel, None, ws, st)
    ab.adapshot_assemble_kv(model, dpool, sel, 0, 1, None, None, 0, off, st)
    torch.cuda.synchronize()
    if st.item() != 0:
        raise SystemExit(f"device status {st.item()} while planning")
    return int(-(-int(off[:, -1].max().item()) // 128) * 128)


def algorithmic_counts(w: wl.Workload, ctx_off: np.ndarray, n_layers: int):
    """Algorithmic bytes / flops of one step from the plan: 2 x bpt bytes per context token and layer
    for the gather, 4 Hq d flops per (query token, key) and layer for attention."""
    L = ctx_off[:, -1].astype(np.float64)                         # longest probe per query
    Lj = np.stack([ctx_off[:, n] for n in w.probes], axis=1).astype(np.float64)
    bpt = w.bytes_per_token_layer
    gather_bytes = float(L.sum()) * bpt * 2 * n_layers            # read + write, K and V
    attn_flops = float((4.0 * w.t_q * (Lj + (w.t_q + 1) / 2.0) * w.n_q_heads * w.head_dim).sum()) * n_layers
    attn_kv_bytes = float(L.sum()) * bpt * n_layers               # K/V of the longest probe read once
    R = w.batch * len(w.probes)
    entropy_bytes = float(R) * w.vocab * (4 if w.logits_dtype == "fp32" else 2)
    select_bytes = float(wl.shot_lengths(w).size) * w.emb_dim * 4
    return {"ctx_tokens": float(L.sum()), "gather_bytes": gather_bytes, "attn_flops": attn_flops,
            "attn_kv_bytes": attn_kv_bytes, "entropy_bytes": entropy_bytes, "select_bytes": select_bytes}


# ------------------------------------------------------------------ CPU oracle legs
def oracle_sample_seconds(w: wl.Workload, pool, qs, row_stride: int):
    """Times the oracle, as it stands, on a bounded sample of the workload: select,
    offsets, assemble and entropy in full for query 0 / layer 0, attention on every
    `row_stride`-th (probe, head, token) row; returns (seconds scaled to one full step,
    description, measured seconds, CPU seconds used per second of wall clock)."""
    from oracle import adapshot_oracle as orc
    f64 = wl.to_f64
    cpu0 = time.process_time()
    t0 = time.perf_counter()
    sel, _ = orc.select_topk(f64(qs["q_emb"]), f64(pool["emb"]), w.k)
    off = orc.plan_offsets(sel, pool["shot_off"])
    t_select = time.perf_counter() - t0
    t0 = time.perf_counter()
    kc, vc, _ = orc.assemble_kv(f64(pool["k"][:1]), f64(pool["v"][:1]), pool["shot_off"], sel[0], w.rope_base)
    t_assemble = time.perf_counter() - t0
    q, kq, vq = f64(qs["q"][0, 0]), f64(qs["kq"][0, 0]), f64(qs["vq"][0, 0])
    rows = [(j, h, t) for j in range(len(w.probes)) for h in range(w.n_q_heads) for t in range(w.t_q)]
    sample = rows[::row_stride]
    t0 = time.perf_counter()
    for j, h, t in sample:
        orc.attn_row(q[j, t, h], kq[j], vq[j], kc[0], vc[0], int(off[0, w.probes[j]]), t, h // w.group, w.rope_base)
    t_attn = time.perf_counter() - t0
    t0 = time.perf_counter()
    orc.entropy(f64(qs["logits"]))
    t_entropy = time.perf_counter() - t0
    units = w.batch * w.n_layers                                   # (query, layer) units are independent
    full = w.batch * (t_select + t_entropy) + units * (t_assemble + t_attn * len(rows) / len(sample))
    measured = t_select + t_assemble + t_attn + t_entropy
    desc = (f"query 0: select and entropy in full (scaled by {w.batch} queries), assemble and attention at layer 0 "
            f"with every {row_stride}th of {len(rows)} attention rows (scaled by rows and by {units} (query, layer) "
            "units)")
    cores_used = (time.process_time() - cpu0) / max(measured, 1e-9)      # CPU seconds per second of wall clock
    return full, desc, measured, cores_used


def job_aggregate(ms: float, tokens: float, dist, device):
    """Replicas share nothing but the clock: the job's time is the slowest rank's, its tokens
    the sum over ranks.  dist = torch.distributed (initialised) or None for one process."""
    if dist is None:
        return ms, tokens
    t = torch.tensor([ms], device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    n = torch.tensor([tokens], device=device, dtype=torch.float64)
    dist.all_reduce(n, op=dist.ReduceOp.SUM)
    return float(t.item()), float(n.item())


def rank_seed(seed: int, rank: int) -> int:
    """Every replica draws its own queries (same pool)."""
    return seed + 100 * rank if rank else seed


def cpu_threads() -> dict:
    """Threads the oracle run can use: its per-row loops are single-threaded Python, the numpy
    products inside them go through the BLAS pool."""
    blas = 1
    try:
        import threadpoolctl
        info = threadpoolctl.threadpool_info()
        blas = max([i.get("num_threads", 1) for i in info] + [1])
    except Exception:
        pass
    return {"python_threads": 1, "blas_threads": blas, "host_cores": os.cpu_count() or 1}


def host_inputs(w: wl.Workload, n_pool_layers: int = 1):
    """CPU copies of a one-layer, one-query slice of the workload for the oracle legs, and the
    oracle's own selection / plan for the whole batch (cheap: one B x N x E product)."""
    from oracle import adapshot_oracle as orc
    ws = w.scaled(batch=1)
    pool = wl.make_pool(ws, "cpu", n_layers=n_pool_layers)
    q_emb_all = wl.make_query_embeddings(w, "cpu")
    if w.k == 0:          # token-budget selection: the longest similarity-ordered prefix within the limit
        order, _ = orc.select_topk(wl.to_f64(q_emb_all), wl.to_f64(pool["emb"]), int(pool["n_shots"]))
        k = int(np.searchsorted(np.cumsum(pool["lengths"][order[0]]), w.ctx_token_limit, side="right"))
        w = w.scaled(k=k, probes=(k,))
        ws = w.scaled(batch=1)
    qs = wl.make_queries(ws, "cpu", n_layers=1)
    sel_all, _ = orc.select_topk(wl.to_f64(q_emb_all), wl.to_f64(pool["emb"]), w.k)
    ctx_tokens = float(orc.plan_offsets(sel_all, pool["shot_off"])[:, -1].sum())
    return w, pool, qs, ctx_tokens


def workload_config(w: wl.Workload, pool_shots: int, pool_tokens: int, ctx_tokens: float, world: int) -> dict:
    """The keys that name the workload: the same in the GPU arm's line and in the reference arm's."""
    return {"workload": w.name, "n_layers": w.n_layers, "batch_per_gpu": w.batch, "k": w.k,
            "probes": list(w.probes), "t_q": w.t_q, "pool_shots": int(pool_shots),
            "pool_tokens": int(pool_tokens), "ctx_tokens_per_step": float(ctx_tokens),
            "parallelism": "replicas" if world > 1 else "single"}      # (the selection is device-independent)


def run_reference(args, w: wl.Workload):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    w, pool, qs, ctx_tokens = host_inputs(w)
    n_rows = len(w.probes) * w.n_q_heads * w.t_q
    stride = max(1, n_rows // 96)
    for _ in range(args.warmup):
        oracle_sample_seconds(w, pool, qs, stride * 8)
    vals, desc, used = [], "", []
    for _ in range(args.steps):
        full, desc, _m, c = oracle_sample_seconds(w, pool, qs, stride)
        vals.append(full)
        used.append(c)
    sec = float(np.mean(vals))
    value = ctx_tokens / sec
    cfg = workload_config(w, pool["n_shots"], pool["pool_tokens"], ctx_tokens, 1)
    cfg["note"] = "oracle timed on host cores; each step is a bounded sample scaled to the full step"
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": sec * 1e3, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": cfg,
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": max(1, round(float(np.mean(used)))),
                             "cpu_seconds_per_second": float(np.mean(used)), "threads": cpu_threads(),
                             "kind": "oracle", "sample": desc},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


# ------------------------------------------------------------------------- GPU arm
def _timed(fn, n, flush):
    """Mean device time of fn() over n calls, L2 flushed before each (CUDA events on the current stream)."""
    tot = 0.0
    for _ in range(n):
        flush.zero_()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        fn()
        b.record()
        torch.cuda.synchronize()
        tot += a.elapsed_time(b)
    return tot / n


def per_probe_costs(ab, path, model, dpool, w, qc, kqc, vqc, ctx_off_np, flush, n_rep=5):
    """What every nested probe costs on its own, on the first full-size layer chunk: the attention of
    that probe alone over its prefix of the shared re-encoded cache, and the gather of the shots it adds
    to the previous probe's prefix (the prefix itself is shared and stays in place)."""
    ci = max(range(len(path.chunks)), key=lambda i: (path.chunks[i][1] - path.chunks[i][0], -i))
    lb, le = path.chunks[ci]
    nl = le - lb
    k_ctx, v_ctx = path.ctx_views(nl)
    out = []
    dev = path.status.device
    prev = 0
    for j, n_j in enumerate(w.probes):
        q_j, kq_j, vq_j = (x[ci][:, :, j:j + 1].contiguous() for x in (qc, kqc, vqc))
        o_j = torch.empty_like(q_j)
        attn_ms = _timed(lambda: path.attend(q_j, kq_j, vq_j, o_j, lb, le, probes=[n_j]), n_rep, flush)
        sel_j = path.sel_idx[:, :n_j].contiguous()
        off_j = torch.empty((w.batch, n_j + 1), dtype=torch.int64, device=dev)
        gflags = ab.ASSEMBLE_K_ONLY if path.vpool else 0
        gather_ms = _timed(lambda: ab.adapshot_assemble_kv_from(model, dpool, sel_j, prev, lb, le, k_ctx, v_ctx,
                                                                path.ctx_cap, off_j, path.status, flags=gflags),
                           n_rep, flush)
        Lj = ctx_off_np[:, n_j].astype(np.float64)
        Lp = ctx_off_np[:, prev].astype(np.float64) if prev else np.zeros_like(Lj)
        flops = float((4.0 * w.t_q * (Lj + (w.t_q + 1) / 2.0) * w.n_q_heads * w.head_dim).sum()) * nl
        out.append({"n_shots": int(n_j), "ctx_tokens": float(Lj.sum()),
                    "attn_ms": attn_ms * w.n_layers / nl, "attn_tflops": flops / (attn_ms * 1e-3) / 1e12,
                    "gather_added_ms": gather_ms * w.n_layers / nl,
                    "gather_added_gbs": float((Lj - Lp).sum()) * w.bytes_per_token_layer * (1 if path.vpool else 2) * nl
                    / (gather_ms * 1e-3) / 1e9})
        prev = n_j
    path.assemble(lb, le, keep_plan=True)        # the cache of the whole selection again
    torch.cuda.synchronize()
    return {"what": "each nested probe alone (attention over its prefix; gather of the shots it adds), "
                    f"measured on layers {lb}..{le - 1} and scaled to {w.n_layers} layers",
            "probes": out,
            "sum_attn_ms": float(sum(p["attn_ms"] for p in out)),
            "sum_gather_ms": float(sum(p["gather_added_ms"] for p in out))}


def measure(args, name: str, steps: int, warmup: int, dev, peaks, dist, rank: int, world: int,
            with_cpu_baseline: bool) -> dict:
    """Builds one workload on the device, times the whole path over it and returns the fields of a
    bench line for it (everything is freed again on return)."""
    from paper_2605_03644_b200 import binding as ab
    from paper_2605_03644_b200.pipeline import ReusePath

    w = resolve_workload(name, args.layers, args.queries)
    if w.dtype != "bf16":   # cfg1: fp32 storage; the attention kernel takes bf16 (the parity tests round its inputs)
        raise SystemExit(f"{w.name} is a parity configuration (fp32 storage); bench workloads: cfg2 cfg3 cfg4 cfg5")

    # ---- resident inputs (every rank: same pool, its own queries)
    pool = wl.make_pool(w, dev)
    so = torch.from_numpy(pool["shot_off"]).to(dev)
    dpool = ab.Pool(so, pool["k"], pool["v"], pool["emb"])
    wq = w.scaled(seed=rank_seed(w.seed, rank))
    if w.k == 0:
        w = resolve_k_by_budget(ab, dpool, wl.make_query_embeddings(wq, dev), w, pool["lengths"])
        wq = w.scaled(seed=wq.seed)
    model = ab.make_model(w.n_layers, w.n_q_heads, w.n_kv_heads, w.head_dim, w.dtype, w.rope_base,
                          k_pos_mode=args.k_pos_mode)
    qs = wl.make_queries(wq, dev)
    ctx_cap = args.ctx_cap or planned_ctx_cap(ab, dpool, qs["q_emb"], w)
    fused = args.variant == "fused"
    vpool, lpc = choose_variant(w, ctx_cap, args.variant, args.layers_per_call)
    if fused and not args.layers_per_call:
        lpc = w.n_layers                      # no assembled cache to fit: all layers in one call
    path = ReusePath(model, dpool, w.batch, w.k, w.probes, w.t_q, w.vocab, ctx_cap, lpc, fused=fused,
                     entropy_overlap=args.entropy_overlap, vpool=vpool, ramp=args.ramp)
    chunk = lambda x: [x[:, lb:le].contiguous() for lb, le in path.chunks]
    q_emb, qc, kqc, vqc, logits = qs["q_emb"], chunk(qs["q"]), chunk(qs["kq"]), chunk(qs["vq"]), qs["logits"]
    del qs
    flush = torch.empty(L2_FLUSH_BYTES, dtype=torch.uint8, device=dev)
    n_sel = 2 if w.n_shots <= 4096 else (3 if w.n_shots > 8192 else 2)
    if fused or vpool:
        launches_per_step = n_sel + 1 + len(path.chunks) * ((1 if vpool else 0) + 4) + 2
    else:
        launches_per_step = n_sel + 1 + len(path.chunks) * (1 + 3) + 2

    use_graph = args.graph == "on" or (args.graph == "auto" and w.n_layers == 1)
    if use_graph:
        path.capture(q_emb, qc, kqc, vqc, logits, args.tau)

    def step():
        if use_graph:
            path.replay()
        else:
            path.run(q_emb, qc, kqc, vqc, logits, args.tau)

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    def check_status(when):
        code = int(path.status.item())
        if code != 0:
            raise SystemExit(f"device status {code} {when}: {ab.adapshot_strerror(code)}")

    step()
    torch.cuda.synchronize()
    check_status("after the first pass")
    ctx_off = path.ctx_off.cpu().numpy()
    counts = algorithmic_counts(w, ctx_off, w.n_layers)
    if vpool:      # the gather moves K only: bpt / 2 read + bpt / 2 written per context token and layer
        counts["gather_bytes"] *= 0.5

    for _ in range(warmup):
        flush.zero_()
        step()
    barrier()

    # ---- timed region: K steps, CUDA events around every step, L2 flushed between steps
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
    with ClockSampler(dev.index) as clocks:
        barrier()
        for a, b in ev:
            flush.zero_()
            a.record()
            step()
            b.record()
        barrier()
    step_ms = np.array([a.elapsed_time(b) for a, b in ev])
    total_ms = float(step_ms.sum())
    total_ms, job_tokens = job_aggregate(total_ms, counts["ctx_tokens"], dist, dev)
    ms_per_step = total_ms / steps
    value = job_tokens / (ms_per_step * 1e-3)
    check_status("after the timed region")

    # ---- per-call device times (second pass, same conditions) for the roofline object
    names = ["select", "assemble", "attn", "entropy"]     # select includes the plan; assemble = gather
    acc = {n: 0.0 for n in names}
    n_prof = min(steps, 50)
    for _ in range(n_prof):
        flush.zero_()
        marks = [torch.cuda.Event(enable_timing=True) for _ in range(2 + 2 * len(path.chunks) + 1)]
        marks[0].record()
        path.select(q_emb)
        path.plan()                              # offsets once per pass, timed with the selection
        marks[1].record()
        mi = 1
        for i, (lb, le) in enumerate(path.chunks):
            if not fused:
                path.assemble(lb, le, keep_plan=True)
            marks[mi + 1].record()
            if fused:
                path.attend_fused(qc[i], kqc[i], vqc[i], path.out[i], lb, le)
            else:
                path.attend(qc[i], kqc[i], vqc[i], path.out[i], lb, le)
            marks[mi + 2].record()
            mi += 2
        path.entropy(logits, args.tau)
        marks[mi + 1].record()
        torch.cuda.synchronize()
        acc["select"] += marks[0].elapsed_time(marks[1])
        mi = 1
        for _c in path.chunks:
            acc["assemble"] += marks[mi].elapsed_time(marks[mi + 1])
            acc["attn"] += marks[mi + 1].elapsed_time(marks[mi + 2])
            mi += 2
        acc["entropy"] += marks[mi].elapsed_time(marks[mi + 1])
    per_call_ms = {n: acc[n] / n_prof for n in names}

    # ---- the dominant kernel alone: CUDA events recorded by the library around attn_main_kernel
    ab.adapshot_profile(True)
    main_ms = 0.0
    for _ in range(n_prof):
        flush.zero_()
        for i, (lb, le) in enumerate(path.chunks):
            if fused:
                if i == 0:
                    path.plan()
                path.attend_fused(qc[i], kqc[i], vqc[i], path.out[i], lb, le)
            else:
                path.assemble(lb, le, keep_plan=i > 0)
                path.attend(qc[i], kqc[i], vqc[i], path.out[i], lb, le)
            main_ms += ab.adapshot_profile_attn_main_ms()
    ab.adapshot_profile(False)
    main_ms /= n_prof
    n_main = len(path.chunks)

    attn_s = main_ms * 1e-3
    call_s = per_call_ms["attn"] * 1e-3
    gather_s = per_call_ms["assemble"] * 1e-3
    attn_tflops = counts["attn_flops"] / attn_s / 1e12
    attn_kv_gbs = counts["attn_kv_bytes"] / attn_s / 1e9
    tensor_bound = counts["attn_flops"] / (peaks["bf16_tflops"] * 1e12) >= \
        counts["attn_kv_bytes"] / (peaks["hbm_gbs"] * 1e9)
    traffic_attn = traffic_gather = None
    cap = NCU_TRAFFIC.get(w.name)
    if cap is not None and args.variant == "auto" and not args.layers and not args.queries and args.k_pos_mode == 0:
        units_per_launch = w.n_layers / n_main * w.batch      # the mean launch, like the other per-launch figures
        if cap[0] is not None:
            traffic_attn = cap[0] / cap[1] * units_per_launch
        if cap[2] is not None:
            traffic_gather = cap[2] / cap[3] * units_per_launch
    call_tflops = counts["attn_flops"] / call_s / 1e12
    roofline = {
        "kernel": "attn_main_kernel" + ("<fused>" if fused else ""),
        "launches_per_step": n_main,
        "bound": "tensor" if tensor_bound else "hbm",
        "achieved": attn_tflops if tensor_bound else attn_kv_gbs,
        "peak": peaks["bf16_tflops"] if tensor_bound else peaks["hbm_gbs"],
        "unit": "TFLOP/s" if tensor_bound else "GB/s",
        "frac": (attn_tflops / peaks["bf16_tflops"]) if tensor_bound else (attn_kv_gbs / peaks["hbm_gbs"]),
        "frac_of_sustained_peak": attn_tflops / peaks["bf16_tflops_sustained"] if tensor_bound else None,
        "peak_source": f"of {peaks['source']}",
        "traffic": traffic_attn,
        "ms_per_launch": main_ms / n_main,
        "algorithmic_flops_per_launch": counts["attn_flops"] / n_main,
        "algorithmic_kv_bytes_per_launch": counts["attn_kv_bytes"] / n_main,
        "whole_call": {"what": "adapshot_query_attn (prep + main + combine)", "ms_per_step": per_call_ms["attn"],
                       "achieved": call_tflops, "unit": "TFLOP/s", "frac": call_tflops / peaks["bf16_tflops"]},
        "gather": None if fused else {
            "bound": "hbm", "achieved": counts["gather_bytes"] / gather_s / 1e9, "peak": peaks["hbm_gbs"],
            "unit": "GB/s", "frac": counts["gather_bytes"] / gather_s / 1e9 / peaks["hbm_gbs"],
            "ms_per_step": per_call_ms["assemble"], "traffic": traffic_gather},
        "select": {"bound": "hbm", "achieved": counts["select_bytes"] / (per_call_ms["select"] * 1e-3) / 1e9,
                   "unit": "GB/s", "ms_per_step": per_call_ms["select"]},
        "entropy": {"bound": "hbm", "achieved": counts["entropy_bytes"] / (per_call_ms["entropy"] * 1e-3) / 1e9,
                    "unit": "GB/s", "ms_per_step": per_call_ms["entropy"]},
    }

    per_probe = None
    if len(w.probes) > 1 and not fused:
        per_probe = per_probe_costs(ab, path, model, dpool, w, qc, kqc, vqc, ctx_off, flush)
        check_status("after the per-probe pass")

    # ---- end to end: pinned host inputs in, results out, inside the timed region
    host = {"q_emb": q_emb.cpu().pin_memory(), "logits": logits.cpu().pin_memory(),
            "q": [x.cpu().pin_memory() for x in qc], "kq": [x.cpu().pin_memory() for x in kqc],
            "vq": [x.cpu().pin_memory() for x in vqc]}
    out_host = [torch.empty_like(x, device="cpu").pin_memory() for x in path.out]
    H_host = torch.empty_like(path.H, device="cpu").pin_memory()
    fo_host = torch.empty_like(path.first_ok, device="cpu").pin_memory()
    sel_host = torch.empty_like(path.sel_idx, device="cpu").pin_memory()
    nbytes = lambda t: t.numel() * t.element_size()
    h2d = nbytes(host["q_emb"]) + nbytes(host["logits"]) + sum(nbytes(x) for k in ("q", "kq", "vq") for x in host[k])
    d2h = sum(nbytes(x) for x in out_host) + nbytes(H_host) + nbytes(fo_host) + nbytes(sel_host)

    dev_in = {"q_emb": q_emb, "logits": logits, "q": qc, "kq": kqc, "vq": vqc}
    host_out = {"out": out_host, "H": H_host, "first_ok": fo_host, "sel_idx": sel_host}
    path.run_host(host, dev_in, host_out, args.tau)
    torch.cuda.synchronize()
    e2e_graph = None
    if use_graph:
        # the copies from and to pinned host memory are graph nodes beside the kernels
        e2e_graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(e2e_graph):
            path.run_host(host, dev_in, host_out, args.tau)

    def e2e_step():
        if e2e_graph is not None:
            e2e_graph.replay()
        else:
            path.run_host(host, dev_in, host_out, args.tau)

    n_e2e = max(3, min(steps, 50))
    for _ in range(3):
        e2e_step()
    barrier()
    ev2 = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(n_e2e)]
    for a, b in ev2:
        flush.zero_()
        a.record()
        e2e_step()
        b.record()
    barrier()
    e2e_ms = float(np.sum([a.elapsed_time(b) for a, b in ev2]))
    e2e_ms, _ = job_aggregate(e2e_ms, 0.0, dist, dev)
    e2e_value = job_tokens / (e2e_ms / n_e2e * 1e-3)
    check_status("after the end-to-end pass")
    e2e_timeline = None
    if args.e2e_timeline:
        # when each step of one plain (uncaptured) end-to-end pass ends on the compute stream, from events
        # recorded after the calls; the copies run on their own streams beside them
        marks = []
        def wrapped(name, fn):
            def call(*a, **k):
                r = fn(*a, **k)
                e = torch.cuda.Event(enable_timing=True)
                e.record()
                marks.append((name, e))
                return r
            return call
        names = ["select", "plan", "assemble", "attend", "attend_fused", "entropy"]
        saved = {n: getattr(path, n) for n in names}
        for n in names:
            setattr(path, n, wrapped(n, saved[n]))
        flush.zero_()
        t0 = torch.cuda.Event(enable_timing=True)
        t0.record()
        path.run_host(host, dev_in, host_out, args.tau)
        t1 = torch.cuda.Event(enable_timing=True)
        t1.record()
        torch.cuda.synchronize()
        for n in names:
            setattr(path, n, saved[n])
        e2e_timeline = [[n, t0.elapsed_time(e)] for n, e in marks] + [["results in host memory", t0.elapsed_time(t1)]]

    config = workload_config(w, pool["n_shots"], pool["pool_tokens"], counts["ctx_tokens"], world)
    config.update({"variant": "fused" if fused else ("vpool" if vpool else "materialise"), "k_pos_mode": args.k_pos_mode, "cuda_graph": use_graph,
                   "ctx_cap": ctx_cap, "layers_per_call": lpc, "layer_chunks": [le - lb for lb, le in path.chunks],
                   "gather_overlaps_attention": path.overlap,
                   "entropy": "side stream, overlapped with the pass" if path.entropy_overlap
                   else "after the last attention call (serial)",
                   "l2": "flushed between steps (512 MiB write)"})
    res = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": steps,
        "warmup": warmup, "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": config, "roofline": roofline,
        "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "graph": e2e_graph is not None},
        "gpu_launches": launches_per_step * steps, "clocks": clocks.summary(),
        "per_call_ms": per_call_ms,
        "step_ms_min_med_max": [float(step_ms.min()), float(np.median(step_ms)), float(step_ms.max())],
        "timed_region_ms": total_ms,
        **({"e2e_timeline_ms": e2e_timeline} if e2e_timeline is not None else {}),
    }
    if per_probe is not None:
        res["per_probe"] = per_probe

    # ---- free everything this workload holds on the device and in pinned memory
    del path, pool, dpool, so, qc, kqc, vqc, logits, q_emb, flush, host, out_host, dev_in, host_out, e2e_graph
    import gc
    gc.collect()
    torch.cuda.empty_cache()

    # ---- CPU oracle beside it (rank 0, N = 1 only)
    if with_cpu_baseline:
        w0, hpool, hqs, ctx_tokens = host_inputs(wl.CONFIGS[name] if not (args.layers or args.queries)
                                                 else resolve_workload(name, args.layers, args.queries))
        n_rows = len(w0.probes) * w0.n_q_heads * w0.t_q
        full, desc, meas, used = oracle_sample_seconds(w0, hpool, hqs, max(1, n_rows // 3000))   # about 15 s of oracle work
        res["cpu_baseline"] = {"value": ctx_tokens / full, "unit": UNIT, "cores": max(1, round(used)),
                               "cpu_seconds_per_second": used, "threads": cpu_threads(),
                               "kind": "oracle", "sample": desc, "measured_seconds": meas}
    else:
        res["cpu_baseline"] = None
    return res


def run_micro(args):
    """One HBM-bound step alone on an input large enough to be bound by bandwidth (the benchmark
    workloads give the entropy and selection steps a few MB, where they are bound by launch latency):
    CUDA events around the call, L2 flushed before each, achieved GB/s against the measured copy peak.
    Prints its own JSON line (not a bench line)."""
    from paper_2605_03644_b200 import binding as ab
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the hot path has no CPU fallback")
    dev = torch.device("cuda", int(os.environ.get("LOCAL_RANK", "0")))
    torch.cuda.set_device(dev)
    peaks = load_peaks()
    flush = torch.empty(L2_FLUSH_BYTES, dtype=torch.uint8, device=dev)
    st = torch.zeros(1, dtype=torch.int32, device=dev)
    steps = args.steps or 20
    g = torch.Generator(device=dev)
    g.manual_seed(5)
    if args.micro == "entropy":
        R, V = args.rows, args.vocab
        dt = torch.bfloat16 if args.logits_dtype == "bf16" else torch.float32
        logits = torch.randn(R, V, generator=g, device=dev).to(dt)
        H = torch.empty(R, dtype=torch.float32, device=dev)
        fo = torch.empty(R, dtype=torch.int32, device=dev)
        ws = torch.empty(max(256, ab.adapshot_entropy_workspace_bytes(R, V)), dtype=torch.uint8, device=dev)
        fn = lambda: ab.adapshot_entropy(logits, H, args.tau, 1, fo, ws, st)
        nbytes = float(R) * V * logits.element_size()
        what = {"rows": R, "vocab": V, "logits_dtype": args.logits_dtype}
    elif args.micro == "relevance":
        # the attention-based selector (Sec. 4.2) over one layer of a workload's pool: tensor-core passes, bound
        # by the exponentials (one per query row and pool key, twice)
        w = wl.CONFIGS["cfg3" if args.workload == "default" else args.workload]
        pool = wl.make_pool(w, dev, n_layers=1)
        so = torch.from_numpy(pool["shot_off"]).to(dev)
        dpool = ab.Pool(so, pool["k"], pool["v"], pool["emb"])
        model = ab.make_model(1, w.n_q_heads, w.n_kv_heads, w.head_dim, w.dtype, w.rope_base)
        q = torch.randn(w.batch, w.t_q, w.n_q_heads, w.head_dim, generator=g, device=dev).to(torch.bfloat16)
        sel = torch.empty((w.batch, w.k), dtype=torch.int32, device=dev)
        ws = torch.empty(max(256, ab.adapshot_select_attn_workspace_bytes(model, dpool, w.batch, w.t_q, w.k)),
                         dtype=torch.uint8, device=dev)
        fn = lambda: ab.adapshot_select_attn(model, dpool, 0, q, w.k, sel, None, ws, st)
        rows = float(w.batch) * w.t_q * w.n_q_heads
        flops = 2.0 * 2.0 * rows * pool["pool_tokens"] * w.head_dim            # two passes of Q K^T
        nbytes = 2.0 * pool["pool_tokens"] * w.n_kv_heads * w.head_dim * 2     # the layer's K, twice
        what = {"workload": w.name, "pool_tokens": int(pool["pool_tokens"]), "query_rows": rows,
                "algorithmic_flops": flops, "exponentials": 2.0 * rows * pool["pool_tokens"]}
    else:
        w = wl.CONFIGS[HEADLINE if args.workload == "default" else args.workload]
        n_shots = int(wl.shot_lengths(w).size)
        emb = torch.randn(n_shots, w.emb_dim, generator=g, device=dev)
        q_emb = torch.randn(w.batch, w.emb_dim, generator=g, device=dev)
        so = torch.arange(n_shots + 1, dtype=torch.int64, device=dev)
        dpool = ab.Pool(so, None, None, emb)
        sel = torch.empty((w.batch, w.k), dtype=torch.int32, device=dev)
        ws = torch.empty(max(256, ab.adapshot_select_workspace_bytes(n_shots, w.batch, w.k)), dtype=torch.uint8,
                         device=dev)
        fn = lambda: ab.adapshot_select(dpool, q_emb, w.k, sel, None, ws, st)
        nbytes = float(n_shots) * w.emb_dim * 4
        what = {"pool_shots": n_shots, "emb_dim": w.emb_dim, "queries": w.batch, "k": w.k}
    for _ in range(3):
        fn()
    torch.cuda.synchronize()
    with ClockSampler(dev.index) as clocks:
        ms = _timed(fn, steps, flush)
    if st.item() != 0:
        raise SystemExit(f"device status {st.item()}")
    gbs = nbytes / (ms * 1e-3) / 1e9
    if args.micro == "relevance":
        what["achieved_tflops"] = what["algorithmic_flops"] / (ms * 1e-3) / 1e12
        what["frac_of_bf16_peak"] = what["achieved_tflops"] / peaks["bf16_tflops"]
        # 16 exponentials per clock and SM at the clock the sampler saw
        what["exp_per_s"] = what["exponentials"] / (ms * 1e-3)
    print(json.dumps({"micro": args.micro, **what, "algorithmic_bytes": nbytes, "ms_per_call": ms, "steps": steps,
                      "achieved_gbs": gbs, "peak_gbs": peaks["hbm_gbs"], "frac": gbs / peaks["hbm_gbs"],
                      "peak_source": f"of {peaks['source']}", "clocks": clocks.summary(),
                      "l2": "flushed before every call (512 MiB write)"}))


def run_ours(args):
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the hot path has no CPU fallback")
    torch.cuda.set_device(local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    peaks = load_peaks()
    dev = torch.device("cuda", local)
    baseline = rank == 0 and world == 1 and not args.no_cpu_baseline

    def steps_for(name, headline):
        small = wl.CONFIGS[name].n_layers == 1 or args.layers == 1
        if headline:
            k = (2000 if small else 10) if args.steps is None else args.steps
        else:       # a sub-workload's timed region lasts a few tenths of a second at least
            k = max(2000 if small else 40, args.steps or 0)
        wu = (20 if small else 3) if args.warmup is None else max(3, args.warmup)
        return k, wu

    if args.workload == "default":
        free_bytes, _ = torch.cuda.mem_get_info()
        headline = HEADLINE if free_bytes > 170e9 else "cfg3"      # cfg5 holds a 140 GB pool
        subs = [n for n in SUB_WORKLOADS if n != headline]
    else:
        headline, subs = args.workload, []
    sub_res = {}
    for name in subs:
        k, wu = steps_for(name, False)
        sub_res[name] = measure(args, name, k, wu, dev, peaks, dist, rank, world, False)
    k, wu = steps_for(headline, True)
    line = measure(args, headline, k, wu, dev, peaks, dist, rank, world, baseline)
    if sub_res:
        line["workloads"] = sub_res
        line["gpu_launches_all_workloads"] = line["gpu_launches"] + sum(r["gpu_launches"] for r in sub_res.values())
    if rank == 0:
        print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=None)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="default",
                    help="default: the headline configuration (cfg5) with cfg2 and cfg3 as sub-objects of the "
                         "same line; or one of cfg2 cfg3 cfg4 cfg5 alone")
    ap.add_argument("--layers", type=int, default=0,
                    help="run only the first N layers of the workload (a smaller case for profiler captures)")
    ap.add_argument("--queries", type=int, default=0,
                    help="run only the first N queries of the workload (a smaller case for profiler captures)")
    ap.add_argument("--layers-per-call", type=int, default=0)
    ap.add_argument("--ctx-cap", type=int, default=0)
    ap.add_argument("--variant", default="auto", choices=["auto", "materialise", "vpool", "fused"],
                    help="materialise: gather + re-encode K and V into a contiguous cache, then attend; "
                         "vpool: gather + re-encode K only, attention takes V tiles from the pool; "
                         "fused: attention reads the pool and re-encodes K in shared memory; "
                         "auto (default): vpool when a call's cache is larger than L2, else materialise")
    ap.add_argument("--k-pos-mode", type=int, default=0, choices=[0, 1],
                    help="0: pool K carries no position (default); 1: pool K rotated at shot-local positions "
                         "(the paper's store), the re-encode is one angle per shot")
    ap.add_argument("--graph", default="auto", choices=["auto", "on", "off"],
                    help="replay the pass as one CUDA graph (auto: single-layer workloads)")
    ap.add_argument("--entropy-overlap", action="store_true",
                    help="run the entropy probe on a side stream beside the pass instead of after the attention")
    ap.add_argument("--e2e-timeline", action="store_true",
                    help="add e2e_timeline_ms to the line: when every step of one end-to-end pass ends")
    ap.add_argument("--ramp", action="store_true",
                    help="make the first and the last layer chunk of a pass a quarter of --layers-per-call: it shortens "
                         "the only upload and download of the end-to-end pass that no kernel runs beside (measured: "
                         "e2e 2-3 percent faster, the device-resident step up to 1.6 percent slower, hence off by default)")
    ap.add_argument("--micro", default=None, choices=["entropy", "select", "relevance"],
                    help="time one HBM-bound step alone on a bandwidth-bound input and print its own JSON line")
    ap.add_argument("--rows", type=int, default=2048, help="--micro entropy: logit rows")
    ap.add_argument("--vocab", type=int, default=128256, help="--micro entropy: vocabulary size")
    ap.add_argument("--logits-dtype", default="bf16", choices=["bf16", "fp32"])
    ap.add_argument("--tau", type=float, default=0.65)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args()
    if args.impl == "reference":
        args.steps = 3 if args.steps is None else args.steps
        args.warmup = 1 if args.warmup is None else args.warmup
        name = HEADLINE if args.workload == "default" else args.workload
        run_reference(args, resolve_workload(name, args.layers, args.queries))
        return
    if args.micro is not None:
        run_micro(args)
        return
    run_ours(args)


if __name__ == "__main__":
    main()
