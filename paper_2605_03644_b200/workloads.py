"""Seeded synthetic inputs shaped like the paper's many-shot workloads.

This module only draws random inputs (shot lengths, cached K/V, embeddings,
query tensors, logits) and lays them out in the pool format; it holds none of
the method's arithmetic and is the one module both the CUDA tests and the CPU
oracle tests take their inputs from.

The shapes stand in for the many-shot prompts of the paper's evaluation
(Sec. 5: CoT-Collection tasks on 3B-8B decoder models): only sizes, length
mixes and value distributions are imitated; no dataset item is reproduced.

Pool layout (Sec. 4.2 "hierarchical" pool, made concrete):
    k, v      : [n_layers][pool_tokens][n_kv_heads][head_dim]
    shot_off  : int64 [n_shots + 1], token offset of every shot in the pool
    emb       : fp32 [n_shots][emb_dim], unit-norm rows
"""
from __future__ import annotations

from dataclasses import dataclass, replace
from typing import Optional, Sequence

import numpy as np
import torch


@dataclass(frozen=True)
class Workload:
    name: str
    n_layers: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    rope_base: float
    dtype: str                 # "fp32" | "bf16": storage of pool / ctx / q / out
    n_shots: int               # 0 => draw shots until pool_token_target is reached
    len_dist: str              # "const" | "uniform" | "lognormal"
    len_lo: int
    len_hi: int
    emb_dim: int
    batch: int                 # B queries
    k: int                     # shots selected per query (0 => by ctx_token_limit)
    probes: Sequence[int]      # nested shot counts n_1 < ... < n_P = k
    t_q: int                   # query (+ probe prompt) tokens
    vocab: int
    logits_dtype: str          # "fp32" | "bf16"
    seed: int
    channel_scale: bool = True  # K/V ~ N(0,1) x per-channel U(0.5, 2)
    len_median: float = 0.0     # lognormal only
    len_sigma: float = 0.0      # lognormal only
    pool_token_target: int = 0  # n_shots == 0 only
    ctx_token_limit: int = 0    # k == 0 only: longest prefix with L <= limit
    logits_std: float = 1.0

    @property
    def group(self) -> int:
        return self.n_q_heads // self.n_kv_heads

    @property
    def elem_size(self) -> int:
        return 4 if self.dtype == "fp32" else 2

    @property
    def torch_dtype(self) -> torch.dtype:
        return torch.float32 if self.dtype == "fp32" else torch.bfloat16

    @property
    def bytes_per_token_layer(self) -> int:
        """K + V bytes of one token at one layer (bpt)."""
        return 2 * self.n_kv_heads * self.head_dim * self.elem_size

    def scaled(self, **kw) -> "Workload":
        return replace(self, **kw)


# The five benchmark configurations.  Values their description leaves open and that are
# fixed here: emb_dim of cfg4/cfg5 (1024), vocab of cfg4/cfg5 (128256), sigma of the
# lognormal of cfg5's shot lengths (0.4).
CONFIGS = {
    "cfg1": Workload("cfg1", 1, 4, 1, 64, 1e4, "fp32", 64, "const", 32, 32, 128,
                     1, 8, (8,), 16, 1024, "fp32", seed=0, channel_scale=False,
                     logits_std=float(np.sqrt(2.0))),
    "cfg2": Workload("cfg2", 1, 32, 8, 128, 5e5, "bf16", 2048, "uniform", 64, 256, 1024,
                     1, 128, (16, 32, 64, 128), 128, 32000, "fp32", seed=1),
    "cfg3": Workload("cfg3", 32, 32, 8, 128, 5e5, "bf16", 4096, "uniform", 64, 192, 1024,
                     8, 256, (256,), 128, 128256, "bf16", seed=2),
    "cfg4": Workload("cfg4", 80, 64, 8, 128, 5e5, "bf16", 0, "uniform", 128, 512, 1024,
                     1, 0, (), 256, 128256, "bf16", seed=3,
                     pool_token_target=98304, ctx_token_limit=65536),
    "cfg5": Workload("cfg5", 32, 32, 8, 128, 5e5, "bf16", 8192, "lognormal", 40, 400, 1024,
                     32, 512, (8, 16, 32, 64, 128, 256, 512), 64, 128256, "bf16", seed=4,
                     len_median=120.0, len_sigma=0.4),
}


def shot_lengths(w: Workload) -> np.ndarray:
    """Token length of every pool shot (numpy Generator seeded by w.seed)."""
    rng = np.random.default_rng(w.seed)
    if w.n_shots == 0:
        out, tot = [], 0
        while tot < w.pool_token_target:
            t = int(rng.integers(w.len_lo, w.len_hi + 1))
            out.append(t)
            tot += t
        return np.asarray(out, dtype=np.int64)
    if w.len_dist == "const":
        return np.full(w.n_shots, w.len_lo, dtype=np.int64)
    if w.len_dist == "uniform":
        return rng.integers(w.len_lo, w.len_hi + 1, size=w.n_shots).astype(np.int64)
    if w.len_dist == "lognormal":
        z = rng.standard_normal(w.n_shots)
        t = np.rint(np.exp(np.log(w.len_median) + w.len_sigma * z))
        return np.clip(t, w.len_lo, w.len_hi).astype(np.int64)
    raise ValueError(w.len_dist)


def shot_offsets(lengths: np.ndarray) -> np.ndarray:
    off = np.zeros(len(lengths) + 1, dtype=np.int64)
    off[1:] = np.cumsum(lengths)
    return off


def _gen(seed: int, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return g


def _unit_rows(n: int, e: int, seed: int, device) -> torch.Tensor:
    """Unit-norm Gaussian rows.  Always drawn by a CPU generator and then moved: the embeddings
    decide the selection (and with it context lengths and token counts), which must not depend on
    the device the large tensors are generated on."""
    x = torch.randn(n, e, generator=_gen(seed, "cpu"), dtype=torch.float32)
    return (x / x.norm(dim=1, keepdim=True)).to(device)


def channel_scales(w: Workload, device, n_layers: Optional[int] = None):
    """One scale per (layer, kv head, channel), separate for K and V."""
    nl = w.n_layers if n_layers is None else n_layers
    shape = (nl, 1, w.n_kv_heads, w.head_dim)
    if not w.channel_scale:
        one = torch.ones(shape, device=device)
        return one, one.clone()
    rng = np.random.default_rng(w.seed + 1000)
    sk = torch.from_numpy(rng.uniform(0.5, 2.0, size=shape).astype(np.float32)).to(device)
    sv = torch.from_numpy(rng.uniform(0.5, 2.0, size=shape).astype(np.float32)).to(device)
    return sk, sv


def make_pool(w: Workload, device="cpu", n_layers: Optional[int] = None):
    """Cached shot pool.  n_layers < w.n_layers generates only that many pool
    layers (callers that alias layers say so in their report)."""
    nl = w.n_layers if n_layers is None else n_layers
    lengths = shot_lengths(w)
    off = shot_offsets(lengths)
    tokens = int(off[-1])
    g = _gen(w.seed * 7919 + 11, device)
    sk, sv = channel_scales(w, device, nl)
    k = torch.empty(nl, tokens, w.n_kv_heads, w.head_dim, dtype=w.torch_dtype, device=device)
    v = torch.empty_like(k)
    for l in range(nl):   # layer by layer: bounds the fp32 staging at full size
        x = torch.randn(tokens, w.n_kv_heads, w.head_dim, generator=g, device=device)
        k[l] = (x * sk[l]).to(w.torch_dtype)
        x = torch.randn(tokens, w.n_kv_heads, w.head_dim, generator=g, device=device)
        v[l] = (x * sv[l]).to(w.torch_dtype)
        del x
    emb = _unit_rows(len(lengths), w.emb_dim, w.seed * 7919 + 13, device)
    return {"lengths": lengths, "shot_off": off, "k": k, "v": v, "emb": emb,
            "pool_tokens": tokens, "n_shots": len(lengths)}


def make_query_embeddings(w: Workload, device="cpu") -> torch.Tensor:
    """The q_emb of make_queries alone, for callers that need the selection of a whole batch
    without the per-layer query tensors."""
    return _unit_rows(w.batch, w.emb_dim, w.seed * 7919 + 29, device)


def make_queries(w: Workload, device="cpu", n_layers: Optional[int] = None,
                 n_probes: Optional[int] = None):
    """Query-side tensors: embeddings, un-rotated Q / K_q / V_q per probe and
    layer, and the last-token logits of every probe."""
    nl = w.n_layers if n_layers is None else n_layers
    P = len(w.probes) if n_probes is None else n_probes
    g = _gen(w.seed * 7919 + 23, device)
    sk, sv = channel_scales(w, device, nl)
    q_emb = make_query_embeddings(w, device)
    shape_q = (w.batch, nl, P, w.t_q, w.n_q_heads, w.head_dim)
    shape_kv = (w.batch, nl, P, w.t_q, w.n_kv_heads, w.head_dim)
    q = torch.randn(shape_q, generator=g, device=device).to(w.torch_dtype)
    skq = sk.view(1, nl, 1, 1, w.n_kv_heads, w.head_dim)
    svq = sv.view(1, nl, 1, 1, w.n_kv_heads, w.head_dim)
    kq = (torch.randn(shape_kv, generator=g, device=device) * skq).to(w.torch_dtype)
    vq = (torch.randn(shape_kv, generator=g, device=device) * svq).to(w.torch_dtype)
    ldt = torch.float32 if w.logits_dtype == "fp32" else torch.bfloat16
    logits = (torch.randn(w.batch * P, w.vocab, generator=g, device=device)
              * w.logits_std).to(ldt)
    return {"q_emb": q_emb, "q": q, "kq": kq, "vq": vq, "logits": logits}


def to_f64(t: torch.Tensor) -> np.ndarray:
    """Exact widening of stored fp32 / bf16 values for the CPU oracle."""
    return t.detach().to("cpu").to(torch.float64).numpy()
