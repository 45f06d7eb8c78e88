"""Host driver that calls the four C-ABI steps in order for a batch of queries.

It owns the device buffers (assembled cache, offsets, workspaces, outputs) so a
caller can run many queries without allocating; it does no arithmetic itself.
Layers are processed in chunks of `layers_per_call`: assemble the chunk's cache,
attend over it, reuse the buffer for the next chunk.  `fused=True` skips the assembled
cache: attention reads the pool and re-encodes K on the fly.  `vpool=True` assembles the
re-encoded K only and lets attention read V from the pool (the re-encode leaves V as it is).  `overlap=True` double-buffers the
cache and enqueues the gather of chunk i+1 on a second stream; on B200 the persistent
attention CTAs leave no room for a second resident kernel, so the two do not actually run
together and the default is off.  Query-side tensors come as one tensor per chunk, [B][layers in chunk][P][T_q][heads][d] (in a model, the queries of a
later layer do not exist before the earlier layers have run).
"""
from __future__ import annotations

from typing import Optional, Sequence

import torch

from . import binding as ab


def layer_chunks(n_layers: int, lpc: int, ramp: bool = False):
    """Layer ranges of one pass: chunks of lpc layers; with ramp (and room for it) the first and the last
    chunk are a quarter of that and their neighbours make up for it ([s, lpc - s, lpc, ..., lpc - s, s]).
    For a caller whose tensors live in host memory the first chunk's upload and the last chunk's download
    are the only copies no kernel runs beside, so they are kept short."""
    small = max(1, lpc // 4)
    if not ramp or lpc < 2 or n_layers < 2 * lpc:
        sizes = [min(lpc, n_layers - lb) for lb in range(0, n_layers, lpc)]
    else:
        middle = n_layers - 2 * lpc
        sizes = [small, lpc - small] + [min(lpc, middle - lb) for lb in range(0, middle, lpc)] + [lpc - small, small]
    out, lb = [], 0
    for n in sizes:
        out.append((lb, lb + n))
        lb += n
    return out


class ReusePath:
    def __init__(self, model: ab.ModelT, pool: ab.Pool, batch: int, k: int, probes: Sequence[int],
                 t_q: int, vocab: int, ctx_cap: int, layers_per_call: Optional[int] = None,
                 overlap: bool = False, fused: bool = False, entropy_overlap: bool = False,
                 vpool: Optional[bool] = False, ramp: bool = False, device="cuda"):
        self.model, self.pool = model, pool
        self.B, self.k, self.probes, self.t_q, self.vocab = batch, k, list(probes), t_q, vocab
        self.P = len(self.probes)
        self.ctx_cap = int(ctx_cap)
        self.nl = model.n_layers
        self.lpc = self.nl if layers_per_call is None else int(layers_per_call)
        dt = torch.float32 if model.dtype == ab.F32 else torch.bfloat16
        hkv, hq, d = model.n_kv_heads, model.n_q_heads, model.head_dim
        u8 = dict(dtype=torch.uint8, device=device)
        self.status = torch.zeros(1, dtype=torch.int32, device=device)
        self.sel_idx = torch.empty((batch, k), dtype=torch.int32, device=device)
        self.sel_score = torch.empty((batch, k), dtype=torch.float32, device=device)
        self.ctx_off = torch.empty((batch, k + 1), dtype=torch.int64, device=device)
        self.chunks = layer_chunks(self.nl, self.lpc, ramp)
        self.fused = bool(fused)
        if vpool is None:
            # measured choice: a cache that stays in L2 between the gather and the attention (a single
            # layer of one query) is cheapest to read in full; anything larger is better off with the
            # K-only cache, whose gather moves half the bytes - unless a KV head has so many query rows
            # (more than 1024) that the gather is a small share of the call anyway
            vpool = (batch * self.lpc * self.ctx_cap * 2 * hkv * d * (4 if model.dtype == ab.F32 else 2) > (128 << 20)
                     and t_q * (hq // hkv) <= 1024)
        self.vpool = bool(vpool) and not self.fused and model.dtype != ab.F32
        self.overlap = bool(overlap) and len(self.chunks) > 1 and not self.fused
        n_ctx = batch * self.lpc * self.ctx_cap * hkv * d
        n_buf = 0 if self.fused else (2 if self.overlap else 1)     # the fused variant has no assembled cache
        self.k_bufs = [torch.empty(n_ctx, dtype=dt, device=device) for _ in range(n_buf)]
        self.v_bufs = [torch.empty(0 if self.vpool else n_ctx, dtype=dt, device=device) for _ in range(n_buf)]
        self.out = [torch.empty((batch, le - lb, self.P, t_q, hq, d), dtype=dt, device=device)
                    for lb, le in self.chunks]
        self.H = torch.empty((batch * self.P,), dtype=torch.float32, device=device)
        self.first_ok = torch.empty((batch,), dtype=torch.int32, device=device)
        self.ws_select = torch.empty(max(256, ab.adapshot_select_workspace_bytes(pool.c.n_shots, batch, k)), **u8)
        ws_fn = (ab.adapshot_attn_fused_workspace_bytes if self.fused else
                 ab.adapshot_attn_vpool_workspace_bytes if self.vpool else ab.adapshot_attn_workspace_bytes)
        self.ws_attn = torch.empty(max(256, ws_fn(model, batch, self.P, t_q, self.lpc, self.ctx_cap)), **u8)
        self.ws_entropy = torch.empty(max(256, ab.adapshot_entropy_workspace_bytes(batch * self.P, vocab)), **u8)
        # In the method the probe's logits come out of the model after the probe attention (Eq. 2
        # follows Eq. 1), so the entropy step runs after the last attention call.  With
        # entropy_overlap=True it runs on a second stream beside the pass instead (for callers
        # whose logits are already there, e.g. those of the previous round of probes).
        self.entropy_overlap = bool(entropy_overlap)
        self.side = torch.cuda.Stream(device=device)
        self.ev_begin, self.ev_entropy = torch.cuda.Event(), torch.cuda.Event()
        if self.overlap:
            self.ev_plan = torch.cuda.Event()
            self.ev_asm = [torch.cuda.Event() for _ in range(2)]
            self.ev_attn = [torch.cuda.Event() for _ in range(2)]

    def select(self, q_emb: torch.Tensor):
        ab.adapshot_select(self.pool, q_emb, self.k, self.sel_idx, self.sel_score, self.ws_select, self.status)

    def plan(self):
        """Destination offsets of the selected shots (and the capacity check)."""
        ab.adapshot_assemble_kv(self.model, self.pool, self.sel_idx, 0, 1, None, None, self.ctx_cap,
                                self.ctx_off, self.status)

    def ctx_views(self, nl: int, buf: int = 0):
        shape = (self.B, nl, self.ctx_cap, self.model.n_kv_heads, self.model.head_dim)
        n = shape[0] * shape[1] * shape[2] * shape[3] * shape[4]
        return self.k_bufs[buf][:n].view(shape), (None if self.vpool else self.v_bufs[buf][:n].view(shape))

    def assemble(self, layer_begin: int, layer_end: int, buf: int = 0, keep_plan: bool = False):
        k_ctx, v_ctx = self.ctx_views(layer_end - layer_begin, buf)
        flags = (ab.ASSEMBLE_KEEP_PLAN if keep_plan else 0) | (ab.ASSEMBLE_K_ONLY if self.vpool else 0)
        ab.adapshot_assemble_kv(self.model, self.pool, self.sel_idx, layer_begin, layer_end,
                                k_ctx, v_ctx, self.ctx_cap, self.ctx_off, self.status, flags=flags)

    def attend(self, q, kq, vq, out, layer_begin: int, layer_end: int, buf: int = 0, probes=None):
        """Attention of the probes (default: all of them; a sub-list must be ascending) over the cache."""
        k_ctx, v_ctx = self.ctx_views(layer_end - layer_begin, buf)
        probes = self.probes if probes is None else list(probes)
        if self.vpool:
            ab.adapshot_query_attn_vpool(self.model, self.pool, self.sel_idx, k_ctx, self.ctx_cap, self.ctx_off,
                                         probes, q, kq, vq, layer_begin, layer_end, out, None,
                                         self.ws_attn, self.status)
            return
        ab.adapshot_query_attn(self.model, k_ctx, v_ctx, self.ctx_cap, self.ctx_off,
                               self.k, probes, q, kq, vq, layer_begin, layer_end, out, None,
                               self.ws_attn, self.status)

    def attend_fused(self, q, kq, vq, out, layer_begin: int, layer_end: int):
        ab.adapshot_query_attn_fused(self.model, self.pool, self.sel_idx, self.ctx_off, self.ctx_cap,
                                     self.probes, q, kq, vq, layer_begin, layer_end, out, None,
                                     self.ws_attn, self.status)

    def entropy(self, logits: torch.Tensor, tau: float):
        ab.adapshot_entropy(logits, self.H, tau, self.P, self.first_ok, self.ws_entropy, self.status)

    def run(self, q_emb, q_chunks, kq_chunks, vq_chunks, logits, tau: float = 0.65):
        """One pass of the whole path; everything is enqueued on the current stream (the
        gathers of a multi-chunk pass on the side stream, ordered by events).
        q_chunks[i] / kq_chunks[i] / vq_chunks[i] belong to layer chunk self.chunks[i]."""
        main = torch.cuda.current_stream()
        if self.entropy_overlap:
            self.ev_begin.record(main)
            self.side.wait_event(self.ev_begin)
            with torch.cuda.stream(self.side):
                self.entropy(logits, tau)
                self.ev_entropy.record(self.side)
        self.select(q_emb)
        if self.fused:
            self.plan()
            for i, (lb, le) in enumerate(self.chunks):
                self.attend_fused(q_chunks[i], kq_chunks[i], vq_chunks[i], self.out[i], lb, le)
        elif not self.overlap:
            self.plan()
            for i, (lb, le) in enumerate(self.chunks):
                self.assemble(lb, le, keep_plan=True)
                self.attend(q_chunks[i], kq_chunks[i], vq_chunks[i], self.out[i], lb, le)
        else:
            self.plan()
            self.ev_plan.record(main)
            self.side.wait_event(self.ev_plan)
            for i, (lb, le) in enumerate(self.chunks):
                buf = i & 1
                with torch.cuda.stream(self.side):
                    if i >= 2:
                        self.side.wait_event(self.ev_attn[buf])     # the buffer's last reader
                    self.assemble(lb, le, buf, keep_plan=True)
                    self.ev_asm[buf].record(self.side)
                main.wait_event(self.ev_asm[buf])
                self.attend(q_chunks[i], kq_chunks[i], vq_chunks[i], self.out[i], lb, le, buf)
                self.ev_attn[buf].record(main)
        if self.entropy_overlap:
            main.wait_event(self.ev_entropy)
        else:
            self.entropy(logits, tau)
        return self.out, self.H, self.first_ok

    # ---- the same pass for a caller whose tensors live in host memory
    def run_host(self, host_in: dict, dev_in: dict, host_out: dict, tau: float = 0.65):
        """One pass with pinned host inputs and pinned host results; no arithmetic here.

        host_in / dev_in: {"q_emb", "logits", "q": [...], "kq": [...], "vq": [...]} (one tensor per
        layer chunk), the same shapes on both sides; host_out: {"out": [...], "H", "first_ok",
        "sel_idx"}.  Every upload goes through one copy stream in the order it is needed (query
        embeddings, the chunks' query-side tensors, the logits), every download through another
        (the selection, each chunk's output while the next chunk is computed, the entropies); the
        compute stream issues no copy itself and waits only for the bytes its next kernel reads
        (with entropy_overlap the logits, the entropy step and its results use the side stream).
        PCIe carries both directions at once.  Everything is
        joined back to the current stream before returning (the results are complete once that
        stream is synchronised), so the pass can also be captured into a graph."""
        if self.overlap:
            raise ValueError("the two-stream gather pass has no host variant")
        if not hasattr(self, "h2d"):
            dev = self.status.device
            self.h2d, self.d2h = torch.cuda.Stream(device=dev), torch.cuda.Stream(device=dev)
            self.ev_in = [torch.cuda.Event() for _ in self.chunks]
            self.ev_out = [torch.cuda.Event() for _ in self.chunks]
            self.ev_d2h = torch.cuda.Event()
            self.ev_qemb, self.ev_sel = torch.cuda.Event(), torch.cuda.Event()
        main = torch.cuda.current_stream()
        self.ev_begin.record(main)
        for s in (self.h2d, self.d2h) + ((self.side,) if self.entropy_overlap else ()):
            s.wait_event(self.ev_begin)
        # The compute stream issues no copy of its own: a copy waits in its engine's queue behind
        # whatever was submitted to that engine before, and a few KB stuck behind gigabytes would stall
        # the kernels that follow it in the stream.  Uploads go through the h2d stream in the order
        # they are needed (the query embeddings first, the logits last unless the entropy step runs
        # beside the pass), downloads through the d2h stream.
        with torch.cuda.stream(self.h2d):
            dev_in["q_emb"].copy_(host_in["q_emb"], non_blocking=True)
            self.ev_qemb.record(self.h2d)
        if self.entropy_overlap:
            with torch.cuda.stream(self.side):
                dev_in["logits"].copy_(host_in["logits"], non_blocking=True)
                self.entropy(dev_in["logits"], tau)
                host_out["H"].copy_(self.H, non_blocking=True)
                host_out["first_ok"].copy_(self.first_ok, non_blocking=True)
                self.ev_entropy.record(self.side)
        with torch.cuda.stream(self.h2d):
            for i in range(len(self.chunks)):
                for name in ("q", "kq", "vq"):
                    dev_in[name][i].copy_(host_in[name][i], non_blocking=True)
                self.ev_in[i].record(self.h2d)
            if not self.entropy_overlap:      # needed only after the last attention call: behind the bulk
                dev_in["logits"].copy_(host_in["logits"], non_blocking=True)
                self.ev_entropy.record(self.h2d)
        main.wait_event(self.ev_qemb)
        self.select(dev_in["q_emb"])
        self.plan()
        self.ev_sel.record(main)
        with torch.cuda.stream(self.d2h):
            self.d2h.wait_event(self.ev_sel)
            host_out["sel_idx"].copy_(self.sel_idx, non_blocking=True)
        for i, (lb, le) in enumerate(self.chunks):
            if not self.fused:
                self.assemble(lb, le, keep_plan=True)
            main.wait_event(self.ev_in[i])
            if self.fused:
                self.attend_fused(dev_in["q"][i], dev_in["kq"][i], dev_in["vq"][i], self.out[i], lb, le)
            else:
                self.attend(dev_in["q"][i], dev_in["kq"][i], dev_in["vq"][i], self.out[i], lb, le)
            self.ev_out[i].record(main)
            with torch.cuda.stream(self.d2h):
                self.d2h.wait_event(self.ev_out[i])
                host_out["out"][i].copy_(self.out[i], non_blocking=True)
        main.wait_event(self.ev_entropy)
        if not self.entropy_overlap:          # the logits are up; the probe follows the last attention call
            self.entropy(dev_in["logits"], tau)
            self.ev_sel.record(main)
            with torch.cuda.stream(self.d2h):
                self.d2h.wait_event(self.ev_sel)
                host_out["H"].copy_(self.H, non_blocking=True)
                host_out["first_ok"].copy_(self.first_ok, non_blocking=True)
        self.ev_d2h.record(self.d2h)
        main.wait_event(self.ev_d2h)
        return host_out

    # ---- the same pass as one CUDA graph: launch-bound small workloads (a few hundred
    # microseconds per pass) lose a visible share to per-launch host work otherwise
    def capture(self, q_emb, q_chunks, kq_chunks, vq_chunks, logits, tau: float = 0.65):
        """Records run(...) on these (static) input tensors into a CUDA graph.  Run one plain
        pass first (first calls query device attributes).  Returns self; replay() launches it."""
        if self.overlap:
            raise ValueError("the two-stream gather pass is not captured")
        self.run(q_emb, q_chunks, kq_chunks, vq_chunks, logits, tau)
        torch.cuda.synchronize()
        self._graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(self._graph):
            self.run(q_emb, q_chunks, kq_chunks, vq_chunks, logits, tau)
        return self

    def replay(self):
        self._graph.replay()
        return self.out, self.H, self.first_ok
