"""Host driver that calls the four C-ABI steps in order for a batch of queries.

It owns the device buffers (assembled cache, offsets, workspaces, outputs) so a
caller can run many queries without allocating; it does no arithmetic itself.
Layers are processed in chunks of `layers_per_call`: assemble the chunk's cache,
attend over it, reuse the buffer for the next chunk.  Query-side tensors come as one
tensor per chunk, [B][layers in chunk][P][T_q][heads][d] (in a model, the queries of a
later layer do not exist before the earlier layers have run).
"""
from __future__ import annotations

from typing import Optional, Sequence

import torch

from . import binding as ab


class ReusePath:
    def __init__(self, model: ab.ModelT, pool: ab.Pool, batch: int, k: int, probes: Sequence[int],
                 t_q: int, vocab: int, ctx_cap: int, layers_per_call: Optional[int] = None,
                 attn_flags: int = 0, device="cuda"):
        self.model, self.pool = model, pool
        self.B, self.k, self.probes, self.t_q, self.vocab = batch, k, list(probes), t_q, vocab
        self.P = len(self.probes)
        self.ctx_cap = int(ctx_cap)
        self.nl = model.n_layers
        self.lpc = self.nl if layers_per_call is None else int(layers_per_call)
        self.attn_flags = attn_flags
        dt = torch.float32 if model.dtype == ab.F32 else torch.bfloat16
        hkv, hq, d = model.n_kv_heads, model.n_q_heads, model.head_dim
        u8 = dict(dtype=torch.uint8, device=device)
        self.status = torch.zeros(1, dtype=torch.int32, device=device)
        self.sel_idx = torch.empty((batch, k), dtype=torch.int32, device=device)
        self.sel_score = torch.empty((batch, k), dtype=torch.float32, device=device)
        self.ctx_off = torch.empty((batch, k + 1), dtype=torch.int64, device=device)
        self.chunks = [(lb, min(self.nl, lb + self.lpc)) for lb in range(0, self.nl, self.lpc)]
        self._ctx_shape = lambda nl: (batch, nl, self.ctx_cap, hkv, d)
        n_ctx = batch * self.lpc * self.ctx_cap * hkv * d
        self.k_buf = torch.empty(n_ctx, dtype=dt, device=device)
        self.v_buf = torch.empty(n_ctx, dtype=dt, device=device)
        self.out = [torch.empty((batch, le - lb, self.P, t_q, hq, d), dtype=dt, device=device)
                    for lb, le in self.chunks]
        self.H = torch.empty((batch * self.P,), dtype=torch.float32, device=device)
        self.first_ok = torch.empty((batch,), dtype=torch.int32, device=device)
        self.ws_select = torch.empty(max(256, ab.adapshot_select_workspace_bytes(pool.c.n_shots, batch, k)), **u8)
        self.ws_attn = torch.empty(max(256, ab.adapshot_attn_workspace_bytes(model, batch, self.P, t_q, self.lpc,
                                                                              self.ctx_cap)), **u8)
        self.ws_entropy = torch.empty(max(256, ab.adapshot_entropy_workspace_bytes(batch * self.P, vocab)), **u8)

    def select(self, q_emb: torch.Tensor):
        ab.adapshot_select(self.pool, q_emb, self.k, self.sel_idx, self.sel_score, self.ws_select, self.status)

    def ctx_views(self, nl: int):
        shape = self._ctx_shape(nl)
        n = shape[0] * shape[1] * shape[2] * shape[3] * shape[4]
        return self.k_buf[:n].view(shape), self.v_buf[:n].view(shape)

    def assemble(self, layer_begin: int, layer_end: int):
        k_ctx, v_ctx = self.ctx_views(layer_end - layer_begin)
        ab.adapshot_assemble_kv(self.model, self.pool, self.sel_idx, layer_begin, layer_end,
                                k_ctx, v_ctx, self.ctx_cap, self.ctx_off, self.status)

    def attend(self, q, kq, vq, out, layer_begin: int, layer_end: int):
        k_ctx, v_ctx = self.ctx_views(layer_end - layer_begin)
        ab.adapshot_query_attn(self.model, k_ctx, v_ctx, self.ctx_cap, self.ctx_off,
                               self.k, self.probes, q, kq, vq, layer_begin, layer_end, out, None,
                               self.ws_attn, self.status, flags=self.attn_flags)

    def entropy(self, logits: torch.Tensor, tau: float):
        ab.adapshot_entropy(logits, self.H, tau, self.P, self.first_ok, self.ws_entropy, self.status)

    def run(self, q_emb, q_chunks, kq_chunks, vq_chunks, logits, tau: float = 0.65):
        """One pass of the whole path; everything is enqueued on the current stream.
        q_chunks[i] / kq_chunks[i] / vq_chunks[i] belong to layer chunk self.chunks[i]."""
        self.select(q_emb)
        for i, (lb, le) in enumerate(self.chunks):
            self.assemble(lb, le)
            self.attend(q_chunks[i], kq_chunks[i], vq_chunks[i], self.out[i], lb, le)
        self.entropy(logits, tau)
        return self.out, self.H, self.first_ok
