"""Multi-round probing (paper Sec. 4.1, "adaptive shot count"): rounds of m nested probes,
shot counts n0, n0 + step, ... ; the answer is the smallest shot count whose last-token
entropy (Eq. 2) is at most tau, and probing stops with the round that finds it.

The driver only sequences the C-ABI steps and keeps the books: selection once for the
largest shot count, then per round the gather of the shots the round adds (nested
prefixes share their re-encoded positions, so the earlier shots stay where they are), the
probe attention of the round's m probes over it and the entropy rule on the logits the
caller's model produced for those probes.  It does no arithmetic on tensors itself.
"""
from __future__ import annotations

from typing import Callable, List, Optional, Sequence

import torch

from . import binding as ab


def probe_schedule(n0: int, step: int, m: int, rounds: int) -> List[List[int]]:
    """Shot counts of every round: round r probes n0 + (r*m + i)*step, i < m."""
    if n0 < 1 or step < 1 or m < 1 or rounds < 1:
        raise ValueError("n0, step, m and rounds must be positive")
    return [[n0 + (r * m + i) * step for i in range(m)] for r in range(rounds)]


def first_stops(first_ok_by_round: Sequence[Sequence[int]]):
    """Per query: (round, probe index) of the first probe that met the threshold, given the
    per-round results of the threshold rule (-1 = none in that round); (-1, -1) if never."""
    n_q = len(first_ok_by_round[0]) if first_ok_by_round else 0
    stops = [(-1, -1)] * n_q
    for r, row in enumerate(first_ok_by_round):
        for b, j in enumerate(row):
            if stops[b] == (-1, -1) and int(j) >= 0:
                stops[b] = (r, int(j))
    return stops


class ProbeRounds:
    """Runs the schedule on one batch of queries (all queries advance round by round; a query
    that has stopped is still carried along, its later results are ignored)."""

    def __init__(self, model: ab.ModelT, pool: ab.Pool, batch: int, n0: int, step: int, m: int,
                 rounds: int, t_q: int, vocab: int, ctx_cap: int, device="cuda"):
        self.model, self.pool = model, pool
        self.B, self.m, self.t_q, self.vocab = batch, m, t_q, vocab
        self.schedule = probe_schedule(n0, step, m, rounds)
        self.k_max = self.schedule[-1][-1]
        self.ctx_cap = int(ctx_cap)
        nl, hkv, hq, d = model.n_layers, model.n_kv_heads, model.n_q_heads, model.head_dim
        dt = torch.float32 if model.dtype == ab.F32 else torch.bfloat16
        u8 = dict(dtype=torch.uint8, device=device)
        self.status = torch.zeros(1, dtype=torch.int32, device=device)
        self.sel_idx = torch.empty((batch, self.k_max), dtype=torch.int32, device=device)
        self.sel_score = torch.empty((batch, self.k_max), dtype=torch.float32, device=device)
        self._ctx_off = torch.empty(batch * (self.k_max + 1), dtype=torch.int64, device=device)
        self.k_ctx = torch.empty((batch, nl, self.ctx_cap, hkv, d), dtype=dt, device=device)
        self.v_ctx = torch.empty_like(self.k_ctx)
        self.out = torch.empty((batch, nl, m, t_q, hq, d), dtype=dt, device=device)
        self.H = torch.empty((batch * m,), dtype=torch.float32, device=device)
        self.first_ok = torch.empty((batch,), dtype=torch.int32, device=device)
        self.ws_select = torch.empty(max(256, ab.adapshot_select_workspace_bytes(pool.c.n_shots, batch, self.k_max)), **u8)
        self.ws_attn = torch.empty(max(256, ab.adapshot_attn_workspace_bytes(model, batch, m, t_q, nl, self.ctx_cap)), **u8)
        self.ws_entropy = torch.empty(max(256, ab.adapshot_entropy_workspace_bytes(batch * m, vocab)), **u8)

    def ctx_off(self, k: int) -> torch.Tensor:
        return self._ctx_off[: self.B * (k + 1)].view(self.B, k + 1)

    def run_round(self, r: int, q, kq, vq, logits, tau: float):
        """Extend the cache to round r's largest probe (rounds must be run in order, from 0),
        attend with its m probes, apply the entropy rule to `logits` ([B*m][V], the model's
        last-token logits of those probes)."""
        probes = self.schedule[r]
        k_r = probes[-1]
        nl = self.model.n_layers
        sel_r = self.sel_idx[:, :k_r].contiguous()
        off_r = self.ctx_off(k_r)
        # the earlier rounds' shots are in place already: only the new ones are gathered
        first_new = self.schedule[r - 1][-1] if r > 0 else 0
        ab.adapshot_assemble_kv_from(self.model, self.pool, sel_r, first_new, 0, nl, self.k_ctx, self.v_ctx,
                                     self.ctx_cap, off_r, self.status)
        ab.adapshot_query_attn(self.model, self.k_ctx, self.v_ctx, self.ctx_cap, off_r, k_r, probes,
                               q, kq, vq, 0, nl, self.out, None, self.ws_attn, self.status)
        ab.adapshot_entropy(logits, self.H, tau, self.m, self.first_ok, self.ws_entropy, self.status)

    def run(self, q_emb: torch.Tensor, round_inputs: Callable[[int, List[int]], tuple], tau: float = 0.65,
            on_round: Optional[Callable[[int, "ProbeRounds"], None]] = None):
        """round_inputs(r, probes) -> (q, kq, vq, logits) of round r.  Returns per query the
        stopping (round, probe index), the shot count n* (-1 if the threshold was never met)
        and the rounds that were run.  on_round(r, self) is called after each round's results
        are complete (a caller that wants that round's outputs reads them there)."""
        ab.adapshot_select(self.pool, q_emb, self.k_max, self.sel_idx, self.sel_score, self.ws_select, self.status)
        per_round = []
        for r, probes in enumerate(self.schedule):
            q, kq, vq, logits = round_inputs(r, probes)
            self.run_round(r, q, kq, vq, logits, tau)
            torch.cuda.current_stream().synchronize()
            if self.status.item() != 0:
                raise RuntimeError(f"device status {self.status.item()}: {ab.adapshot_strerror(self.status.item())}")
            per_round.append(self.first_ok.cpu().tolist())
            if on_round is not None:
                on_round(r, self)
            if all(s != (-1, -1) for s in first_stops(per_round)):
                break
        stops = first_stops(per_round)
        n_star = [self.schedule[r][j] if r >= 0 else -1 for r, j in stops]
        return {"stops": stops, "n_star": n_star, "rounds_run": len(per_round)}
