"""Multi-round probing (Sec. 4.1; the case study of Sec. 5): host logic on the CPU, the driver
against the oracle chain on the GPU."""
import numpy as np
import pytest
import torch

from oracle import adapshot_oracle as orc
from paper_2605_03644_b200 import workloads as wl
from tests import helpers as hp


def test_schedule_and_stop_bookkeeping():
    from paper_2605_03644_b200.adaptive import first_stops, probe_schedule
    # the case study's schedule: four probes per round, step 4, from 4 shots
    assert probe_schedule(4, 4, 4, 2) == [[4, 8, 12, 16], [20, 24, 28, 32]]
    assert probe_schedule(1, 1, 1, 3) == [[1], [2], [3]]
    with pytest.raises(ValueError):
        probe_schedule(0, 4, 4, 2)
    # per-round results of the threshold rule -> first (round, probe) per query
    assert first_stops([[-1, 0, -1], [2, 1, -1]]) == [(1, 2), (0, 0), (-1, -1)]
    assert first_stops([]) == []
    # the same bookkeeping as the oracle's rule on the paper's printed entropies
    rows = [l.split() for l in open(hp.golden("paper_case_study_entropies.txt")) if l.strip() and l[0] != "#"]
    H = np.array([float(r[1]) for r in rows])
    per_round = [orc.first_ok(H[:4], 0.65, 4).tolist(), orc.first_ok(H[4:], 0.65, 4).tolist()]
    assert first_stops(per_round) == [(1, 2)]


@pytest.mark.gpu
def test_probe_rounds_driver_against_the_oracle():
    from paper_2605_03644_b200 import binding as ab
    from paper_2605_03644_b200.adaptive import ProbeRounds
    nl, n0, step, m, rounds = 2, 4, 4, 4, 2
    base = wl.CONFIGS["cfg2"].scaled(n_shots=96, batch=3, k=32, probes=(32,), t_q=32, vocab=1500, seed=53)
    pool = wl.make_pool(base, n_layers=nl)
    schedule = [[n0 + (r * m + i) * step for i in range(m)] for r in range(rounds)]
    # per-round query tensors from the seeded generator; logits scaled so that the entropy falls
    # with the shot count and crosses the threshold at a different probe for every query
    ws = [base.scaled(k=s[-1], probes=tuple(s), seed=53) for s in schedule]
    qs = [wl.make_queries(w, n_layers=nl) for w in ws]
    q_emb = qs[0]["q_emb"]
    sharp = torch.tensor([[1.0, 1.0, 1.0, 1.0, 1.0, 1.0, 6.0, 6.0],      # query 0: 28 shots (round 2)
                          [1.0, 6.0, 6.0, 6.0, 6.0, 6.0, 6.0, 6.0],      # query 1: 8 shots (round 1)
                          [1.0, 1.0, 1.0, 1.0, 1.0, 1.0, 1.0, 1.0]])     # query 2: never
    for r in range(rounds):
        lg = qs[r]["logits"].view(base.batch, m, -1)
        qs[r]["logits"] = (lg * sharp[:, r * m:(r + 1) * m, None]).reshape(base.batch * m, -1).contiguous()
        qs[r]["q_emb"] = q_emb
    H_rounds = [orc.entropy(hp.f64(qs[r]["logits"])).reshape(base.batch, m) for r in range(rounds)]
    tau = float(0.5 * (H_rounds[1][0, 2] + H_rounds[1][0, 1]))          # between query 0's 24- and 28-shot probes
    want_stops, want_rounds = orc.probe_rounds(H_rounds, schedule, tau)
    assert [s[2] for s in want_stops] == [28, 8, -1] and want_rounds == 2   # the generator does what the comments say

    model = hp.model_of(ab, base, n_layers=nl)
    dp = hp.dev_pool(ab, pool)
    drv = ProbeRounds(model, dp, base.batch, n0, step, m, rounds, base.t_q, base.vocab, schedule[-1][-1] * base.len_hi)
    outs, Hs = [], []

    def inputs(r, probes):
        assert probes == schedule[r]
        return (qs[r]["q"].cuda(), qs[r]["kq"].cuda(), qs[r]["vq"].cuda(), qs[r]["logits"].cuda())

    def grab(r, d):
        outs.append(d.out.cpu().clone())
        Hs.append(d.H.cpu().numpy().reshape(base.batch, m).copy())

    res = drv.run(q_emb.cuda(), inputs, tau, on_round=grab)
    assert res["rounds_run"] == want_rounds
    assert res["stops"] == [(s[0], s[1]) for s in want_stops]
    assert res["n_star"] == [s[2] for s in want_stops]
    for r in range(res["rounds_run"]):
        assert np.all(np.abs(Hs[r] - H_rounds[r]) <= 1e-4 * np.abs(H_rounds[r]))
    # the rounds' attention outputs against the oracle chain (selection, re-encode, attention)
    from tests.test_gpu_path import oracle_path
    for r in range(res["rounds_run"]):
        w_r = ws[r].scaled(dtype="bf16")
        sel, off, out_want, _, _ = oracle_path(w_r, pool, qs[r], nl, tau)
        assert np.array_equal(drv.sel_idx.cpu().numpy()[:, :schedule[r][-1]], sel)      # nested prefixes
        # (a 4-shot context averages so few values that |O| reaches 4 and more: the shared bound
        # allows the bf16 result's own rounding on top of the stated tolerance)
        hp.assert_attn_close(outs[r].double().numpy(), out_want, what=r)
