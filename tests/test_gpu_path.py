"""The whole hot path (select -> assemble -> attention -> entropy) through the host
driver against the oracle chain, at the tolerances stated for each step."""
import numpy as np
import pytest
import torch

from oracle import adapshot_oracle as orc
from paper_2605_03644_b200 import workloads as wl
from tests import helpers as hp

pytestmark = pytest.mark.gpu


def oracle_path(w, pool, qs, nl, tau, k_pos_mode=0):
    """Oracle results for every query of the workload (K' kept in fp64, never rounded)."""
    sel, _ = orc.select_topk(hp.f64(qs["q_emb"]), hp.f64(pool["emb"]), w.k)
    off = orc.plan_offsets(sel, pool["shot_off"])
    kp, vp = hp.f64(pool["k"][:nl]), hp.f64(pool["v"][:nl])
    outs = []
    for b in range(w.batch):
        kc, vc, _ = orc.assemble_kv(kp, vp, pool["shot_off"], sel[b], w.rope_base, k_pos_mode)
        L_list = [int(off[b, n]) for n in w.probes]
        per_layer = [orc.query_attn(hp.f64(qs["q"][b, l]), hp.f64(qs["kq"][b, l]), hp.f64(qs["vq"][b, l]),
                                    kc[l], vc[l], L_list, w.rope_base)[0] for l in range(nl)]
        outs.append(np.stack(per_layer))
    H = orc.entropy(hp.f64(qs["logits"]))
    return sel, off, np.stack(outs), H, orc.first_ok(H, tau, len(w.probes))


def run_gpu_path(w, pool, qs, nl, tau, layers_per_call=None, ctx_cap=None, overlap=False, fused=False, vpool=False):
    from paper_2605_03644_b200 import binding as ab
    from paper_2605_03644_b200.pipeline import ReusePath
    dp = hp.dev_pool(ab, pool)
    model = hp.model_of(ab, w, n_layers=nl)
    cap = ctx_cap or w.k * w.len_hi
    path = ReusePath(model, dp, w.batch, w.k, w.probes, w.t_q, w.vocab, cap, layers_per_call, overlap=overlap,
                     fused=fused, vpool=vpool)
    chunk = lambda x: [x[:, lb:le].contiguous().cuda() for lb, le in path.chunks]
    out, H, fo = path.run(qs["q_emb"].cuda(), chunk(qs["q"]), chunk(qs["kq"]), chunk(qs["vq"]),
                          qs["logits"].cuda(), tau)
    torch.cuda.synchronize()
    assert path.status.item() == 0
    return path, torch.cat(out, dim=1)


def _to_bf16_inputs(w, pool, qs):
    for key in ("k", "v"):
        pool[key] = pool[key].to(torch.bfloat16)
    for key in ("q", "kq", "vq"):
        qs[key] = qs[key].to(torch.bfloat16)
    return w.scaled(dtype="bf16")


def _check(w, nl, layers_per_call=None, tau=None, overlap=False, fused=False, vpool=False):
    pool, qs = wl.make_pool(w, n_layers=nl), wl.make_queries(w, n_layers=nl)
    if w.dtype == "fp32":     # the attention kernel is bf16: both sides get the same rounded inputs
        w = _to_bf16_inputs(w, pool, qs)
    H_want = orc.entropy(hp.f64(qs["logits"]))
    tau = float(np.median(H_want)) + 1e-2 if tau is None else tau
    sel, off, out_want, H_want, fo_want = oracle_path(w, pool, qs, nl, tau)
    path, out = run_gpu_path(w, pool, qs, nl, tau, layers_per_call, overlap=overlap, fused=fused, vpool=vpool)
    assert np.array_equal(path.sel_idx.cpu().numpy(), sel)
    assert np.array_equal(path.ctx_off.cpu().numpy(), off)
    hp.assert_attn_close(out.cpu().double().numpy(), out_want, own_rounding=False)      # the stated bounds alone
    assert np.all(np.abs(path.H.cpu().numpy() - H_want) <= 1e-4 * np.abs(H_want))
    assert np.array_equal(path.first_ok.cpu().numpy(), fo_want)


def test_cfg1_whole_path():
    _check(wl.CONFIGS["cfg1"], 1)


def test_8b_shape_nested_probes_two_layer_chunks():
    w = wl.CONFIGS["cfg2"].scaled(n_shots=96, n_layers=3, batch=2, k=24, probes=(3, 6, 12, 24), t_q=48,
                                  vocab=4000, seed=31)
    _check(w, 3, layers_per_call=2)


def test_two_stream_pipeline_three_chunks():
    # gathers on the side stream into two alternating buffers, ordered by events
    w = wl.CONFIGS["cfg2"].scaled(n_shots=80, n_layers=3, batch=2, k=20, probes=(5, 20), t_q=32,
                                  vocab=3000, seed=33)
    _check(w, 3, layers_per_call=1, overlap=True)


@pytest.mark.parametrize("cfg", ["cfg1", "8b", "d64"])
def test_fused_variant_whole_path(cfg):
    # attention straight from the pool, K re-encoded in shared memory: same oracle, same tolerances
    if cfg == "cfg1":
        _check(wl.CONFIGS["cfg1"], 1, fused=True)
    elif cfg == "8b":
        w = wl.CONFIGS["cfg2"].scaled(n_shots=96, n_layers=3, batch=2, k=24, probes=(3, 6, 12, 24), t_q=48,
                                      vocab=4000, seed=31)
        _check(w, 3, layers_per_call=2, fused=True)
    else:
        # head_dim 64, T_q > 128 (two own-token tiles), G = 2, 1-token shots among the lengths
        w = wl.CONFIGS["cfg2"].scaled(n_shots=50, len_lo=1, len_hi=80, n_layers=2, batch=2, k=30, probes=(7, 30),
                                      t_q=150, head_dim=64, n_q_heads=6, n_kv_heads=3, vocab=2000, seed=35)
        _check(w, 2, fused=True)


@pytest.mark.parametrize("cfg", ["cfg1", "8b", "d64"])
def test_v_from_pool_variant_whole_path(cfg):
    # K-only cache (gathered and re-encoded), V tiles copied from the pool inside attention: same oracle,
    # same tolerances
    if cfg == "cfg1":
        _check(wl.CONFIGS["cfg1"], 1, vpool=True)
    elif cfg == "8b":
        w = wl.CONFIGS["cfg2"].scaled(n_shots=96, n_layers=3, batch=2, k=24, probes=(3, 6, 12, 24), t_q=48,
                                      vocab=4000, seed=31)
        _check(w, 3, layers_per_call=2, vpool=True)
    else:
        w = wl.CONFIGS["cfg2"].scaled(n_shots=50, len_lo=1, len_hi=80, n_layers=2, batch=2, k=30, probes=(7, 30),
                                      t_q=150, head_dim=64, n_q_heads=6, n_kv_heads=3, vocab=2000, seed=35)
        _check(w, 2, vpool=True)


def test_v_from_pool_equals_the_full_cache_bit_for_bit():
    # the same values reach the tensor cores in the same order: the two variants' outputs are identical
    w = wl.CONFIGS["cfg2"].scaled(n_shots=128, n_layers=2, batch=2, k=40, probes=(5, 13, 40), t_q=128, vocab=2000,
                                  seed=39)
    pool, qs = wl.make_pool(w, n_layers=2), wl.make_queries(w, n_layers=2)
    _, out_full = run_gpu_path(w, pool, qs, 2, 5.0)
    _, out_vpool = run_gpu_path(w, pool, qs, 2, 5.0, vpool=True)
    assert torch.equal(out_full, out_vpool)


def test_cuda_graph_replay_equals_the_plain_pass():
    from paper_2605_03644_b200 import binding as ab
    from paper_2605_03644_b200.pipeline import ReusePath
    w = wl.CONFIGS["cfg2"].scaled(n_shots=64, batch=1, k=16, probes=(4, 16), t_q=32, vocab=2000, seed=37)
    pool, qs = wl.make_pool(w), wl.make_queries(w)
    dp = hp.dev_pool(ab, pool)
    path = ReusePath(hp.model_of(ab, w), dp, w.batch, w.k, w.probes, w.t_q, w.vocab, w.k * w.len_hi)
    args = [qs["q_emb"].cuda(), [qs["q"].cuda()], [qs["kq"].cuda()], [qs["vq"].cuda()], qs["logits"].cuda()]
    path.run(*args)
    torch.cuda.synchronize()
    want = (path.out[0].clone(), path.H.clone(), path.sel_idx.clone())
    path.capture(*args)
    path.out[0].zero_(); path.H.zero_(); path.sel_idx.zero_()
    path.replay()
    torch.cuda.synchronize()
    assert path.status.item() == 0
    assert torch.equal(path.out[0], want[0]) and torch.equal(path.H, want[1]) and torch.equal(path.sel_idx, want[2])


@pytest.mark.parametrize("fused", [False, True])
def test_host_buffer_pass_equals_the_device_pass(fused):
    """run_host (pinned host tensors in and out, copies on their own streams) returns what
    run returns on device tensors, as a plain pass and as a captured graph, three chunks."""
    from paper_2605_03644_b200 import binding as ab
    from paper_2605_03644_b200.pipeline import ReusePath
    nl = 3
    w = wl.CONFIGS["cfg2"].scaled(n_shots=64, batch=2, k=16, probes=(4, 16), t_q=32, vocab=2000, seed=41)
    pool, qs = wl.make_pool(w, n_layers=nl), wl.make_queries(w, n_layers=nl)
    dp = hp.dev_pool(ab, pool)
    path = ReusePath(hp.model_of(ab, w, n_layers=nl), dp, w.batch, w.k, w.probes, w.t_q, w.vocab,
                     w.k * w.len_hi, 1, fused=fused)
    chunk = lambda x: [x[:, lb:le].contiguous() for lb, le in path.chunks]
    host_in = {"q_emb": qs["q_emb"].pin_memory(), "logits": qs["logits"].pin_memory(),
               "q": [x.pin_memory() for x in chunk(qs["q"])], "kq": [x.pin_memory() for x in chunk(qs["kq"])],
               "vq": [x.pin_memory() for x in chunk(qs["vq"])]}
    on_dev = lambda v: [x.cuda() for x in v] if isinstance(v, list) else v.cuda()
    dev_ref = {n: on_dev(v) for n, v in host_in.items()}
    path.run(dev_ref["q_emb"], dev_ref["q"], dev_ref["kq"], dev_ref["vq"], dev_ref["logits"])
    torch.cuda.synchronize()
    want = {"out": [o.cpu() for o in path.out], "H": path.H.cpu(), "first_ok": path.first_ok.cpu(),
            "sel_idx": path.sel_idx.cpu()}
    dev_in = {n: ([torch.zeros_like(x) for x in v] if isinstance(v, list) else torch.zeros_like(v))
              for n, v in dev_ref.items()}
    host_out = {n: ([torch.zeros_like(x).pin_memory() for x in v] if isinstance(v, list)
                    else torch.zeros_like(v).pin_memory()) for n, v in want.items()}

    def same():
        torch.cuda.synchronize()
        assert path.status.item() == 0
        for n, v in want.items():
            pairs = zip(v, host_out[n]) if isinstance(v, list) else [(v, host_out[n])]
            assert all(torch.equal(a, b) for a, b in pairs), n

    path.run_host(host_in, dev_in, host_out)
    same()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        path.run_host(host_in, dev_in, host_out)
    for v in host_out.values():
        for x in (v if isinstance(v, list) else [v]):
            x.zero_()
    graph.replay()
    same()


@pytest.mark.parametrize("fused", [False, True])
def test_paper_literal_key_store_whole_path(fused):
    """k_pos_mode 1 (pool K stored rotated at shot-local positions, angle = the shot's offset,
    Eq. 7 as printed), materialised and fused, against the oracle chain in the same mode."""
    from paper_2605_03644_b200 import binding as ab
    from paper_2605_03644_b200.pipeline import ReusePath
    nl = 2
    w = wl.CONFIGS["cfg2"].scaled(n_shots=80, batch=2, k=24, probes=(5, 24), t_q=40, vocab=1800, seed=61)
    pool, qs = wl.make_pool(w, n_layers=nl), wl.make_queries(w, n_layers=nl)
    tau = 7.0
    sel, off, out_want, H_want, fo_want = oracle_path(w, pool, qs, nl, tau, k_pos_mode=1)
    # the mode matters: the same stored values read as position-free keys give another result
    _, _, out_mode0, _, _ = oracle_path(w, pool, qs, nl, tau, k_pos_mode=0)
    assert np.abs(out_mode0 - out_want).max() > 0.1
    dp = hp.dev_pool(ab, pool)
    model = hp.model_of(ab, w, n_layers=nl, k_pos_mode=1)
    path = ReusePath(model, dp, w.batch, w.k, w.probes, w.t_q, w.vocab, w.k * w.len_hi, 1, fused=fused)
    chunk = lambda x: [x[:, lb:le].contiguous().cuda() for lb, le in path.chunks]
    out, H, fo = path.run(qs["q_emb"].cuda(), chunk(qs["q"]), chunk(qs["kq"]), chunk(qs["vq"]), qs["logits"].cuda(), tau)
    torch.cuda.synchronize()
    assert path.status.item() == 0
    assert np.array_equal(path.sel_idx.cpu().numpy(), sel) and np.array_equal(path.ctx_off.cpu().numpy(), off)
    hp.assert_attn_close(torch.cat(out, dim=1).cpu().double().numpy(), out_want, own_rounding=False)
