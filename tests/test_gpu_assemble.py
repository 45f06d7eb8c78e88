"""adapshot_assemble_kv vs the fp64 oracle: offsets and V bit-exact; fp32 K within
1e-5 max-abs; bf16 K within half a bf16 step (+1e-5) of the oracle, >= 99 % bit-equal."""
import numpy as np
import pytest
import torch

from oracle import adapshot_oracle as orc
from paper_2605_03644_b200 import workloads as wl
from tests import helpers as hp

pytestmark = pytest.mark.gpu

K_TOL_FP32 = 1e-5     # stated tolerance of the fp32 re-encode


def _compare(w, pool, sel_np, kc, vc, off, nl_begin, nl_end, k_pos_mode=0):
    B = sel_np.shape[0]
    want_off = orc.plan_offsets(sel_np, pool["shot_off"])
    assert np.array_equal(off.cpu().numpy(), want_off), "offsets must be bit-exact"
    kp, vp = hp.f64(pool["k"][nl_begin:nl_end]), hp.f64(pool["v"][nl_begin:nl_end])
    for b in range(B):
        ok, ov, _ = orc.assemble_kv(kp, vp, pool["shot_off"], sel_np[b], w.rope_base, k_pos_mode)
        L = int(want_off[b, -1])
        got_v = vc[b, :, :L].cpu()
        assert torch.equal(got_v.double(), torch.from_numpy(ov)), "V must be a bit copy"
        got_k = kc[b, :, :L].cpu()
        if w.dtype == "fp32":
            err = (got_k.double() - torch.from_numpy(ok)).abs().max().item()
            assert err <= K_TOL_FP32, err
        else:
            # bf16 store: one round-to-nearest-even of the fp32 rotation, so the error is
            # at most half a bf16 step (2^-8 relative) plus the fp32 slack; and nearly
            # every element must equal the rounded oracle value bit for bit
            want = torch.from_numpy(ok)
            err = (got_k.double() - want).abs()
            assert (err <= want.abs() * 2.0 ** -8 + K_TOL_FP32).all(), err.max().item()
            ref = want.to(torch.float32).to(torch.bfloat16)
            assert (hp.bf16_ulp_diff(got_k, ref) == 0).float().mean().item() >= 0.99
        # zero padding up to the 128-token tile edge, untouched canary after it
        pad_end = min((L + 127) // 128 * 128, kc.shape[2])
        assert (kc[b, :, L:pad_end] == 0).all() and (vc[b, :, L:pad_end] == 0).all()
        assert (kc[b, :, pad_end:] == 7.0).all() and (vc[b, :, pad_end:] == 7.0).all()


def test_cfg1_full():
    ab = hp.gpu_binding()
    w = wl.CONFIGS["cfg1"]
    pool = wl.make_pool(w)
    q = wl.make_queries(w)
    dp = hp.dev_pool(ab, pool)
    sel, _, _ = hp.run_select(ab, dp, q["q_emb"], w.k)
    kc, vc, off, st = hp.run_assemble(ab, hp.model_of(ab, w), dp, sel, 300, 0, 1, torch.float32)
    assert st == 0
    _compare(w, pool, sel.cpu().numpy(), kc, vc, off, 0, 1)


@pytest.mark.parametrize("dtype,d,hkv", [("bf16", 128, 8), ("bf16", 64, 2), ("fp32", 128, 3), ("fp32", 64, 1),
                                         ("bf16", 128, 1), ("bf16", 64, 5)])
@pytest.mark.parametrize("k_pos_mode", [0, 1])
def test_ragged_shapes_layers_and_modes(dtype, d, hkv, k_pos_mode):
    ab = hp.gpu_binding()
    w = wl.CONFIGS["cfg2"].scaled(n_layers=3, n_shots=40, len_lo=1, len_hi=70, n_kv_heads=hkv,
                                  n_q_heads=hkv * 2, head_dim=d, dtype=dtype, batch=3, k=17, seed=11 + d + hkv)
    pool = wl.make_pool(w)
    dp = hp.dev_pool(ab, pool)
    rng = np.random.default_rng(3)
    sel_np = rng.integers(0, 40, size=(3, 17)).astype(np.int32)      # arbitrary order, duplicates allowed
    sel_np[1] = np.arange(17)                                        # identity prefix
    sel = torch.from_numpy(sel_np).cuda()
    model = hp.model_of(ab, w, k_pos_mode=k_pos_mode)
    cap = int(orc.plan_offsets(sel_np, pool["shot_off"])[:, -1].max()) + 130
    kc, vc, off, st = hp.run_assemble(ab, model, dp, sel, cap, 1, 3, w.torch_dtype)
    assert st == 0
    _compare(w, pool, sel_np, kc, vc, off, 1, 3, k_pos_mode)


def test_cfg2_shape_spans_many_tiles():
    ab = hp.gpu_binding()
    w = wl.CONFIGS["cfg2"].scaled(n_shots=256)
    pool = wl.make_pool(w)
    q = wl.make_queries(w, n_probes=1)
    dp = hp.dev_pool(ab, pool)
    sel, _, _ = hp.run_select(ab, dp, q["q_emb"], 64)
    cap = 64 * 256
    kc, vc, off, st = hp.run_assemble(ab, hp.model_of(ab, w), dp, sel, cap, 0, 1, torch.bfloat16)
    assert st == 0
    _compare(w, pool, sel.cpu().numpy(), kc, vc, off, 0, 1)


def test_identity_order_reproduces_the_pool_and_large_positions():
    ab = hp.gpu_binding()
    # 70 shots of 1000 tokens: positions reach 70K, the regime where fp32 angles would fail
    w = wl.CONFIGS["cfg1"].scaled(n_shots=70, len_lo=1000, len_hi=1000, k=70)
    pool = wl.make_pool(w)
    dp = hp.dev_pool(ab, pool)
    sel = torch.arange(70, dtype=torch.int32, device="cuda")[None]
    kc, vc, off, st = hp.run_assemble(ab, hp.model_of(ab, w), dp, sel, 70000, 0, 1, torch.float32)
    assert st == 0 and torch.equal(vc[0, 0], pool["v"][0].cuda())
    _compare(w, pool, sel.cpu().numpy(), kc, vc, off, 0, 1)


def test_plan_only_capacity_and_bad_ids():
    ab = hp.gpu_binding()
    w = wl.CONFIGS["cfg1"]
    pool = wl.make_pool(w)
    dp = hp.dev_pool(ab, pool)
    model = hp.model_of(ab, w)
    sel = torch.tensor([[3, 1, 2]], dtype=torch.int32, device="cuda")
    off = torch.zeros((1, 4), dtype=torch.int64, device="cuda")
    st = hp.new_status()
    ab.adapshot_assemble_kv(model, dp, sel, 0, 1, None, None, 0, off, st)
    assert off.tolist() == [[0, 32, 64, 96]] and st.item() == 0
    # capacity too small: reported on the device, nothing written past the capacity
    kc, vc, off, st = hp.run_assemble(ab, model, dp, sel, 80, 0, 1, torch.float32)
    assert st == ab.ECAPACITY
    assert torch.equal(vc[0, 0, :80], torch.cat([pool["v"][0, 96:128], pool["v"][0, 32:64], pool["v"][0, 64:80]]).cuda())
    # an id outside the pool: reported, the slot counts as empty
    bad = torch.tensor([[3, 99, 2]], dtype=torch.int32, device="cuda")
    kc, vc, off, st = hp.run_assemble(ab, model, dp, bad, 128, 0, 1, torch.float32)
    assert st == ab.EINDEX and off.tolist() == [[0, 32, 32, 64]]
    assert torch.equal(vc[0, 0, 32:64], pool["v"][0, 64:96].cuda())


@pytest.mark.parametrize("k_pos_mode", [0, 1])
def test_extending_a_nested_prefix_equals_one_gather(k_pos_mode):
    """adapshot_assemble_kv_from: a cache assembled for the first k1 shots and extended with
    shots k1 .. k2-1 is, bit for bit, the cache assembled for k2 shots at once (K, V, the zero
    fill and the untouched canary), and the extension leaves the first positions alone."""
    ab = hp.gpu_binding()
    w = wl.CONFIGS["cfg2"].scaled(n_shots=60, batch=3, k=20, probes=(20,), seed=71)
    nl = 3
    pool = wl.make_pool(w, n_layers=nl)
    dp = hp.dev_pool(ab, pool)
    rng = np.random.default_rng(71)
    sel_np = np.stack([rng.permutation(w.n_shots)[:w.k] for _ in range(w.batch)]).astype(np.int32)
    sel = torch.from_numpy(sel_np).cuda()
    model = hp.model_of(ab, w, n_layers=nl, k_pos_mode=k_pos_mode)
    cap = w.k * w.len_hi
    want_k, want_v, want_off, st = hp.run_assemble(ab, model, dp, sel, cap, 0, nl, torch.bfloat16)
    assert st == 0
    for k1 in (1, 7, 19):
        sel1 = sel[:, :k1].contiguous()
        kc, vc, off1, st = hp.run_assemble(ab, model, dp, sel1, cap, 0, nl, torch.bfloat16)
        assert st == 0
        # poison the first positions: the extension must not rewrite them
        first = off1[:, k1].cpu().numpy()
        keep_k, keep_v = kc.clone(), vc.clone()
        off2 = torch.full((w.batch, w.k + 1), -1, dtype=torch.int64, device="cuda")
        status = hp.new_status()
        ab.adapshot_assemble_kv_from(model, dp, sel, k1, 0, nl, kc, vc, cap, off2, status)
        torch.cuda.synchronize()
        assert status.item() == 0
        assert torch.equal(off2, want_off)
        assert torch.equal(kc, want_k) and torch.equal(vc, want_v)
        for b in range(w.batch):
            assert torch.equal(kc[b, :, :first[b]], keep_k[b, :, :first[b]])
            assert torch.equal(vc[b, :, :first[b]], keep_v[b, :, :first[b]])
