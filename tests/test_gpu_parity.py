"""CUDA path vs the CPU oracle, element by element, through the C ABI."""
import dataclasses

import pytest
import torch

from oracle import specexit_oracle as orc
from paper_2509_24248_b200 import binding, synth
from tests import harness, parity

pytestmark = pytest.mark.gpu


def _wl(**kw):
    return harness.tiny_workload(**kw)


@pytest.mark.parametrize("B,K,lo,hi", [(1, 1, 5, 5), (1, 4, 33, 33), (2, 3, 5, 40), (3, 5, 16, 16), (5, 2, 1, 70)])
def test_chain_tiny(B, K, lo, hi):
    rep = parity.run_chain(harness.build_case(_wl(B=B, K=K, len_lo=lo, len_hi=hi)))
    assert all(0 <= l <= K for l in rep.accept_len)


def test_chain_zero_cached_tokens():
    parity.run_chain(harness.build_case(_wl(B=2, K=3, len_lo=0, len_hi=0)))


@pytest.mark.parametrize("tiled", [False, True])
def test_chain_config0_exact(tiled):
    """The tiny exactness configuration, held to the whole free-running pass: the oracle runs all K rounds
    on its own (no hook) and every draft token, accepted length, exit flag and recover token must be equal,
    every hidden within 2e-2 relative L2 and every signal within 1e-2."""
    wl = synth.workload("C0")
    parity.TILED = tiled
    try:
        rep = parity.run_chain(harness.build_case(wl), strict_free=True)
    finally:
        parity.TILED = False
    print(rep.free.table("C0"))
    assert rep.exempt == [] and rep.exit_near_threshold == []
    assert rep.free.diverged == [] and rep.free.tail_equal is True
    assert rep.free.in_step == [wl.B] * wl.K


@pytest.mark.parametrize("shape_kw", [dict(H=128, n_q=8, n_kv=1, d=16, F=200, V=333),
                                      dict(H=64, n_q=2, n_kv=2, d=32, F=72, V=129),
                                      dict(H=256, n_q=4, n_kv=1, d=64, F=688, V=1000),
                                      dict(H=256, n_q=2, n_kv=1, d=128, F=264, V=515, page=64)])
def test_chain_odd_shapes(shape_kw):
    sh = synth.ModelShape(**{"page": 16, **shape_kw})
    wl = synth.Workload("odd", sh, B=3, mode=synth.CHAIN, K=3, len_lo=3, len_hi=150, seed=5,
                        sigma_lo=0.1, sigma_hi=0.6)
    parity.run_chain(harness.build_case(wl))


@pytest.mark.parametrize("thr", [0.3, 0.5, 0.7, 0.9])
@pytest.mark.parametrize("mask", [0b001, 0b111])
def test_exit_threshold_sweep(thr, mask):
    wl = _wl(B=4, K=4, len_lo=10, len_hi=50, sigma_lo=0.05, sigma_hi=0.3)
    case = harness.build_case(wl)
    # head weights scaled up so that the signals spread over (0, 1)
    w = dict(case.weights)
    w["head"] = (w["head"].to(torch.float32) * 8.0).to(torch.bfloat16)
    case = dataclasses.replace(case, weights=w)
    cfg = harness.default_exit_cfg(wl, thr=(thr, thr, 0.5), dir=(orc.DIR_GT, orc.DIR_GT, orc.DIR_LT), enable_mask=mask)
    parity.run_chain(case, cfg)


def test_exit_split_bitmap_first_only_and_expm1():
    wl = _wl(B=4, K=5, len_lo=10, len_hi=50, sigma_lo=0.0, sigma_hi=0.1)
    case = harness.build_case(wl)
    bm = synth.split_bitmap(wl.shape.V, 3)
    cfg = harness.default_exit_cfg(wl, thr=(0.45, 0.0, 0.0), split_bitmap=bm)
    parity.run_chain(case, cfg)
    cfg = harness.default_exit_cfg(wl, thr=(0.45, 0.0, 0.0), ema_positions=orc.EMA_FIRST_ONLY)
    parity.run_chain(case, cfg)
    # remaining length through exp(z) - 1, thresholded from above
    act = (orc.ACT_SIGMOID, orc.ACT_SIGMOID, orc.ACT_EXPM1)
    cfg = harness.default_exit_cfg(wl, thr=(0.4, 0.4, 0.2), dir=(orc.DIR_GT, orc.DIR_GT, orc.DIR_LT), enable_mask=0b111)
    parity.run_chain(case, cfg, act=act)
    # a sequence that already left the reasoning phase is passed through
    st = orc.ExitState.fresh(wl.B)
    st.thinking[1] = 0
    st.x[2] = torch.tensor([0.9, 0.1, 0.3], dtype=torch.float64)
    st.n_updates[2] = 4
    parity.run_chain(case, harness.default_exit_cfg(wl, thr=(0.45, 0.0, 0.0)), state0=st)


def test_multi_iteration_loop_carries_state():
    wl = _wl(B=3, K=3, len_lo=10, len_hi=30, sigma_lo=0.0, sigma_hi=0.2)
    case = harness.build_case(wl)
    cfg = harness.default_exit_cfg(wl, thr=(0.52, 0.0, 0.0))
    st = orc.ExitState.fresh(wl.B)
    for it in range(3):
        c2 = dataclasses.replace(case, f0=synth._randn_bf16(wl.B, wl.shape.H, 1.0, 0.0, torch.Generator().manual_seed(100 + it)))
        before = st.clone()
        parity.run_chain(c2, cfg, state0=before)
        # advance the oracle-side state the same way for the next round
        model = harness.oracle_model(c2)
        d = orc.draft_chain(model, harness.oracle_kv(c2), c2.f0, c2.t0, wl.K)
        v = orc.verify(model, harness.chain_target_hidden(c2, d), d.cand_tok)
        orc.exit_update(cfg, st, d.slot_signal, d.cand_tok, v.path, v.accept_len, v.recover_tok)


@pytest.mark.parametrize("topk,depth,nodes,B", [(2, 3, 5, 1), (3, 4, 14, 2), (8, 3, 20, 2), (4, 5, 30, 3)])
def test_tree_tiny(topk, depth, nodes, B):
    sh = synth.ModelShape(H=64, n_q=4, n_kv=2, d=16, F=96, V=300, page=16)
    wl = synth.Workload("t", sh, B=B, mode=synth.TREE, K=depth, topk=topk, max_nodes=nodes, len_lo=9, len_hi=60,
                        seed=21, sigma_lo=0.0, sigma_hi=0.3)
    case = harness.build_case(wl)
    w = dict(case.weights)
    w["head"] = (w["head"].to(torch.float32) * 20.0).to(torch.bfloat16)      # peaked distributions
    rep = parity.run_tree(dataclasses.replace(case, weights=w))
    print("tree exempt:", rep.exempt, "accept:", rep.accept_len)


def test_tree_top1_equals_chain_on_gpu():
    sh = synth.ModelShape(H=64, n_q=4, n_kv=2, d=16, F=96, V=300, page=16)
    wl = synth.Workload("t1", sh, B=2, mode=synth.TREE, K=4, topk=1, max_nodes=4, len_lo=9, len_hi=60, seed=22)
    parity.run_tree(harness.build_case(wl))


def test_standalone_entry_points():
    wl = _wl(B=2, K=3, len_lo=7, len_hi=21)
    case = harness.build_case(wl)
    model = harness.oracle_model(case)
    d = orc.draft_chain(model, harness.oracle_kv(case), case.f0, case.t0, wl.K)
    th = harness.chain_target_hidden(case, d)
    sx = parity.make_gpu(case)
    dev = sx.dev
    feat, tok = case.f0.to(dev), case.t0.to(dev)
    for k in range(1, wl.K + 1):
        hid, tok_out, _, sig = sx.sx_draft_step(k, feat, tok)
        torch.cuda.synchronize()
        sx.check_status()
        assert tok_out[:, 0].cpu().tolist() == d.cand_tok[:, k].tolist()
        assert (sig.cpu().double() - d.slot_signal[:, k - 1]).abs().max() < 1e-2
        for b in range(wl.B):
            assert parity._rel_l2(hid[b].cpu().double(), d.hidden[b, k - 1]) < 2e-2
        feat, tok = hid, tok_out[:, 0].contiguous()
    cand = d.cand_tok.to(torch.int32).to(dev)
    tt, L, path, rec = sx.sx_verify(th.to(dev), cand)
    v = orc.verify(model, th, d.cand_tok)
    assert tt.cpu().tolist() == v.target_tok.tolist() and L.cpu().tolist() == v.accept_len.tolist()
    assert rec.cpu().tolist() == v.recover_tok.tolist()
    cfg = harness.default_exit_cfg(wl, thr=(0.5, 0, 0))
    st = sx.new_state(wl.B)
    ef, Lo, ro, sm = sx.sx_exit_update(parity.to_params(sx, cfg), st, d.slot_signal.to(torch.float32).to(dev), cand,
                                       path, L, rec)
    e = orc.exit_update(cfg, orc.ExitState.fresh(wl.B), d.slot_signal, d.cand_tok, v.path, v.accept_len, v.recover_tok)
    assert ef.cpu().tolist() == e.exit_flag.tolist() and Lo.cpu().tolist() == e.accept_len.tolist()
    assert ro.cpu().tolist() == e.recover_tok.tolist()
    assert (sm.cpu().double() - e.smoothed).abs().max() < 1e-6
    sx.check_status()


def test_verify_many_rows_and_ties():
    # more verify rows than one head launch holds; duplicated head rows tie, lower index wins
    sh = synth.ModelShape(H=64, n_q=4, n_kv=2, d=16, F=96, V=777, page=16)
    wl = synth.Workload("v", sh, B=37, mode=synth.CHAIN, K=7, len_lo=4, len_hi=4, seed=9)
    case = harness.build_case(wl)
    w = dict(case.weights)
    w["head"] = w["head"].clone()
    w["head"][600] = w["head"][17]
    w["head"][300] = w["head"][17]
    case = dataclasses.replace(case, weights=w)
    model = harness.oracle_model(case)
    g = torch.Generator().manual_seed(3)
    th = torch.randn(wl.B, wl.K + 1, sh.H, generator=g).to(torch.bfloat16)
    th[0, 0] = (w["head"][17].to(torch.float32) * 40).to(torch.bfloat16)      # argmax lands on the tied rows
    cand = torch.randint(0, sh.V, (wl.B, wl.K + 1), generator=g, dtype=torch.int32)
    sx = parity.make_gpu(case)
    tt, L, path, rec = sx.sx_verify(th.to(sx.dev), cand.to(sx.dev))
    torch.cuda.synchronize()
    o_tt, gap = orc.target_argmax(model, th)
    assert int(tt[0, 0]) == 17 and int(o_tt[0, 0]) == 17
    diff = (tt.cpu().to(torch.int64) != o_tt)
    assert bool((gap[diff] < parity.REL_GAP).all())


def test_bit_identical_on_repeat_and_poisoned_workspace():
    wl = _wl(B=2, K=3, len_lo=20, len_hi=45)
    case = harness.build_case(wl)
    sx = parity.make_gpu(case)
    model = harness.oracle_model(case)
    th = harness.chain_target_hidden(case, orc.draft_chain(model, harness.oracle_kv(case), case.f0, case.t0, wl.K))
    outs = []
    for rep in range(2):
        sx.ws.fill_(0xFF if rep else 0x00)            # scratch content must not matter
        sx.set_kv(case.kv)
        out, st = sx.new_outputs(wl.B), sx.new_state(wl.B)
        sx.sx_spec_exit_iter(parity.to_params(sx, harness.default_exit_cfg(wl)), st, case.f0.to(sx.dev),
                             case.t0.to(sx.dev), th.to(sx.dev), out)
        torch.cuda.synchronize()
        sx.check_status()
        outs.append({k: v.cpu() for k, v in out.items()})
    for k in outs[0]:
        a, b = outs[0][k], outs[1][k]
        if a.dtype.is_floating_point:
            assert torch.equal(a.view(torch.int16 if a.element_size() == 2 else torch.int32),
                               b.view(torch.int16 if b.element_size() == 2 else torch.int32)), k
        else:
            assert torch.equal(a, b), k


def test_errors_are_reported_not_fatal():
    wl = _wl(B=2, K=3, len_lo=20, len_hi=45)
    case = harness.build_case(wl)
    sx = parity.make_gpu(case)
    lib = sx.lib
    # host-detectable: workspace too small
    code = lib.sx_verify(sx.h, 1, 2, 16, 16, None, 16, 16, 16, 3, 16, sx.ws_ptr, 8, sx.status.data_ptr(), 0)
    assert code == -4
    code = lib.sx_verify(sx.h, 1, 2, None, 16, None, 16, 16, 16, 3, 16, sx.ws_ptr, sx.ws_bytes, sx.status.data_ptr(), 0)
    assert code == -1
    # device-detectable: page table too short for the new slots -> status word, no fault
    kv = synth.make_kv(wl.shape, case.kv["cache_len"], 0, wl.seed)
    lens = kv["cache_len"].clone()
    lens[:] = kv["page_table"].shape[1] * wl.shape.page      # cache full, nowhere to append
    kv["cache_len"] = lens
    sx.set_kv(kv)
    out, st = sx.new_outputs(wl.B), sx.new_state(wl.B)
    th = torch.zeros(wl.B, wl.K + 1, wl.shape.H, dtype=torch.bfloat16, device=sx.dev)
    sx.sx_spec_exit_iter(parity.to_params(sx, harness.default_exit_cfg(wl)), st, case.f0.to(sx.dev),
                         case.t0.to(sx.dev), th, out)
    torch.cuda.synchronize()
    assert int(sx.status.item()) == -3
    sx.status.zero_()
    # an out-of-vocabulary token id is reported the same way
    sx.set_kv(case.kv)
    bad = torch.full_like(case.t0, wl.shape.V + 5).to(sx.dev)
    sx.sx_spec_exit_iter(parity.to_params(sx, harness.default_exit_cfg(wl)), st, case.f0.to(sx.dev), bad, th, out)
    torch.cuda.synchronize()
    assert int(sx.status.item()) == -3
    sx.status.zero_()
    # the context is still usable
    parity.run_chain(case, sx=sx)


def test_chain_of_maximum_length():
    """K = 63 draft rounds (64 verify slots): the limit of the per-sequence slot masks."""
    wl = _wl(B=2, K=63, len_lo=1, len_hi=30, sigma_lo=0.0, sigma_hi=0.05)
    rep = parity.run_chain(harness.build_case(wl))
    print("K=63 accept:", rep.accept_len, "exempt:", len(rep.exempt))


@pytest.mark.parametrize("topk,depth", [(8, 8), (7, 10), (1, 64)])
def test_tree_at_the_row_and_slot_limits(topk, depth):
    """1 + topk (depth - 1) drafted rows per sequence up to the 64-row limit, 63 kept nodes (64 slots)."""
    sh = synth.ModelShape(H=64, n_q=4, n_kv=2, d=16, F=96, V=300, page=16)
    rows = 1 + topk * (depth - 1)
    assert rows <= 64
    nodes = min(63, topk + (depth - 1) * topk * topk)
    wl = synth.Workload("tmax", sh, B=2, mode=synth.TREE, K=depth, topk=topk, max_nodes=nodes, len_lo=3, len_hi=40,
                        seed=81, sigma_lo=0.0, sigma_hi=0.1)
    case = harness.build_case(wl)
    w = dict(case.weights)
    w["head"] = (w["head"].to(torch.float32) * 20.0).to(torch.bfloat16)
    rep = parity.run_tree(dataclasses.replace(case, weights=w))
    print("tree", topk, depth, "accept:", rep.accept_len, "exempt:", len(rep.exempt))
