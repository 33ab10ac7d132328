"""Stochastic acceptance (speculative sampling with deterministic drafts): the CUDA verify head's
Gumbel-max draw vs the CPU oracle's, token by token, through the C ABI."""
import dataclasses

import pytest
import torch

from oracle import specexit_oracle as orc
from paper_2509_24248_b200 import binding, synth
from tests import harness, parity

pytestmark = pytest.mark.gpu


def _peaked(case: harness.Case, scale: float) -> harness.Case:
    w = dict(case.weights)
    w["head"] = (w["head"].to(torch.float32) * scale).to(torch.bfloat16)
    return dataclasses.replace(case, weights=w)


@pytest.mark.parametrize("tau,seed,offset", [(0.05, 1, 0), (0.3, 2, 7), (1.0, (5 << 32) + 9, 1), (4.0, 3, 2 ** 32 - 1)])
def test_chain_sampled_verification(tau, seed, offset):
    wl = harness.tiny_workload(B=3, K=5, len_lo=5, len_hi=50, sigma_lo=0.0, sigma_hi=0.01)
    case = _peaked(harness.build_case(wl), 30.0)
    rep = parity.run_chain(case, sample=orc.SampleCfg(tau, seed, offset))
    print("tau", tau, "accept:", rep.accept_len, "exempt:", rep.exempt)


def test_sampled_acceptance_shrinks_as_the_temperature_rises():
    wl = harness.tiny_workload(B=4, K=5, len_lo=5, len_hi=50, sigma_lo=0.0, sigma_hi=0.0)
    case = _peaked(harness.build_case(wl), 30.0)
    sx = parity.make_gpu(case)
    tot = []
    for tau in (0.0, 0.2, 50.0):
        n = 0
        for it in range(6):
            rep = parity.run_chain(case, sx=sx, sample=orc.SampleCfg(tau, 11, it))
            n += sum(rep.accept_len)
        tot.append(n)
    sx.close()
    print("accepted tokens at tau = 0, 0.2, 50:", tot)
    assert tot[0] >= tot[1] >= tot[2] and tot[0] > tot[2]


@pytest.mark.parametrize("topk,depth,nodes,B,tau", [(3, 4, 14, 2, 0.5), (8, 3, 20, 2, 1.0)])
def test_tree_sampled_verification(topk, depth, nodes, B, tau):
    sh = synth.ModelShape(H=64, n_q=4, n_kv=2, d=16, F=96, V=300, page=16)
    wl = synth.Workload("ts", sh, B=B, mode=synth.TREE, K=depth, topk=topk, max_nodes=nodes, len_lo=9, len_hi=60,
                        seed=41, sigma_lo=0.0, sigma_hi=0.2)
    rep = parity.run_tree(_peaked(harness.build_case(wl), 20.0), sample=orc.SampleCfg(tau, 17, 4))
    print("tree accept:", rep.accept_len, "exempt:", rep.exempt)


def test_sampled_verification_over_many_rows_and_an_odd_vocabulary():
    # 5 sequences x 64 verify rows (> 256 rows: two head launches, the row offset enters the counter)
    sh = synth.ModelShape(H=64, n_q=2, n_kv=1, d=32, F=72, V=1031, page=16)
    wl = synth.Workload("sv", sh, B=5, mode=synth.CHAIN, K=63, len_lo=3, len_hi=9, seed=43)
    case = harness.build_case(wl)
    model = harness.oracle_model(case)
    g = torch.Generator().manual_seed(3)
    th = torch.randn(wl.B, wl.P, sh.H, generator=g).to(torch.bfloat16)
    cand = torch.randint(0, sh.V, (wl.B, wl.P), generator=g, dtype=torch.int32)
    smp = orc.SampleCfg(0.7, 123456789012345, 77)
    want, gap = orc.target_sample(model, th, smp)
    sx = parity.make_gpu(case)
    sx.sx_set_sampling(smp.temperature, smp.seed, smp.offset)
    tt, L, path, rec = sx.sx_verify(th.to(sx.dev), cand.to(sx.dev), path_stride=wl.P)
    torch.cuda.synchronize()
    sx.check_status("sx_verify")
    got = tt.cpu().to(torch.int64)
    bad = (got != want) & (gap >= parity.REL_GAP)
    assert not bool(bad.any()), (got[bad], want[bad])
    assert int((got != want).sum()) <= 3
    # the draws are not the greedy choices
    greedy, _ = orc.target_argmax(model, th)
    assert int((want != greedy).sum()) > wl.B * wl.P // 4
    sx.close()


def test_set_sampling_rejects_bad_temperatures():
    wl = harness.tiny_workload(B=1, K=2)
    sx = parity.make_gpu(harness.build_case(wl))
    assert sx.lib.sx_set_sampling(sx.h, -1.0, 0, 0) == -1
    assert sx.lib.sx_set_sampling(sx.h, float("nan"), 0, 0) == -1
    assert sx.lib.sx_set_sampling(sx.h, float("inf"), 0, 0) == -1
    sx.close()


# ---------------------------------------------------------------------------------------
# sampled drafts: the rule in its general form (accept test min(1, p/q), residual draw)
# ---------------------------------------------------------------------------------------
@pytest.mark.parametrize("tau,seed,offset,scale", [(0.3, 1, 0, 30.0), (1.0, 2, 5, 30.0), (1.0, (7 << 32) + 1, 9, 100.0),
                                                   (2.5, 3, 1, 100.0)])
def test_chain_sampled_drafts(tau, seed, offset, scale):
    wl = harness.tiny_workload(B=4, K=5, len_lo=5, len_hi=50, sigma_lo=0.0, sigma_hi=0.02)
    case = _peaked(harness.build_case(wl), scale)
    rep = parity.run_chain(case, sample=orc.SampleCfg(tau, seed, offset, True))
    print("tau", tau, "accept:", rep.accept_len, "exempt:", rep.exempt)


def test_sampled_drafts_are_all_kept_when_target_and_draft_distributions_coincide():
    # noise-free target hiddens: p == q at every slot, so the accept test passes whatever the temperature
    wl = harness.tiny_workload(B=4, K=4, len_lo=5, len_hi=50, sigma_lo=0.0, sigma_hi=0.0)
    case = _peaked(harness.build_case(wl), 60.0)
    cfg = harness.default_exit_cfg(wl, thr=(2.0, 0.0, 0.0))          # the exit rule never fires
    sx = parity.make_gpu(case, sample_drafts=True)
    for tau in (0.05, 1.0, 20.0):
        for it in range(3):
            rep = parity.run_chain(case, cfg, sx=sx, sample=orc.SampleCfg(tau, 31, it, True))
            assert rep.accept_len == [wl.K] * wl.B
    # zero temperature on the same context is plain greedy verification
    parity.run_chain(case, cfg, sx=sx)
    # with noisy target hiddens some drafts are refused
    sx.close()
    wl2 = harness.tiny_workload(B=4, K=4, len_lo=5, len_hi=50, sigma_lo=0.5, sigma_hi=1.0)
    case2 = _peaked(harness.build_case(wl2), 60.0)
    cfg2 = harness.default_exit_cfg(wl2, thr=(2.0, 0.0, 0.0))
    sx = parity.make_gpu(case2, sample_drafts=True)
    n = 0
    for it in range(5):
        n += sum(parity.run_chain(case2, cfg2, sx=sx, sample=orc.SampleCfg(0.5, 32, it, True)).accept_len)
    sx.close()
    print("accepted with noisy targets:", n, "of", 5 * wl2.B * wl2.K)
    assert 0 < n < 5 * wl2.B * wl2.K


def test_sampled_drafts_on_an_odd_vocabulary_and_the_three_feature_layer():
    sh = synth.ModelShape(H=128, n_q=8, n_kv=1, d=16, F=200, V=333, page=16, arch=1)
    wl = synth.Workload("sd", sh, B=3, mode=synth.CHAIN, K=3, len_lo=3, len_hi=90, seed=71, sigma_lo=0.0, sigma_hi=0.05)
    case = _peaked(harness.build_case(wl), 40.0)
    parity.run_chain(case, sample=orc.SampleCfg(0.8, 5, 3, True))


def test_sampled_drafts_need_a_full_draft_vocabulary():
    sh2 = synth.ModelShape(H=64, n_q=4, n_kv=2, d=16, F=96, V=300, page=16, Vd=100)
    wl2 = synth.Workload("sdv", sh2, B=1, mode=synth.CHAIN, K=3, len_lo=9, len_hi=9, seed=73)
    with pytest.raises(binding.SxError):
        parity.make_gpu(harness.build_case(wl2), sample_drafts=True)


@pytest.mark.parametrize("topk,depth,nodes,tau", [(2, 3, 2 + 2 * 4, 1.0), (3, 3, 3 + 2 * 9, 0.7), (4, 3, 20, 1.5), (8, 2, 30, 1.0)])
def test_tree_with_sampled_children(topk, depth, nodes, tau):
    """Children drawn without replacement (the Gumbel-top-k of every drafted row) and the sequential accept /
    residual walk over the laid-out tree: candidates, layout, the tokens of the visited slots, accepted
    length, path, recover token and the exit decision against the oracle; the first two trees are unpruned."""
    sh = synth.ModelShape(H=64, n_q=4, n_kv=2, d=16, F=96, V=300, page=16)
    wl = synth.Workload("stc", sh, B=3, mode=synth.TREE, K=depth, topk=topk, max_nodes=nodes, len_lo=9, len_hi=60,
                        seed=70 + topk, sigma_lo=0.0, sigma_hi=0.05)
    case = harness.build_case(wl)
    w = dict(case.weights)
    w["head"] = (w["head"].to(torch.float32) * 20.0).to(torch.bfloat16)       # a peaked head: some children get accepted
    case = dataclasses.replace(case, weights=w)
    accepted = 0
    for offset in (1, 2, 3):
        rep = parity.run_tree(case, sample=orc.SampleCfg(tau, 4242, offset, True))
        accepted += sum(rep.accept_len)
        print("sampled children tau", tau, "offset", offset, "accept:", rep.accept_len, "exempt:", rep.exempt)
        assert len(rep.exempt) <= 2
    assert accepted > 0


def test_sampled_children_on_an_odd_vocabulary_cut_into_several_chunks():
    """V = 2501: the top-k pass cuts a row into three chunks (the last one ragged) and merges them; the walk's
    eight vocabulary slices are 316 ids wide with a short last one.  Five sequences, a deep narrow tree."""
    sh = synth.ModelShape(H=64, n_q=4, n_kv=2, d=16, F=96, V=2501, page=16)
    wl = synth.Workload("stv", sh, B=5, mode=synth.TREE, K=5, topk=2, max_nodes=2 + 4 * 4, len_lo=9, len_hi=60,
                        seed=91, sigma_lo=0.0, sigma_hi=0.05)
    case = harness.build_case(wl)
    w = dict(case.weights)
    w["head"] = (w["head"].to(torch.float32) * 25.0).to(torch.bfloat16)
    case = dataclasses.replace(case, weights=w)
    accepted = 0
    for offset in (1, 2):
        rep = parity.run_tree(case, sample=orc.SampleCfg(0.8, 99, offset, True))
        accepted += sum(rep.accept_len)
        print("odd vocabulary, offset", offset, "accept:", rep.accept_len, "exempt:", rep.exempt)
        assert len(rep.exempt) <= 2
    assert accepted > 0


def test_sampled_children_need_the_full_vocabulary_and_a_positive_temperature_to_act():
    sh = synth.ModelShape(H=64, n_q=4, n_kv=2, d=16, F=96, V=300, page=16)
    wl = synth.Workload("stx", sh, B=2, mode=synth.TREE, K=3, topk=3, max_nodes=12, len_lo=9, len_hi=40, seed=75)
    case = harness.build_case(wl)
    # temperature 0 in a context created for sampled children: the deterministic tree and the greedy walk
    sx = parity.make_gpu(case, sample_drafts=True)
    parity.run_tree(case, sx=sx)
    sx.close()
    # a reduced draft vocabulary cannot be combined with sampled drafts
    wl2 = dataclasses.replace(wl, shape=dataclasses.replace(sh, Vd=100))
    case2 = harness.build_case(wl2)
    with pytest.raises(binding.SxError, match="not supported"):
        parity.make_gpu(case2, sample_drafts=True)
