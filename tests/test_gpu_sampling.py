"""Stochastic acceptance (speculative sampling with deterministic drafts): the CUDA verify head's
Gumbel-max draw vs the CPU oracle's, token by token, through the C ABI."""
import dataclasses

import pytest
import torch

from oracle import specexit_oracle as orc
from paper_2509_24248_b200 import synth
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
