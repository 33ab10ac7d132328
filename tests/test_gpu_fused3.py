"""The draft layer with three-feature fusion and a concatenated attention input: CUDA path vs
the CPU oracle through the C ABI (chain, tree, standalone rounds, larger shapes)."""
import dataclasses

import pytest
import torch

from oracle import specexit_oracle as orc
from paper_2509_24248_b200 import binding, synth
from tests import harness, parity

pytestmark = pytest.mark.gpu

_SH = synth.ModelShape(H=64, n_q=4, n_kv=2, d=16, F=96, V=200, page=16, arch=1)


@pytest.mark.parametrize("B,K,lo,hi", [(1, 1, 5, 5), (2, 4, 5, 40), (3, 5, 0, 70)])
def test_chain_fused3(B, K, lo, hi):
    wl = synth.Workload("f3", _SH, B=B, mode=synth.CHAIN, K=K, len_lo=lo, len_hi=hi, seed=61,
                        sigma_lo=0.0, sigma_hi=0.2)
    rep = parity.run_chain(harness.build_case(wl))
    print("accept:", rep.accept_len, "hidden rel:", rep.max_hidden_rel, "exempt:", rep.exempt)


@pytest.mark.parametrize("shape_kw", [dict(H=128, n_q=8, n_kv=1, d=16, F=200, V=333),
                                      dict(H=256, n_q=4, n_kv=1, d=64, F=688, V=1000, Vd=300),
                                      dict(H=256, n_q=2, n_kv=1, d=128, F=264, V=515, page=64)])
def test_chain_fused3_odd_shapes(shape_kw):
    sh = synth.ModelShape(**{"page": 16, "arch": 1, **shape_kw})
    wl = synth.Workload("f3o", sh, B=3, mode=synth.CHAIN, K=3, len_lo=3, len_hi=150, seed=62,
                        sigma_lo=0.1, sigma_hi=0.6)
    parity.run_chain(harness.build_case(wl))


@pytest.mark.parametrize("topk,depth,nodes,B", [(2, 3, 5, 1), (8, 3, 20, 2), (4, 5, 30, 2)])
def test_tree_fused3(topk, depth, nodes, B):
    sh = dataclasses.replace(_SH, V=300)
    wl = synth.Workload("f3t", sh, B=B, mode=synth.TREE, K=depth, topk=topk, max_nodes=nodes, len_lo=9, len_hi=60,
                        seed=63, sigma_lo=0.0, sigma_hi=0.3)
    case = harness.build_case(wl)
    w = dict(case.weights)
    w["head"] = (w["head"].to(torch.float32) * 20.0).to(torch.bfloat16)
    rep = parity.run_tree(dataclasses.replace(case, weights=w))
    print("tree accept:", rep.accept_len, "exempt:", rep.exempt)


def test_standalone_rounds_take_three_features_then_the_previous_output():
    wl = synth.Workload("f3s", _SH, B=2, mode=synth.CHAIN, K=3, len_lo=7, len_hi=21, seed=64)
    case = harness.build_case(wl)
    model = harness.oracle_model(case)
    d = orc.draft_chain(model, harness.oracle_kv(case), case.f0, case.t0, wl.K)
    sx = parity.make_gpu(case)
    feat, tok = case.f0.to(sx.dev), case.t0.to(sx.dev)
    assert feat.shape[1] == 3 * _SH.H
    for k in range(1, wl.K + 1):
        hid, tok_out, _, sig = sx.sx_draft_step(k, feat, tok)
        torch.cuda.synchronize()
        sx.check_status()
        assert hid.shape[1] == _SH.H
        assert tok_out[:, 0].cpu().tolist() == d.cand_tok[:, k].tolist()
        for b in range(wl.B):
            assert parity._rel_l2(hid[b].cpu().double(), d.hidden[b, k - 1]) < 2e-2
        feat, tok = hid, tok_out[:, 0].contiguous()
    sx.close()


def test_fused3_without_the_embedding_gain_is_refused():
    wl = synth.Workload("f3e", _SH, B=1, mode=synth.CHAIN, K=2, len_lo=5, len_hi=5, seed=65)
    case = harness.build_case(wl)
    w = {k: v for k, v in case.weights.items() if k != "norm_e"}
    with pytest.raises(binding.SxError):
        parity.make_gpu(dataclasses.replace(case, weights=w))
