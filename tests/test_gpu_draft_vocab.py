"""Reduced draft vocabulary (the draft head scores Vd < V ids, an id map names their tokens, the
target head is a matrix of its own): CUDA path vs the CPU oracle through the C ABI."""
import dataclasses

import pytest
import torch

from paper_2509_24248_b200 import binding, synth
from tests import harness, parity

pytestmark = pytest.mark.gpu


def _aligned_target_head(case: harness.Case, scale: float = 1.0) -> harness.Case:
    """A target head that agrees with the draft head on the mapped ids (row map[i] = draft row i)
    and is small elsewhere, so that acceptance lengths are not all zero."""
    w = dict(case.weights)
    sh = case.wl.shape
    Vd = sh.Vd or sh.V
    head = (w["head"].to(torch.float32) * scale).to(torch.bfloat16)
    w["head"] = head
    th = (w["target_head"].to(torch.float32) * 0.25).to(torch.bfloat16)
    th[w["draft_to_token"].to(torch.int64)] = head[:Vd]
    w["target_head"] = th
    return dataclasses.replace(case, weights=w)


@pytest.mark.parametrize("V,Vd,B,K", [(200, 64, 2, 3), (515, 129, 3, 4), (1000, 999, 1, 5)])
def test_chain_reduced_draft_vocabulary(V, Vd, B, K):
    sh = synth.ModelShape(H=64, n_q=4, n_kv=2, d=16, F=96, V=V, page=16, Vd=Vd)
    wl = synth.Workload("dv", sh, B=B, mode=synth.CHAIN, K=K, len_lo=5, len_hi=70, seed=31,
                        sigma_lo=0.0, sigma_hi=0.2)
    case = harness.build_case(wl)
    rep = parity.run_chain(case)                      # unrelated target head: mostly rejections
    assert all(0 <= l <= K for l in rep.accept_len)
    rep = parity.run_chain(_aligned_target_head(case))
    print("aligned accept:", rep.accept_len)
    assert max(rep.accept_len) > 0


@pytest.mark.parametrize("topk,depth,nodes,B", [(2, 3, 5, 1), (8, 3, 20, 2), (4, 5, 30, 2)])
def test_tree_reduced_draft_vocabulary(topk, depth, nodes, B):
    sh = synth.ModelShape(H=64, n_q=4, n_kv=2, d=16, F=96, V=300, page=16, Vd=77)
    wl = synth.Workload("dvt", sh, B=B, mode=synth.TREE, K=depth, topk=topk, max_nodes=nodes, len_lo=9, len_hi=60,
                        seed=32, sigma_lo=0.0, sigma_hi=0.3)
    rep = parity.run_tree(_aligned_target_head(harness.build_case(wl), scale=20.0))
    print("tree accept:", rep.accept_len)


def test_full_size_permutation_map():
    """Vd == V with a map that is a permutation: every token that leaves the library is mapped."""
    wl = harness.tiny_workload(B=2, K=4, len_lo=10, len_hi=40)
    case = harness.build_case(wl)
    w = dict(case.weights)
    g = torch.Generator().manual_seed(5)
    perm = torch.randperm(wl.shape.V, generator=g).to(torch.int32)
    w["draft_to_token"] = perm
    th = torch.empty(wl.shape.V, wl.shape.H, dtype=torch.bfloat16)
    th[perm.to(torch.int64)] = w["head"][:wl.shape.V]
    w["target_head"] = th
    rep = parity.run_chain(dataclasses.replace(case, weights=w))
    assert max(rep.accept_len) > 0


def test_reduced_vocabulary_without_a_map_is_refused():
    sh = synth.ModelShape(H=64, n_q=4, n_kv=2, d=16, F=96, V=200, page=16, Vd=64)
    wl = synth.Workload("dv", sh, B=1, mode=synth.CHAIN, K=2, len_lo=5, len_hi=5, seed=33)
    case = harness.build_case(wl)
    w = {k: v for k, v in case.weights.items() if k != "draft_to_token"}
    with pytest.raises(binding.SxError):
        parity.make_gpu(dataclasses.replace(case, weights=w))
