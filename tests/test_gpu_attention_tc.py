"""The tensor-core decode attention (head dimension 128, 64-slot pages) against the oracle, forced on for
shapes small enough for the CPU: runs of blocks that start and end inside a (sequence, KV head) pair, CTAs
that cross several pairs, ragged last blocks behind which the cache holds NaN, zero cached tokens, lengths
on block boundaries, ancestor masks of a tree with 8, 16 and 32 queries per pair, and the refusal of
shapes it does not cover.  The same cases run with the split kernel forced, so both stay covered whatever
the automatic choice is."""
import pytest
import torch

from paper_2509_24248_b200 import binding, synth
from tests import harness, parity

pytestmark = pytest.mark.gpu


@pytest.fixture(params=[binding.ATTN_TC, binding.ATTN_SPLIT], ids=["tc", "split"])
def kernel(request):
    parity.ATTN = request.param
    yield request.param
    parity.ATTN = None


def _shape(n_q=4, n_kv=2, page=64, V=515):
    return synth.ModelShape(H=256, n_q=n_q, n_kv=n_kv, d=128, F=264, V=V, page=page)


@pytest.mark.parametrize("B,K,lo,hi", [(1, 2, 0, 0), (2, 3, 128, 128), (3, 3, 5, 700), (2, 4, 125, 131),
                                       (40, 2, 150, 400), (8, 2, 3000, 3300)])
def test_chain_attention(kernel, B, K, lo, hi):
    wl = synth.Workload("atc", _shape(), B=B, mode=synth.CHAIN, K=K, len_lo=lo, len_hi=hi, seed=50 + B)
    rep = parity.run_chain(harness.build_case(wl))
    assert rep.max_hidden_rel < 2e-2


def test_chain_attention_with_128_slot_pages_and_group_of_eight(kernel):
    wl = synth.Workload("atc8", _shape(n_q=8, n_kv=1, page=128), B=3, mode=synth.CHAIN, K=3, len_lo=60, len_hi=900, seed=58)
    parity.run_chain(harness.build_case(wl))


@pytest.mark.parametrize("n_q,n_kv,topk,depth,nodes,B,lo,hi", [(4, 2, 4, 3, 10, 2, 9, 300), (4, 2, 8, 3, 20, 3, 100, 1000),
                                                             (8, 2, 8, 4, 30, 2, 250, 260), (8, 2, 8, 3, 16, 6, 1500, 1700)])
def test_tree_attention(kernel, n_q, n_kv, topk, depth, nodes, B, lo, hi):
    wl = synth.Workload("att", _shape(n_q=n_q, n_kv=n_kv), B=B, mode=synth.TREE, K=depth, topk=topk, max_nodes=nodes,
                        len_lo=lo, len_hi=hi, seed=60 + topk, sigma_lo=0.0, sigma_hi=0.3)
    parity.run_tree(harness.build_case(wl))


def test_forcing_the_tensor_core_kernel_on_an_unsupported_shape_is_refused():
    sh = synth.ModelShape(H=64, n_q=4, n_kv=2, d=16, F=96, V=200, page=16)
    wl = synth.Workload("atx", sh, B=2, mode=synth.CHAIN, K=2, len_lo=5, len_hi=40, seed=3)
    case = harness.build_case(wl)
    sx = parity.make_gpu(case)
    sx.sx_set_attention(binding.ATTN_TC)
    with pytest.raises(binding.SxError, match="not supported"):
        sx.sx_draft_step(1, case.f0.to(sx.dev), case.t0.to(sx.dev))
    sx.sx_set_attention(binding.ATTN_AUTO)
    sx.sx_draft_step(1, case.f0.to(sx.dev), case.t0.to(sx.dev))
    torch.cuda.synchronize()
    sx.check_status()
    with pytest.raises(binding.SxError):
        sx.sx_set_attention(7)
    sx.close()
