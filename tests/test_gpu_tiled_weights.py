"""GEMM weights stored tile by tile (sx_tile_weight, sx_model_cfg.tiled_weights): the repack is exact and
every path gives the oracle's results with that layout as it does with row-major weights."""
import dataclasses

import pytest
import torch

from oracle import specexit_oracle as orc
from paper_2509_24248_b200 import binding, synth
from tests import harness, parity

pytestmark = pytest.mark.gpu


@pytest.fixture(autouse=True)
def _tiled_contexts():
    parity.TILED = True
    yield
    parity.TILED = False


@pytest.mark.parametrize("N,K", [(128, 64), (333, 200), (1, 8), (515, 4096), (1000, 72)])
def test_tile_weight_layout_is_exact(N, K):
    g = torch.Generator().manual_seed(N * 1000 + K)
    w = torch.randn(N, K, generator=g).to(torch.bfloat16)
    got = binding.sx_tile_weight(w.cuda()).cpu()
    T, KB = (N + 127) // 128, (K + 63) // 64
    pad = torch.zeros(T * 128, KB * 64, dtype=torch.bfloat16)
    pad[:N, :K] = w
    want = pad.view(T, 128, KB, 64).permute(0, 2, 1, 3).contiguous().view(-1)
    assert got.numel() == want.numel() == binding.load_library().sx_tiled_weight_bytes(N, K) // 2
    assert torch.equal(got.view(torch.int16), want.view(torch.int16))


@pytest.mark.parametrize("B,K,lo,hi", [(1, 1, 5, 5), (2, 4, 5, 40), (3, 5, 0, 70)])
def test_chain_with_tiled_weights(B, K, lo, hi):
    parity.run_chain(harness.build_case(harness.tiny_workload(B=B, K=K, len_lo=lo, len_hi=hi)))


@pytest.mark.parametrize("shape_kw", [dict(H=128, n_q=8, n_kv=1, d=16, F=200, V=333),
                                      dict(H=64, n_q=2, n_kv=2, d=32, F=72, V=129),
                                      dict(H=256, n_q=4, n_kv=1, d=64, F=688, V=1000, Vd=300, arch=1)])
def test_odd_shapes_with_tiled_weights(shape_kw):
    sh = synth.ModelShape(**{"page": 16, **shape_kw})
    wl = synth.Workload("to", sh, B=3, mode=synth.CHAIN, K=3, len_lo=3, len_hi=150, seed=5, sigma_lo=0.1, sigma_hi=0.6)
    parity.run_chain(harness.build_case(wl))


def test_tree_commit_and_sampling_with_tiled_weights():
    sh = synth.ModelShape(H=64, n_q=4, n_kv=2, d=16, F=96, V=300, page=16)
    wl = synth.Workload("tt", sh, B=2, mode=synth.TREE, K=4, topk=4, max_nodes=20, len_lo=9, len_hi=60, seed=21,
                        sigma_lo=0.0, sigma_hi=0.3)
    case = harness.build_case(wl)
    w = dict(case.weights)
    w["head"] = (w["head"].to(torch.float32) * 20.0).to(torch.bfloat16)
    parity.run_tree(dataclasses.replace(case, weights=w))
    wl2 = harness.tiny_workload(B=3, K=4, len_lo=5, len_hi=50, sigma_lo=0.0, sigma_hi=0.02)
    parity.run_chain(harness.build_case(wl2), sample=orc.SampleCfg(0.7, 5, 2, True))
    # a commit re-keys through the tiled fc and q/k/v weights
    case3 = harness.build_case(wl2, poison_tail=False)
    case3.kv.update(synth.make_kv(wl2.shape, synth.cache_lengths(wl2), 2 * wl2.K + 2, wl2.seed, poison_tail=False))
    g = torch.Generator().manual_seed(6)
    th = torch.randn(wl2.B, wl2.P, wl2.shape.H, generator=g).to(torch.bfloat16)
    cand = torch.randint(0, wl2.shape.V, (wl2.B, wl2.P), generator=g, dtype=torch.int32)
    path = torch.tensor([[0, 1, 2, 3, 4], [0, 1, -1, -1, -1], [0, -1, -1, -1, -1]], dtype=torch.int32)
    L = torch.tensor([4, 1, 0], dtype=torch.int32)
    rec = torch.tensor([3, 4, 5], dtype=torch.int32)
    okv = harness.oracle_kv(case3)
    n0 = list(okv.len)
    oc = orc.commit(harness.oracle_model(case3), okv, th, cand, path, L, rec)
    sx = parity.make_gpu(case3)
    feat0, tok0 = sx.sx_commit(th.to(sx.dev), cand.to(sx.dev), path.to(sx.dev), L.to(sx.dev), rec.to(sx.dev))
    torch.cuda.synchronize()
    sx.check_status()
    assert sx.kv["cache_len"].cpu().tolist() == oc.cache_len
    kg = sx.kv["k_pages"].cpu()
    for b in range(wl2.B):
        for j in range(1, int(L[b]) + 1):
            pp, off = okv._loc(b, n0[b] + j)
            a, want = kg[pp, :, off].double(), okv.k[pp, :, off].double()
            assert float((a - want).norm() / want.norm()) < 2e-2
    sx.close()


def test_config1_with_tiled_weights():
    wl = synth.workload("C1")
    rep = parity.run_chain(harness.build_case(wl, poison_tail=True))
    print(f"C1 tiled: accept_len {rep.accept_len} exempt {rep.exempt} hidden rel-L2 {rep.max_hidden_rel:.2e}")
    assert len(rep.exempt) <= 2
