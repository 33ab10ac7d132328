"""sx_commit against the oracle's commit on the same inputs: new cached lengths and the next
iteration's first row exactly, the re-keyed K/V of every accepted token within the hidden-state
tolerance, every other cache slot untouched; and a three-iteration loop on the GPU alone."""
import pytest
import torch

from oracle import specexit_oracle as orc
from paper_2509_24248_b200 import synth
from tests import harness, parity

pytestmark = pytest.mark.gpu


def _random_paths(B, P, M, gen, tree):
    L = torch.randint(0, M + 1, (B,), generator=gen)
    L[0] = M                                   # the longest possible path
    if B > 1:
        L[1] = 0                               # nothing accepted
    path = torch.full((B, M + 1), -1, dtype=torch.int32)
    for b in range(B):
        if tree:
            slots = sorted(torch.randperm(P - 1, generator=gen)[: int(L[b])].add(1).tolist())
        else:
            slots = list(range(1, int(L[b]) + 1))
        path[b, 0] = 0
        for j, s in enumerate(slots):
            path[b, j + 1] = s
    return L.to(torch.int32), path


@pytest.mark.parametrize("tree", [False, True])
@pytest.mark.parametrize("shape_kw,B,K", [(dict(H=64, n_q=4, n_kv=2, d=16, F=96, V=300, page=16), 5, 4),
                                          (dict(H=256, n_q=4, n_kv=2, d=64, F=688, V=4096, page=64), 3, 6),
                                          (dict(H=64, n_q=4, n_kv=2, d=16, F=96, V=300, page=16, arch=1), 5, 4),
                                          (dict(H=256, n_q=4, n_kv=2, d=64, F=688, V=4096, page=64, arch=1), 3, 6)])
def test_commit_matches_oracle(shape_kw, B, K, tree):
    # with the three-feature layer (arch=1) the rows handed to the commit are [.., 3H] target features
    sh = synth.ModelShape(**shape_kw)
    wl = synth.Workload("cm", sh, B=B, mode=synth.TREE if tree else synth.CHAIN, K=K, topk=2 if tree else 1,
                        max_nodes=9 if tree else 0, len_lo=3, len_hi=70, seed=17)
    case = harness.build_case(wl)
    P = wl.P
    g = torch.Generator().manual_seed(23)
    th = torch.randn(B, P, (3 if sh.arch else 1) * sh.H, generator=g).to(torch.bfloat16)
    cand = torch.randint(0, sh.V, (B, P), generator=g, dtype=torch.int32)
    rec = torch.randint(0, sh.V, (B,), generator=g, dtype=torch.int32)
    L, path = _random_paths(B, P, K, g, tree)
    # oracle
    model = harness.oracle_model(case)
    okv = harness.oracle_kv(case)
    n0 = list(okv.len)
    oc = orc.commit(model, okv, th, cand, path, L, rec)
    # GPU
    sx = parity.make_gpu(case)
    dev = sx.dev
    k_before = sx.kv["k_pages"].clone()
    feat0, tok0 = sx.sx_commit(th.to(dev), cand.to(dev), path.to(dev), L.to(dev), rec.to(dev))
    torch.cuda.synchronize()
    sx.check_status()
    assert sx.kv["cache_len"].cpu().tolist() == oc.cache_len == [n0[b] + int(L[b]) + 1 for b in range(B)]
    assert tok0.cpu().tolist() == oc.tok0.tolist()
    assert torch.equal(feat0.cpu().to(torch.float64), oc.feat0)
    kg, vg = sx.kv["k_pages"].cpu(), sx.kv["v_pages"].cpu()
    touched = torch.zeros(kg.shape[0], kg.shape[2], dtype=torch.bool)
    for b in range(B):
        for j in range(1, int(L[b]) + 1):
            pp, off = okv._loc(b, n0[b] + j)
            touched[pp, off] = True
            for got, want in ((kg, okv.k), (vg, okv.v)):
                a, w = got[pp, :, off].double(), want[pp, :, off].double()
                assert float((a - w).norm() / w.norm()) < 2e-2, (b, j)
    kb = k_before.cpu()
    keep = ~touched[:, None, :, None].expand_as(kg)
    same = (kg == kb) | (torch.isnan(kg) & torch.isnan(kb))
    assert bool(same[keep].all())


@pytest.mark.parametrize("arch", [0, 1])
def test_three_iterations_with_commit_on_the_gpu(arch):
    wl = synth.Workload("loop", synth.ModelShape(H=64, n_q=4, n_kv=2, d=16, F=96, V=300, page=16, arch=arch), B=3,
                        mode=synth.CHAIN, K=3, len_lo=5, len_hi=20, seed=3)
    case = harness.build_case(wl, poison_tail=False)
    # room for three iterations of K + 1 new tokens each
    case.kv.update(synth.make_kv(wl.shape, synth.cache_lengths(wl), 3 * (wl.K + 1) + wl.K, wl.seed, poison_tail=False))
    sx = parity.make_gpu(case)
    dev = sx.dev
    params = parity.to_params(sx, harness.default_exit_cfg(wl, thr=(0.99, 0.0, 0.0)))
    state, out = sx.new_state(wl.B), sx.new_outputs(wl.B)
    feat, tok = case.f0.to(dev), case.t0.to(dev)
    n = sx.kv["cache_len"].cpu().clone()
    g = torch.Generator().manual_seed(4)
    for it in range(3):
        th = torch.randn(wl.B, wl.P, wl.shape.H, generator=g).to(torch.bfloat16).to(dev)
        sx.sx_spec_exit_iter(params, state, feat, tok, th, out)
        if arch:                                   # the target's three features of every verify slot
            th = torch.randn(wl.B, wl.P, 3 * wl.shape.H, generator=g).to(torch.bfloat16).to(dev)
        feat, tok = sx.sx_commit(th, out["cand_tok_d"], out["path_d"], out["accept_len_out_d"], out["recover_tok_out_d"])
        torch.cuda.synchronize()
        sx.check_status()
        n = n + out["accept_len_out_d"].cpu() + 1
        assert sx.kv["cache_len"].cpu().tolist() == n.tolist()
        assert tok.cpu().tolist() == out["recover_tok_out_d"].cpu().tolist()


@pytest.mark.parametrize("arch", [0, 1])
def test_second_iteration_after_a_commit_matches_the_oracle(arch):
    """Iteration 1 and its commit run on the GPU; iteration 2 then starts from the committed cache
    and the returned first row, and is compared with the oracle element by element."""
    sh = synth.ModelShape(H=64, n_q=4, n_kv=2, d=16, F=96, V=300, page=16, arch=arch)
    wl = synth.Workload("it2", sh, B=3, mode=synth.CHAIN, K=3, len_lo=5, len_hi=40, seed=9,
                        sigma_lo=0.0, sigma_hi=0.0)
    case = harness.build_case(wl, poison_tail=False)
    case.kv.update(synth.make_kv(sh, synth.cache_lengths(wl), 2 * (wl.K + 1) + wl.K, wl.seed, poison_tail=False))
    w = dict(case.weights)
    w["head"] = (w["head"].to(torch.float32) * 30.0).to(torch.bfloat16)       # peaked: some drafts get accepted
    case = harness.Case(wl, w, case.kv, case.f0, case.t0, case.sigma)
    sx = parity.make_gpu(case)
    dev = sx.dev
    params = parity.to_params(sx, harness.default_exit_cfg(wl, thr=(0.99, 0.0, 0.0)))
    state, out = sx.new_state(wl.B), sx.new_outputs(wl.B)
    # iteration 1 on the oracle gives the target hiddens the harness would use; the GPU runs on them
    model = harness.oracle_model(case)
    d = orc.draft_chain(model, harness.oracle_kv(case), case.f0, case.t0, wl.K)
    th = harness.chain_target_hidden(case, d)
    sx.sx_spec_exit_iter(params, state, case.f0.to(dev), case.t0.to(dev), th.to(dev), out)
    g = torch.Generator().manual_seed(10)
    tf = th if not arch else torch.randn(wl.B, wl.P, 3 * sh.H, generator=g).to(torch.bfloat16)
    feat, tok = sx.sx_commit(tf.to(dev), out["cand_tok_d"], out["path_d"], out["accept_len_out_d"],
                             out["recover_tok_out_d"])
    torch.cuda.synchronize()
    sx.check_status()
    assert int(out["accept_len_out_d"].sum()) > 0
    kv2 = {"k_pages": sx.kv["k_pages"].cpu(), "v_pages": sx.kv["v_pages"].cpu(),
           "page_table": sx.kv["page_table"].cpu(), "cache_len": sx.kv["cache_len"].cpu(),
           "max_pages": case.kv["max_pages"]}
    case2 = harness.Case(wl, w, kv2, feat.cpu(), tok.cpu(), case.sigma)
    sx.close()
    rep = parity.run_chain(case2)
    print("iteration 2 accept:", rep.accept_len, "hidden rel:", rep.max_hidden_rel)
