"""sx_verify_noalloc: verification for callers that cannot allocate device memory.

A server whose memory pool owns the whole device, or code running where cudaMalloc is forbidden,
has no workspace to hand to sx_verify.  The no-allocation entry point keeps its scratch in a fixed
array inside the library image instead; here it is checked against sx_verify (same inputs, exact
equality of every integer result) on two calls in a row with different inputs, so that the second
call sees the first call's leftovers in the shared scratch.  This file sorts last on purpose: a run
that stops at the first failure has already been through every other test.
"""
import torch
import pytest

from paper_2509_24248_b200 import binding, synth
from tests import harness, parity

pytestmark = pytest.mark.gpu


def _outputs(B, P, stride, dev):
    return {"target_tok": torch.full((B, P), -7, dtype=torch.int32, device=dev),
            "accept_len": torch.full((B,), -7, dtype=torch.int32, device=dev),
            "path": torch.full((B, stride), -7, dtype=torch.int32, device=dev),
            "recover_tok": torch.full((B,), -7, dtype=torch.int32, device=dev)}


def _compare(sx, head, th, cand, parent, stride):
    dev = sx.dev
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    out = _outputs(cand.shape[0], cand.shape[1], stride, dev)
    binding.sx_verify_noalloc(head, th, cand, parent, out, status)
    tt, L, path, rec = sx.sx_verify(th, cand, parent, path_stride=stride)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    sx.check_status()
    assert torch.equal(out["target_tok"], tt)
    assert torch.equal(out["accept_len"], L)
    assert torch.equal(out["path"], path)
    assert torch.equal(out["recover_tok"], rec)
    return L


def test_noalloc_verify_matches_sx_verify_twice_in_a_row():
    sh = synth.ModelShape(H=256, n_q=4, n_kv=2, d=64, F=688, V=4096, page=64)
    wl = synth.Workload("na", sh, B=5, mode=synth.CHAIN, K=6, len_lo=8, len_hi=8, seed=41)
    case = harness.build_case(wl)
    sx = parity.make_gpu(case)
    dev = sx.dev
    head = sx.w["target_head"][: sh.V]
    g = torch.Generator().manual_seed(5)
    P = wl.K + 1
    # call 1: chain, 35 rows; candidates copied from the target's own choices so that some prefixes are accepted
    th1 = torch.randn(wl.B, P, sh.H, generator=g).to(torch.bfloat16).to(dev)
    tt_ref, _, _, _ = sx.sx_verify(th1, torch.zeros(wl.B, P, dtype=torch.int32, device=dev))
    cand1 = torch.randint(0, sh.V, (wl.B, P), generator=g, dtype=torch.int32).to(dev)
    cand1[:, 1:4] = tt_ref[:, 0:3]
    cand1[0, 2] = (cand1[0, 2] + 1) % sh.V
    L1 = _compare(sx, head, th1, cand1, None, P)
    assert sorted(set(L1.cpu().tolist())) != [0]
    # call 2: tree, the full 64 rows, other hidden states; the scratch still holds call 1's partials
    B2, P2 = 4, 16
    th2 = torch.randn(B2, P2, sh.H, generator=g).to(torch.bfloat16).to(dev)
    tt2, _, _, _ = sx.sx_verify(th2, torch.zeros(B2, P2, dtype=torch.int32, device=dev))
    parent = torch.tensor([[-1] + [(s - 1) // 2 for s in range(1, P2)]] * B2, dtype=torch.int32, device=dev)
    cand2 = torch.randint(0, sh.V, (B2, P2), generator=g, dtype=torch.int32).to(dev)
    cand2[:, 2] = tt2[:, 0]          # slot 2 is a child of the root
    cand2[:, 5] = tt2[:, 2]          # slot 5 is a child of slot 2
    L2 = _compare(sx, head, th2, cand2, parent, 7)
    assert L2.cpu().tolist() == [2] * B2 or min(L2.cpu().tolist()) >= 2


def test_noalloc_rejects_more_rows_than_the_built_in_scratch_holds():
    lib = binding.load_library()
    dev = torch.device("cuda:0")
    buf = torch.zeros(4096, dtype=torch.int32, device=dev)
    p = buf.data_ptr()
    code = lib.sx_verify_noalloc(p, 64, 64, 13, 5, p, p, None, p, p, p, 5, p, p, 0)
    assert code == -7 and b"built-in scratch" in lib.sx_strerror(code)
    assert lib.sx_verify_noalloc(None, 64, 64, 1, 2, p, p, None, p, p, p, 2, p, p, 0) == -1
    torch.cuda.synchronize()
