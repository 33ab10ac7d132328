"""Ties in the head epilogues when a CTA of the head kernel owns several vocabulary tiles.

The head kernel is persistent: with more 128-row tiles than SMs a CTA takes tiles b, b + G, b + 2G
... (G CTAs), and inside a tile each epilogue thread scans one 32-row quarter.  Equal logits must
go to the LOWER vocabulary index (larger value first, then lower index - the rule both sides
follow for argmax and top-k).  The head used here is periodic with period M = 128 G - 32, so a row
in quarter q >= 1 of tile t has a bit-identical twin in quarter q - 1 of tile t + G: same CTA,
earlier quarter, higher index.  A merge that ranks quarters instead of indices picks the twin.
Every path through the head epilogues is checked against the oracle's argmax_low / topk_low with
no near-tie adoption: verification, a chain draft round, a tree draft round (top-8 + log-sum-exp).
"""
import pytest
import torch

from oracle import specexit_oracle as orc
from paper_2509_24248_b200 import synth
from tests import harness, parity

pytestmark = pytest.mark.gpu


def test_verify_argmax_takes_the_lower_index_across_tiles_of_one_cta():
    case, M = parity.periodic_head_case(synth.CHAIN, B=9, K=6)
    wl = case.wl
    model = harness.oracle_model(case)
    g = torch.Generator().manual_seed(8)
    th = torch.randn(wl.B, wl.P, wl.shape.H, generator=g).to(torch.bfloat16)
    cand = torch.randint(0, wl.shape.V, (wl.B, wl.P), generator=g, dtype=torch.int32)
    sx = parity.make_gpu(case)
    tt, L, path, rec = sx.sx_verify(th.to(sx.dev), cand.to(sx.dev))
    torch.cuda.synchronize()
    sx.check_status()
    o_tt, _ = orc.target_argmax(model, th)
    assert int(o_tt.max()) < M, "every maximum has its lowest copy in the first period"
    # three quarters of the winners sit in a quarter >= 1 and have a twin in an earlier quarter
    assert int(((o_tt % 128) >= 32).sum()) > wl.B * wl.P // 2
    assert torch.equal(tt.cpu().to(torch.int64), o_tt)
    sx.close()


def test_chain_draft_argmax_takes_the_lower_index():
    case, M = parity.periodic_head_case(synth.CHAIN, B=12, K=2)
    wl = case.wl
    model = harness.oracle_model(case)
    sx = parity.make_gpu(case)
    hid, tok_out, _, sig = sx.sx_draft_step(1, case.f0.to(sx.dev), case.t0.to(sx.dev))
    torch.cuda.synchronize()
    sx.check_status()
    ho = model.head(hid.cpu().to(torch.float64))
    want = [orc.argmax_low(ho.logits[r]) for r in range(wl.B)]
    assert max(want) < M and sum(1 for i in want if i % 128 >= 32) >= 3
    assert tok_out[:, 0].cpu().tolist() == want
    assert float((sig.cpu().double() - ho.s).abs().max()) < 1e-2
    sx.close()


def test_tree_top8_orders_equal_logits_by_index():
    case, M = parity.periodic_head_case(synth.TREE, B=6, K=2, topk=8, max_nodes=12)
    wl = case.wl
    model = harness.oracle_model(case)
    sx = parity.make_gpu(case)
    hid, tok_out, logp, _ = sx.sx_draft_step(1, case.f0.to(sx.dev), case.t0.to(sx.dev))
    torch.cuda.synchronize()
    sx.check_status()
    ho = model.head(hid.cpu().to(torch.float64))
    for r in range(wl.B):
        want = orc.topk_low(ho.logits[r], 8)
        # copies of one row are consecutive in the ranking: i, i + M, i + 2M
        assert want[1] == want[0] + M and want[2] == want[0] + 2 * M
        assert tok_out[r].cpu().tolist() == want, f"row {r}"
        lse = torch.logsumexp(ho.logits[r], dim=0)
        got = logp[r].cpu().double()
        assert float((got - (ho.logits[r][want] - lse)).abs().max()) < 1e-3
    sx.close()
