"""The smoothing rules of Appendix A.1 (none, sliding window, momentum, paragraph mean, EWMA) in
sx_exit_update against the oracle, over many iterations with the state carried on both sides."""
import pytest
import torch

from oracle import specexit_oracle as orc
from paper_2509_24248_b200 import synth
from tests import harness, parity

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("rule,window", [(orc.SMOOTH_EWMA, 10), (orc.SMOOTH_NONE, 10), (orc.SMOOTH_WINDOW, 10),
                                         (orc.SMOOTH_WINDOW, 3), (orc.SMOOTH_MOMENTUM, 10), (orc.SMOOTH_MOMENTUM, 4),
                                         (orc.SMOOTH_PARAGRAPH, 10)])
def test_smoothing_rule_matches_oracle_over_a_long_run(rule, window):
    wl = harness.tiny_workload(B=6, K=4)
    case = harness.build_case(wl)
    sx = parity.make_gpu(case)
    dev = sx.dev
    B, P, S, V = wl.B, wl.K + 1, wl.shape.S, wl.shape.V
    bm = torch.zeros((V + 31) // 32, dtype=torch.int32)
    for t in range(0, V, 4):
        bm[t // 32] |= (1 << (t % 32)) if (t % 32) < 31 else -(1 << 31)
    cfg = orc.ExitCfg(alpha=0.1, thr=(0.8, 0.3, 0.9), dir=(orc.DIR_GT, orc.DIR_GT, orc.DIR_LT), enable_mask=0b011,
                      split_bitmap=bm, stop_think_token=3, smoothing=rule, window=window)
    params = parity.to_params(sx, cfg)
    ost = orc.ExitState.fresh(B, S)
    gst = sx.new_state(B)
    g = torch.Generator().manual_seed(100 + rule * 7 + window)
    exits = 0
    for it in range(40):
        sig = torch.rand(B, P, S, generator=g).to(torch.float32)
        sig[:, :, 0] = 0.55 + 0.45 * sig[:, :, 0]            # confidence mostly high
        L = torch.randint(0, P, (B,), generator=g)
        for b in range(B):
            if L[b] == P - 1:
                sig[b, P - 1] = float("nan")                # the last slot was never drafted from
        cand = torch.randint(0, V, (B, P), generator=g, dtype=torch.int32)
        rec = torch.randint(0, V, (B,), generator=g, dtype=torch.int32)
        paths = [list(range(int(L[b]) + 1)) for b in range(B)]
        path_t = torch.full((B, P), -1, dtype=torch.int32)
        for b in range(B):
            path_t[b, : len(paths[b])] = torch.tensor(paths[b], dtype=torch.int32)
        want = orc.exit_update(cfg, ost, sig.double(), cand.long(), paths, L, rec.long())
        ef, Lo, ro, sm = sx.sx_exit_update(params, gst, sig.to(dev), cand.to(dev), path_t.to(dev),
                                           L.to(torch.int32).to(dev), rec.to(dev))
        torch.cuda.synchronize()
        sx.check_status()
        assert ef.cpu().tolist() == want.exit_flag.tolist(), it
        assert Lo.cpu().tolist() == want.accept_len.tolist() and ro.cpu().tolist() == want.recover_tok.tolist()
        assert (sm.cpu().double() - want.smoothed).abs().max() < 1e-6
        assert gst["n_updates"].cpu().tolist() == ost.n_updates.tolist()
        assert gst["thinking"].cpu().tolist() == ost.thinking.tolist()
        exits += int(want.exit_flag.sum())
        if it == 19:                                         # start a fresh batch half way: exits freeze sequences
            ost = orc.ExitState.fresh(B, S)
            gst = sx.new_state(B)
    assert exits > 0
    if rule == orc.SMOOTH_PARAGRAPH:
        assert gst["par_n"].cpu().tolist() == ost.par_n.tolist()
        assert (gst["par_sum"].cpu().double() - ost.par_sum).abs().max() < 1e-6
