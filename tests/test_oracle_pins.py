"""Pins for the CPU oracle: hand-worked values, closed forms, textbook special cases,
invariants and brute force.  None of these re-types the oracle's own formula: each expected
value is derived independently (by hand, by a closed form, by enumeration, or by numpy)."""
import dataclasses
import itertools
import math
import os
import random

import numpy as np
import pytest
import torch

from oracle import specexit_oracle as orc
from paper_2509_24248_b200 import synth
from tests import harness

F64 = torch.float64
GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _rows(name):
    out = []
    with open(os.path.join(GOLD, name)) as f:
        for line in f:
            line = line.strip()
            if line and not line.startswith("#"):
                out.append(line.split())
    return out


# ---------------------------------------------------------------- EWMA (Appendix A.1)
def test_ewma_hand_worked_values():
    rows = [(float(a), float(s), float(x)) for a, s, x in _rows("ewma_worked.txt")]
    # first block: alpha 0.3, first sample initialises
    cfg = orc.ExitCfg(alpha=0.3)
    x, n = torch.zeros(1, dtype=F64), 0
    for a, s, want in rows[:3]:
        x = orc.ewma(cfg, x, n, torch.tensor([s], dtype=F64))
        n += 1
        assert abs(float(x) - want) < 1e-6
    # second block: the paper's alpha 0.1, state seeded with 0.5 (n_updates > 0)
    cfg = orc.ExitCfg(alpha=0.1)
    x, n = torch.tensor([0.5], dtype=F64), 1
    for a, s, want in rows[3:]:
        x = orc.ewma(cfg, x, n, torch.tensor([s], dtype=F64))
        n += 1
        assert abs(float(x) - want) < 1e-6


@pytest.mark.parametrize("alpha", [0.1, 0.3, 0.75])
def test_ewma_closed_form_constant_signal(alpha):
    cfg = orc.ExitCfg(alpha=alpha)
    c, x0 = 0.8, 0.1
    x = torch.tensor([x0], dtype=F64)
    for n in range(1, 30):
        x = orc.ewma(cfg, x, n, torch.tensor([c], dtype=F64))
        assert abs(float(x) - (c + (1 - alpha) ** n * (x0 - c))) < 1e-5
    # first-sample initialisation keeps a constant signal constant
    x = orc.ewma(cfg, torch.zeros(1, dtype=F64), 0, torch.tensor([c], dtype=F64))
    assert abs(float(x) - c) < 1e-7


# ---------------------------------------------------------------- activations (Eq. 3-5)
def test_activations():
    z = torch.tensor([[0.0, math.log(3.0), math.log(101.0)]], dtype=F64)
    s = orc.activate(z, (orc.ACT_SIGMOID, orc.ACT_SIGMOID, orc.ACT_EXPM1))
    assert abs(float(s[0, 0]) - 0.5) < 1e-12          # sigmoid(0) = 1/2
    assert abs(float(s[0, 1]) - 0.75) < 1e-12         # sigmoid(ln 3) = 3/4
    assert abs(float(s[0, 2]) - 100.0) < 1e-9         # head regresses log(1+r): r = 100
    s = orc.activate(z, (orc.ACT_IDENTITY,) * 3)
    assert torch.equal(s, z)


# ---------------------------------------------------------------- exit decision (Alg. 1, Sec. 3.3)
def _exit_once(cfg, sig_conf, toks, L, state=None, S=3):
    P = len(toks)
    ss = torch.full((1, P, S), float("nan"), dtype=F64)
    for j, c in enumerate(sig_conf):
        if c is not None:
            ss[0, j] = torch.tensor([c, 0.5, 0.5], dtype=F64)
    st = state if state is not None else orc.ExitState.fresh(1, S)
    out = orc.exit_update(cfg, st, ss, torch.tensor([toks]), [list(range(P))],
                          torch.tensor([L]), torch.tensor([99]))
    return out, st


def test_exit_hand_worked_scenario():
    # x: 0.5 ; 0.3*0.95+0.7*0.5 = 0.635 ; 0.3*0.99+0.7*0.635 = 0.7415   (alpha 0.3)
    cfg = orc.ExitCfg(alpha=0.3, thr=(0.6, 0, 0), enable_mask=1, stop_think_token=42)
    out, st = _exit_once(cfg, [0.5, 0.95, 0.99, None], [10, 11, 12, 13], L=3)
    assert int(out.exit_flag[0]) == 1 and int(out.accept_len[0]) == 1
    assert int(out.recover_tok[0]) == 42 and int(st.thinking[0]) == 0
    assert abs(float(out.smoothed[0, 0]) - 0.635) < 1e-6 and int(st.n_updates[0]) == 2
    # only token 12 is a step-split token: exit moves to slot 2 with x = 0.7415
    bm = torch.zeros(1, dtype=torch.int32)
    bm[0] = 1 << 12
    cfg2 = orc.ExitCfg(alpha=0.3, thr=(0.6, 0, 0), enable_mask=1, stop_think_token=42, split_bitmap=bm)
    out, st = _exit_once(cfg2, [0.5, 0.95, 0.99, None], [10, 11, 12, 13], L=3)
    assert int(out.exit_flag[0]) == 1 and int(out.accept_len[0]) == 2
    assert abs(float(out.smoothed[0, 0]) - 0.7415) < 1e-6
    # the draft stopped at slot 1: slot 2 is outside the accepted prefix, no exit
    out, st = _exit_once(cfg2, [0.5, 0.95, 0.99, None], [10, 11, 12, 13], L=1)
    assert int(out.exit_flag[0]) == 0 and int(out.accept_len[0]) == 1 and int(out.recover_tok[0]) == 99
    assert int(st.thinking[0]) == 1 and int(st.n_updates[0]) == 2
    # threshold higher than anything reached
    cfg3 = orc.ExitCfg(alpha=0.3, thr=(0.75, 0, 0), enable_mask=1, stop_think_token=42)
    out, st = _exit_once(cfg3, [0.5, 0.95, 0.99, None], [10, 11, 12, 13], L=3)
    assert int(out.exit_flag[0]) == 0 and int(out.accept_len[0]) == 3
    assert int(st.n_updates[0]) == 3      # slot 3 carries no signal: smoothing stops there


def test_exit_first_only_mode_and_and_combination():
    # paper-literal: only the signal of the last accepted token (slot 0) is smoothed
    cfg = orc.ExitCfg(alpha=0.3, thr=(0.6, 0, 0), enable_mask=1, stop_think_token=1,
                      ema_positions=orc.EMA_FIRST_ONLY)
    out, st = _exit_once(cfg, [0.5, 0.95, 0.99, None], [10, 11, 12, 13], L=3)
    assert int(out.exit_flag[0]) == 0 and int(st.n_updates[0]) == 1
    assert abs(float(out.smoothed[0, 0]) - 0.5) < 1e-7
    # SpecExit*-style: conf > .8 AND prog > .3 AND rem < 200 ; signals (c, .5, .5)
    cfg = orc.ExitCfg(alpha=1.0, thr=(0.8, 0.3, 200.0), dir=(orc.DIR_GT, orc.DIR_GT, orc.DIR_LT),
                      enable_mask=0b111, stop_think_token=1)
    out, _ = _exit_once(cfg, [0.9], [3], L=0)
    assert int(out.exit_flag[0]) == 1
    cfg = orc.ExitCfg(alpha=1.0, thr=(0.8, 0.6, 200.0), dir=(orc.DIR_GT, orc.DIR_GT, orc.DIR_LT),
                      enable_mask=0b111, stop_think_token=1)
    out, _ = _exit_once(cfg, [0.9], [3], L=0)
    assert int(out.exit_flag[0]) == 0           # progress 0.5 is not > 0.6
    cfg = orc.ExitCfg(alpha=1.0, thr=(0.8, 0.3, 0.4), dir=(orc.DIR_GT, orc.DIR_GT, orc.DIR_LT),
                      enable_mask=0b111, stop_think_token=1)
    out, _ = _exit_once(cfg, [0.9], [3], L=0)
    assert int(out.exit_flag[0]) == 0           # remaining 0.5 is not < 0.4
    # strictness: "greater than 0.9" is false at exactly 0.9 (fp32 compare)
    cfg = orc.ExitCfg(alpha=1.0, thr=(0.5, 0, 0), enable_mask=1, stop_think_token=1)
    out, _ = _exit_once(cfg, [0.5], [3], L=0)
    assert int(out.exit_flag[0]) == 0


def test_exit_invariants_random():
    rng = random.Random(5)
    for trial in range(200):
        K = rng.randint(1, 6)
        L = rng.randint(0, K)
        conf = [rng.random() for _ in range(K)] + [None]
        toks = [rng.randrange(64) for _ in range(K + 1)]
        bm = torch.tensor([rng.getrandbits(31), rng.getrandbits(31)], dtype=torch.int32)
        prev_flag = 1
        for thr in [0.0, 0.2, 0.4, 0.6, 0.8, 1.0]:
            cfg = orc.ExitCfg(alpha=0.3, thr=(thr, 0, 0), enable_mask=1, stop_think_token=5,
                              split_bitmap=bm)
            out, st = _exit_once(cfg, conf, toks, L)
            flag = int(out.exit_flag[0])
            assert flag <= prev_flag                      # monotone in a "greater than" threshold
            prev_flag = flag
            assert 0 <= int(out.accept_len[0]) <= L <= K
            if flag:
                assert int(out.recover_tok[0]) == 5 and int(st.thinking[0]) == 0
                assert orc.is_split(cfg, toks[int(out.accept_len[0])])
            else:
                assert int(out.recover_tok[0]) == 99 and int(out.accept_len[0]) == L
        # an empty split set never exits
        cfg = orc.ExitCfg(alpha=0.3, thr=(0.0, 0, 0), enable_mask=1,
                          split_bitmap=torch.zeros(2, dtype=torch.int32))
        out, _ = _exit_once(cfg, conf, toks, L)
        assert int(out.exit_flag[0]) == 0
        # a sequence that left the reasoning phase is frozen
        st = orc.ExitState.fresh(1)
        st.thinking[0] = 0
        st.x[0] = torch.tensor([0.1, 0.2, 0.3], dtype=F64)
        before = st.clone()
        cfg = orc.ExitCfg(alpha=0.3, thr=(0.0, 0, 0), enable_mask=1)
        out, st = _exit_once(cfg, conf, toks, L, state=st)
        assert int(out.exit_flag[0]) == 0 and int(out.accept_len[0]) == L
        assert torch.equal(st.x, before.x) and torch.equal(st.n_updates, before.n_updates)


def test_exit_lt_direction_monotone():
    for thr_lo, thr_hi in [(10.0, 50.0), (50.0, 150.0)]:
        flags = []
        for thr in (thr_lo, thr_hi):
            cfg = orc.ExitCfg(alpha=1.0, thr=(0, 0, thr), dir=(orc.DIR_GT, orc.DIR_GT, orc.DIR_LT),
                              enable_mask=0b100)
            ss = torch.tensor([[[0.5, 0.5, 40.0]]], dtype=F64)
            out = orc.exit_update(cfg, orc.ExitState.fresh(1), ss, torch.tensor([[1]]), [[0]],
                                  torch.tensor([0]), torch.tensor([9]))
            flags.append(int(out.exit_flag[0]))
        assert flags[0] <= flags[1]                        # non-decreasing in a "less than" threshold
    assert flags == [1, 1]


# ---------------------------------------------------------------- acceptance (Alg. 1)
@pytest.mark.parametrize("K", [1, 2, 3, 4, 5, 6])
def test_accept_chain_brute_force(K):
    for bits in itertools.product("01", repeat=K):
        pattern = "".join(bits)
        cand = [7] + [100 + j for j in range(1, K + 1)]
        target = [(cand[j + 1] if pattern[j] == "1" else 999) for j in range(K)] + [555]
        L, path, rec = orc.accept_chain(cand, target)
        want = pattern.find("0") if "0" in pattern else K          # length of the all-ones prefix
        assert L == want and path == list(range(want + 1)) and rec == target[want] and L <= K


def test_accept_tree_brute_force():
    rng = random.Random(3)
    for trial in range(300):
        P = rng.randint(1, 12)
        parent = [-1] + [rng.randrange(s) for s in range(1, P)]
        tok = [0] * P
        for s in range(1, P):       # siblings carry distinct tokens, as top-k children do
            used = {tok[c] for c in range(1, s) if parent[c] == parent[s]}
            tok[s] = rng.choice([t for t in range(12) if t not in used])
        target = [rng.randrange(4) for _ in range(P)]
        # enumerate every root path, keep the fully accepted ones
        accepted = []
        for s in range(P):
            chain = [s]
            while parent[chain[-1]] >= 0:
                chain.append(parent[chain[-1]])
            chain.reverse()
            if all(tok[chain[i]] == target[chain[i - 1]] for i in range(1, len(chain))):
                accepted.append(chain)
        best = max(len(c) for c in accepted)
        longest = [c for c in accepted if len(c) == best]
        assert len(longest) == 1
        L, path, rec = orc.accept_tree(tok, parent, target)
        assert path == longest[0] and L == best - 1 and rec == target[path[-1]]


# ---------------------------------------------------------------- building blocks: textbook cases
def test_rmsnorm_constant_vector_and_scaling():
    g = torch.tensor([1.0, 2.0, -1.0, 0.5], dtype=F64)
    out = orc.rmsnorm(torch.full((1, 4), -3.0, dtype=F64), g, 0.0)
    assert torch.allclose(out, -g.view(1, 4))
    x = torch.randn(3, 16, dtype=F64)
    a = orc.rmsnorm(x, torch.ones(16, dtype=F64), 0.0)
    assert torch.allclose((a * a).mean(dim=1), torch.ones(3, dtype=F64))         # unit RMS
    assert torch.allclose(orc.rmsnorm(5.0 * x, torch.ones(16, dtype=F64), 0.0), a)  # scale-free
    # eps enters under the root: x = (2, 2), eps = 5 -> 2 / sqrt(4 + 5) = 2/3
    out = orc.rmsnorm(torch.tensor([[2.0, 2.0]], dtype=F64), torch.ones(2, dtype=F64), 5.0)
    assert torch.allclose(out, torch.full((1, 2), 2.0 / 3.0, dtype=F64))


def test_rope_rotation_values_and_properties():
    # d = 2: one pair, frequency theta^0 = 1: (1, 0) at position 1 -> (cos 1, sin 1)
    out = orc.rope(torch.tensor([[1.0, 0.0]], dtype=F64), 1, 10000.0)
    assert torch.allclose(out, torch.tensor([[0.5403023058681398, 0.8414709848078965]], dtype=F64))
    # d = 4, theta = 1e4: pairs (0,2) at frequency 1 and (1,3) at 1e4^(-2/4) = 0.01
    out = orc.rope(torch.tensor([[0.0, 1.0, 0.0, 0.0]], dtype=F64), 100, 10000.0)
    assert torch.allclose(out, torch.tensor([[0.0, math.cos(1.0), 0.0, math.sin(1.0)]], dtype=F64))
    out = orc.rope(torch.tensor([[1.0, 0.0, 0.0, 0.0]], dtype=F64), 3, 10000.0)
    assert torch.allclose(out, torch.tensor([[math.cos(3.0), 0.0, math.sin(3.0), 0.0]], dtype=F64))
    q, k = torch.randn(2, 32, dtype=F64), torch.randn(2, 32, dtype=F64)
    assert torch.allclose(orc.rope(q, 0, 1e6), q)                                   # identity at 0
    assert torch.allclose(orc.rope(q, 977, 1e6).norm(dim=1), q.norm(dim=1))         # an isometry
    d1 = (orc.rope(q, 40, 1e6) * orc.rope(k, 33, 1e6)).sum()
    d2 = (orc.rope(q, 1007, 1e6) * orc.rope(k, 1000, 1e6)).sum()
    assert abs(float(d1 - d2)) < 1e-9                                               # relative only


def test_silu_values():
    x = torch.tensor([0.0, math.log(3.0), -math.log(3.0)], dtype=F64)
    want = torch.tensor([0.0, 0.75 * math.log(3.0), -0.25 * math.log(3.0)], dtype=F64)
    assert torch.allclose(orc.silu(x), want)


def _mini_model(H=8, n_q=2, n_kv=1, d=4, F=8, V=5, S=1, page=4, eps=1e-12, theta=1e4):
    sh = synth.ModelShape(H=H, n_q=n_q, n_kv=n_kv, d=d, F=F, V=V, S=S, eps=eps, theta=theta, page=page)
    z = lambda *s: torch.zeros(*s, dtype=torch.bfloat16)
    w = {"embed": z(V, H), "fc": z(H, 2 * H), "norm1": torch.ones(H, dtype=torch.bfloat16),
         "norm2": torch.ones(H, dtype=torch.bfloat16), "normf": torch.ones(H, dtype=torch.bfloat16),
         "wqkv": z(sh.qkv_rows, H), "wo": z(H, n_q * d), "wgate_up": z(2 * F, H), "wdown": z(H, F),
         "head": z(V + S, H)}
    w["fc"][:, :H] = torch.eye(H, dtype=torch.bfloat16)       # x = feature
    return sh, w


def _mini_kv(sh, n, kval=None, vval=None, extra=4, seed=0):
    lens = torch.tensor([n], dtype=torch.int32)
    kv = synth.make_kv(sh, lens, extra, seed, poison_tail=True)
    if kval is not None:
        kv["k_pages"][:] = kval
    if vval is not None:
        kv["v_pages"][:] = vval
    return orc.PagedKV(kv["k_pages"], kv["v_pages"], kv["page_table"], kv["cache_len"])


def test_one_token_hand_example():
    g = {r[0]: [float(v) for v in r[1:]] for r in _rows("one_token_example.txt")}
    sh, w = _mini_model(H=2, n_q=1, n_kv=1, d=2, F=2, V=3, S=1)
    w["head"][:] = torch.tensor([[1, 0], [0, 1], [1, 1], [1, -1]], dtype=torch.bfloat16)
    w["wqkv"][:] = 0.37                                     # attention runs, W_o = 0 discards it
    model = orc.DraftModel(sh, w, act=(orc.ACT_SIGMOID,))
    kv = _mini_kv(sh, 3)
    d = orc.draft_chain(model, kv, torch.tensor([[3.0, 4.0]], dtype=torch.bfloat16),
                        torch.tensor([1]), K=1)
    assert torch.allclose(d.hidden[0, 0], torch.tensor(g["g_bf16"], dtype=F64), atol=0, rtol=0)
    assert (d.hidden[0, 0] - torch.tensor(g["g_exact"], dtype=F64)).abs().max() < 4e-3
    assert int(d.cand_tok[0, 1]) == int(g["token"][0])
    assert abs(float(d.z[0, 0, 0]) - g["z_bf16"][0]) < 1e-7
    assert abs(float(d.slot_signal[0, 0, 0]) - g["sigmoid_bf16"][0]) < 1e-6
    assert abs(float(d.slot_signal[0, 0, 0]) - g["sigmoid_exact"][0]) < 2e-3
    assert bool(torch.isnan(d.slot_signal[0, 1]).all())     # slot K was never drafted from


def test_layer_residual_only_closed_form():
    # W_o = 0 and W_down = 0: the layer adds nothing, g = RMSNorm(feature) * gain
    sh, w = _mini_model()
    w["wqkv"][:] = 0.25
    w["wgate_up"][:] = 0.5
    w["normf"][:] = torch.tensor([1, 2, 1, 2, 1, 2, 1, 2], dtype=torch.bfloat16)
    model = orc.DraftModel(sh, w, act=(orc.ACT_SIGMOID,))
    f = torch.tensor([[1, -1, 2, -2, 1, -1, 2, -2]], dtype=torch.bfloat16)
    g, _ = model.round(_mini_kv(sh, 5), [orc.Row(0, f[0].to(F64), 0, 5, 5, [5])])
    rms = math.sqrt(2.5)
    want = torch.tensor([1, -2, 2, -4, 1, -2, 2, -4], dtype=F64) / rms
    assert (g[0] - want).abs().max() < 8e-3 * want.abs().max()


def test_attention_uniform_scores_closed_form():
    # W_qkv = 0: q = k_new = v_new = 0, every score is 0, softmax is uniform over the n cached
    # entries plus the row's own new (zero) entry: o = n/(n+1) * c.  W_o = permutation, so
    # a = x + perm(o); W_down = 0; no final gain.
    sh, w = _mini_model()
    n, c = 7, 2.0
    perm = [3, 0, 1, 2, 7, 4, 5, 6]                        # (W_o o)[i] = o[perm[i]]: not an involution
    for i, p in enumerate(perm):
        w["wo"][i, p] = 1.0
    kv = _mini_kv(sh, n)
    kv.v[:] = torch.arange(4, dtype=torch.bfloat16) + c    # v[dim j] = c + j for every cached slot
    kv.v[:] = torch.where(torch.isnan(kv.k), torch.full_like(kv.v, float("nan")), kv.v)
    f = torch.tensor([[1, 2, 3, 4, 5, 6, 7, 8]], dtype=torch.bfloat16)
    model = orc.DraftModel(sh, w, act=(orc.ACT_SIGMOID,))
    g, _ = model.round(kv, [orc.Row(0, f[0].to(F64), 0, n, n, [n])])
    o = np.array([(c + j) * n / (n + 1) for j in range(4)] * 2)    # both q heads share the kv head
    a = np.arange(1, 9, dtype=np.float64) + o[perm]
    want = a / math.sqrt((a * a).mean())
    assert np.abs(g[0].numpy() - want).max() < 1e-2 * np.abs(want).max()


def test_attention_textbook_cases():
    sh, w = _mini_model(n_q=4, n_kv=2, d=4, H=16)
    model = orc.DraftModel(sh, w)
    # (a) all keys equal -> plain mean of V ; GQA: q heads 0,1 read kv head 0, heads 2,3 kv head 1
    kv = _mini_kv(sh, 6, kval=1.0)
    kv.v[:, 0] = 10.0
    kv.v[:, 1] = 20.0
    kv.len = [6]
    row = orc.Row(0, None, 0, 0, 0, [])
    out = model.attention(kv, row, torch.randn(4, 4, dtype=F64))
    assert torch.allclose(out[:2], torch.full((2, 4), 10.0, dtype=F64))
    assert torch.allclose(out[2:], torch.full((2, 4), 20.0, dtype=F64))
    # (b) one cached entry -> exactly its V
    kv = _mini_kv(sh, 1)
    out = model.attention(kv, row, torch.randn(4, 4, dtype=F64))
    assert torch.allclose(out[0], kv.prefix(0)[1][0, 0])
    # (c) adding one vector to every key shifts all scores alike: output unchanged
    kv = _mini_kv(sh, 9, seed=4)
    q = torch.randn(4, 4, dtype=F64)
    base = model.attention(kv, row, q)
    kv2 = _mini_kv(sh, 9, seed=4)
    kv2.k[:] = (kv2.k.to(torch.float32) + 0.5).to(torch.bfloat16)
    kv3 = orc.PagedKV(kv2.k, kv2.v, kv2.table, kv2.len)
    # bf16 re-rounding of the shifted keys perturbs slightly; compare against the definition
    Kp, Vp = kv3.prefix(0)
    for h in range(4):
        sc = (Kp[h // 2] @ q[h]) / 2.0                       # sqrt(d) = 2
        e = np.exp(sc.numpy() - sc.numpy().max())
        want = (e / e.sum()) @ Vp[h // 2].numpy()
        assert np.abs(model.attention(kv3, row, q)[h].numpy() - want).max() < 1e-12
    # (d) a dominant key wins: q = 50 * k_3 -> output ~ v_3
    Kp, Vp = kv.prefix(0)
    q = torch.stack([50.0 * Kp[0, 3], 50.0 * Kp[0, 3], 50.0 * Kp[1, 3], 50.0 * Kp[1, 3]])
    out = model.attention(kv, row, q)
    sc = (Kp[0] @ q[0]) / 2.0
    if float(sc[3] - torch.cat([sc[:3], sc[4:]]).max()) > 30:
        assert torch.allclose(out[0], Vp[0, 3], atol=1e-9)
    # (e) visible extra slots enter, invisible ones do not
    kv = _mini_kv(sh, 4, kval=1.0, vval=1.0)
    kv.write(0, 4, torch.ones(2, 4), torch.full((2, 4), 6.0))
    kv.write(0, 5, torch.ones(2, 4), torch.full((2, 4), 600.0))
    out = model.attention(kv, orc.Row(0, None, 0, 0, 0, [4]), torch.randn(4, 4, dtype=F64))
    assert torch.allclose(out, torch.full((4, 4), 2.0, dtype=F64))    # (4*1 + 6)/5


def test_mlp_closed_form_with_permutations():
    # W_o = 0; gate = n2[pg], up = n2[pu]; y = a + (silu(gate)*up)[pd]; distinct non-involutive perms
    sh, w = _mini_model()
    pg = [1, 2, 3, 4, 5, 6, 7, 0]
    pu = [2, 3, 4, 5, 6, 7, 0, 1]
    pd = [5, 6, 7, 0, 1, 2, 3, 4]
    for i in range(8):
        w["wgate_up"][i, pg[i]] = 1.0
        w["wgate_up"][8 + i, pu[i]] = 1.0
        w["wdown"][i, pd[i]] = 1.0
    f = np.array([1, -2, 3, -4, 0.5, 1.5, -0.5, 2], dtype=np.float64)
    model = orc.DraftModel(sh, w, act=(orc.ACT_SIGMOID,))
    g, _ = model.round(_mini_kv(sh, 3), [orc.Row(0, torch.tensor(f, dtype=F64), 0, 3, 3, [3])])
    n2 = f / math.sqrt((f * f).mean())
    gate, up = n2[pg], n2[pu]
    m = gate / (1 + np.exp(-gate)) * up
    y = f + m[pd]
    want = y / math.sqrt((y * y).mean())
    assert np.abs(g[0].numpy() - want).max() < 1e-2 * np.abs(want).max()


def test_fc_takes_feature_first_then_embedding():
    # x = W_fc [f ; E[t]] with W_fc = [0 | I]: x is the embedding row of the token
    sh, w = _mini_model()
    w["fc"][:] = 0
    w["fc"][:, 8:] = torch.eye(8, dtype=torch.bfloat16)
    w["embed"][3] = torch.tensor([2, 0, 0, 0, 0, 0, 0, 2], dtype=torch.bfloat16)
    model = orc.DraftModel(sh, w, act=(orc.ACT_SIGMOID,))
    g, _ = model.round(_mini_kv(sh, 3), [orc.Row(0, torch.full((8,), 9.0, dtype=F64), 3, 3, 3, [3])])
    assert torch.allclose(g[0], torch.tensor([2, 0, 0, 0, 0, 0, 0, 2], dtype=F64), atol=1e-2)


def test_paging_layout_invariance():
    # the same logical cache under page sizes 16 / 64 / 128 and shuffled tables: same result
    base = harness.tiny_workload(B=1, len_lo=37, len_hi=37)
    outs = []
    logical = None
    for page, seed in [(16, 1), (64, 2), (128, 3)]:
        wl = synth.Workload(**{**base.__dict__, "shape": synth.ModelShape(
            **{**base.shape.__dict__, "page": page})})
        case = harness.build_case(wl)
        kvd = synth.make_kv(wl.shape, case.kv["cache_len"], wl.draft_rows, seed, poison_tail=True)
        n = 37
        gk = torch.randn(n, wl.shape.n_kv, wl.shape.d, generator=torch.Generator().manual_seed(9)).to(torch.bfloat16)
        gv = torch.randn(n, wl.shape.n_kv, wl.shape.d, generator=torch.Generator().manual_seed(10)).to(torch.bfloat16)
        for s in range(n):
            pp = int(kvd["page_table"][0, s // page])
            kvd["k_pages"][pp, :, s % page] = gk[s]
            kvd["v_pages"][pp, :, s % page] = gv[s]
        kv = orc.PagedKV(kvd["k_pages"], kvd["v_pages"], kvd["page_table"], kvd["cache_len"])
        d = orc.draft_chain(harness.oracle_model(case), kv, case.f0, case.t0, wl.K)
        outs.append(d)
    for d in outs[1:]:
        assert torch.equal(d.cand_tok, outs[0].cand_tok)
        assert torch.equal(d.hidden, outs[0].hidden)


# ---------------------------------------------------------------- extended head (Eq. 1)
def test_head_against_numpy_scan_ties_and_concat():
    torch.manual_seed(0)
    sh = synth.ModelShape(H=64, n_q=4, n_kv=2, d=16, F=96, V=4096)
    w = {"head": (torch.randn(sh.V + 3, sh.H) * 0.02).to(torch.bfloat16)}
    g = torch.randn(5, sh.H).to(torch.bfloat16).to(F64)
    model = orc.DraftModel(sh, w)
    ho = model.head(g)
    Wn = w["head"].to(torch.float64).numpy()
    for r in range(5):
        dense = Wn @ g[r].numpy()
        best, arg = -np.inf, -1
        for i in range(sh.V):                     # linear scan, strict '>' keeps the lower index
            v = np.float32(dense[i])
            if v > best:
                best, arg = v, i
        assert orc.argmax_low(ho.logits[r]) == arg
        # Eq. 1: the signal outputs are the last rows of the same product
        sep = w["head"][sh.V:].to(F64) @ g[r]
        assert torch.allclose(ho.z[r], sep.to(torch.float32).to(F64))
        assert torch.allclose(ho.s[r], (1 / (1 + torch.exp(-ho.z[r]))).to(torch.float32).to(F64))
    # duplicated best row at a lower and a higher index: the lower one wins
    w2 = {"head": w["head"].clone()}
    a = orc.argmax_low(ho.logits[0])
    lo, hi = (5, 4000) if a not in (5, 4000) else (6, 4001)
    w2["head"][lo] = w2["head"][a]
    w2["head"][hi] = w2["head"][a]
    ho2 = orc.DraftModel(sh, w2).head(g[:1])
    assert orc.argmax_low(ho2.logits[0]) == min(lo, a)
    assert orc.top_gap(ho2.logits[0]) == 0.0
    # signal rows never take part in the argmax: make them huge
    w3 = {"head": w["head"].clone()}
    w3["head"][sh.V:] = 50.0 * torch.sign(g[0]).to(torch.bfloat16)
    ho3 = orc.DraftModel(sh, w3).head(g[:1])
    assert orc.argmax_low(ho3.logits[0]) == a and ho3.logits.shape[1] == sh.V


def test_topk_low_order_and_large_vocab_path():
    v = torch.tensor([1.0, 3.0, 3.0, 2.0, 3.0, 0.0], dtype=F64)
    assert orc.topk_low(v, 4) == [1, 2, 4, 3]
    torch.manual_seed(1)
    big = torch.randn(10000, dtype=F64).to(torch.float32).to(F64)
    big[77] = big[9000] = big.max() + 1
    got = orc.topk_low(big, 8)
    want = sorted(range(10000), key=lambda i: (-float(big[i]), i))[:8]
    assert got == want and got[:2] == [77, 9000]


# ---------------------------------------------------------------- tree drafting
def _tree_case(topk, depth, nodes, B=2, V=40):
    sh = synth.ModelShape(H=32, n_q=2, n_kv=1, d=16, F=48, V=V, page=16)
    wl = synth.Workload("t", sh, B=B, mode=synth.TREE, K=depth, topk=topk, max_nodes=nodes,
                        len_lo=9, len_hi=30, seed=21)
    return harness.build_case(wl)


def test_tree_invariants():
    case = _tree_case(topk=3, depth=4, nodes=14)
    wl = case.wl
    model = harness.oracle_model(case)
    model.w = {k: (v.to(torch.float32) * (25.0 if k in ("head",) else 1.0)).to(torch.bfloat16)
               for k, v in case.weights.items()}            # spread the logits a little
    t = orc.draft_tree(model, harness.oracle_kv(case), case.f0, case.t0, wl.K, wl.topk, wl.max_nodes)
    for b in range(wl.B):
        cs = t.cands[b]
        assert len(cs) == 3 + 3 * 9
        for c in cs:
            assert c.logp <= 0.0
            if c.parent >= 0:
                assert c.score <= cs[c.parent].score + 1e-7      # scores fall along a path
                assert cs[c.parent].row == c.src_row              # produced by its parent's row
        kept = {int(x) for x in t.slot_cid[b, 1:]}
        assert len(kept) == wl.max_nodes
        for cid in kept:
            assert cs[cid].parent < 0 or cs[cid].parent in kept   # ancestor-closed
        for s in range(1, wl.P):
            p = int(t.parent[b, s])
            assert 0 <= p < s and int(t.depth[b, s]) == int(t.depth[b, p]) + 1
        worst_kept = min(cs[c].score for c in kept)
        assert all(c.score <= worst_kept for c in cs if c.cid not in kept)
        # children of one parent carry distinct tokens
        for p in range(wl.P):
            ch = [int(t.cand_tok[b, s]) for s in range(1, wl.P) if int(t.parent[b, s]) == p]
            assert len(ch) == len(set(ch))


def test_tree_logprobs_sum_to_one_over_full_vocab():
    case = _tree_case(topk=8, depth=1, nodes=8, B=1, V=8)
    wl = case.wl
    t = orc.draft_tree(harness.oracle_model(case), harness.oracle_kv(case), case.f0, case.t0,
                       1, 8, 8)
    assert abs(sum(math.exp(c.logp) for c in t.cands[0]) - 1.0) < 1e-6
    assert sorted(c.tok for c in t.cands[0]) == list(range(8))


def test_tree_top1_degenerates_to_chain():
    case = _tree_case(topk=1, depth=4, nodes=4)
    wl = case.wl
    model = harness.oracle_model(case)
    t = orc.draft_tree(model, harness.oracle_kv(case), case.f0, case.t0, 4, 1, 4)
    c = orc.draft_chain(model, harness.oracle_kv(case), case.f0, case.t0, 4)
    assert torch.equal(t.cand_tok, c.cand_tok)
    assert torch.equal(t.hidden, c.hidden)
    assert torch.equal(t.slot_signal[:, :4], c.slot_signal[:, :4])
    assert torch.equal(t.parent[:, 1:], torch.arange(4).repeat(wl.B, 1))


# ---------------------------------------------------------------- whole forward vs an independent restatement
def _np_bf16(v):
    """Round-to-nearest-even to bf16 on the bit pattern of the fp32 value (numpy only)."""
    u = np.asarray(v, dtype=np.float64).astype(np.float32).view(np.uint32).astype(np.uint64)
    u = (u + 0x7FFF + ((u >> 16) & 1)) & 0xFFFF0000
    return u.astype(np.uint32).view(np.float32).astype(np.float64)


def _np_forward(case, f, tok, b, n_extra_k, n_extra_v, fused3=False, rnd=lambda v: v):
    """float64 numpy restatement of one draft position, written against the logical (un-paged) cache.
    By default nothing is rounded on the way; ``rnd`` is applied at the points where the method stores a
    bf16 activation (x, the normed inputs, q / k / v, the attention output, a, m, y, the final hidden).
    ``fused3``: the layer with three-feature fusion (f of length 3H goes through fc, f of length H is the
    residual stream itself) and [norm(embedding) ; norm(x)] as the attention input; then y is returned as
    well."""
    sh, w = case.wl.shape, {k: v.to(torch.float64).numpy() for k, v in case.weights.items()}
    page = sh.page
    n = int(case.kv["cache_len"][b])
    K = np.zeros((n, sh.n_kv, sh.d))
    Vv = np.zeros((n, sh.n_kv, sh.d))
    for s in range(n):
        pp = int(case.kv["page_table"][b, s // page])
        K[s] = case.kv["k_pages"][pp, :, s % page].to(torch.float64).numpy()
        Vv[s] = case.kv["v_pages"][pp, :, s % page].to(torch.float64).numpy()
    K = np.concatenate([K] + n_extra_k, axis=0) if n_extra_k else K
    Vv = np.concatenate([Vv] + n_extra_v, axis=0) if n_extra_v else Vv
    pos = K.shape[0]
    def norm(v, g):
        return v / np.sqrt((v ** 2).mean() + sh.eps) * g

    if fused3:
        x = w["fc"] @ f if f.size == 3 * sh.H else f
        att_in = np.concatenate([norm(w["embed"][tok], w["norm_e"]), norm(x, w["norm1"])])
    else:
        x = rnd(w["fc"] @ np.concatenate([f, w["embed"][tok]]))
        att_in = rnd(norm(x, w["norm1"]))

    def rot(v):
        out = v.copy()
        h = sh.d // 2
        for i in range(h):
            ang = pos * sh.theta ** (-2.0 * i / sh.d)
            out[:, i] = v[:, i] * math.cos(ang) - v[:, i + h] * math.sin(ang)
            out[:, i + h] = v[:, i + h] * math.cos(ang) + v[:, i] * math.sin(ang)
        return out

    qkv = w["wqkv"] @ att_in
    q = rnd(rot(qkv[:sh.n_q * sh.d].reshape(sh.n_q, sh.d)))
    k = rnd(rot(qkv[sh.n_q * sh.d:(sh.n_q + sh.n_kv) * sh.d].reshape(sh.n_kv, sh.d)))
    v = rnd(qkv[(sh.n_q + sh.n_kv) * sh.d:].reshape(sh.n_kv, sh.d))
    K = np.concatenate([K, k[None]], axis=0)
    Vv = np.concatenate([Vv, v[None]], axis=0)
    o = np.zeros((sh.n_q, sh.d))
    for h in range(sh.n_q):
        kvh = h // (sh.n_q // sh.n_kv)
        sc = K[:, kvh] @ q[h] / math.sqrt(sh.d)
        p = np.exp(sc - sc.max())
        o[h] = (p / p.sum()) @ Vv[:, kvh]
    o = rnd(o)
    a = rnd(x + w["wo"] @ o.reshape(-1))
    gu = w["wgate_up"] @ rnd(norm(a, w["norm2"]))
    gate, up = gu[:sh.F], gu[sh.F:]
    y = rnd(a + w["wdown"] @ rnd(gate / (1 + np.exp(-gate)) * up))
    g = rnd(norm(y, w["normf"]))
    if fused3:
        return g, w["head"] @ g, k[None], v[None], y
    return g, w["head"] @ g, k[None], v[None]


def test_full_forward_against_float64_restatement():
    wl = synth.workload("C0")
    case = harness.build_case(wl)
    model = harness.oracle_model(case)
    d = orc.draft_chain(model, harness.oracle_kv(case), case.f0, case.t0, 2)
    f = case.f0[0].to(torch.float64).numpy()
    g1, logits1, k1, v1 = _np_forward(case, f, int(case.t0[0]), 0, [], [])
    rel = np.linalg.norm(d.hidden[0, 0].numpy() - g1) / np.linalg.norm(g1)
    assert rel < 1e-2
    assert int(np.argmax(logits1[:wl.shape.V])) == int(d.cand_tok[0, 1]) or float(d.gap[0, 0]) < 5e-2
    s1 = 1 / (1 + np.exp(-logits1[wl.shape.V:]))
    assert np.abs(s1 - d.slot_signal[0, 0].numpy()).max() < 5e-3
    # second position: attends to the first position's fresh K/V as well
    g2, _, _, _ = _np_forward(case, g1, int(d.cand_tok[0, 1]), 0, [k1], [v1])
    rel = np.linalg.norm(d.hidden[0, 1].numpy() - g2) / np.linalg.norm(g2)
    assert rel < 2e-2


def test_full_forward_against_float64_restatement_with_the_rounding_points():
    """The same restatement with bf16 rounding (its own bit-level implementation) at exactly the points
    where an activation is stored: now the two agree to float64 noise except where a value sits on a
    rounding boundary, so a misplaced, missing or extra rounding point (an error of a bf16 ulp, 4e-3, on
    every element of a row) fails, as does any wrong operand."""
    wl = synth.workload("C0")
    case = harness.build_case(wl)
    model = harness.oracle_model(case)
    d = orc.draft_chain(model, harness.oracle_kv(case), case.f0, case.t0, 3)
    f, tok, ks, vs = case.f0[0].to(torch.float64).numpy(), int(case.t0[0]), [], []
    for k in range(3):
        g, logits, k1, v1 = _np_forward(case, f, tok, 0, ks, vs, rnd=_np_bf16)
        got = d.hidden[0, k].numpy()
        rel = np.linalg.norm(got - g) / np.linalg.norm(g)
        assert rel < 1e-3, (k, rel)
        assert np.mean(got == g) > 0.97, (k, np.mean(got == g))    # nearly every element bit-identical
        lg = logits[:wl.shape.V].astype(np.float32)
        assert int(np.argmax(lg)) == int(d.cand_tok[0, k + 1]) or float(d.gap[0, k]) < 1e-3
        s1 = 1 / (1 + np.exp(-logits[wl.shape.V:]))
        assert np.abs(s1 - d.slot_signal[0, k].numpy()).max() < 1e-3
        # continue from the oracle's own state so that each position is checked on identical inputs
        f, tok = got, int(d.cand_tok[0, k + 1])
        ks.append(k1)
        vs.append(v1)


def test_top_gap_is_the_kth_margin_over_the_largest_value():
    """The margin that decides whether a differing decision is exempt: (k-th largest - (k+1)-th largest) /
    |largest|, checked for k = 1 and k = 8 against a sorted list, on values with a known answer and on random
    ones; an off-by-one in k or another denominator fails."""
    v = torch.tensor([0.5, -4.0, 2.0, 1.0, 8.0, 7.5, 3.0, 2.5, 6.0, 5.0, 4.0, 0.0], dtype=F64)
    # sorted: 8, 7.5, 6, 5, 4, 3, 2.5, 2, 1, 0.5, 0, -4
    assert orc.top_gap(v) == pytest.approx((8.0 - 7.5) / 8.0)
    assert orc.top_gap(v, 1) == pytest.approx(0.0625)
    assert orc.top_gap(v, 8) == pytest.approx((2.0 - 1.0) / 8.0)
    assert orc.top_gap(v, 3) == pytest.approx((6.0 - 5.0) / 8.0)
    assert orc.top_gap(-v) == pytest.approx((4.0 - 0.0) / 4.0)          # largest is 4, runner-up 0
    g = torch.Generator().manual_seed(77)
    for _ in range(20):
        x = torch.randn(500, generator=g, dtype=F64) * 3 - 1.0
        srt = sorted((float(t) for t in x), reverse=True)
        for k in (1, 8):
            assert orc.top_gap(x, k) == pytest.approx((srt[k - 1] - srt[k]) / abs(srt[0]), rel=1e-12)
    assert orc.top_gap(torch.tensor([2.0, 2.0, 1.0], dtype=F64)) == 0.0
    assert orc.top_gap(torch.tensor([2.0, 2.0, 1.0], dtype=F64), 2) == pytest.approx(0.5)


def test_order_gap_is_the_smallest_neighbour_gap_among_the_first_k_plus_one():
    v = torch.tensor([0.5, -4.0, 2.0, 1.0, 8.0, 7.5, 3.0, 2.5, 6.0, 5.0, 4.0, 0.0], dtype=F64)
    # sorted: 8, 7.5, 6, 5, 4, 3, 2.5, 2, 1 | 0.5, 0, -4
    assert orc.order_gap(v, 1) == pytest.approx(0.5 / 8.0)
    assert orc.order_gap(v, 3) == pytest.approx(0.5 / 8.0)            # 8 - 7.5 is the smallest among 8, 7.5, 6, 5
    assert orc.order_gap(v, 8) == pytest.approx(0.5 / 8.0)
    w = torch.tensor([10.0, 7.0, 6.9, 1.0, 0.0], dtype=F64)
    assert orc.order_gap(w, 1) == pytest.approx(0.3)                  # cut between 10 and 7
    assert orc.order_gap(w, 2) == pytest.approx(0.01)                 # 7 vs 6.9 decides the cut
    assert orc.order_gap(w, 3) == pytest.approx(0.01)                 # ... and then the order inside the list
    assert orc.order_gap(torch.tensor([3.0, 3.0, 1.0], dtype=F64), 2) == 0.0
    g = torch.Generator().manual_seed(78)
    for _ in range(10):
        x = torch.randn(300, generator=g, dtype=F64)
        srt = sorted((float(t) for t in x), reverse=True)
        want = min(srt[i] - srt[i + 1] for i in range(8)) / abs(srt[0])
        assert orc.order_gap(x, 8) == pytest.approx(want, rel=1e-12)


def test_chain_iteration_end_to_end_properties():
    wl = harness.tiny_workload(B=3, K=4)
    case = harness.build_case(wl)
    model = harness.oracle_model(case)
    d = orc.draft_chain(model, harness.oracle_kv(case), case.f0, case.t0, wl.K)
    th = harness.chain_target_hidden(case, d)
    v = orc.verify(model, th, d.cand_tok)
    assert bool((v.accept_len <= wl.K).all()) and bool((v.accept_len >= 0).all())
    # zero noise: the target hidden IS the draft hidden, so every draft token is accepted
    case0 = harness.Case(wl, case.weights, case.kv, case.f0, case.t0, torch.zeros(wl.B))
    v0 = orc.verify(model, harness.chain_target_hidden(case0, d), d.cand_tok)
    assert bool((v0.accept_len == wl.K).all())
    # forcing a draft token changes everything after it and nothing before it
    alt = (int(d.cand_tok[1, 2]) + 1) % wl.shape.V
    d2 = orc.draft_chain(model, harness.oracle_kv(case), case.f0, case.t0, wl.K, forced={(1, 2): alt})
    assert torch.equal(d2.hidden[1, :2], d.hidden[1, :2]) and int(d2.cand_tok[1, 2]) == alt
    assert not torch.equal(d2.hidden[1, 2], d.hidden[1, 2])
    assert torch.equal(d2.hidden[0], d.hidden[0])


# ---------------------------------------------------------------- commit (Algorithm 1, KV-cache update)
def test_commit_bookkeeping_and_pairing_on_a_tree_path():
    # x = feature (fc = [I | 0]), k = first d components of rmsnorm(x) rotated, v = next d components
    sh, w = _mini_model(H=4, n_q=1, n_kv=1, d=2, F=2, V=6, S=1, page=4, theta=1e4)
    w["wqkv"][2, 0] = 1.0   # k0 <- n1[0]
    w["wqkv"][3, 1] = 1.0   # k1 <- n1[1]
    w["wqkv"][4, 2] = 1.0   # v0 <- n1[2]
    w["wqkv"][5, 3] = 1.0   # v1 <- n1[3]
    model = orc.DraftModel(sh, w, act=(orc.ACT_SIGMOID,))
    n = 5
    kv = _mini_kv(sh, n, extra=6)
    before_k, before_v = kv.k.clone(), kv.v.clone()
    P = 8
    th = torch.zeros(1, P, 4, dtype=torch.bfloat16)
    for s in range(P):
        th[0, s] = torch.tensor([1.0 + s, 2.0, -1.0, 0.5 * s], dtype=torch.bfloat16)
    cand = torch.tensor([[9, 1, 2, 3, 4, 5, 0, 1]])
    path = torch.tensor([[0, 3, 6, -1]])            # accepted: slot 3 (child of the root), then slot 6
    out = orc.commit(model, kv, th, cand, path, torch.tensor([2]), torch.tensor([4]))
    assert out.cache_len == [n + 3] and kv.len == [n + 3]
    assert torch.equal(out.feat0[0], th[0, 6].to(F64)) and int(out.tok0[0]) == 4
    # slot n + 1 pairs the hidden of path slot 0 with the token of path slot 3; the embedding is zero, so
    # only the hidden matters: k = rot(n1[0:2], pos = n + 1), v = n1[2:4]
    for j, src in ((1, 0), (2, 3)):
        x = th[0, src].to(F64)
        n1 = x / torch.sqrt((x * x).mean() + sh.eps)
        n1 = n1.to(torch.bfloat16).to(F64)
        pos = n + j
        ang = pos * sh.theta ** (-0.0)               # d = 2: a single frequency, exponent 0
        want_k = torch.tensor([n1[0] * math.cos(ang) - n1[1] * math.sin(ang),
                               n1[1] * math.cos(ang) + n1[0] * math.sin(ang)], dtype=F64)
        got_k, got_v = kv.read(0, n + j)
        assert (got_k[0] - want_k).abs().max() < 1e-2 * max(1.0, float(want_k.abs().max()))
        assert (got_v[0] - n1[2:4]).abs().max() < 1e-2
    # nothing but the two catch-up slots was written
    kv2 = kv.k.clone()
    for j in (1, 2):
        pp, off = kv._loc(0, n + j)
        kv2[pp, :, off] = before_k[pp, :, off]
    same = (kv2 == before_k) | (torch.isnan(kv2) & torch.isnan(before_k))
    assert bool(same.all())


def test_commit_with_nothing_accepted_keeps_the_cache_and_moves_on_by_one():
    sh, w = _mini_model(H=4, n_q=1, n_kv=1, d=2, F=2, V=6, S=1, page=4)
    model = orc.DraftModel(sh, w, act=(orc.ACT_SIGMOID,))
    kv = _mini_kv(sh, 3, extra=4)
    k0 = kv.k.clone()
    th = torch.randn(1, 3, 4, generator=torch.Generator().manual_seed(1)).to(torch.bfloat16)
    out = orc.commit(model, kv, th, torch.tensor([[1, 2, 3]]), torch.tensor([[0, -1, -1]]), torch.tensor([0]),
                     torch.tensor([5]))
    assert out.cache_len == [4] and int(out.tok0[0]) == 5 and torch.equal(out.feat0[0], th[0, 0].to(F64))
    assert bool(((kv.k == k0) | (torch.isnan(kv.k) & torch.isnan(k0))).all())


def test_commit_kv_against_float64_restatement_and_next_iteration_consistency():
    # C0: after an iteration and its commit, every catch-up slot holds the K/V that the unrounded numpy
    # restatement computes for (target hidden of the previous path slot, accepted token) at that position
    wl = synth.workload("C0")
    case = harness.build_case(wl, poison_tail=False)
    model = harness.oracle_model(case)
    kv = harness.oracle_kv(case)
    d = orc.draft_chain(model, kv, case.f0, case.t0, wl.K)
    th = harness.chain_target_hidden(case, d)
    cand = d.cand_tok.clone()
    cand[0, 1] = int(orc.target_argmax(model, th)[0][0, 0])        # make at least two tokens accepted
    cand[0, 2] = int(orc.target_argmax(model, th)[0][0, 1])
    v = orc.verify(model, th, cand)
    L = int(v.accept_len[0])
    assert L >= 2
    n = int(case.kv["cache_len"][0])
    out = orc.commit(model, kv, th, cand, v.path, v.accept_len, v.recover_tok)
    assert out.cache_len[0] == n + L + 1
    for j in range(1, L + 1):
        f = th[0, j - 1].to(torch.float64).numpy()
        pad = [np.zeros((1, wl.shape.n_kv, wl.shape.d))] * j          # position n + j
        _, _, k_np, v_np = _np_forward(case, f, int(cand[0, j]), 0, pad, pad)
        got_k, got_v = kv.read(0, n + j)
        rel = lambda a, b: float(np.linalg.norm(a - b) / np.linalg.norm(b))
        assert rel(got_k.numpy(), k_np[0]) < 1e-2 and rel(got_v.numpy(), v_np[0]) < 1e-2
    # the next iteration drafts from the committed context without error and its first row sits at n + L + 1
    d2 = orc.draft_chain(model, kv, out.feat0.to(torch.bfloat16), out.tok0, 2)
    assert d2.cand_tok.shape == (1, 3) and kv.len[0] == n + L + 1


# ---------------------------------------------------------------- smoothing rules (Appendix A.1)
def _run_rule(rule, samples, window=3, split_at=()):
    """Feeds one sample per iteration (slot 0 only) and returns the smoothed values."""
    V = 64
    bm = torch.zeros(V // 32, dtype=torch.int32)
    bm[0] = 1 << 5                                         # token 5 is the only step-split token
    cfg = orc.ExitCfg(alpha=0.5, thr=(1e9, 0, 0), enable_mask=1, split_bitmap=bm, stop_think_token=1,
                      smoothing=rule, window=window)
    st = orc.ExitState.fresh(1, S=1)
    xs = []
    for i, s in enumerate(samples):
        sig = torch.tensor([[[s], [float("nan")]]], dtype=F64)
        tok = 5 if i in split_at else 7
        out = orc.exit_update(cfg, st, sig, torch.tensor([[tok, 0]]), [[0]], torch.tensor([0]), torch.tensor([3]))
        assert int(out.exit_flag[0]) == 0
        xs.append(float(out.smoothed[0, 0]))
    return xs


def test_sliding_window_hand_values():
    assert _run_rule(orc.SMOOTH_WINDOW, [1, 2, 3, 4, 5], window=3) == [1.0, 1.5, 2.0, 3.0, 4.0]


def test_momentum_hand_values_and_linear_sequences_are_predicted_exactly():
    # x_t = s_{t-1} + (s_{t-1} - s_{t-N}) / (N - 1) once N + 1 samples exist; fewer differences before
    assert _run_rule(orc.SMOOTH_MOMENTUM, [1, 2, 4, 7, 11], window=3) == [1.0, 1.0, 3.0, 5.5, 9.5]
    # literal form of the printed sum for t = 3, N = 3: s_2 + ((s_1 - s_0) + (s_2 - s_1)) / 2
    assert 4 + ((2 - 1) + (4 - 2)) / 2 == 5.5
    lin = [0.25 + 0.125 * i for i in range(14)]
    xs = _run_rule(orc.SMOOTH_MOMENTUM, lin, window=10)
    assert xs[2:] == lin[2:]


def test_paragraph_mean_resets_at_a_split_token_and_none_passes_through():
    assert _run_rule(orc.SMOOTH_PARAGRAPH, [2, 4, 6, 10], split_at=(1,)) == [2.0, 3.0, 6.0, 8.0]
    assert _run_rule(orc.SMOOTH_NONE, [0.5, 0.25, 0.75]) == [0.5, 0.25, 0.75]


@pytest.mark.parametrize("rule", [orc.SMOOTH_EWMA, orc.SMOOTH_NONE, orc.SMOOTH_WINDOW, orc.SMOOTH_MOMENTUM,
                                  orc.SMOOTH_PARAGRAPH])
def test_every_rule_is_the_identity_on_a_constant_signal(rule):
    assert _run_rule(rule, [0.625] * 14, window=10) == [0.625] * 14


def test_window_longer_than_the_ring_history_wraps_correctly():
    s = [float(i % 7) for i in range(40)]
    xs = _run_rule(orc.SMOOTH_WINDOW, s, window=10)
    for t in range(40):
        lo = max(0, t - 9)
        want = float(torch.tensor(sum(s[lo:t + 1]) / (t + 1 - lo), dtype=torch.float32))
        assert abs(xs[t] - want) < 1e-6


# ---------------------------------------------------------------- reduced draft vocabulary (id map)
def test_permuted_full_size_id_map_leaves_the_drafted_tokens_unchanged():
    # head'[i] = head[pi[i]] with draft_to_token = pi scores the same tokens: chain and tree drafts agree
    wl = harness.tiny_workload(B=2, K=3)
    case = harness.build_case(wl, poison_tail=False)
    sh = wl.shape
    pi = torch.randperm(sh.V, generator=torch.Generator().manual_seed(8))
    w2 = dict(case.weights)
    w2["head"] = torch.cat([case.weights["head"][:sh.V][pi], case.weights["head"][sh.V:]], dim=0)
    w2["draft_to_token"] = pi.to(torch.int32)
    w2["target_head"] = case.weights["head"][:sh.V]
    m1, m2 = orc.DraftModel(sh, case.weights), orc.DraftModel(sh, w2)
    d1 = orc.draft_chain(m1, harness.oracle_kv(case), case.f0, case.t0, wl.K)
    d2 = orc.draft_chain(m2, harness.oracle_kv(case), case.f0, case.t0, wl.K)
    assert torch.equal(d1.cand_tok, d2.cand_tok)
    assert (d1.hidden - d2.hidden).abs().max() == 0 and (d1.slot_signal[:, :-1] - d2.slot_signal[:, :-1]).abs().max() == 0
    wt = harness.tiny_workload(B=2, K=3, mode=synth.TREE, topk=3, max_nodes=8)
    ct = harness.build_case(wt, poison_tail=False, weights=case.weights)
    t1 = orc.draft_tree(m1, harness.oracle_kv(ct), ct.f0, ct.t0, 3, 3, 8)
    t2 = orc.draft_tree(m2, harness.oracle_kv(ct), ct.f0, ct.t0, 3, 3, 8)
    assert torch.equal(t1.cand_tok, t2.cand_tok) and torch.equal(t1.parent, t2.parent)


def test_reduced_draft_vocabulary_drafts_the_best_token_among_its_rows_only():
    sh = synth.ModelShape(H=64, n_q=4, n_kv=2, d=16, F=96, V=200, page=16, Vd=37)
    wl = synth.Workload("rv", sh, B=3, mode=synth.CHAIN, K=2, len_lo=4, len_hi=20, seed=13)
    case = harness.build_case(wl, poison_tail=False)
    assert case.weights["head"].shape[0] == 37 + sh.S and case.weights["target_head"].shape[0] == 200
    model = harness.oracle_model(case)
    d = orc.draft_chain(model, harness.oracle_kv(case), case.f0, case.t0, wl.K)
    allowed = set(case.weights["draft_to_token"].tolist())
    assert set(d.cand_tok[:, 1:].reshape(-1).tolist()) <= allowed
    # brute force for round 1: numpy scan over the 37 rows on the oracle's own hidden
    W = case.weights["head"][:37].to(torch.float64).numpy()
    for b in range(wl.B):
        logits = (W @ d.hidden[b, 0].numpy()).astype(np.float32)
        assert int(case.weights["draft_to_token"][int(np.argmax(logits))]) == int(d.cand_tok[b, 1])
    # the signal rows follow the 37 vocabulary rows
    Wsig = case.weights["head"][37:].to(torch.float64).numpy()
    z = (Wsig @ d.hidden[0, 0].numpy()).astype(np.float32)
    assert np.allclose(z, d.z[0, 0].numpy(), atol=1e-6)
    # verification uses the target's own full-vocabulary head
    v = orc.verify(model, harness.chain_target_hidden(case, d), d.cand_tok)
    assert int(v.target_tok.max()) < 200


# ---------------------------------------------------------------------------------------
# stochastic verification (speculative sampling with deterministic drafts)
# ---------------------------------------------------------------------------------------
def test_philox_known_answers():
    for row in _rows("philox4x32_10_kat.txt"):
        w = [int(x, 16) for x in row]
        out = orc.philox4x32_10(w[0:4], w[4:6])
        assert [int(x) for x in out] == w[6:10]


def test_philox_is_vectorised_over_counters_consistently():
    ctr = np.arange(7, dtype=np.uint64)
    blk = orc.philox4x32_10((ctr, 3, 5, 9), (11, 13))
    for i in range(7):
        one = orc.philox4x32_10((i, 3, 5, 9), (11, 13))
        assert [int(x) for x in one] == [int(blk[k][i]) for k in range(4)]


def test_uniform_is_strictly_inside_the_unit_interval_and_exact_in_float32():
    w = np.array([0, 1, 511, 512, 0x7FFFFFFF, 0x80000000, 0xFFFFFFFF], dtype=np.uint64)
    u = orc.uniform_open(w)
    assert u.min() > 0.0 and u.max() < 1.0
    assert np.array_equal(u.astype(np.float32).astype(np.float64), u)
    assert u[0] == 2.0 ** -24 and u[-1] == 1.0 - 2.0 ** -24 and u[3] == 1.5 * 2.0 ** -23


class _IdentityHead:
    """Stand-in model whose target logits are the hidden state itself."""
    def __init__(self, V):
        self.target_head = torch.eye(V, dtype=torch.bfloat16)


def _draws(logits, tau, n, seed=77, offset=3):
    V = len(logits)
    hid = torch.tensor(logits, dtype=torch.bfloat16).view(1, 1, V).repeat(1, n, 1)
    tok, _ = orc.target_sample(_IdentityHead(V), hid, orc.SampleCfg(tau, seed, offset))
    return tok.view(-1).numpy()


def test_sampled_target_token_follows_the_softmax_at_that_temperature():
    logits = [1.0, -0.5, 2.0, 0.25, 1.5, -2.0]            # exact in bf16
    for tau in (0.5, 1.0, 2.0):
        n = 20000
        t = _draws(logits, tau, n)
        p = np.exp(np.array(logits) / tau)
        p /= p.sum()
        f = np.bincount(t, minlength=len(logits)) / n
        sd = np.sqrt(p * (1 - p) / n)
        assert np.all(np.abs(f - p) < 5 * sd), (tau, f, p)


def test_acceptance_law_of_speculative_sampling_with_a_point_mass_draft():
    # accept x with probability min(1, p(x) / q(x)); otherwise draw from norm(max(0, p - q))
    logits = [0.5, 1.75, -1.0, 1.0, 0.0]
    x, n = 1, 30000
    p = np.exp(np.array(logits))
    p /= p.sum()
    q = np.zeros_like(p)
    q[x] = 1.0
    accept_prob = min(1.0, p[x] / q[x])
    resid = np.maximum(0.0, p - q)
    resid /= resid.sum()
    t = _draws(logits, 1.0, n, seed=5, offset=0)
    cand = [9, x]                                             # slot 0: last accepted token; slot 1: the draft
    acc, rec = [], []
    for i in range(n):
        L, path, r = orc.accept_chain(cand, [int(t[i]), 0])
        acc.append(L)
        if L == 0:
            rec.append(r)
    fa = np.mean(acc)
    assert abs(fa - accept_prob) < 5 * math.sqrt(accept_prob * (1 - accept_prob) / n)
    fr = np.bincount(np.array(rec), minlength=len(p)) / len(rec)
    assert fr[x] == 0.0
    assert np.all(np.abs(fr - resid) < 5 * np.sqrt(resid * (1 - resid) / len(rec)) + 1e-12)


def test_tree_children_tried_in_turn_against_the_residual_keep_child_i_with_probability_p_i():
    # closed form of the sequential rule: child i is reached when all earlier ones were refused,
    # and is then kept with probability p(c_i) / (1 - p(c_1) - ... - p(c_{i-1}))
    logits = [0.5, 1.75, -1.0, 1.0, 0.0, 0.75]
    p = np.exp(np.array(logits))
    p /= p.sum()
    children = [3, 1, 4]
    reach, gone = 1.0, 0.0
    for c in children:
        keep = p[c] / (1.0 - gone)
        assert abs(reach * keep - p[c]) < 1e-15
        reach *= 1.0 - keep
        gone += p[c]
    # ... and the coupled draw reproduces it: one level of a tree, children in slots 1..3
    n = 30000
    t = _draws(logits, 1.0, n, seed=6, offset=1)
    cand, parent = [9] + children, [-1, 0, 0, 0]
    kept = np.zeros(len(children) + 1)
    for i in range(n):
        L, path, r = orc.accept_tree(cand, parent, [int(t[i]), 0, 0, 0])
        kept[path[1] if L else 0] += 1
    f = kept / n
    want = np.array([1.0 - p[children].sum()] + [p[c] for c in children])
    assert np.all(np.abs(f - want) < 5 * np.sqrt(want * (1 - want) / n))


def test_zero_temperature_is_greedy_verification_and_draws_differ_by_slot_sequence_and_offset():
    wl = harness.tiny_workload(B=2, K=3, len_lo=6, len_hi=20)
    case = harness.build_case(wl, poison_tail=False)
    model = harness.oracle_model(case)
    d = orc.draft_chain(model, harness.oracle_kv(case), case.f0, case.t0, wl.K)
    th = harness.chain_target_hidden(case, d)
    v0 = orc.verify(model, th, d.cand_tok)
    v1 = orc.verify(model, th, d.cand_tok, sample=orc.SampleCfg(0.0, 1, 2))
    assert torch.equal(v0.target_tok, v1.target_tok) and torch.equal(v0.accept_len, v1.accept_len)
    g = [orc.gumbel_noise(orc.SampleCfg(1.0, s, o), b, j, 50) for (s, o, b, j) in
         [(1, 0, 0, 0), (1, 0, 0, 1), (1, 0, 1, 0), (1, 1, 0, 0), (2, 0, 0, 0), (1 + (1 << 32), 0, 0, 0)]]
    for a, b in itertools.combinations(range(len(g)), 2):
        assert not torch.equal(g[a], g[b])
    # a very high temperature makes the draw nearly uniform: it leaves the greedy choice often
    hot = orc.verify(model, th, d.cand_tok, sample=orc.SampleCfg(50.0, 1, 0))
    assert not torch.equal(hot.target_tok, v0.target_tok)


# ---------------------------------------------------------------------------------------
# the draft layer with three-feature fusion and a concatenated attention input
# ---------------------------------------------------------------------------------------
_SH_F3 = synth.ModelShape(H=64, n_q=4, n_kv=2, d=16, F=96, V=200, page=16, arch=1)


def test_fused3_round_one_reduces_to_the_concat_layer_when_the_extra_inputs_are_switched_off():
    # concat layer whose fc ignores the embedding  ==  fused layer fed [f ; 0 ; 0] whose q/k/v
    # projection ignores the (normalised) embedding half: same x, same residual, same y
    wl0 = harness.tiny_workload(B=2, K=1, len_lo=7, len_hi=21)
    c0 = harness.build_case(wl0, poison_tail=False)
    sh0, H = wl0.shape, wl0.shape.H
    w0 = dict(c0.weights)
    fc0 = w0["fc"].clone()
    fc0[:, H:] = 0
    w0["fc"] = fc0
    wl1 = dataclasses.replace(wl0, shape=dataclasses.replace(sh0, arch=1))
    w1 = synth.make_weights(wl1.shape, wl1.seed)
    for k in ("embed", "norm1", "norm2", "normf", "wo", "wgate_up", "wdown", "head"):
        w1[k] = w0[k]
    fc1 = w1["fc"].clone()
    fc1[:, :H] = fc0[:, :H]
    w1["fc"] = fc1
    wq = torch.zeros_like(w1["wqkv"])
    wq[:, H:] = w0["wqkv"]
    w1["wqkv"] = wq
    f3 = torch.cat([c0.f0, torch.zeros(wl0.B, 2 * H, dtype=c0.f0.dtype)], dim=1)
    m0, m1 = orc.DraftModel(sh0, w0), orc.DraftModel(wl1.shape, w1)
    kv0, kv1 = harness.oracle_kv(c0), harness.oracle_kv(c0)
    d0 = orc.draft_chain(m0, kv0, c0.f0, c0.t0, 1)
    d1 = orc.draft_chain(m1, kv1, f3, c0.t0, 1)
    assert torch.equal(d0.cand_tok, d1.cand_tok)
    assert torch.equal(d0.slot_signal[:, 0], d1.slot_signal[:, 0])
    g_from_y = orc.bf16r(orc.rmsnorm(d1.hidden[:, 0], w1["normf"], sh0.eps))
    assert torch.equal(g_from_y, d0.hidden[:, 0])
    for b in range(wl0.B):
        ka, va = kv0.read(b, kv0.len[b])
        kb, vb = kv1.read(b, kv1.len[b])
        assert torch.equal(ka, kb) and torch.equal(va, vb)
    # ... and switching the other half off instead changes the result: the halves are not symmetric
    wq2 = torch.zeros_like(wq)
    wq2[:, :H] = w0["wqkv"]
    w2 = dict(w1)
    w2["wqkv"] = wq2
    d2 = orc.draft_chain(orc.DraftModel(wl1.shape, w2), harness.oracle_kv(c0), f3, c0.t0, 1)
    assert not torch.equal(d2.hidden, d1.hidden)


def test_fused3_two_rounds_against_float64_restatement():
    wl = synth.Workload("f3", _SH_F3, B=2, mode=synth.CHAIN, K=2, len_lo=9, len_hi=30, seed=51)
    case = harness.build_case(wl, poison_tail=False)
    assert case.f0.shape == (2, 3 * 64) and case.weights["fc"].shape == (64, 192)
    assert case.weights["wqkv"].shape == (_SH_F3.qkv_rows, 128)
    model = harness.oracle_model(case)
    d = orc.draft_chain(model, harness.oracle_kv(case), case.f0, case.t0, 2)
    for b in range(wl.B):
        f = case.f0[b].to(torch.float64).numpy()
        g1, logits1, k1, v1, y1 = _np_forward(case, f, int(case.t0[b]), b, [], [], fused3=True)
        assert np.linalg.norm(d.hidden[b, 0].numpy() - y1) / np.linalg.norm(y1) < 1e-2
        s1 = 1 / (1 + np.exp(-logits1[wl.shape.V:]))
        assert np.abs(s1 - d.slot_signal[b, 0].numpy()).max() < 5e-3
        assert int(np.argmax(logits1[:wl.shape.V])) == int(d.cand_tok[b, 1]) or float(d.gap[b, 0]) < 5e-2
        # round 2 continues from y (not from its final norm, and without fc)
        g2, logits2, _, _, y2 = _np_forward(case, y1, int(d.cand_tok[b, 1]), b, [k1], [v1], fused3=True)
        assert np.linalg.norm(d.hidden[b, 1].numpy() - y2) / np.linalg.norm(y2) < 2e-2
        wrong = _np_forward(case, g1, int(d.cand_tok[b, 1]), b, [k1], [v1], fused3=True)[4]
        assert np.linalg.norm(d.hidden[b, 1].numpy() - wrong) / np.linalg.norm(wrong) > 5e-2


def test_fused3_tree_with_one_child_per_node_is_the_chain():
    wl = synth.Workload("f3t", _SH_F3, B=2, mode=synth.TREE, K=3, topk=1, max_nodes=3, len_lo=9, len_hi=30, seed=52)
    case = harness.build_case(wl, poison_tail=False)
    model = harness.oracle_model(case)
    t = orc.draft_tree(model, harness.oracle_kv(case), case.f0, case.t0, 3, 1, 3)
    c = orc.draft_chain(model, harness.oracle_kv(case), case.f0, case.t0, 3)
    assert torch.equal(t.cand_tok, c.cand_tok)
    assert torch.equal(t.hidden, c.hidden)


def test_fused3_commit_rekeys_from_the_three_target_features():
    wl = synth.Workload("f3c", _SH_F3, B=2, mode=synth.CHAIN, K=2, len_lo=9, len_hi=30, seed=53)
    case = harness.build_case(wl, poison_tail=False)
    case.kv.update(synth.make_kv(wl.shape, synth.cache_lengths(wl), wl.K + 2, wl.seed, poison_tail=False))
    model = harness.oracle_model(case)
    kv = harness.oracle_kv(case)
    n0 = list(kv.len)
    g = torch.Generator().manual_seed(2)
    tf = torch.randn(wl.B, wl.P, 3 * _SH_F3.H, generator=g).to(torch.bfloat16)
    cand = torch.randint(0, _SH_F3.V, (wl.B, wl.P), generator=g)
    path = torch.tensor([[0, 1, 2], [0, 1, -1]])
    L, rec = torch.tensor([2, 1]), torch.tensor([7, 8])
    oc = orc.commit(model, kv, tf, cand, path, L, rec)
    assert oc.cache_len == [n0[0] + 3, n0[1] + 2] and oc.feat0.shape == (2, 3 * _SH_F3.H)
    assert torch.equal(oc.feat0[0], tf[0, 2].to(torch.float64)) and torch.equal(oc.feat0[1], tf[1, 1].to(torch.float64))
    # the K/V of accepted token j: the restatement fed (features of path slot j - 1, token of slot j)
    for b, j in ((0, 1), (0, 2), (1, 1)):
        f = tf[b, j - 1].to(torch.float64).numpy()
        extra_k = [kv.read(b, n0[b] + i)[0].numpy()[None] for i in range(0, j)]
        extra_v = [kv.read(b, n0[b] + i)[1].numpy()[None] for i in range(0, j)]
        _, _, k1, v1, _ = _np_forward(case, f, int(cand[b, j]), b, extra_k, extra_v, fused3=True)
        kk, vv = kv.read(b, n0[b] + j)
        assert np.linalg.norm(kk.numpy() - k1[0]) / np.linalg.norm(k1[0]) < 1e-2
        assert np.linalg.norm(vv.numpy() - v1[0]) / np.linalg.norm(v1[0]) < 1e-2


# ---------------------------------------------------------------------------------------
# speculative sampling with sampled drafts (accept test + residual draw)
# ---------------------------------------------------------------------------------------
class _IdentityModel(_IdentityHead):
    def __init__(self, V):
        super().__init__(V)
        self.map = None
        self.sh = synth.ModelShape(H=V, n_q=1, n_kv=1, d=8, F=8, V=V)


def test_speculative_sampling_emits_the_target_distribution_whatever_the_draft_distribution():
    # the defining property of the rule: x ~ q, kept with min(1, p/q), else a draw from norm(max(0, p - q))
    # gives a token distributed as p; the acceptance rate is sum_i min(p_i, q_i)
    lp = [1.0, -0.5, 2.0, 0.25, 1.5, -2.0]
    lq = [0.5, 1.0, 0.0, 2.0, -1.0, 0.25]
    V, n = 6, 20000
    for tau in (1.0, 0.5):
        cfg = orc.SampleCfg(tau, 99, 5, True)
        p = np.exp(np.array(lp) / tau)
        p /= p.sum()
        q = np.exp(np.array(lq) / tau)
        q /= q.sum()
        cand = torch.zeros(n, 2, dtype=torch.int64)
        for b in range(n):          # one draft draw per sequence, as draft_chain makes it
            s = torch.tensor(lq, dtype=F64) + tau * orc.gumbel_noise(cfg, b, orc.DRAFT_STREAM, V)
            cand[b, 1] = orc.argmax_low(s)
        fq = np.bincount(cand[:, 1].numpy(), minlength=V) / n
        assert np.all(np.abs(fq - q) < 5 * np.sqrt(q * (1 - q) / n))
        dl = torch.tensor(lq, dtype=F64).view(1, 1, V).repeat(n, 1, 1)
        hid = torch.tensor(lp, dtype=torch.bfloat16).view(1, 1, V).repeat(n, 2, 1)
        so = orc.speculative_sample(_IdentityModel(V), hid, cand, dl, cfg)
        f = np.bincount(so.target_tok[:, 0].numpy(), minlength=V) / n
        assert np.all(np.abs(f - p) < 5 * np.sqrt(p * (1 - p) / n)), (tau, f, p)
        rate = float(so.accepted[:, 0].float().mean())
        want = float(np.minimum(p, q).sum())
        assert abs(rate - want) < 5 * math.sqrt(want * (1 - want) / n)
        # the last slot has no draft: a plain draw from p
        f1 = np.bincount(so.target_tok[:, 1].numpy(), minlength=V) / n
        assert np.all(np.abs(f1 - p) < 5 * np.sqrt(p * (1 - p) / n))
        assert not bool(so.accepted[:, 1].any())
        # a refused draft token is never drawn again when q exceeds p there
        refused = ~so.accepted[:, 0]
        over = torch.tensor(q > p)[cand[:, 1]]
        assert not bool((so.target_tok[:, 0] == cand[:, 1])[refused & over].any())


def test_speculative_sampling_keeps_every_draft_when_draft_and_target_agree():
    lp = [1.0, -0.5, 2.0, 0.25]
    V, n = 4, 300
    cfg = orc.SampleCfg(0.7, 3, 1, True)
    cand = torch.zeros(n, 2, dtype=torch.int64)
    cand[:, 1] = torch.arange(n) % V
    dl = torch.tensor(lp, dtype=F64).view(1, 1, V).repeat(n, 1, 1)
    hid = torch.tensor(lp, dtype=torch.bfloat16).view(1, 1, V).repeat(n, 2, 1)
    so = orc.speculative_sample(_IdentityModel(V), hid, cand, dl, cfg)
    assert bool(so.accepted[:, 0].all()) and torch.equal(so.target_tok[:, 0], cand[:, 1])


# ---------------------------------------------------------------------------------------
# sampled children in a tree: draws without replacement, the sequential accept / residual rule
# ---------------------------------------------------------------------------------------
def _one_level_tree(n, V, k, lq, cfg):
    """n sequences, each a root (slot 0) with k children drawn from softmax(lq / tau) the way draft_tree
    draws them: the k best of lq + tau * Gumbel noise of the stream TREE_STREAM + 0, best first."""
    tau = cfg.temperature
    cand = torch.zeros(n, 1 + k, dtype=torch.int64)
    rl = {}
    for b in range(n):
        sc = torch.tensor(lq, dtype=F64) + tau * orc.gumbel_noise(cfg, b, orc.TREE_STREAM, V)
        cand[b, 1:] = torch.tensor(orc.topk_low(sc, k))
        rl[(b, 0)] = torch.tensor(lq, dtype=F64)
    parent = torch.tensor([[-1] + [0] * k] * n)
    slot_row = torch.tensor([[0] + [-1] * k] * n)
    return orc.TreeDraft(cands=None, cand_tok=cand, parent=parent, depth=None, slot_row=slot_row, slot_src_row=None,
                         hidden=None, slot_signal=None, row_logits=rl)


def test_children_drawn_with_the_gumbel_top_k_are_a_draw_without_replacement():
    # P(first = i, second = j) = q_i q_j / (1 - q_i): the law of sequential draws without replacement
    lq, V, n, tau = [0.5, 1.0, 0.0, 2.0, -1.0], 5, 20000, 0.8
    cfg = orc.SampleCfg(tau, 17, 3, True)
    d = _one_level_tree(n, V, 2, lq, cfg)
    q = np.exp(np.array(lq) / tau)
    q /= q.sum()
    pair = np.zeros((V, V))
    for a, b2 in d.cand_tok[:, 1:].numpy():
        pair[a, b2] += 1
    pair /= n
    for i in range(V):
        assert pair[i, i] == 0.0
        for j in range(V):
            if i != j:
                want = q[i] * q[j] / (1 - q[i])
                assert abs(pair[i, j] - want) < 5 * math.sqrt(want * (1 - want) / n), (i, j)


def test_tree_walk_with_sampled_children_emits_the_target_distribution():
    # the defining property of the sequential rule: whatever q is and however many children are tried, the
    # token emitted at the root (an accepted child or the final draw) follows p; one child = the chain's rule
    lp = [1.0, -0.5, 2.0, 0.25, 1.5, -2.0]
    lq = [0.5, 1.0, 0.0, 2.0, -1.0, 0.25]
    V, n = 6, 12000
    model = _IdentityModel(V)
    for tau, k in ((1.0, 1), (1.0, 3), (0.6, 2), (1.3, 5)):
        cfg = orc.SampleCfg(tau, 1234, 7, True)
        p = np.exp(np.array(lp) / tau)
        p /= p.sum()
        q = np.exp(np.array(lq) / tau)
        q /= q.sum()
        d = _one_level_tree(n, V, k, lq, cfg)
        hid = torch.tensor(lp, dtype=torch.bfloat16).view(1, 1, V).repeat(n, 1 + k, 1)
        w = orc.tree_speculative_walk(model, hid, d, cfg)
        f = np.bincount(w.target_tok[:, 0].numpy(), minlength=V) / n
        assert np.all(np.abs(f - p) < 5 * np.sqrt(p * (1 - p) / n)), (tau, k, f, p)
        # an accepted child is the root's emitted token and the walk moved there; its own draw follows p again
        moved = w.accept_len == 1
        for b in range(0, n, 97):
            if moved[b]:
                s = w.path[b][1]
                assert int(w.target_tok[b, 0]) == int(d.cand_tok[b, s]) and int(w.target_tok[b, s]) == int(w.recover_tok[b])
            else:
                assert w.path[b] == [0] and int(w.recover_tok[b]) == int(w.target_tok[b, 0])
        if k == 1:
            rate, want = float(moved.float().mean()), float(np.minimum(p, q).sum())
            assert abs(rate - want) < 5 * math.sqrt(want * (1 - want) / n)
        leaf = torch.stack([w.target_tok[b, w.path[b][-1]] for b in range(n) if w.accept_len[b] == 1])
        f2 = np.bincount(leaf.numpy(), minlength=V) / max(1, leaf.numel())
        assert np.all(np.abs(f2 - p) < 5 * np.sqrt(p * (1 - p) / max(1, leaf.numel())) + 1e-9)


def test_tree_walk_accepts_the_first_child_when_draft_and_target_agree_and_can_be_steered():
    lp = [1.0, -0.5, 2.0, 0.25]
    V, n, k = 4, 200, 2
    cfg = orc.SampleCfg(0.7, 3, 1, True)
    d = _one_level_tree(n, V, k, lp, cfg)
    hid = torch.tensor(lp, dtype=torch.bfloat16).view(1, 1, V).repeat(n, 1 + k, 1)
    w = orc.tree_speculative_walk(_IdentityModel(V), hid, d, cfg)
    assert bool((w.accept_len == 1).all()) and all(pth == [0, 1] for pth in w.path)      # p / q = 1 for every token
    # the decision hook (used by the GPU comparison at near-ties) replaces single decisions and is recorded
    w2 = orc.tree_speculative_walk(_IdentityModel(V), hid[:3], d, cfg,
                                   decide=lambda kind, key, default, margin: (False if (kind == "accept" and key == (1, 1)) else default))
    assert w2.path[0] == [0, 1] and w2.path[1] == [0, 2] and w2.exempt == ["accept test b=1 slot=1"]


def test_sampled_tree_children_run_through_the_draft_model():
    sh = synth.ModelShape(H=64, n_q=4, n_kv=2, d=16, F=96, V=300, page=16)
    wl = synth.Workload("st", sh, B=2, mode=synth.TREE, K=3, topk=3, max_nodes=3 + 2 * 9, len_lo=9, len_hi=40, seed=5)
    case = harness.build_case(wl, poison_tail=False)
    w = dict(case.weights)
    w["head"] = (w["head"].to(torch.float32) * 20.0).to(torch.bfloat16)
    case = dataclasses.replace(case, weights=w)
    model = harness.oracle_model(case)
    smp = orc.SampleCfg(1.0, 8, 4, True)
    d = orc.draft_tree(model, harness.oracle_kv(case), case.f0, case.t0, wl.K, wl.topk, wl.max_nodes, sample=smp)
    g = orc.draft_tree(model, harness.oracle_kv(case), case.f0, case.t0, wl.K, wl.topk, wl.max_nodes)
    assert g.row_logits is None and len(d.row_logits) == wl.B * (1 + wl.topk * (wl.K - 1))
    assert torch.equal(d.hidden[:, 0], g.hidden[:, 0])               # the root row does not depend on a draw
    assert not torch.equal(d.cand_tok, g.cand_tok)                   # ... its children do
    for b in range(wl.B):                                            # siblings are distinct tokens; scores stay log-probabilities
        for c in d.cands[b]:
            sib = [x.tok for x in d.cands[b] if x.parent == c.parent and x.src_row == c.src_row]
            assert len(set(sib)) == len(sib)
            lg = d.row_logits[(b, c.src_row)]
            assert abs(c.logp - float(lg[c.tok] - torch.logsumexp(lg, dim=0))) < 1e-5
    th = harness.tree_target_hidden(case, d)
    v = orc.tree_speculative_walk(model, th, d, smp)
    for b in range(wl.B):
        pth = v.path[b]
        assert pth[0] == 0 and all(int(d.parent[b, pth[i + 1]]) == pth[i] for i in range(len(pth) - 1))
        assert int(v.accept_len[b]) == len(pth) - 1 and int(v.recover_tok[b]) == int(v.target_tok[b, pth[-1]])


def test_sampled_chain_drafts_and_their_verification_run_end_to_end():
    wl = harness.tiny_workload(B=2, K=3, len_lo=6, len_hi=20)
    case = harness.build_case(wl, poison_tail=False)
    model = harness.oracle_model(case)
    smp = orc.SampleCfg(0.8, 21, 2, True)
    d = orc.draft_chain(model, harness.oracle_kv(case), case.f0, case.t0, wl.K, sample=smp)
    g = orc.draft_chain(model, harness.oracle_kv(case), case.f0, case.t0, wl.K)
    assert d.logits.shape == (2, 3, wl.shape.V) and g.logits is None
    assert torch.equal(d.hidden[:, 0], g.hidden[:, 0])               # round 1 does not depend on a draw
    assert not torch.equal(d.cand_tok, g.cand_tok)
    th = harness.chain_target_hidden(case, d)
    v = orc.verify(model, th, d.cand_tok, sample=smp, draft_logits=d.logits)
    for b in range(wl.B):
        L = int(v.accept_len[b])
        assert all(int(v.target_tok[b, j]) == int(d.cand_tok[b, j + 1]) for j in range(L))
        assert L == wl.K or int(v.target_tok[b, L]) != int(d.cand_tok[b, L + 1])
        assert int(v.recover_tok[b]) == int(v.target_tok[b, L])
