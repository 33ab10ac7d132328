"""Shared test plumbing: builds a seeded case, runs the CPU oracle on it and derives the
target hiddens the verification step takes as input.  Nothing here comes from the CUDA path."""
from __future__ import annotations

import dataclasses
from dataclasses import dataclass
from typing import Dict, List, Optional

import torch

from oracle import specexit_oracle as orc
from paper_2509_24248_b200 import synth


@dataclass
class Case:
    wl: synth.Workload
    weights: Dict[str, torch.Tensor]
    kv: Dict[str, torch.Tensor]
    f0: torch.Tensor
    t0: torch.Tensor
    sigma: torch.Tensor


def build_case(wl: synth.Workload, poison_tail: bool = True, weights=None) -> Case:
    lens = synth.cache_lengths(wl)
    kv = synth.make_kv(wl.shape, lens, wl.draft_rows, wl.seed, poison_tail=poison_tail)
    f0, t0 = synth.make_f0_t0(wl)
    if weights is None:
        weights = synth.make_weights(wl.shape, wl.seed)
    return Case(wl, weights, kv, f0, t0, synth.noise_sigmas(wl))


def oracle_model(case: Case, act=(orc.ACT_SIGMOID,) * 3) -> orc.DraftModel:
    return orc.DraftModel(case.wl.shape, case.weights, act=act)


def oracle_kv(case: Case) -> orc.PagedKV:
    return orc.PagedKV(case.kv["k_pages"], case.kv["v_pages"], case.kv["page_table"],
                       case.kv["cache_len"])


def chain_target_hidden(case: Case, draft: "orc.ChainDraft") -> torch.Tensor:
    """Target final hidden per verify slot: slot j < K predicts slot j+1, so it is the draft
    hidden of round j+1 plus noise; slot K (never drafted from) reuses round K's hidden with
    its own noise draw.  bf16 ``[B, K+1, H]``."""
    wl = case.wl
    K = wl.K
    eps = synth.unit_noise(wl, K + 1)
    base = torch.empty(wl.B, K + 1, wl.shape.H, dtype=torch.bfloat16)
    hid = draft.hidden.to(torch.bfloat16)
    base[:, :K] = hid
    base[:, K] = hid[:, K - 1]
    return synth.noisy_hidden(base, eps, case.sigma.view(-1, 1, 1))


def tree_target_hidden(case: Case, draft: "orc.TreeDraft") -> torch.Tensor:
    """Slot s: the hidden of the row drafted from it when there is one (it predicts the slot's
    child), else the hidden of the row that produced its token; each with its own noise."""
    wl = case.wl
    P = wl.P
    eps = synth.unit_noise(wl, P)
    hid = draft.hidden.to(torch.bfloat16)
    base = torch.empty(wl.B, P, wl.shape.H, dtype=torch.bfloat16)
    for b in range(wl.B):
        for s in range(P):
            r = int(draft.slot_row[b, s])
            if r < 0:
                r = int(draft.slot_src_row[b, s])
            base[b, s] = hid[b, r]
    return synth.noisy_hidden(base, eps, case.sigma.view(-1, 1, 1))


def default_exit_cfg(wl: synth.Workload, **kw) -> "orc.ExitCfg":
    """Confidence-only gate at the workload's threshold; every token is a boundary."""
    base = dict(alpha=wl.alpha, thr=(wl.thr, 0.8, 100.0), dir=(orc.DIR_GT, orc.DIR_GT, orc.DIR_LT),
                enable_mask=0b001, stop_think_token=min(7, wl.shape.V - 1))
    base.update(kw)
    return orc.ExitCfg(**base)


def tiny_workload(**kw) -> synth.Workload:
    sh = synth.ModelShape(H=64, n_q=4, n_kv=2, d=16, F=96, V=200, page=16)
    base = dict(name="tiny", shape=sh, B=2, mode=synth.CHAIN, K=3, len_lo=5, len_hi=40, seed=11)
    base.update(kw)
    return synth.Workload(**base)
