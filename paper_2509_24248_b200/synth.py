"""Seeded synthetic inputs for the speculative-exit step.

This module only draws random numbers and lays buffers out; it holds none of
the method's arithmetic.  It is the one piece of code that both the CUDA path
and the CPU checker are fed from, so that both see bit-identical bf16 inputs.

Everything is produced on the CPU with ``torch.Generator`` objects whose seed is
derived from ``(workload.seed, item)``, which makes every item independent of
the order in which the others are drawn.  Values are rounded to bf16 once, here.

Workloads (shapes follow the five benchmark configurations):

* ``C0``  tiny exactness case (H=256, vocab 4096, B=1, 128 cached tokens, chain K=4)
* ``C1``  8B-shaped draft, B=1, 4096 cached tokens, chain K=6
* ``C2``  8B-shaped draft, B=32, cached lengths U[2048, 8192], chain K=4, per-sequence noise
* ``C3``  32B-shaped draft, B=8, 16384 cached tokens, chain K=6
* ``C4``  8B-shaped draft, tree (top-8, depth 6, 60 nodes), B=4, 32768 cached tokens
"""
from __future__ import annotations

import dataclasses
from dataclasses import dataclass
from typing import Dict, Optional, Tuple

import torch

CHAIN = 0
TREE = 1

# item ids for the per-item generators
_IT = {"embed": 1, "fc": 2, "norm1": 3, "norm2": 4, "normf": 5, "wqkv": 6, "wo": 7,
       "wgate_up": 8, "wdown": 9, "head": 10, "k": 11, "v": 12, "f0": 13, "t0": 14,
       "noise": 15, "sigma": 16, "lens": 17, "perm": 18, "noise2": 19, "d2t": 20, "target_head": 21,
       "norm_e": 22}


@dataclass(frozen=True)
class ModelShape:
    H: int
    n_q: int
    n_kv: int
    d: int
    F: int
    V: int
    S: int = 3
    eps: float = 1e-6
    theta: float = 1e6
    page: int = 64
    Vd: int = 0          # rows of a reduced draft vocabulary (0: the draft head covers all V ids)
    arch: int = 0        # 0: fc over [hidden ; embedding] every round; 1: three-feature fusion in
    #                      round 1 and [norm(embedding) ; norm(hidden)] as the attention input

    @property
    def qkv_rows(self) -> int:
        return (self.n_q + 2 * self.n_kv) * self.d


@dataclass(frozen=True)
class Workload:
    name: str
    shape: ModelShape
    B: int
    mode: int            # CHAIN | TREE
    K: int               # chain length, or tree depth
    topk: int = 1        # tree: children per expanded node
    max_nodes: int = 0   # tree: nodes kept for verification (without the root)
    alpha: float = 0.3
    thr: float = 0.9
    len_lo: int = 128
    len_hi: int = 128    # cached length is uniform in [len_lo, len_hi]
    sigma_lo: float = 0.5
    sigma_hi: float = 0.5
    seed: int = 0

    @property
    def draft_rows(self) -> int:
        """Rows drafted per sequence over the whole iteration (= new KV slots)."""
        if self.mode == CHAIN:
            return self.K
        return 1 + self.topk * (self.K - 1)

    @property
    def P(self) -> int:
        """Verify positions per sequence."""
        return self.K + 1 if self.mode == CHAIN else 1 + self.max_nodes


SHAPE_TINY = ModelShape(H=256, n_q=4, n_kv=2, d=64, F=688, V=4096)
SHAPE_8B = ModelShape(H=4096, n_q=32, n_kv=8, d=128, F=12288, V=151936)
SHAPE_32B = ModelShape(H=5120, n_q=64, n_kv=8, d=128, F=25600, V=151936)

_WORKLOADS = {
    "C0": Workload("C0", SHAPE_TINY, B=1, mode=CHAIN, K=4, len_lo=128, len_hi=128, seed=0),
    "C1": Workload("C1", SHAPE_8B, B=1, mode=CHAIN, K=6, len_lo=4096, len_hi=4096, seed=1),
    "C2": Workload("C2", SHAPE_8B, B=32, mode=CHAIN, K=4, len_lo=2048, len_hi=8192,
                   sigma_lo=0.2, sigma_hi=1.0, seed=2),
    "C3": Workload("C3", SHAPE_32B, B=8, mode=CHAIN, K=6, len_lo=16384, len_hi=16384, seed=3),
    "C4": Workload("C4", SHAPE_8B, B=4, mode=TREE, K=6, topk=8, max_nodes=60,
                   len_lo=32768, len_hi=32768, seed=4),
}


def workload(name: str, **overrides) -> Workload:
    w = _WORKLOADS[name]
    return dataclasses.replace(w, **overrides) if overrides else w


def _gen(seed: int, item: str) -> torch.Generator:
    g = torch.Generator(device="cpu")
    g.manual_seed(seed * 1000 + _IT[item])
    return g


def _randn_bf16(rows: int, cols: int, std: float, mean: float, g: torch.Generator) -> torch.Tensor:
    """N(mean, std^2) drawn in fp32, row-chunked to bound the temporary, rounded to bf16."""
    out = torch.empty(rows, cols, dtype=torch.bfloat16)
    step = max(1, (1 << 26) // max(cols, 1))
    for r0 in range(0, rows, step):
        r1 = min(rows, r0 + step)
        t = torch.randn(r1 - r0, cols, generator=g, dtype=torch.float32)
        if std != 1.0:
            t.mul_(std)
        if mean != 0.0:
            t.add_(mean)
        out[r0:r1] = t.to(torch.bfloat16)
    return out


def make_weights(shape: ModelShape, seed: int, std: float = 0.02) -> Dict[str, torch.Tensor]:
    """All draft weights, bf16, row-major ``[out, in]``.

    Matrices are N(0, std^2); the three RMSNorm gains are 1 + N(0, std^2).
    ``head`` has ``V + S`` rows: the vocabulary rows first, the signal rows last.
    """
    s = shape
    w = {
        "embed": _randn_bf16(s.V, s.H, std, 0.0, _gen(seed, "embed")),
        "fc": _randn_bf16(s.H, (3 if s.arch else 2) * s.H, std, 0.0, _gen(seed, "fc")),
        "norm1": _randn_bf16(1, s.H, std, 1.0, _gen(seed, "norm1")).reshape(s.H),
        "norm2": _randn_bf16(1, s.H, std, 1.0, _gen(seed, "norm2")).reshape(s.H),
        "normf": _randn_bf16(1, s.H, std, 1.0, _gen(seed, "normf")).reshape(s.H),
        "wqkv": _randn_bf16(s.qkv_rows, (2 if s.arch else 1) * s.H, std, 0.0, _gen(seed, "wqkv")),
        "wo": _randn_bf16(s.H, s.n_q * s.d, std, 0.0, _gen(seed, "wo")),
        "wgate_up": _randn_bf16(2 * s.F, s.H, std, 0.0, _gen(seed, "wgate_up")),
        "wdown": _randn_bf16(s.H, s.F, std, 0.0, _gen(seed, "wdown")),
        "head": _randn_bf16((s.Vd or s.V) + s.S, s.H, std, 0.0, _gen(seed, "head")),
    }
    if s.arch:
        w["norm_e"] = _randn_bf16(1, s.H, std, 1.0, _gen(seed, "norm_e")).reshape(s.H)
    if s.Vd:
        # reduced draft vocabulary: Vd distinct token ids in increasing order, and a target head of its own
        w["draft_to_token"] = torch.sort(torch.randperm(s.V, generator=_gen(seed, "d2t"))[:s.Vd]).values.to(torch.int32)
        w["target_head"] = _randn_bf16(s.V, s.H, std, 0.0, _gen(seed, "target_head"))
    return w


def cache_lengths(w: Workload) -> torch.Tensor:
    if w.len_lo == w.len_hi:
        return torch.full((w.B,), w.len_lo, dtype=torch.int32)
    return torch.randint(w.len_lo, w.len_hi + 1, (w.B,), generator=_gen(w.seed, "lens"),
                         dtype=torch.int32)


def noise_sigmas(w: Workload) -> torch.Tensor:
    if w.sigma_lo == w.sigma_hi:
        return torch.full((w.B,), w.sigma_lo, dtype=torch.float32)
    u = torch.rand(w.B, generator=_gen(w.seed, "sigma"), dtype=torch.float32)
    return w.sigma_lo + (w.sigma_hi - w.sigma_lo) * u


def make_kv(shape: ModelShape, lens: torch.Tensor, extra_slots: int, seed: int,
            poison_tail: bool = False) -> Dict[str, torch.Tensor]:
    """Paged KV cache ``[num_pages, n_kv, page, d]`` (bf16) with a shuffled page table.

    Sequence ``b`` owns ``ceil((lens[b] + extra_slots) / page)`` physical pages; the
    page table maps its logical pages to a random permutation of the physical ones.
    K and V are N(0,1) (K as if already rotated).  With ``poison_tail`` every slot at
    or beyond ``lens[b]`` holds NaN, so that a read past the valid length shows up.
    """
    s = shape
    B = int(lens.numel())
    pages_b = [(int(lens[b]) + extra_slots + s.page - 1) // s.page for b in range(B)]
    num_pages = sum(pages_b)
    max_pages = max(pages_b)
    perm = torch.randperm(num_pages, generator=_gen(seed, "perm")).to(torch.int32)
    table = torch.full((B, max_pages), -1, dtype=torch.int32)
    o = 0
    for b in range(B):
        table[b, :pages_b[b]] = perm[o:o + pages_b[b]]
        o += pages_b[b]
    k = _randn_bf16(num_pages * s.n_kv, s.page * s.d, 1.0, 0.0, _gen(seed, "k")).view(
        num_pages, s.n_kv, s.page, s.d)
    v = _randn_bf16(num_pages * s.n_kv, s.page * s.d, 1.0, 0.0, _gen(seed, "v")).view(
        num_pages, s.n_kv, s.page, s.d)
    if poison_tail:
        for b in range(B):
            n = int(lens[b])
            for lp in range(n // s.page, pages_b[b]):
                lo = max(0, n - lp * s.page)
                pp = int(table[b, lp])
                k[pp, :, lo:, :] = float("nan")
                v[pp, :, lo:, :] = float("nan")
    return {"k_pages": k, "v_pages": v, "page_table": table, "cache_len": lens.clone(),
            "max_pages": max_pages}


def make_f0_t0(w: Workload) -> Tuple[torch.Tensor, torch.Tensor]:
    """Target feature of the last accepted token (N(0,1), bf16) and that token's id."""
    f0 = _randn_bf16(w.B, (3 if w.shape.arch else 1) * w.shape.H, 1.0, 0.0, _gen(w.seed, "f0"))
    t0 = torch.randint(0, w.shape.V, (w.B,), generator=_gen(w.seed, "t0"), dtype=torch.int32)
    return f0, t0


def unit_noise(w: Workload, rows_per_seq: int, which: str = "noise") -> torch.Tensor:
    """Standard-normal draws ``[B, rows_per_seq, H]`` (fp32) for the target hiddens."""
    return torch.randn(w.B, rows_per_seq, w.shape.H, generator=_gen(w.seed, which),
                       dtype=torch.float32)


def noisy_hidden(base_bf16: torch.Tensor, eps: torch.Tensor, sigma) -> torch.Tensor:
    """``bf16(base + sigma * eps)`` in fp32 arithmetic: a stand-in for the target trunk's
    final hidden state at a verify position."""
    return (base_bf16.to(torch.float32) + sigma * eps).to(torch.bfloat16)


def split_bitmap(V: int, modulus: Optional[int]) -> Optional[torch.Tensor]:
    """Bitmap over token ids (uint32 words as int32 storage) marking ``id % modulus == 0``
    as step-split tokens; ``None`` means every token is a boundary."""
    if modulus is None:
        return None
    ids = torch.arange(V, dtype=torch.int64)
    bits = (ids % modulus == 0)
    words = (V + 31) // 32
    pad = torch.zeros(words * 32, dtype=torch.int64)
    pad[:V] = bits.to(torch.int64)
    sh = torch.arange(32, dtype=torch.int64)
    vals = (pad.view(words, 32) << sh).sum(dim=1)            # < 2^32
    vals = torch.where(vals >= 2 ** 31, vals - 2 ** 32, vals)  # two's complement
    return vals.to(torch.int32)
