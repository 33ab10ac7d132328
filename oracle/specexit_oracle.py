"""CPU oracle for the speculative-exit step.  TEST INFRASTRUCTURE ONLY.

A plain, slow, step-by-step restatement of what one iteration of signal-guided
speculative decoding computes (Algorithm 1 of the paper, the body of its loop without
the target trunk): the draft pass run autoregressively, the extended head of Eq. 1
(token logits plus the confidence / progress / remaining rows), the activations of
Eq. 3-5, greedy verification against the target head, and the smoothed, thresholded
exit decision (Section 3.3, Appendix A.1).  Only the tests, the smoke check and the
benchmark's CPU-baseline leg may use it; the product never does, and it shares no code
with the CUDA path.

Arithmetic.  Every contraction and every elementwise step is evaluated in float64 with
library matmuls as single steps, so a result does not depend on summation order.  Values
are then rounded to the storage type the method fixes: activations handed from one layer
to the next are bf16 (via fp32, round-to-nearest-even) at exactly these points -
x, n1, q, k, v (q and k after the rotation), o, a, n2, m, y, g - and logits, signal
values, log-probabilities, scores and the smoothed state are fp32.  An argmax is taken on
the fp32 logits; ties go to the lower index.

Parity status.  The paper prints no numeric example of the draft forward, so that part is
"parity unpinned" by the paper itself; tests pin it against closed forms, textbook special
cases, brute force and an independent float64 restatement instead.  The smoothing rule, the
activations, the threshold logic and the acceptance rule are pinned by hand-worked values
and invariants (see tests/).
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field
from typing import Dict, List, Optional, Sequence, Tuple

import torch

F64 = torch.float64

# signal activations (Eq. 3-5): sigmoid for confidence/progress; the remaining-length row
# regresses log(1 + r), so r = exp(z) - 1
ACT_SIGMOID, ACT_EXPM1, ACT_IDENTITY = 0, 1, 2
DIR_GT, DIR_LT = 0, 1
EMA_VERIFIED_CONTEXT, EMA_FIRST_ONLY = 0, 1

EXEMPT_REL_GAP = 1e-3

# Draft layer shapes.  ARCH_CONCAT (the layer the rest of this file describes): the previous
# hidden state and the token embedding are concatenated and mixed by fc (2H -> H) in every round.
# ARCH_FUSED3 (the EAGLE-3-shaped layer; the paper trains its draft with that recipe but does not
# describe the layer, so this follows that publication): round 1 receives three target features
# (low / middle / high layer, 3H) fused by fc (3H -> H); the attention input is the
# concatenation [RMSNorm_e(embedding) ; RMSNorm_1(x)] (2H) while the residual stream starts
# from x itself; later rounds take the layer's own output y (before the final norm) as x,
# without fc.  The head still reads RMSNorm_f(y).
ARCH_CONCAT, ARCH_FUSED3 = 0, 1


def bf16r(x: torch.Tensor) -> torch.Tensor:
    """Round to bf16 the way a kernel holding an fp32 value would; result kept as f64."""
    return x.to(torch.float32).to(torch.bfloat16).to(F64)


def f32r(x: torch.Tensor) -> torch.Tensor:
    return x.to(torch.float32).to(F64)


def linear(x: torch.Tensor, W: torch.Tensor, chunk: int = 8192) -> torch.Tensor:
    """``x @ W^T`` in float64.  ``x`` is ``[R, K]`` f64, ``W`` is ``[N, K]`` (bf16 storage).
    ``W`` is widened a slab of rows at a time only to bound memory."""
    R, N = x.shape[0], W.shape[0]
    out = torch.empty(R, N, dtype=F64)
    for n0 in range(0, N, chunk):
        n1 = min(N, n0 + chunk)
        out[:, n0:n1] = x @ W[n0:n1].to(F64).t()
    return out


def rmsnorm(x: torch.Tensor, gamma: torch.Tensor, eps: float) -> torch.Tensor:
    """Root-mean-square normalisation over the last axis, then the gain."""
    ms = (x * x).mean(dim=-1, keepdim=True)
    return x * torch.rsqrt(ms + eps) * gamma.to(F64)


def rope(x: torch.Tensor, pos: int, theta: float) -> torch.Tensor:
    """Rotary embedding, rotate-half pairing (i, i + d/2), absolute position ``pos``.
    ``x`` is ``[heads, d]``."""
    d = x.shape[-1]
    half = d // 2
    i = torch.arange(half, dtype=F64)
    ang = float(pos) * torch.pow(torch.tensor(theta, dtype=F64), -2.0 * i / d)
    c, s = torch.cos(ang), torch.sin(ang)
    x1, x2 = x[..., :half], x[..., half:]
    return torch.cat([x1 * c - x2 * s, x2 * c + x1 * s], dim=-1)


def silu(x: torch.Tensor) -> torch.Tensor:
    return x / (1.0 + torch.exp(-x))


def activate(z: torch.Tensor, act: Sequence[int]) -> torch.Tensor:
    """Eq. 3-5: map the raw signal rows ``z [..., S]`` to signal values."""
    out = torch.empty_like(z)
    for i, a in enumerate(act):
        zi = z[..., i]
        if a == ACT_SIGMOID:
            out[..., i] = 1.0 / (1.0 + torch.exp(-zi))
        elif a == ACT_EXPM1:
            out[..., i] = torch.expm1(zi)
        else:
            out[..., i] = zi
    return out


def argmax_low(v: torch.Tensor) -> int:
    """Index of the maximum; the lowest index among equals."""
    m = v.max()
    return int(torch.nonzero(v == m)[0, 0])


def top_gap(v: torch.Tensor, k: int = 1) -> float:
    """(k-th largest - (k+1)-th largest) / |largest| on fp32 logits: the deciding margin."""
    t = torch.topk(v, k + 1).values
    den = abs(float(t[0]))
    return float(t[k - 1] - t[k]) / den if den > 0 else 0.0


def order_gap(v: torch.Tensor, k: int) -> float:
    """Smallest gap between neighbours among the k + 1 largest values, over |largest|: the margin by which
    an ordered top-k list (its order and its cut) is decided."""
    t = torch.topk(v, min(k + 1, v.numel())).values
    den = abs(float(t[0]))
    if t.numel() < 2 or den == 0:
        return 0.0 if den == 0 else 1.0
    return float((t[:-1] - t[1:]).min()) / den


def topk_low(v: torch.Tensor, k: int) -> List[int]:
    """The k largest entries, larger value first, lower index first among equals."""
    order = sorted(range(v.numel()), key=lambda i: (-float(v[i]), i)) if v.numel() <= 4096 else None
    if order is not None:
        return order[:k]
    # large vocabularies: take a candidate pool, then order it exactly
    pool = torch.topk(v, min(v.numel(), k + 32)).indices.tolist()
    kth = sorted((float(v[i]) for i in pool), reverse=True)[k - 1]
    pool = torch.nonzero(v >= kth).flatten().tolist()
    pool.sort(key=lambda i: (-float(v[i]), i))
    return pool[:k]


# --------------------------------------------------------------------------------------
# paged KV cache
# --------------------------------------------------------------------------------------
class PagedKV:
    """Private copy of a paged bf16 KV cache ``[num_pages, n_kv, page, d]``."""

    def __init__(self, k_pages, v_pages, page_table, cache_len):
        self.k = k_pages.clone()
        self.v = v_pages.clone()
        self.table = page_table.clone()
        self.len = [int(n) for n in cache_len]
        self.page = int(k_pages.shape[2])
        self._prefix: Dict[int, Tuple[torch.Tensor, torch.Tensor]] = {}

    def _loc(self, b: int, slot: int) -> Tuple[int, int]:
        lp, off = divmod(slot, self.page)
        if lp >= self.table.shape[1] or int(self.table[b, lp]) < 0:
            raise IndexError(f"slot {slot} of sequence {b} is beyond its page table")
        return int(self.table[b, lp]), off

    def write(self, b: int, slot: int, k: torch.Tensor, v: torch.Tensor) -> None:
        pp, off = self._loc(b, slot)
        self.k[pp, :, off, :] = k.to(torch.bfloat16)
        self.v[pp, :, off, :] = v.to(torch.bfloat16)

    def read(self, b: int, slot: int) -> Tuple[torch.Tensor, torch.Tensor]:
        pp, off = self._loc(b, slot)
        return self.k[pp, :, off, :].to(F64), self.v[pp, :, off, :].to(F64)

    def prefix(self, b: int) -> Tuple[torch.Tensor, torch.Tensor]:
        """K, V of slots [0, len[b]) as ``[n_kv, len, d]`` f64 (kept: the prefix is fixed
        for the whole iteration)."""
        if b not in self._prefix:
            n = self.len[b]
            npg = (n + self.page - 1) // self.page
            pages = self.table[b, :npg].to(torch.int64)
            kk = self.k[pages].permute(1, 0, 2, 3).reshape(self.k.shape[1], npg * self.page, self.k.shape[3])
            vv = self.v[pages].permute(1, 0, 2, 3).reshape(self.v.shape[1], npg * self.page, self.v.shape[3])
            self._prefix[b] = (kk[:, :n].to(F64), vv[:, :n].to(F64))
        return self._prefix[b]


# --------------------------------------------------------------------------------------
# the draft model: concat(feature, embedding) -> fc -> one pre-norm decoder layer -> norm
# -> extended head (Eq. 1)
# --------------------------------------------------------------------------------------
@dataclass
class Row:
    b: int                 # sequence
    feat: torch.Tensor     # [H] f64 holding bf16 values: hidden of the previous position
    tok: int               # token at this position
    pos: int               # absolute rotary position
    slot: int              # cache slot its K/V are written to
    visible: List[int]     # slots beyond the cached prefix it may attend to (incl. its own)


@dataclass
class HeadOut:
    logits: torch.Tensor   # [R, V] fp32 values in f64
    z: torch.Tensor        # [R, S] raw signal rows, fp32 values
    s: torch.Tensor        # [R, S] activated signals, fp32 values


class DraftModel:
    def __init__(self, shape, weights: Dict[str, torch.Tensor], act=(ACT_SIGMOID,) * 3,
                 target_head: Optional[torch.Tensor] = None):
        self.sh = shape
        self.w = weights
        self.act = tuple(act)
        self.arch = int(getattr(shape, "arch", ARCH_CONCAT))
        # The draft head may cover a reduced vocabulary: its first Vd rows score the draft ids
        # 0..Vd-1, `draft_to_token` maps a draft id to the token id it stands for (identity when
        # absent); the signal rows of Eq. 1 follow the Vd vocabulary rows.
        self.Vd = int(weights["head"].shape[0]) - shape.S
        m = weights.get("draft_to_token")
        self.map = None if m is None else [int(t) for t in m]
        assert self.map is None or len(self.map) == self.Vd
        # the target's LM head; by default the draft's vocabulary rows (full vocabulary only)
        if target_head is None:
            target_head = weights.get("target_head")
        if target_head is None:
            assert self.Vd == shape.V, "a reduced draft vocabulary needs the target's own head"
            target_head = weights["head"][:shape.V]
        self.target_head = target_head

    def to_token(self, draft_id: int) -> int:
        return int(draft_id) if self.map is None else self.map[int(draft_id)]

    # Eq. 1: one matrix, vocabulary rows first, signal rows last, same hidden state
    def head(self, g: torch.Tensor) -> HeadOut:
        V, S = self.Vd, self.sh.S
        full = f32r(linear(g, self.w["head"]))
        z = full[:, V:V + S]
        return HeadOut(logits=full[:, :V], z=z, s=f32r(activate(z, self.act)))

    def attention(self, kv: PagedKV, row: Row, q: torch.Tensor) -> torch.Tensor:
        """softmax(q K^T / sqrt(d)) V over the cached prefix and the visible new slots.
        ``q`` is ``[n_q, d]``; returns ``[n_q, d]``."""
        sh = self.sh
        group = sh.n_q // sh.n_kv
        Kp, Vp = kv.prefix(row.b)
        extra = [kv.read(row.b, s) for s in row.visible]
        if extra:
            Ke = torch.stack([e[0] for e in extra], dim=1)   # [n_kv, E, d]
            Ve = torch.stack([e[1] for e in extra], dim=1)
            Kall, Vall = torch.cat([Kp, Ke], dim=1), torch.cat([Vp, Ve], dim=1)
        else:
            Kall, Vall = Kp, Vp
        out = torch.empty(sh.n_q, sh.d, dtype=F64)
        for h in range(sh.n_q):
            kvh = h // group
            sc = (Kall[kvh] @ q[h]) / math.sqrt(sh.d)
            p = torch.softmax(sc, dim=0)
            out[h] = p @ Vall[kvh]
        return out

    def layer_input(self, rows: List[Row]) -> Tuple[torch.Tensor, torch.Tensor]:
        """u = [feature ; embedding], x = fc u, n1 = RMSNorm(x), and the fused q/k/v projection of
        n1.  Returns ``x [R, H]`` (bf16 values) and ``qkv [R, (n_q + 2 n_kv) d]`` (unrounded)."""
        sh, w = self.sh, self.w
        toks = torch.tensor([r.tok for r in rows], dtype=torch.int64)
        if self.arch == ARCH_FUSED3:
            # a row that carries the three target features (3H) goes through fc; a row that
            # carries a draft hidden state (H) is x as it stands
            x = torch.stack([bf16r(linear(r.feat.view(1, -1), w["fc"]))[0] if r.feat.numel() == 3 * sh.H
                             else bf16r(r.feat) for r in rows])
            e = w["embed"][toks].to(F64)
            u = torch.cat([bf16r(rmsnorm(e, w["norm_e"], sh.eps)), bf16r(rmsnorm(x, w["norm1"], sh.eps))], dim=1)
            return x, linear(u, w["wqkv"])
        u = torch.cat([torch.stack([r.feat for r in rows]), w["embed"][toks].to(F64)], dim=1)
        x = bf16r(linear(u, w["fc"]))
        n1 = bf16r(rmsnorm(x, w["norm1"], sh.eps))
        return x, linear(n1, w["wqkv"])

    def append_kv(self, kv: PagedKV, rows: List[Row]) -> None:
        """Writes the rows' K (rotated at their positions) and V into their cache slots.  With one
        decoder layer the K/V of a position depend on that position's input only."""
        sh = self.sh
        nq, nk, d = sh.n_q, sh.n_kv, sh.d
        _, qkv = self.layer_input(rows)
        for i, r in enumerate(rows):
            k = qkv[i, nq * d:(nq + nk) * d].view(nk, d)
            v = qkv[i, (nq + nk) * d:].view(nk, d)
            kv.write(r.b, r.slot, bf16r(rope(k, r.pos, sh.theta)), bf16r(v))

    def round(self, kv: PagedKV, rows: List[Row], head_input=None) -> Tuple[torch.Tensor, HeadOut]:
        """One draft pass over ``rows``; appends their K/V to the cache.  Returns the
        final-normed hidden ``g [R, H]`` (bf16 values) and the head outputs.
        ``head_input(rows, g)`` (replay hook) may name the hidden the head is evaluated on, so
        that a test can check the head's decisions on another implementation's hidden."""
        sh, w = self.sh, self.w
        R = len(rows)
        x, qkv = self.layer_input(rows)
        nq, nk, d = sh.n_q, sh.n_kv, sh.d
        o = torch.empty(R, nq * d, dtype=F64)
        qs = []
        for i, r in enumerate(rows):          # all rows' K/V land first: siblings never see
            q = qkv[i, :nq * d].view(nq, d)   # each other unless listed in `visible`
            k = qkv[i, nq * d:(nq + nk) * d].view(nk, d)
            v = qkv[i, (nq + nk) * d:].view(nk, d)
            qs.append(bf16r(rope(q, r.pos, sh.theta)))
            kv.write(r.b, r.slot, bf16r(rope(k, r.pos, sh.theta)), bf16r(v))
        for i, r in enumerate(rows):
            o[i] = bf16r(self.attention(kv, r, qs[i])).reshape(-1)
        a = bf16r(x + linear(o, w["wo"]))
        n2 = bf16r(rmsnorm(a, w["norm2"], sh.eps))
        gu = linear(n2, w["wgate_up"])
        m = bf16r(silu(gu[:, :sh.F]) * gu[:, sh.F:])
        y = bf16r(a + linear(m, w["wdown"]))
        if self.arch == ARCH_FUSED3:
            # the hidden handed on (and compared) is y; the head reads its final norm
            yh = y if head_input is None else head_input(rows, y)
            return y, self.head(bf16r(rmsnorm(yh, w["normf"], sh.eps)))
        g = bf16r(rmsnorm(y, w["normf"], sh.eps))
        return g, self.head(g if head_input is None else head_input(rows, g))


# --------------------------------------------------------------------------------------
# chain drafting
# --------------------------------------------------------------------------------------
@dataclass
class ChainDraft:
    cand_tok: torch.Tensor      # [B, K+1] slot 0 = last accepted token, slot j = j-th draft token
    hidden: torch.Tensor        # [B, K, H] g of round k (bf16 values, f64)
    slot_signal: torch.Tensor   # [B, K+1, S]; slot j carries the signal computed from the
    #                             position of slot j's token (round j+1); slot K: NaN
    gap: torch.Tensor           # [B, K] relative top-2 gap at each draft argmax
    z: torch.Tensor             # [B, K, S] raw signal rows per round
    logits: Optional[torch.Tensor] = None   # [B, K, Vd] draft logits, kept when drafts are sampled


def draft_chain(model: DraftModel, kv: PagedKV, f0: torch.Tensor, t0: torch.Tensor, K: int,
                forced: Optional[Dict[Tuple[int, int], int]] = None, chooser=None,
                before_round=None, head_input=None, sample=None) -> ChainDraft:
    """K autoregressive draft rounds per sequence.  ``forced[(b, k)]`` (k = 1..K) replaces
    the k-th draft token of sequence b (used to replay a near-tie the other way);
    ``chooser("tok", (b, k), logits, 1, [tok]) -> [tok]`` may do the same on the fly."""
    B, H, S = f0.shape[0], model.sh.H, model.sh.S
    cand = torch.zeros(B, K + 1, dtype=torch.int64)
    cand[:, 0] = t0.to(torch.int64)
    hidden = torch.empty(B, K, H, dtype=F64)
    sig = torch.full((B, K + 1, S), float("nan"), dtype=F64)
    zz = torch.empty(B, K, S, dtype=F64)
    gap = torch.empty(B, K, dtype=F64)
    feat = f0.to(F64)
    # sampled drafts: token k of sequence b is a Gumbel-max draw from softmax(logits / tau), with
    # the draws of verify slot k - 1 of the draft stream (see speculative_sample)
    sampling = sample is not None and sample.sample_drafts and sample.temperature > 0.0
    kept = torch.empty(B, K, model.Vd, dtype=F64) if sampling else None
    tau = float(torch.tensor(sample.temperature, dtype=torch.float32)) if sampling else 0.0
    for k in range(1, K + 1):
        if before_round is not None and k > 1:
            # replay hook: lets a test restart round k from another implementation's state
            # (its previous hidden and the K/V it appended), so that each round is compared
            # on identical inputs; returns the feature to use
            feat = before_round(k, kv, feat)
        rows = [Row(b=b, feat=feat[b], tok=int(cand[b, k - 1]), pos=kv.len[b] + k - 1,
                    slot=kv.len[b] + k - 1,
                    visible=[kv.len[b] + j for j in range(k)]) for b in range(B)]
        g, ho = model.round(kv, rows, head_input)
        for b in range(B):
            score = ho.logits[b]
            if sampling:
                kept[b, k - 1] = ho.logits[b]
                score = score + tau * gumbel_noise(sample, b, DRAFT_STREAM + k - 1, model.Vd)
            tok = argmax_low(score)
            gap[b, k - 1] = top_gap(score)
            if forced and (b, k) in forced:
                tok = int(forced[(b, k)])
            if chooser is not None:
                tok = int(chooser("tok", (b, k), score, 1, [tok])[0])
            cand[b, k] = model.to_token(tok)      # decisions are taken on draft ids, tokens are stored
        hidden[:, k - 1] = g
        sig[:, k - 1] = ho.s
        zz[:, k - 1] = ho.z
        feat = g
    return ChainDraft(cand, hidden, sig, gap, zz, kept)


# --------------------------------------------------------------------------------------
# tree drafting: top-k children per expanded node, `depth` levels, best `max_nodes` kept
# --------------------------------------------------------------------------------------
@dataclass
class Cand:
    cid: int          # generation order: depth 1 first, then by expanding row, then by rank
    depth: int
    parent: int       # candidate id of the parent, -1 for children of the root
    tok: int
    logp: float
    score: float      # fp32 sum of log-probabilities along the path
    src_row: int      # drafted row whose head produced it
    row: int = -1     # drafted row that took it as input (-1: never expanded)


@dataclass
class TreeDraft:
    cands: List[List[Cand]]         # per sequence, all candidates
    cand_tok: torch.Tensor          # [B, P] slot 0 = root (last accepted token)
    parent: torch.Tensor            # [B, P] parent slot, -1 for the root
    depth: torch.Tensor             # [B, P]
    slot_row: torch.Tensor          # [B, P] drafted row with this slot's token as input, else -1
    slot_src_row: torch.Tensor      # [B, P] drafted row whose head produced the slot's token
    hidden: torch.Tensor            # [B, rows, H]
    slot_signal: torch.Tensor       # [B, P, S], NaN where the slot was never expanded
    margins: Dict[Tuple, float] = field(default_factory=dict)  # deciding margin per decision
    slot_cid: Optional[torch.Tensor] = None
    row_logits: Optional[Dict[Tuple[int, int], torch.Tensor]] = None   # (b, row) -> draft logits, when children are sampled


def draft_tree(model: DraftModel, kv: PagedKV, f0: torch.Tensor, t0: torch.Tensor, depth: int,
               topk: int, max_nodes: int, override: Optional[Dict[Tuple, List[int]]] = None,
               chooser=None, before_round=None, head_input=None, sample=None) -> TreeDraft:
    """Tree drafting.  Round 1 drafts the root; round r >= 2 expands the `topk` best
    candidates of depth r-1 (score = sum of log-probabilities; ties: lower candidate id).
    After the last round the `max_nodes` best candidates overall are kept and laid out in
    candidate-id order behind the root.  ``override`` replaces single decisions by the
    given choice: ``("topk", b, row) -> token ids``, ``("expand", b, depth) -> cand ids``,
    ``("keep", b) -> cand ids``.  ``chooser(kind, key, values, k, default) -> choice`` is
    asked at every decision instead (values: the row's logits for "topk", else a list of
    (cand id, score)); it lets a test adopt another implementation's choice at a near-tie."""
    sh = model.sh
    B, H, S = f0.shape[0], sh.H, sh.S
    ov = override or {}
    # Sampled children (``sample.sample_drafts`` with a positive temperature): the children of a drafted row
    # are the topk largest of logit + tau * Gumbel noise, best first, which is a draw of topk tokens WITHOUT
    # replacement, in order, from softmax(logits / tau) (the Gumbel-top-k identity).  The noise of the
    # children of drafted row `row` of sequence b is the stream with slot word TREE_STREAM + row.  Scores
    # stay sums of (unperturbed) log-probabilities.  The rows' logits are kept for the verification walk.
    sampling = sample is not None and sample.sample_drafts and sample.temperature > 0.0
    tau = float(torch.tensor(sample.temperature, dtype=torch.float32)) if sampling else 0.0
    row_logits: Dict[Tuple[int, int], torch.Tensor] = {}
    n_rows = 1 + topk * (depth - 1)
    P = 1 + max_nodes
    hidden = torch.empty(B, n_rows, H, dtype=F64)
    row_sig = torch.full((B, n_rows, S), float("nan"), dtype=F64)
    cands: List[List[Cand]] = [[] for _ in range(B)]
    margins: Dict[Tuple, float] = {}
    row_vis: List[Dict[int, List[int]]] = [dict() for _ in range(B)]

    def emit(b, row, par_cid, par_score, dep, logits):
        rank_by = logits
        if sampling:
            assert model.map is None, "sampled children need a full-vocabulary draft head"
            row_logits[(b, row)] = logits
            rank_by = logits + tau * gumbel_noise(sample, b, TREE_STREAM + row, logits.numel())
        ids = topk_low(rank_by, topk)
        margins[("topk", b, row)] = order_gap(rank_by, topk)     # order of the k children and the cut behind them
        if ("topk", b, row) in ov:
            ids = list(ov[("topk", b, row)])
        if chooser is not None:
            ids = list(chooser("topk", (b, row), rank_by, topk, ids))
        lse = torch.logsumexp(logits, dim=0)
        for t in ids:
            lp = f32r(logits[t] - lse)
            sc = f32r(torch.tensor(par_score, dtype=F64) + lp)
            cands[b].append(Cand(cid=len(cands[b]), depth=dep, parent=par_cid, tok=model.to_token(t),
                                 logp=float(lp), score=float(sc), src_row=row))

    # round 1: the root row
    rows = [Row(b=b, feat=f0[b].to(F64), tok=int(t0[b]), pos=kv.len[b], slot=kv.len[b],
                visible=[kv.len[b]]) for b in range(B)]
    for b in range(B):
        row_vis[b][0] = [kv.len[b]]
    g, ho = model.round(kv, rows, head_input)
    for b in range(B):
        hidden[b, 0] = g[b]
        row_sig[b, 0] = ho.s[b]
        emit(b, 0, -1, 0.0, 1, ho.logits[b])

    for r in range(2, depth + 1):
        feat_src = hidden
        if before_round is not None:
            feat_src = before_round(r, kv, hidden)   # replay hook, see draft_chain
        rows, owner = [], []
        for b in range(B):
            level = [c for c in cands[b] if c.depth == r - 1]
            level.sort(key=lambda c: (-c.score, c.cid))
            if len(level) > 1:
                # the chosen candidates take their rows in rank order: order and cut both decide
                margins[("expand", b, r - 1)] = order_gap(torch.tensor([c.score for c in level], dtype=F64), topk)
            chosen = level[:topk]
            if ("expand", b, r - 1) in ov:
                byid = {c.cid: c for c in cands[b]}
                chosen = [byid[i] for i in ov[("expand", b, r - 1)]]
            if chooser is not None:
                byid = {c.cid: c for c in cands[b]}
                pick = chooser("expand", (b, r - 1), [(c.cid, c.score) for c in level], topk,
                               [c.cid for c in chosen])
                chosen = [byid[i] for i in pick]
            for j, c in enumerate(chosen):
                rid = 1 + (r - 2) * topk + j
                c.row = rid
                vis = list(row_vis[b][c.src_row]) + [kv.len[b] + rid]
                row_vis[b][rid] = vis
                rows.append(Row(b=b, feat=feat_src[b, c.src_row], tok=c.tok,
                                pos=kv.len[b] + r - 1, slot=kv.len[b] + rid, visible=vis))
                owner.append((b, rid, c))
        g, ho = model.round(kv, rows, head_input)
        for i, (b, rid, c) in enumerate(owner):
            hidden[b, rid] = g[i]
            row_sig[b, rid] = ho.s[i]
            emit(b, rid, c.cid, c.score, r, ho.logits[i])

    cand_tok = torch.zeros(B, P, dtype=torch.int64)
    parent = torch.full((B, P), -1, dtype=torch.int64)
    dep = torch.zeros(B, P, dtype=torch.int64)
    slot_row = torch.full((B, P), -1, dtype=torch.int64)
    slot_src = torch.full((B, P), -1, dtype=torch.int64)
    slot_cid = torch.full((B, P), -1, dtype=torch.int64)
    slot_sig = torch.full((B, P, S), float("nan"), dtype=F64)
    for b in range(B):
        ranked = sorted(cands[b], key=lambda c: (-c.score, c.cid))
        if len(ranked) > max_nodes:
            den = abs(ranked[0].score)
            margins[("keep", b)] = ((ranked[max_nodes - 1].score - ranked[max_nodes].score) / den
                                    if den > 0 else 0.0)
        keep = sorted(c.cid for c in ranked[:max_nodes])
        if ("keep", b) in ov:
            keep = sorted(ov[("keep", b)])
        if chooser is not None:
            keep = sorted(chooser("keep", (b,), [(c.cid, c.score) for c in ranked], max_nodes, keep))
        slot_of = {-1: 0}
        cand_tok[b, 0] = int(t0[b])
        slot_row[b, 0] = 0
        slot_sig[b, 0] = row_sig[b, 0]
        for s, cid in enumerate(keep, start=1):
            c = cands[b][cid]
            slot_of[cid] = s
            cand_tok[b, s] = c.tok
            parent[b, s] = slot_of[c.parent]     # parents precede children in id order
            dep[b, s] = c.depth
            slot_row[b, s] = c.row
            slot_src[b, s] = c.src_row
            slot_cid[b, s] = cid
            if c.row >= 0:
                slot_sig[b, s] = row_sig[b, c.row]
    return TreeDraft(cands, cand_tok, parent, dep, slot_row, slot_src, hidden, slot_sig, margins,
                     slot_cid, row_logits if sampling else None)


# --------------------------------------------------------------------------------------
# verification (Algorithm 1: accept tokens, accept length, recover token)
# --------------------------------------------------------------------------------------
@dataclass
class VerifyOut:
    target_tok: torch.Tensor   # [B, P]
    accept_len: torch.Tensor   # [B]
    path: List[List[int]]      # per sequence: accepted slots, starting with slot 0
    recover_tok: torch.Tensor  # [B]
    gap: torch.Tensor          # [B, P] relative top-2 gap of the target argmax


def target_argmax(model: DraftModel, target_hidden: torch.Tensor) -> Tuple[torch.Tensor, torch.Tensor]:
    B, P, H = target_hidden.shape
    logits = f32r(linear(target_hidden.reshape(B * P, H).to(F64), model.target_head))
    tok = torch.tensor([argmax_low(logits[i]) for i in range(B * P)], dtype=torch.int64)
    gap = torch.tensor([top_gap(logits[i]) for i in range(B * P)], dtype=F64)
    return tok.view(B, P), gap.view(B, P)


# --------------------------------------------------------------------------------------
# stochastic verification: speculative sampling with deterministic drafts
# --------------------------------------------------------------------------------------
# Speculative sampling (the acceptance rule the paper's background section cites) keeps a draft
# token x with probability min(1, p(x) / q(x)) and otherwise draws from the normalised
# max(0, p - q); p is the target's distribution at temperature tau, q the draft's.  The drafts
# here are deterministic (the draft's argmax, or its top-k children in a tree), so q is a point
# mass: x is kept with probability p(x), and a rejection draws from p with x removed.  Drawing
# one token t ~ p and keeping x exactly when t == x has that joint law (P(t = x) = p(x); given
# t != x, t follows p without x), and for the children c_1..c_m of a tree node tried one after
# the other against the shrinking residual, P(c_i kept) = p(c_i) again, so "keep the child that
# equals t, else recover t" is the same law.  The verification below is therefore the greedy
# walk with the target's argmax replaced by a sample t ~ softmax(logits / tau).
#
# The sample is a Gumbel-max draw so that it depends on the random numbers element by element
# and not on a summation order:  t = argmax_i (logit_i + tau * g_i),  g_i = -ln(-ln(u_i)),
# with u_i a uniform on (0, 1) taken from the counter-based generator Philox4x32-10 (Salmon et
# al., "Parallel random numbers: as easy as 1, 2, 3", 2011): the draw for sequence b, verify
# slot j and token id i is word (i mod 4) of the block with counter (i div 4, j, b, offset) and
# key (seed mod 2^32, seed div 2^32).  tau = 0 is greedy verification.
PHILOX_M0, PHILOX_M1 = 0xD2511F53, 0xCD9E8D57
PHILOX_W0, PHILOX_W1 = 0x9E3779B9, 0xBB67AE85


def philox4x32_10(counter, key):
    """Philox4x32 with 10 rounds on numpy arrays of uint64 holding 32-bit words.
    ``counter``: four arrays (or ints), ``key``: two.  Returns the four output words."""
    import numpy as np
    m32 = np.uint64(0xFFFFFFFF)
    c = [np.asarray(x, dtype=np.uint64) & m32 for x in counter]
    c = list(np.broadcast_arrays(*c))
    k0, k1 = np.uint64(int(key[0]) & 0xFFFFFFFF), np.uint64(int(key[1]) & 0xFFFFFFFF)
    for rnd in range(10):
        if rnd:
            k0 = (k0 + np.uint64(PHILOX_W0)) & m32
            k1 = (k1 + np.uint64(PHILOX_W1)) & m32
        p0 = np.uint64(PHILOX_M0) * c[0]            # 32 x 32 -> 64 bit products
        p1 = np.uint64(PHILOX_M1) * c[2]
        hi0, lo0 = p0 >> np.uint64(32), p0 & m32
        hi1, lo1 = p1 >> np.uint64(32), p1 & m32
        c = [hi1 ^ c[1] ^ k0, lo1, hi0 ^ c[3] ^ k1, lo0]
    return c


def uniform_open(word):
    """A 32-bit word to a uniform strictly inside (0, 1): the top 23 bits k give (k + 1/2) / 2^23,
    a value that float32 holds exactly."""
    import numpy as np
    return ((np.asarray(word, dtype=np.uint64) >> np.uint64(9)).astype(np.float64) + 0.5) / float(1 << 23)


@dataclass
class SampleCfg:
    temperature: float = 0.0
    seed: int = 0
    offset: int = 0          # e.g. the iteration number: a fresh set of draws per iteration
    sample_drafts: bool = False   # chain drafts are drawn from the draft's softmax as well


# The slot word of the counter separates three streams of draws: verify slot j itself (the
# target-side Gumbel noise), ACCEPT_STREAM + j (the uniform of the accept test) and
# DRAFT_STREAM + j (the Gumbel noise that draws the draft token proposed at slot j).
ACCEPT_STREAM, DRAFT_STREAM = 0x20000000, 0x40000000
# TREE_STREAM + r: the Gumbel noise that draws the children of drafted row r of a tree
TREE_STREAM = 0x50000000


def gumbel_noise(cfg: SampleCfg, b: int, j: int, V: int) -> torch.Tensor:
    """g_i for i in [0, V) of sequence b, verify slot j (float64)."""
    import numpy as np
    nblk = (V + 3) // 4
    w = philox4x32_10((np.arange(nblk, dtype=np.uint64), j, b, cfg.offset),
                      (cfg.seed & 0xFFFFFFFF, (cfg.seed >> 32) & 0xFFFFFFFF))
    u = uniform_open(np.stack(w, axis=1).reshape(-1)[:V])
    return torch.from_numpy(-np.log(-np.log(u)))


def target_sample(model: DraftModel, target_hidden: torch.Tensor, cfg: SampleCfg
                  ) -> Tuple[torch.Tensor, torch.Tensor]:
    """t[b, j] ~ softmax(logits[b, j] / tau) by Gumbel-max, and the relative top-2 gap of the
    perturbed scores.  The temperature enters as its float32 value."""
    B, P, H = target_hidden.shape
    logits = f32r(linear(target_hidden.reshape(B * P, H).to(F64), model.target_head))
    tau = float(torch.tensor(cfg.temperature, dtype=torch.float32))
    tok = torch.zeros(B * P, dtype=torch.int64)
    gap = torch.zeros(B * P, dtype=F64)
    for r in range(B * P):
        s = logits[r]
        if tau > 0.0:
            s = s + tau * gumbel_noise(cfg, r // P, r % P, s.numel())
        tok[r] = argmax_low(s)
        gap[r] = top_gap(s)
    return tok.view(B, P), gap.view(B, P)


@dataclass
class SpecSampleOut:
    target_tok: torch.Tensor   # [B, P] the kept draft token where the test passed, else the residual draw
    accepted: torch.Tensor     # [B, P] bool
    margin: torch.Tensor       # [B, P] |u - min(1, p(x)/q(x))| of the accept test (inf at the last slot)
    gap: torch.Tensor          # [B, P] relative top-2 gap of the residual draw (inf where accepted)


def speculative_sample(model: DraftModel, target_hidden: torch.Tensor, cand_tok: torch.Tensor,
                       draft_logits: torch.Tensor, cfg: SampleCfg) -> SpecSampleOut:
    """Speculative sampling with sampled drafts, slot by slot (chain).  The draft token x
    proposed at slot j (cand_tok[b, j + 1], drawn from q_j = softmax(draft_logits[b, j] / tau)) is
    kept when u_j < min(1, p_j(x) / q_j(x)), p_j = softmax(target logits / tau); otherwise the slot's
    token is drawn from the normalised max(0, p_j - q_j).  The last slot has no draft: its token is
    drawn from p itself.  Draws: u_j from word 0 of the block with counter (0, ACCEPT_STREAM + j, b,
    offset); the residual draw is a Gumbel-max over log max(0, p - q) with the noise of slot j.
    Probabilities are float64 functions of the float32 logits."""
    import numpy as np
    B, P, H = target_hidden.shape
    K = P - 1
    assert model.map is None and draft_logits.shape[-1] == model.sh.V, "needs a full-vocabulary draft head"
    logits = f32r(linear(target_hidden.reshape(B * P, H).to(F64), model.target_head)).view(B, P, -1)
    tau = float(torch.tensor(cfg.temperature, dtype=torch.float32))
    key = (cfg.seed & 0xFFFFFFFF, (cfg.seed >> 32) & 0xFFFFFFFF)
    tok = torch.zeros(B, P, dtype=torch.int64)
    acc = torch.zeros(B, P, dtype=torch.bool)
    margin = torch.full((B, P), float("inf"), dtype=F64)
    gap = torch.full((B, P), float("inf"), dtype=F64)
    for b in range(B):
        for j in range(P):
            lp = logits[b, j] / tau
            logp = lp - torch.logsumexp(lp, dim=0)
            p = torch.exp(logp)
            q = torch.zeros_like(p)
            x = -1
            if j < K:
                lq = draft_logits[b, j].to(F64) / tau
                logq = lq - torch.logsumexp(lq, dim=0)
                q = torch.exp(logq)
                x = int(cand_tok[b, j + 1])
                ratio = min(1.0, math.exp(float(logp[x] - logq[x])))
                u = float(uniform_open(philox4x32_10((0, ACCEPT_STREAM + j, b, cfg.offset), key)[0]))
                margin[b, j] = abs(u - ratio)
                if u < ratio:
                    acc[b, j] = True
                    tok[b, j] = x
                    continue
            r = p - q
            if not bool((r > 0).any()):
                tok[b, j] = x              # p == q: nothing is left to draw from (x >= 0 here)
                continue
            g = gumbel_noise(cfg, b, j, r.numel())
            s = torch.where(r > 0, torch.log(r.clamp_min(1e-300)) + g, torch.full_like(r, -float("inf")))
            tok[b, j] = argmax_low(s)
            t2 = torch.topk(s, 2).values
            gap[b, j] = float(t2[0] - t2[1])          # absolute: the scores are logarithms
    return SpecSampleOut(tok, acc, margin, gap)


@dataclass
class TreeWalkOut:
    target_tok: torch.Tensor   # [B, P] at a visited slot: the accepted child's token, or the token drawn there; else -1
    accept_len: torch.Tensor   # [B]
    path: List[List[int]]      # accepted slots, starting with slot 0
    recover_tok: torch.Tensor  # [B]
    exempt: List[str]          # decisions adopted from `decide` (see below)


def tree_speculative_walk(model: DraftModel, target_hidden: torch.Tensor, draft: "TreeDraft", cfg: SampleCfg,
                          decide=None) -> TreeWalkOut:
    """Speculative sampling down a tree whose children were drawn from the draft (see draft_tree).

    At the current slot, with p = softmax(target logits / tau) and q = softmax(the logits of the drafted row
    that produced the slot's children / tau), the kept children are tried in the order they were drawn:
    child token x is accepted when u < min(1, p(x) / q(x)); a refusal replaces p by the normalised
    max(0, p - q) and takes x out of q (renormalised), which is the law of the next draw without replacement.
    When a child is accepted the walk continues from it; when all are refused (or the slot has none) the
    recover token is drawn from the p that is left, and the walk ends.  The emitted token then follows the
    target's distribution exactly as long as every child drawn at a visited slot is still in the tree (a
    child pruned away for its score is simply not tried: with pruning the rule is approximate).
    Draws: u of slot s from word 0 of the block with counter (0, ACCEPT_STREAM + s, b, offset); the final draw
    at slot s is a Gumbel-max over the logarithm of what is left of p, with the noise of slot s - for a
    slot where nothing was refused that is argmax(logit + tau g), the draw of `target_sample`.
    ``decide(kind, key, default, margin)`` may replace a decision whose margin is small (tests): kind
    "accept" with key (b, slot) and a bool, kind "draw" with key (b, slot) and a token."""
    B, P, H = target_hidden.shape
    assert draft.row_logits is not None and model.map is None
    logits = f32r(linear(target_hidden.reshape(B * P, H).to(F64), model.target_head)).view(B, P, -1)
    tau = float(torch.tensor(cfg.temperature, dtype=torch.float32))
    key = (cfg.seed & 0xFFFFFFFF, (cfg.seed >> 32) & 0xFFFFFFFF)
    tt = torch.full((B, P), -1, dtype=torch.int64)
    L = torch.zeros(B, dtype=torch.int64)
    rec = torch.zeros(B, dtype=torch.int64)
    paths, exempt = [], []
    for b in range(B):
        cur, path = 0, [0]
        while True:
            lp = logits[b, cur] / tau
            p = torch.exp(lp - torch.logsumexp(lp, dim=0))
            kids = [s for s in range(cur + 1, P) if int(draft.parent[b, s]) == cur]
            row = int(draft.slot_row[b, cur])
            nxt = -1
            if kids:
                lq = draft.row_logits[(b, row)].to(F64) / tau
                q = torch.exp(lq - torch.logsumexp(lq, dim=0))
                for s in kids:
                    x = int(draft.cand_tok[b, s])
                    ratio = min(1.0, float(p[x]) / float(q[x]))
                    u = float(uniform_open(philox4x32_10((0, ACCEPT_STREAM + s, b, cfg.offset), key)[0]))
                    ok = u < ratio
                    if decide is not None:
                        ok2 = bool(decide("accept", (b, s), ok, abs(u - ratio)))
                        if ok2 != ok:
                            exempt.append(f"accept test b={b} slot={s}")
                        ok = ok2
                    if ok:
                        nxt = s
                        break
                    p = (p - q).clamp_min(0.0)
                    p = p / p.sum()
                    q = q.clone()
                    q[x] = 0.0
                    q = q / q.sum()
            if nxt >= 0:
                tt[b, cur] = int(draft.cand_tok[b, nxt])
                cur = nxt
                path.append(cur)
                continue
            g = gumbel_noise(cfg, b, cur, p.numel())
            sc = torch.where(p > 0, torch.log(p.clamp_min(1e-300)) + g, torch.full_like(p, -float("inf")))
            t = argmax_low(sc)
            if decide is not None:
                t2 = torch.topk(sc, 2).values
                tnew = int(decide("draw", (b, cur), t, float(t2[0] - t2[1])))
                if tnew != t:
                    exempt.append(f"draw b={b} slot={cur}")
                t = tnew
            tt[b, cur] = t
            rec[b] = t
            break
        L[b] = len(path) - 1
        paths.append(path)
    return TreeWalkOut(tt, L, paths, rec, exempt)


def accept_chain(cand_tok: Sequence[int], target_tok: Sequence[int]) -> Tuple[int, List[int], int]:
    """Longest prefix of draft tokens that equal the target's greedy choice one slot
    earlier; the recover token is the target's choice after the last accepted slot."""
    K = len(cand_tok) - 1
    L = 0
    while L < K and int(cand_tok[L + 1]) == int(target_tok[L]):
        L += 1
    return L, list(range(L + 1)), int(target_tok[L])


def accept_tree(cand_tok: Sequence[int], parent: Sequence[int], target_tok: Sequence[int]
                ) -> Tuple[int, List[int], int]:
    """Walk from the root to the child whose token is the target's greedy choice at the
    current slot, until there is none."""
    P = len(cand_tok)
    cur, path = 0, [0]
    while True:
        nxt = [s for s in range(1, P) if int(parent[s]) == cur and int(cand_tok[s]) == int(target_tok[cur])]
        if not nxt:
            break
        cur = nxt[0]
        path.append(cur)
    return len(path) - 1, path, int(target_tok[cur])


def verify(model: DraftModel, target_hidden: torch.Tensor, cand_tok: torch.Tensor,
           parent: Optional[torch.Tensor] = None,
           forced_target: Optional[Dict[Tuple[int, int], int]] = None,
           sample: Optional[SampleCfg] = None, draft_logits: Optional[torch.Tensor] = None) -> VerifyOut:
    """Greedy verification, or (``sample`` with a positive temperature) speculative sampling:
    with deterministic drafts through one draw per slot, with sampled drafts (chain only,
    ``draft_logits`` given) through the accept test and the residual draw."""
    if sample is not None and sample.temperature > 0.0 and sample.sample_drafts:
        assert parent is None and draft_logits is not None
        so = speculative_sample(model, target_hidden, cand_tok, draft_logits, sample)
        tt, gap = so.target_tok, so.gap
    elif sample is not None and sample.temperature > 0.0:
        tt, gap = target_sample(model, target_hidden, sample)
    else:
        tt, gap = target_argmax(model, target_hidden)
    if forced_target:
        for (b, j), t in forced_target.items():
            tt[b, j] = t
    B = tt.shape[0]
    L = torch.zeros(B, dtype=torch.int64)
    rec = torch.zeros(B, dtype=torch.int64)
    paths = []
    for b in range(B):
        if parent is None:
            l, p, r = accept_chain(cand_tok[b].tolist(), tt[b].tolist())
        else:
            l, p, r = accept_tree(cand_tok[b].tolist(), parent[b].tolist(), tt[b].tolist())
        L[b], rec[b] = l, r
        paths.append(p)
    return VerifyOut(tt, L, paths, rec, gap)


# --------------------------------------------------------------------------------------
# end of an iteration: Algorithm 1, "Update KV-cache and hidden states accordingly"
# --------------------------------------------------------------------------------------
@dataclass
class CommitOut:
    cache_len: List[int]      # cached length per sequence after the commit
    feat0: torch.Tensor       # [B, H] feature of the next iteration's first draft row
    tok0: torch.Tensor        # [B] its token (the recover token)


def commit(model: DraftModel, kv: PagedKV, target_hidden: torch.Tensor, cand_tok: torch.Tensor,
           path: torch.Tensor, accept_len_out: torch.Tensor, recover_tok_out: torch.Tensor) -> CommitOut:
    """Makes the verified tokens of an iteration part of the draft model's cached context.

    Before the iteration sequence b had n cached positions.  Slot n holds the K/V of the last
    accepted token of the previous iteration, computed in draft round 1 from its true feature:
    it is kept.  The L accepted draft tokens (path slots 1..L) were drafted from draft hidden
    states, so their K/V are recomputed ("catch-up") from the target's hidden states: the token
    of path slot j is paired with the target hidden of path slot j - 1, the hidden that
    predicted it, at position n + j.  The cached length becomes n + L + 1, and the next
    iteration starts from (target hidden of path slot L, recover token).  ``accept_len_out`` and
    ``recover_tok_out`` are the values after the exit rule (a cut path commits fewer tokens)."""
    B = cand_tok.shape[0]
    feat0 = torch.empty(B, target_hidden.shape[-1], dtype=F64)
    tok0 = torch.empty(B, dtype=torch.int64)
    rows: List[Row] = []
    new_len = []
    for b in range(B):
        n, L = kv.len[b], int(accept_len_out[b])
        pb = [int(s) for s in path[b]]              # accepted slots, slot 0 first (tensor row or list)
        for j in range(1, L + 1):
            rows.append(Row(b=b, feat=bf16r(target_hidden[b, pb[j - 1]].to(F64)),
                            tok=int(cand_tok[b, pb[j]]), pos=n + j, slot=n + j, visible=[]))
        feat0[b] = bf16r(target_hidden[b, pb[L]].to(F64))
        tok0[b] = int(recover_tok_out[b])
        new_len.append(n + L + 1)
    if rows:
        model.append_kv(kv, rows)
    kv.len = list(new_len)
    kv._prefix.clear()
    return CommitOut(new_len, feat0, tok0)


# --------------------------------------------------------------------------------------
# exit decision (Section 3.3; Appendix A.1: EWMA x_t = alpha s_t + (1 - alpha) x_{t-1})
# --------------------------------------------------------------------------------------
SMOOTH_EWMA, SMOOTH_NONE, SMOOTH_WINDOW, SMOOTH_MOMENTUM, SMOOTH_PARAGRAPH = 0, 1, 2, 3, 4
HIST = 16        # samples of history kept per sequence (window and momentum rules, N <= 15)


@dataclass
class ExitCfg:
    alpha: float = 0.3
    thr: Tuple[float, float, float] = (0.9, 0.8, 100.0)
    dir: Tuple[int, int, int] = (DIR_GT, DIR_GT, DIR_LT)
    enable_mask: int = 0b001           # bit i: signal i takes part (AND over enabled ones)
    ema_positions: int = EMA_VERIFIED_CONTEXT
    split_bitmap: Optional[torch.Tensor] = None   # int32 words, bit t%32 of word t//32; None = all
    stop_think_token: int = 0
    smoothing: int = SMOOTH_EWMA       # Appendix A.1, "Signal Smoothing"
    window: int = 10                   # N of the sliding-window and momentum rules


@dataclass
class ExitState:
    x: torch.Tensor          # [B, S] smoothed signals (fp32 values)
    n_updates: torch.Tensor  # [B]
    thinking: torch.Tensor   # [B] 1 while inside the reasoning phase
    hist: Optional[torch.Tensor] = None      # [B, HIST, S] ring of the latest samples; sample i at i % HIST
    par_sum: Optional[torch.Tensor] = None   # [B, S] sum of the samples of the current paragraph (fp32 values)
    par_n: Optional[torch.Tensor] = None     # [B] their number

    @staticmethod
    def fresh(B: int, S: int = 3) -> "ExitState":
        return ExitState(torch.zeros(B, S, dtype=F64), torch.zeros(B, dtype=torch.int64),
                         torch.ones(B, dtype=torch.int64), torch.zeros(B, HIST, S, dtype=F64),
                         torch.zeros(B, S, dtype=F64), torch.zeros(B, dtype=torch.int64))

    def clone(self) -> "ExitState":
        c = lambda t: None if t is None else t.clone()
        return ExitState(self.x.clone(), self.n_updates.clone(), self.thinking.clone(), c(self.hist),
                         c(self.par_sum), c(self.par_n))


def is_split(cfg: ExitCfg, tok: int) -> bool:
    if cfg.split_bitmap is None:
        return True
    word = int(cfg.split_bitmap[tok // 32]) & 0xFFFFFFFF
    return bool((word >> (tok % 32)) & 1)


def thresholds_pass(cfg: ExitCfg, x: torch.Tensor) -> bool:
    """AND over the enabled signals; 'greater than' / 'less than' are strict."""
    x32 = x.to(torch.float32)
    for i in range(x.numel()):
        if not (cfg.enable_mask >> i) & 1:
            continue
        thr = torch.tensor(cfg.thr[i], dtype=torch.float32)
        ok = bool(x32[i] > thr) if cfg.dir[i] == DIR_GT else bool(x32[i] < thr)
        if not ok:
            return False
    return True


def ewma(cfg: ExitCfg, x: torch.Tensor, n_updates: int, s: torch.Tensor) -> torch.Tensor:
    """One smoothing step in fp32 storage; the first sample initialises the state."""
    if n_updates == 0:
        return f32r(s)
    a = float(torch.tensor(cfg.alpha, dtype=torch.float32))   # alpha as the fp32 the kernel holds
    return f32r(a * s + (1.0 - a) * x)


def smooth(cfg: ExitCfg, state: ExitState, b: int, s: torch.Tensor) -> torch.Tensor:
    """Folds sample ``s`` (the n-th of sequence b, n = n_updates) into the state and returns the
    smoothed score x_t of Appendix A.1.  Sums run oldest to newest in f64; x is stored as fp32.
    Where fewer samples exist than a rule asks for, it uses those that exist (the paper does not
    say): the window averages what it has; the momentum rule, which as printed predicts step t
    from the samples before it, returns the sample itself while there is no earlier one."""
    n = int(state.n_updates[b])
    if cfg.smoothing == SMOOTH_EWMA:
        return ewma(cfg, state.x[b], n, s)
    if cfg.smoothing == SMOOTH_NONE:
        return f32r(s)
    if cfg.smoothing == SMOOTH_PARAGRAPH:
        state.par_sum[b] = f32r(state.par_sum[b] + s)
        state.par_n[b] += 1
        return f32r(state.par_sum[b] / float(state.par_n[b]))
    N = int(cfg.window)
    assert 2 <= N < HIST
    state.hist[b, n % HIST] = f32r(s)
    at = lambda i: state.hist[b, i % HIST]          # sample i, i in (n - HIST, n]
    if cfg.smoothing == SMOOTH_WINDOW:
        m = min(n + 1, N)
        acc = torch.zeros_like(s)
        for i in range(n - m + 1, n + 1):
            acc = acc + at(i)
        return f32r(acc / float(m))
    # momentum: x_t = s_{t-1} + (1 / (N - 1)) sum_{i = t-N+1}^{t-1} (s_i - s_{i-1}); the sum telescopes
    if n == 0:
        return f32r(s)
    k = min(N - 1, n - 1)                            # differences available behind s_{t-1}
    prev = at(n - 1)
    if k == 0:
        return f32r(prev)
    return f32r(prev + (prev - at(n - 1 - k)) / float(k))


@dataclass
class ExitOut:
    exit_flag: torch.Tensor       # [B]
    accept_len: torch.Tensor      # [B] after truncation
    recover_tok: torch.Tensor     # [B] after substitution
    smoothed: torch.Tensor        # [B, S]


def exit_update(cfg: ExitCfg, state: ExitState, slot_signal: torch.Tensor, cand_tok: torch.Tensor,
                paths: List[List[int]], accept_len: torch.Tensor, recover_tok: torch.Tensor) -> ExitOut:
    """Walk the accepted slots in path order.  Each slot that carries a signal updates the
    smoothed state; the first slot whose token is a step-split token while the smoothed
    signals pass the thresholds ends the reasoning phase: the accepted length is cut at
    that slot and the recover token becomes the stop-think token.  ``state`` is updated
    in place; a sequence that is no longer thinking is left untouched."""
    B = len(paths)
    ef = torch.zeros(B, dtype=torch.int64)
    Lo = accept_len.clone().to(torch.int64)
    ro = recover_tok.clone().to(torch.int64)
    for b in range(B):
        if int(state.thinking[b]) == 0:
            continue
        L = int(accept_len[b])
        for idx in range(L + 1):
            slot = paths[b][idx]
            sig = slot_signal[b, slot]
            if cfg.ema_positions == EMA_VERIFIED_CONTEXT or idx == 0:
                if bool(torch.isnan(sig).any()):
                    break                     # never drafted from this slot: nothing new to smooth
                state.x[b] = smooth(cfg, state, b, sig)
                state.n_updates[b] += 1
            split = is_split(cfg, int(cand_tok[b, slot]))
            if split and thresholds_pass(cfg, state.x[b]):
                ef[b], Lo[b], ro[b] = 1, idx, cfg.stop_think_token
                state.thinking[b] = 0
                break
            if split and cfg.smoothing == SMOOTH_PARAGRAPH:
                state.par_sum[b] = 0.0            # a paragraph delimiter went by: a new paragraph starts
                state.par_n[b] = 0
    return ExitOut(ef, Lo, ro, state.x.clone())
