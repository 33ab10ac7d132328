"""Benchmark of the speculative-exit step.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload C1] [--impl reference]

One step = one whole speculative-exit iteration (all draft rounds, verification, acceptance,
exit decision) over one batch of synthetic input.  Prints ONE JSON line (rank 0).

value      iterations/s with every input resident in HBM, timed with CUDA events over K steps
e2e        the same through the host-buffer entry point: pinned host inputs are copied in and
           the step's results copied out inside the timed region
roofline   the dominant kernel (extended LM head of a draft round): algorithmic bytes of one
           launch / its mean duration, against the measured HBM copy bandwidth
cpu_baseline  the CPU oracle on the same workload (a bounded sample), host cores of this machine

Multi-GPU (torchrun): the path shards by sequence with no exchange step, so every rank runs an
independent replica of the workload ("weak" scaling); the time is the max over ranks.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2509_24248_b200 import synth  # noqa: E402

METRIC = "spec-exit iterations/s"


def measured_peaks() -> dict:
    """Roofline denominators: the copy bandwidth and the bf16 GEMM throughput measured on this machine's GPUs
    (burst figure), else the stated fallback."""
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return {"hbm_gbs": float(d["hbm_gbs"]), "bf16_tflops": float(d["bf16_tflops"]), "kind": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "kind": "fallback"}


def algorithmic_bytes(wl: synth.Workload, lens) -> dict:
    """Bytes one iteration has to move: every weight matrix once per dependent draft round,
    every live KV byte once per round, the verify head once."""
    s = wl.shape
    head = ((s.Vd or s.V) + s.S) * s.H
    rounds = wl.K
    kv_round = int(sum(int(n) for n in lens)) * s.n_kv * s.d * 2 * 2
    if s.arch:
        # three-feature layer: fc (3H -> H) in round 1 only, q/k/v projection over 2H every round
        layer = 2 * s.H * s.qkv_rows + s.n_q * s.d * s.H + 3 * s.H * s.F
        w_round = 2 * (layer + head)
        total = rounds * (w_round + kv_round) + 2 * 3 * s.H * s.H + 2 * s.V * s.H
    else:
        layer = 2 * s.H * s.H + s.H * s.qkv_rows + s.n_q * s.d * s.H + 3 * s.H * s.F
        w_round = 2 * (layer + head)
        total = rounds * (w_round + kv_round) + 2 * s.V * s.H
    return {"total": total, "head_launch": 2 * head, "w_round": w_round, "kv_round": kv_round}


def workload_config(args, wl: synth.Workload, lens) -> dict:
    """The `config` entry of the JSON line: what was run.  Both arms print the same dictionary for the same
    command-line options."""
    ab = algorithmic_bytes(wl, lens)
    return {"workload": wl.name, "batch": wl.B, "K": wl.K, "mode": "chain" if wl.mode == synth.CHAIN else "tree",
            "cached_tokens": int(sum(int(n) for n in lens)),
            "weights": "tiled at load (sx_tile_weight)" if args.weights == "tiled" else "row-major",
            "l2": "no flush: each iteration streams %.2f GB of weights and KV, far beyond the 126 MB L2"
                  % (ab["total"] / 1e9)}


def _oracle_sample(args):
    """Sampling settings of the CPU legs (None: greedy)."""
    from oracle import specexit_oracle as orc
    if args.temperature <= 0.0:
        return None
    return orc.SampleCfg(args.temperature, 1234, 1, bool(args.sample_drafts))


def max_over_ranks(ms_local: float, dist, device) -> float:
    """Replicas share nothing on the data path; the job's time is the slowest rank's."""
    if dist is None:
        return float(ms_local)
    t = torch.tensor([ms_local], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def sum_over_ranks(x: float, dist, device) -> float:
    if dist is None:
        return float(x)
    t = torch.tensor([x], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.item())


def whole_job_rate(units_all_ranks: float, ms_total: float) -> float:
    """Units processed by all ranks per second of the slowest rank's time."""
    return units_all_ranks / (ms_total / 1e3)


class ClockSampler:
    """nvidia-smi clocks and throttle reasons while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.rows, self.proc = index, [], None
        self.t0 = self.t1 = None

    def wait_ready(self, timeout: float = 10.0):
        """nvidia-smi takes a second or two to start and perturbs launches while it does; the timed
        region begins only after its first sample has arrived."""
        t = time.time()
        while self.proc is not None and not self.rows and time.time() - t < timeout:
            time.sleep(0.05)

    def mark_begin(self):
        self.t0 = time.time()

    def mark_end(self):
        self.t1 = time.time()

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "200"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.th = threading.Thread(target=self._read, daemon=True)
            self.th.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append((time.time(), [c.strip() for c in line.split(",")]))

    def stop(self) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], None, set()
        inside = [r for (t, r) in self.rows if self.t0 is not None and self.t0 <= t <= (self.t1 or t) + 0.1]
        if not inside:                      # region shorter than the sampling period: nearest samples
            inside = [r for (_, r) in self.rows[-2:]]
        for r in inside:
            try:
                sm.append(float(r[0]))
                mx = float(r[1])
                for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), r[3:7]):
                    if v.lower().startswith("active"):
                        reasons.add(name)
            except Exception:
                pass
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": mx, "samples": len(sm),
                "reasons": sorted(reasons)}


def write_timeline(path: str, step, name: str) -> None:
    """Three iterations under the CUPTI activity tracer; the middle one is written out.  A kernel's
    'adds' is its completion time minus the latest completion before it: with programmatic dependent
    launch kernels start early and wait, so durations overlap and only completions are meaningful."""
    import collections
    from torch.profiler import ProfilerActivity, profile
    with profile(activities=[ProfilerActivity.CUDA]) as prof:
        for _ in range(3):
            step()
        torch.cuda.synchronize()
    ev = sorted((e for e in prof.events() if e.device_type.name == "CUDA" and e.name.startswith(("sx_", "void sx_"))),
                key=lambda e: e.time_range.start)
    n = len(ev) // 3
    it = ev[n:2 * n]
    t0 = it[0].time_range.start
    prev_end = t0
    agg = collections.OrderedDict()
    lines = [f"workload {name}: one iteration, {len(it)} kernels; times in us", f"{'start':>9s} {'end':>9s} {'adds':>8s}  kernel"]
    for e in it:
        nm = e.name.split("(")[0].replace("void ", "")[:44]
        end = e.time_range.end
        adds = max(0.0, end - prev_end)
        lines.append(f"{e.time_range.start - t0:9.2f} {end - t0:9.2f} {adds:8.2f}  {nm}")
        a = agg.setdefault(nm, [0, 0.0])
        a[0] += 1
        a[1] += adds
        prev_end = max(prev_end, end)
    tot = sum(a[1] for a in agg.values())
    lines.append("")
    lines.append("sum of 'adds' per kernel (the first kernel absorbs the tail of the previous iteration):")
    for k, a in sorted(agg.items(), key=lambda x: -x[1][1]):
        lines.append(f"  {k:46s} n={a[0]:3d} {a[1]:9.1f} us {a[1] / tot * 100:5.1f} %  avg {a[1] / a[0]:7.2f}")
    lines.append(f"  total {tot:.1f} us")
    with open(path, "w") as f:
        f.write("\n".join(lines) + "\n")


def run_reference(args, wl):
    """The CPU oracle as it stands, on this machine's host cores; each step is a bounded sample."""
    from oracle import specexit_oracle as orc
    from tests import harness
    case = harness.build_case(wl, poison_tail=False)
    model = harness.oracle_model(case)
    cfg = harness.default_exit_cfg(wl)

    def one():
        kv = harness.oracle_kv(case)
        if wl.mode == synth.CHAIN:
            d = orc.draft_chain(model, kv, case.f0, case.t0, wl.K, sample=_oracle_sample(args))
            th = harness.chain_target_hidden(case, d)
            v = orc.verify(model, th, d.cand_tok, sample=_oracle_sample(args), draft_logits=d.logits)
        else:
            d = orc.draft_tree(model, kv, case.f0, case.t0, wl.K, wl.topk, wl.max_nodes)
            th = harness.tree_target_hidden(case, d)
            v = orc.verify(model, th, d.cand_tok, d.parent, sample=_oracle_sample(args))
        e = orc.exit_update(cfg, orc.ExitState.fresh(wl.B), d.slot_signal, d.cand_tok, v.path, v.accept_len,
                            v.recover_tok)
        return int((e.accept_len + 1).sum())

    for _ in range(args.warmup):
        one()
    t0 = time.perf_counter()
    toks = 0
    for _ in range(args.steps):
        toks += one()
    dt = time.perf_counter() - t0
    ms = dt / args.steps * 1e3
    val = 1e3 / ms
    cores = torch.get_num_threads()
    line = {"impl": "reference", "metric": METRIC, "value": val, "unit": "iterations/s", "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "verified_tokens_per_s": toks / dt,
            "config": workload_config(args, wl, synth.cache_lengths(wl)),
            "cpu_baseline": {"value": val, "unit": "iterations/s", "cores": cores, "kind": "oracle",
                             "sample": f"{args.steps} whole iteration(s) of {wl.name} (draft rounds + verify + exit)"},
            "e2e": {"value": val, "unit": "iterations/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line), flush=True)

NOMINAL_HBM_GBS = 7700.0          # HBM3e of the HGX B200, for context beside the measured copy bandwidth
NOMINAL_BF16_TFLOPS = 2250.0      # dense bf16 tensor peak, for context


def step_flops(wl: synth.Workload, lens) -> float:
    """Multiply-adds x 2 of one iteration: every weight matrix times the rows of its round, the two attention
    products over the cached keys, and the verify head over all verify slots."""
    s = wl.shape
    head = ((s.Vd or s.V) + s.S) * s.H
    if s.arch:
        layer = 2 * s.H * s.qkv_rows + s.n_q * s.d * s.H + 3 * s.H * s.F
    else:
        layer = 2 * s.H * s.H + s.H * s.qkv_rows + s.n_q * s.d * s.H + 3 * s.H * s.F
    nsum = float(sum(int(n) for n in lens))
    total = 0.0
    for r in range(1, wl.K + 1):
        rows_per_seq = 1 if (wl.mode == synth.CHAIN or r == 1) else wl.topk
        total += 2.0 * (layer + head) * wl.B * rows_per_seq + 4.0 * rows_per_seq * s.n_q * s.d * nsum
    if s.arch:
        total += 2.0 * 3 * s.H * s.H * wl.B
    return total + 2.0 * s.V * s.H * wl.B * wl.P


def apply_variants(args, wl):
    import dataclasses
    if args.draft_vocab:
        wl = dataclasses.replace(wl, name=f"{wl.name}+Vd{args.draft_vocab}",
                                 shape=dataclasses.replace(wl.shape, Vd=args.draft_vocab))
    if args.temperature > 0.0:
        wl = dataclasses.replace(wl, name=f"{wl.name}+tau{args.temperature:g}" + ("+sampled-drafts" if args.sample_drafts else ""))
    if args.layer == "fused3":
        wl = dataclasses.replace(wl, name=f"{wl.name}+fused3", shape=dataclasses.replace(wl.shape, arch=1))
    return wl


def measure(args, wl, dev, dist, world, local, rank, steps, warmup, timeline=None):
    """Builds the workload on `dev`, times `steps` iterations and returns the record of that workload."""
    from paper_2509_24248_b200 import binding
    lens = synth.cache_lengths(wl)
    # two spare slots behind the drafted rows: a commit re-keys up to K positions behind slot n
    kv = synth.make_kv(wl.shape, lens, wl.draft_rows + 2, wl.seed)
    weights = synth.make_weights(wl.shape, wl.seed)
    f0, t0 = synth.make_f0_t0(wl)
    sx = binding.SpecExit(wl.shape, weights, wl.B, wl.mode, wl.K, wl.topk if wl.mode == synth.TREE else 1,
                          wl.max_nodes, device=str(dev), sample_drafts=args.sample_drafts,
                          tiled=args.weights == "tiled")
    sx.set_kv(kv)
    sx.sx_set_attention({"auto": binding.ATTN_AUTO, "split": binding.ATTN_SPLIT, "tc": binding.ATTN_TC}[args.attention])
    del weights
    P, H, S = wl.P, wl.shape.H, wl.shape.S
    FW = (3 if wl.shape.arch else 1) * H
    params = binding.ExitParams(alpha=wl.alpha, thr=(wl.thr, 0.8, 100.0), enable_mask=0b001,
                                stop_think_token=min(7, wl.shape.V - 1))
    out = sx.new_outputs(wl.B)
    state = sx.new_state(wl.B)
    state0 = state["_all"].clone()
    len0 = sx.kv["cache_len"].clone()
    f0_d, t0_d = f0.to(dev), t0.to(dev)

    # target hiddens: the draft hiddens of a set-up pass plus the workload's noise (outside the timed region)
    th_d = torch.zeros(wl.B, P, H, dtype=torch.bfloat16, device=dev)
    sx.sx_spec_exit_iter(params, state, f0_d, t0_d, th_d, out)
    torch.cuda.synchronize()
    sx.check_status("set-up pass")
    hid = out["hidden_d"].float().cpu()
    base = torch.empty(wl.B, P, H)
    if wl.mode == synth.CHAIN:
        base[:, :wl.K] = hid
        base[:, wl.K] = hid[:, wl.K - 1]
    else:
        row = out["slot_row_d"].cpu().long()
        src = out["slot_src_row_d"].cpu().long().clamp_min(0)
        pick = torch.where(row >= 0, row, src)
        base = torch.gather(hid, 1, pick.unsqueeze(-1).expand(-1, -1, H))
    th = synth.noisy_hidden(base.to(torch.bfloat16), synth.unit_noise(wl, P), synth.noise_sigmas(wl).view(-1, 1, 1))
    th_d.copy_(th)

    def reset_state():
        state["_all"].copy_(state0)          # one copy: all state arrays are views of this buffer

    draws = [0]

    def step():
        reset_state()
        if args.temperature > 0.0:
            draws[0] += 1
            sx.sx_set_sampling(args.temperature, 1234, draws[0])     # fresh draws every iteration
        sx.sx_spec_exit_iter(params, state, f0_d, t0_d, th_d, out)

    sampler = ClockSampler(local)
    sampler.start()
    for _ in range(max(3, warmup)):
        step()
    torch.cuda.synchronize()
    sx.check_status("warm-up")
    sampler.wait_ready()

    if dist is not None:
        dist.barrier()
    torch.cuda.synchronize()
    sampler.mark_begin()
    launches0 = sx.launch_count()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    accepted = torch.zeros(steps, wl.B, dtype=torch.int32, device=dev)
    ev0.record()
    for i in range(steps):
        step()
        accepted[i].copy_(out["accept_len_out_d"])
    ev1.record()
    torch.cuda.synchronize()
    sampler.mark_end()
    if dist is not None:
        dist.barrier()
    launches = sx.launch_count() - launches0
    sx.check_status("timed region")
    # per-iteration percentiles: a second pass with one event per iteration (kept out of the timed region: an
    # event record between two iterations costs microseconds and stops the first kernel of the next iteration
    # from overlapping the last one of this)
    n_marks = max(3, min(steps, 200))
    mark0 = torch.cuda.Event(enable_timing=True)
    marks = [torch.cuda.Event(enable_timing=True) for _ in range(n_marks)]
    mark0.record()
    for i in range(n_marks):
        step()
        marks[i].record()
    torch.cuda.synchronize()
    # per-kernel durations: the same steps again with the library's per-launch CUDA events on (kept
    # out of the timed region above: an event record between back-to-back kernels costs microseconds)
    prof_steps = min(steps, 30)
    sx.profile_begin()
    for _ in range(prof_steps):
        step()
    torch.cuda.synchronize()
    prof = sx.profile_end()
    clocks = sampler.stop()
    per_step = sorted(a.elapsed_time(b) for a, b in zip([mark0] + marks[:-1], marks))
    pct = lambda q: per_step[min(len(per_step) - 1, int(q * len(per_step)))]
    ms_total = max_over_ranks(ev0.elapsed_time(ev1), dist, dev)
    ms = ms_total / steps
    value = whole_job_rate(world * steps, ms_total)
    vtok = whole_job_rate(sum_over_ranks(float((accepted.sum() + accepted.numel()).item()), dist, dev), ms_total)

    # the loop a server runs: iteration, then the commit of its verified tokens (Algorithm 1, "Update KV-cache
    # and hidden states accordingly"); the cached lengths are put back before every step so that the cache
    # does not grow.  The commit alone is bracketed by events in a second pass.
    commit = None
    if args.temperature <= 0.0:
        th_commit = th_d if not wl.shape.arch else th_d.repeat(1, 1, 3).contiguous()
        n_loop = max(3, min(steps, 200))

        def loop_step(ev=None):
            reset_state()
            sx.kv["cache_len"].copy_(len0)
            sx.sx_spec_exit_iter(params, state, f0_d, t0_d, th_d, out)
            if ev is not None:
                ev[0].record()
            sx.sx_commit(th_commit, out["cand_tok_d"], out["path_d"], out["accept_len_out_d"], out["recover_tok_out_d"])
            if ev is not None:
                ev[1].record()

        for _ in range(3):
            loop_step()
        torch.cuda.synchronize()
        sx.check_status("iteration + commit warm-up")
        la0 = sx.launch_count()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(n_loop):
            loop_step()
        e1.record()
        torch.cuda.synchronize()
        la1 = sx.launch_count()
        pairs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(min(n_loop, 50))]
        for pr in pairs:
            loop_step(pr)
        torch.cuda.synchronize()
        sx.check_status("iteration + commit")
        sx.kv["cache_len"].copy_(len0)
        s_ = wl.shape
        # a commit streams fc and the K/V rows of the projection once
        cbytes = 2 * ((3 if s_.arch else 2) * s_.H * s_.H + 2 * s_.n_kv * s_.d * (2 if s_.arch else 1) * s_.H)
        cms = statistics.median(a.elapsed_time(b) for a, b in pairs)
        commit = {"iteration_plus_commit_ms": max_over_ranks(e0.elapsed_time(e1) / n_loop, dist, dev),
                  "commit_alone_ms": cms, "commit_weight_bytes": cbytes,
                  "commit_gbs": cbytes / (cms * 1e-3) / 1e9, "launches_per_loop_step": (la1 - la0) / n_loop}

    # the same iteration captured once into a CUDA graph and replayed (what a serving loop would do: the
    # library only enqueues kernels, so the capture needs nothing special); reported beside `value`
    graph_rec = None
    if args.temperature <= 0.0:
        n_graph = max(3, min(steps, 300))
        reset_state()
        torch.cuda.synchronize()
        cg = torch.cuda.CUDAGraph()
        with torch.cuda.graph(cg):
            reset_state()
            sx.sx_spec_exit_iter(params, state, f0_d, t0_d, th_d, out)
        for _ in range(3):
            cg.replay()
        torch.cuda.synchronize()
        sx.check_status("graph warm-up")
        g0, g1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        g0.record()
        for _ in range(n_graph):
            cg.replay()
        g1.record()
        torch.cuda.synchronize()
        sx.check_status("graph replay")
        graph_rec = {"ms_per_step": max_over_ranks(g0.elapsed_time(g1) / n_graph, dist, dev), "steps": n_graph}
        del cg

    if timeline and rank == 0:
        write_timeline(timeline, step, wl.name)

    # end to end: host buffers in, results out, through the host entry point
    stage = {"feat0": torch.empty_like(f0_d), "tok0": torch.empty_like(t0_d), "target_hidden": torch.empty_like(th_d)}
    f0_h, t0_h, th_h = f0.pin_memory(), t0.pin_memory(), th.pin_memory()
    res_h = {"accept_len": torch.zeros(wl.B, dtype=torch.int32).pin_memory(),
             "recover_tok": torch.zeros(wl.B, dtype=torch.int32).pin_memory(),
             "exit_flag": torch.zeros(wl.B, dtype=torch.int32).pin_memory(),
             "smoothed": torch.zeros(wl.B, S, dtype=torch.float32).pin_memory()}
    e2e_steps = max(3, min(steps, 200))
    for _ in range(3):
        reset_state()
        sx.sx_spec_exit_iter_host(params, state, f0_h, t0_h, th_h, stage, out, res_h)
    torch.cuda.synchronize()
    if dist is not None:
        dist.barrier()
    t_start = time.perf_counter()
    for _ in range(e2e_steps):
        reset_state()
        sx.sx_spec_exit_iter_host(params, state, f0_h, t0_h, th_h, stage, out, res_h)
    torch.cuda.synchronize()
    e2e_ms = (time.perf_counter() - t_start) * 1e3 / e2e_steps
    e2e_ms = max_over_ranks(e2e_ms, dist, dev)
    h2d = int(f0_h.numel()) * 2 + wl.B * 4 + wl.B * P * H * 2
    d2h = wl.B * (3 * 4 + S * 4)
    sx.close()
    del sx, kv
    torch.cuda.empty_cache()

    ab = algorithmic_bytes(wl, lens)
    fl = step_flops(wl, lens)
    pk = measured_peaks()
    hbm_ms = ab["total"] / (pk["hbm_gbs"] * 1e9) * 1e3
    flop_ms = fl / (pk["bf16_tflops"] * 1e12) * 1e3
    bound_ms = max(hbm_ms, flop_ms)
    nominal_ms = max(ab["total"] / (NOMINAL_HBM_GBS * 1e9), fl / (NOMINAL_BF16_TFLOPS * 1e12)) * 1e3
    head = prof.get("head_draft", {"ms": None, "n": 0})
    head_ms = head["ms"] / head["n"] if head["n"] else None
    achieved = ab["head_launch"] / (head_ms * 1e-3) / 1e9 if head_ms else None
    traffic = None
    tp = os.path.join(ROOT, "profiles", "dominant_kernel_traffic.txt")
    if os.path.exists(tp):
        for line in open(tp):
            if line.startswith(f"{wl.name}.head_draft.dram_bytes_per_launch="):
                traffic = float(line.split("=")[1])
    return {
        "value": value, "ms_per_step": ms, "steps": steps, "warmup": max(3, warmup),
        "verified_tokens_per_s": vtok, "sequence_iterations_per_s": value * wl.B,
        "ms_per_step_percentiles": {"p10": pct(0.10), "p50": pct(0.50), "p90": pct(0.90)},
        "config": workload_config(args, wl, lens),
        # the step's bound is the slower of its bytes at the HBM bandwidth and its flops at the bf16 tensor peak
        "step_roofline": {"bytes_per_iteration": ab["total"], "flops_per_iteration": fl,
                          "hbm_bound_ms": hbm_ms, "flop_bound_ms": flop_ms, "bound": "hbm" if hbm_ms >= flop_ms else "tensor",
                          "frac": bound_ms / ms, "peak_gbs": pk["hbm_gbs"], "peak_tflops": pk["bf16_tflops"],
                          "peak_kind": pk["kind"],
                          "frac_of_nominal": nominal_ms / ms, "nominal_gbs": NOMINAL_HBM_GBS,
                          "nominal_tflops": NOMINAL_BF16_TFLOPS},
        "roofline": {"kernel": "extended LM head of one draft round", "bound": "hbm", "achieved": achieved,
                     "peak": pk["hbm_gbs"], "unit": "GB/s", "frac": achieved / pk["hbm_gbs"] if achieved else None,
                     "traffic": traffic, "launch_ms": head_ms, "peak_kind": pk["kind"],
                     "frac_of_nominal": achieved / NOMINAL_HBM_GBS if achieved else None},
        "kernel_ms_per_step": {k: (v["ms"] / prof_steps) for k, v in prof.items()},
        "commit": commit,
        "graph_replay": graph_rec,
        "clocks": clocks,
        "e2e": {"value": world * 1e3 / e2e_ms, "unit": "iterations/s", "ms_per_step": e2e_ms,
                "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h},
        "gpu_launches": int(launches),
    }


def oracle_iteration(args, wl, case, model):
    from oracle import specexit_oracle as orc
    from tests import harness
    if wl.mode == synth.CHAIN:
        d = orc.draft_chain(model, harness.oracle_kv(case), case.f0, case.t0, wl.K, sample=_oracle_sample(args))
        v = orc.verify(model, harness.chain_target_hidden(case, d), d.cand_tok,
                       sample=_oracle_sample(args), draft_logits=d.logits)
    else:
        d = orc.draft_tree(model, harness.oracle_kv(case), case.f0, case.t0, wl.K, wl.topk, wl.max_nodes)
        v = orc.verify(model, harness.tree_target_hidden(case, d), d.cand_tok, d.parent,
                       sample=_oracle_sample(args))
    orc.exit_update(harness.default_exit_cfg(wl), orc.ExitState.fresh(wl.B), d.slot_signal, d.cand_tok, v.path,
                    v.accept_len, v.recover_tok)


def cpu_baseline(args, wl) -> dict:
    """The oracle as it stands on this machine's host cores: whole iterations until about 10 s have been timed,
    then one iteration on a single thread."""
    from tests import harness
    case = harness.build_case(wl, poison_tail=False)
    model = harness.oracle_model(case)
    t2 = time.perf_counter()
    n_it = 0
    while n_it < 20:
        oracle_iteration(args, wl, case, model)
        n_it += 1
        if time.perf_counter() - t2 >= 10.0:
            break
    dt = time.perf_counter() - t2
    cores = torch.get_num_threads()
    rec = {"value": n_it / dt, "unit": "iterations/s", "cores": cores, "kind": "oracle",
           "sample": f"{n_it} whole iteration(s) of {wl.name} ({dt:.1f} s)"}
    if not args.no_one_thread:
        torch.set_num_threads(1)
        t3 = time.perf_counter()
        oracle_iteration(args, wl, case, model)
        rec["one_thread"] = {"value": 1.0 / (time.perf_counter() - t3), "unit": "iterations/s", "cores": 1,
                             "sample": f"1 whole iteration of {wl.name}"}
        torch.set_num_threads(cores)
    return rec


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=1000)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--workload", default="C1", help="the headline workload of the JSON line")
    ap.add_argument("--also", default="C2,C3,C4",
                    help="at one GPU: workloads timed after the headline and added to the line as sub-records "
                         "(\"other_workloads\"), each with --also-steps iterations; empty string = none")
    ap.add_argument("--also-steps", type=int, default=300)
    ap.add_argument("--impl", default="b200")
    ap.add_argument("--temperature", type=float, default=0.0,
                    help="verify with stochastic acceptance at this temperature (0 = greedy, the headline setting)")
    ap.add_argument("--weights", choices=["tiled", "rowmajor"], default="tiled",
                    help="layout of the GEMM weights in HBM: repacked tile by tile at load (sx_tile_weight) or "
                         "row-major as handed in")
    ap.add_argument("--sample-drafts", action="store_true",
                    help="with --temperature: draw the chain's draft tokens too and verify with the accept "
                         "test min(1, p/q) and the residual draw")
    ap.add_argument("--layer", choices=["concat", "fused3"], default="concat",
                    help="draft layer: fc over [hidden ; embedding] every round (the headline setting), or "
                         "three-feature fusion in round 1 with [norm(embedding) ; norm(hidden)] as attention input")
    ap.add_argument("--draft-vocab", type=int, default=0, metavar="VD",
                    help="reduce the draft head to VD ids (id map + the target's own head); 0 = the workload as defined")
    ap.add_argument("--attention", choices=["auto", "split", "tc"], default="auto",
                    help="decode-attention kernel: the library's own choice, the split kernel, or the tensor-memory kernel")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-one-thread", action="store_true", help="skip the single-thread figure of the CPU baseline")
    ap.add_argument("--timeline", default=None, metavar="FILE",
                    help="also write a per-kernel timeline of one iteration (CUPTI through torch.profiler): when "
                         "each kernel completed and how long after its predecessor, i.e. what it adds to the "
                         "dependent chain once programmatic dependent launch has overlapped the rest")
    args = ap.parse_args()
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    wl = apply_variants(args, synth.workload(args.workload))

    if args.impl == "reference":
        if rank == 0:
            if args.steps > 3:
                args.steps = 3
            args.warmup = min(args.warmup, 1)
            run_reference(args, wl)
        return

    dist = None
    if world > 1:
        import torch.distributed as dist
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("nccl", device_id=torch.device(f"cuda:{local}"))
    dev = torch.device(f"cuda:{local}")
    torch.cuda.set_device(dev)

    rec = measure(args, wl, dev, dist, world, local, rank, args.steps, args.warmup, timeline=args.timeline)
    others = {}
    if world == 1:
        for name in [n for n in args.also.split(",") if n and n != args.workload]:
            r = measure(args, apply_variants(args, synth.workload(name)), dev, None, 1, local, 0, args.also_steps,
                        args.warmup)
            r.update({"metric": METRIC, "unit": "iterations/s"})
            others[name] = r
    if rank != 0:
        return
    line = {"metric": METRIC, "value": rec["value"], "unit": "iterations/s", "n_gpus": world, "steps": rec["steps"],
            "warmup": rec["warmup"], "ms_per_step": rec["ms_per_step"], "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic"}
    line.update({k: v for k, v in rec.items() if k not in line})
    if others:
        line["other_workloads"] = others
    if not args.no_cpu_baseline and world == 1:
        line["cpu_baseline"] = cpu_baseline(args, wl)
    print(json.dumps(line), flush=True)


if __name__ == "__main__":
    main()
