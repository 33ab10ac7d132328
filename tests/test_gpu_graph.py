"""One whole iteration captured into a CUDA graph and replayed.

`sx_spec_exit_iter` only enqueues kernels on the caller's stream (no allocation, no synchronisation, no
host read of device data), so a serving loop can capture it once and replay it.  The replay must give
bit-identical results to the direct call on the same inputs and state, chain and tree, and again after the
inputs in the captured buffers have been replaced."""
import pytest
import torch

from paper_2509_24248_b200 import synth
from tests import harness, parity

pytestmark = pytest.mark.gpu

KEYS = ("cand_tok_d", "hidden_d", "slot_signal_d", "target_tok_d", "accept_len_d", "path_d", "recover_tok_d",
        "exit_flag_d", "accept_len_out_d", "recover_tok_out_d", "smoothed_d")


def _snapshot(out, gst):
    snap = {k: out[k].clone() for k in KEYS if k in out and out[k] is not None}
    snap.update({"state." + k: v.clone() for k, v in gst.items()})
    return snap


def _same(a, b):
    assert a.keys() == b.keys()
    for k in a:
        x, y = a[k], b[k]
        if x.is_floating_point():
            assert torch.equal(x.view(torch.int16 if x.element_size() == 2 else torch.int32),
                               y.view(torch.int16 if y.element_size() == 2 else torch.int32)), k
        else:
            assert torch.equal(x, y), k


@pytest.mark.parametrize("mode", ["chain", "tree"])
def test_iteration_replayed_from_a_graph_matches_the_direct_call(mode):
    if mode == "chain":
        wl = harness.tiny_workload(B=3, K=5, len_lo=5, len_hi=70, sigma_lo=0.0, sigma_hi=0.05)
    else:
        sh = synth.ModelShape(H=64, n_q=4, n_kv=2, d=16, F=96, V=300, page=16)
        wl = synth.Workload("gt", sh, B=2, mode=synth.TREE, K=3, topk=4, max_nodes=14, len_lo=9, len_hi=60, seed=77,
                            sigma_lo=0.0, sigma_hi=0.1)
    case = harness.build_case(wl)
    sx = parity.make_gpu(case)
    params = parity.to_params(sx, harness.default_exit_cfg(wl))
    g = torch.Generator().manual_seed(5)
    f0, t0 = case.f0.to(sx.dev), case.t0.to(sx.dev)
    th = torch.randn(wl.B, wl.P, wl.shape.H, generator=g).to(torch.bfloat16).to(sx.dev)
    out, gst = sx.new_outputs(wl.B), sx.new_state(wl.B)
    fresh = {k: v.clone() for k, v in gst.items()}

    def reset():
        for k, v in fresh.items():
            gst[k].copy_(v)
        for k in KEYS:
            if k in out and out[k] is not None:
                out[k].fill_(-7 if not out[k].is_floating_point() else float("nan"))

    reset()
    sx.sx_spec_exit_iter(params, gst, f0, t0, th, out)
    torch.cuda.synchronize()
    sx.check_status("direct call")
    want = _snapshot(out, gst)

    # capture (torch switches the current stream to its capture stream, which the binding passes on)
    reset()
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        sx.sx_spec_exit_iter(params, gst, f0, t0, th, out)
    for _ in range(3):
        reset()
        graph.replay()
        torch.cuda.synchronize()
        sx.check_status("graph replay")
        _same(_snapshot(out, gst), want)

    # other inputs in the same buffers: the graph reads the buffers, not the values seen at capture
    th.copy_(torch.randn(wl.B, wl.P, wl.shape.H, generator=g).to(torch.bfloat16).to(sx.dev))
    reset()
    sx.sx_spec_exit_iter(params, gst, f0, t0, th, out)
    torch.cuda.synchronize()
    want2 = _snapshot(out, gst)
    reset()
    graph.replay()
    torch.cuda.synchronize()
    sx.check_status("graph replay, second input")
    _same(_snapshot(out, gst), want2)
    assert not torch.equal(want2["target_tok_d"], want["target_tok_d"])
    sx.close()
