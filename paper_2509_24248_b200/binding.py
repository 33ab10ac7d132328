"""ctypes binding of libspecexit.so: argument marshalling only.

Every step of the speculative-exit iteration runs inside the library's CUDA kernels; torch is
used here for device buffers and streams.  There is no fallback: if the library cannot be
loaded, or a call returns an error, an exception is raised.
"""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass
from typing import Dict, Optional

import torch

from . import synth

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libspecexit.so")

SX_MAX_SIGNALS = 3
MODE_CHAIN, MODE_TREE = 0, 1
ACT_SIGMOID, ACT_EXPM1, ACT_IDENTITY = 0, 1, 2
DIR_GT, DIR_LT = 0, 1
EMA_VERIFIED_CONTEXT, EMA_FIRST_ONLY = 0, 1
ATTN_AUTO, ATTN_SPLIT, ATTN_TC = 0, 1, 2
SMOOTH_EWMA, SMOOTH_NONE, SMOOTH_WINDOW, SMOOTH_MOMENTUM, SMOOTH_PARAGRAPH = 0, 1, 2, 3, 4
HIST = 16

EXPORTS = ["sx_create", "sx_destroy", "sx_workspace_bytes", "sx_strerror", "sx_launch_count",
           "sx_draft_step", "sx_verify", "sx_exit_update", "sx_spec_exit_iter",
           "sx_spec_exit_iter_host", "sx_profile_begin", "sx_profile_end", "sx_verify_noalloc", "sx_commit",
           "sx_set_sampling", "sx_tiled_weight_bytes", "sx_tile_weight", "sx_selftest_bounded_wait", "sx_set_attention"]
PROF_CLASSES = ["head_draft", "head_verify", "gemm_fc", "gemm_qkv", "gemm_o", "gemm_gate_up", "gemm_down",
                "attention"]


class SxError(RuntimeError):
    pass


class ModelCfg(C.Structure):
    _fields_ = [("H", C.c_int32), ("n_q_heads", C.c_int32), ("n_kv_heads", C.c_int32),
                ("head_dim", C.c_int32), ("ffn", C.c_int32), ("vocab", C.c_int32),
                ("n_signals", C.c_int32), ("rms_eps", C.c_float), ("rope_theta", C.c_float),
                ("page_size", C.c_int32), ("act", C.c_int32 * SX_MAX_SIGNALS), ("draft_vocab", C.c_int32),
                ("arch", C.c_int32), ("tiled_weights", C.c_int32)]


class Weights(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in ("embed_d", "fc_d", "norm1_d", "wqkv_d", "wo_d", "norm2_d",
                                          "wgate_up_d", "wdown_d", "normf_d", "head_d", "target_head_d",
                                          "draft_to_token_d", "norm_e_d")]


class KV(C.Structure):
    _fields_ = [("batch", C.c_int32), ("cache_len_d", C.c_void_p), ("page_table_d", C.c_void_p),
                ("max_pages", C.c_int32), ("num_pages", C.c_int32), ("k_pages_d", C.c_void_p),
                ("v_pages_d", C.c_void_p)]


class DraftCfg(C.Structure):
    _fields_ = [("mode", C.c_int32), ("K", C.c_int32), ("topk", C.c_int32), ("max_nodes", C.c_int32),
                ("sample_drafts", C.c_int32)]


class ExitCfg(C.Structure):
    _fields_ = [("alpha", C.c_float), ("thr", C.c_float * SX_MAX_SIGNALS),
                ("dir", C.c_int32 * SX_MAX_SIGNALS), ("enable_mask", C.c_uint32),
                ("ema_positions", C.c_int32), ("split_bitmap_d", C.c_void_p),
                ("stop_think_token", C.c_int32), ("smoothing", C.c_int32), ("window", C.c_int32)]


class ExitState(C.Structure):
    _fields_ = [("x_d", C.c_void_p), ("n_updates_d", C.c_void_p), ("thinking_d", C.c_void_p),
                ("hist_d", C.c_void_p), ("par_sum_d", C.c_void_p), ("par_n_d", C.c_void_p)]


_ITER_FIELDS = ("cand_tok_d", "parent_d", "depth_d", "slot_row_d", "slot_src_row_d", "hidden_d",
                "slot_signal_d", "target_tok_d", "accept_len_d", "path_d", "recover_tok_d",
                "exit_flag_d", "accept_len_out_d", "recover_tok_out_d", "smoothed_d",
                "tree_cand_tok_d", "tree_cand_score_d", "tree_cand_row_d")


class IterOut(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in _ITER_FIELDS]


_lib = None


def load_library() -> C.CDLL:
    """Loads the shared library (built in-tree by ``build.py``).  Raises if it is missing."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise SxError(f"{LIB_PATH} is missing: run `python -m paper_2509_24248_b200.build` "
                      "(there is no CPU fallback)")
    lib = C.CDLL(LIB_PATH)
    vp, i32, sz = C.c_void_p, C.c_int32, C.c_size_t
    lib.sx_create.restype = i32
    lib.sx_create.argtypes = [C.POINTER(ModelCfg), C.POINTER(Weights), i32, C.POINTER(DraftCfg), i32,
                              C.POINTER(vp)]
    lib.sx_destroy.restype = None
    lib.sx_destroy.argtypes = [vp]
    lib.sx_workspace_bytes.restype = sz
    lib.sx_workspace_bytes.argtypes = [vp]
    lib.sx_strerror.restype = C.c_char_p
    lib.sx_strerror.argtypes = [i32]
    lib.sx_tiled_weight_bytes.restype = sz
    lib.sx_tiled_weight_bytes.argtypes = [i32, i32]
    lib.sx_tile_weight.restype = i32
    lib.sx_tile_weight.argtypes = [vp, i32, i32, vp, vp]
    lib.sx_set_sampling.restype = i32
    lib.sx_set_sampling.argtypes = [vp, C.c_float, C.c_uint64, C.c_uint32]
    lib.sx_launch_count.restype = C.c_int64
    lib.sx_launch_count.argtypes = [vp]
    lib.sx_draft_step.restype = i32
    lib.sx_draft_step.argtypes = [vp, C.POINTER(KV), i32, i32, vp, vp, vp, vp, vp, vp, vp, vp, sz, vp, vp]
    lib.sx_verify.restype = i32
    lib.sx_verify.argtypes = [vp, i32, i32, vp, vp, vp, vp, vp, vp, i32, vp, vp, sz, vp, vp]
    lib.sx_exit_update.restype = i32
    lib.sx_exit_update.argtypes = [vp, i32, i32, C.POINTER(ExitCfg), C.POINTER(ExitState), vp, vp, vp, i32,
                                   vp, vp, vp, vp, vp, vp, vp, vp]
    lib.sx_spec_exit_iter.restype = i32
    lib.sx_spec_exit_iter.argtypes = [vp, C.POINTER(KV), C.POINTER(ExitCfg), C.POINTER(ExitState), vp, vp,
                                      vp, C.POINTER(IterOut), vp, sz, vp, vp]
    lib.sx_spec_exit_iter_host.restype = i32
    lib.sx_spec_exit_iter_host.argtypes = [vp, C.POINTER(KV), C.POINTER(ExitCfg), C.POINTER(ExitState), vp, vp,
                                           vp, vp, vp, vp, C.POINTER(IterOut), vp, vp, vp, vp, vp, sz, vp, vp]
    lib.sx_profile_begin.restype = i32
    lib.sx_profile_begin.argtypes = [vp]
    lib.sx_profile_end.restype = i32
    lib.sx_profile_end.argtypes = [vp, vp, vp]
    lib.sx_commit.restype = i32
    lib.sx_commit.argtypes = [vp, C.POINTER(KV), i32, vp, vp, vp, i32, vp, vp, vp, vp, vp, sz, vp, vp]
    lib.sx_set_attention.restype = i32
    lib.sx_set_attention.argtypes = [vp, i32]
    lib.sx_selftest_bounded_wait.restype = i32
    lib.sx_selftest_bounded_wait.argtypes = [C.c_uint32, i32, vp, vp, vp]
    lib.sx_verify_noalloc.restype = i32
    lib.sx_verify_noalloc.argtypes = [vp, i32, i32, i32, i32, vp, vp, vp, vp, vp, vp, i32, vp, vp, vp]
    _lib = lib
    return lib


def _check(code: int, what: str) -> None:
    if code != 0:
        msg = load_library().sx_strerror(code).decode()
        raise SxError(f"{what} failed: {msg} ({code})")


def _p(t: Optional[torch.Tensor]) -> Optional[int]:
    return None if t is None else t.data_ptr()


@dataclass
class ExitParams:
    alpha: float = 0.3
    thr: tuple = (0.9, 0.8, 100.0)
    dir: tuple = (DIR_GT, DIR_GT, DIR_LT)
    enable_mask: int = 0b001
    ema_positions: int = EMA_VERIFIED_CONTEXT
    split_bitmap: Optional[torch.Tensor] = None     # int32 words on the device, or None
    stop_think_token: int = 0
    smoothing: int = SMOOTH_EWMA
    window: int = 10

    def struct(self) -> ExitCfg:
        c = ExitCfg()
        c.alpha = self.alpha
        for i in range(SX_MAX_SIGNALS):
            c.thr[i] = self.thr[i]
            c.dir[i] = self.dir[i]
        c.enable_mask = self.enable_mask
        c.ema_positions = self.ema_positions
        c.split_bitmap_d = _p(self.split_bitmap)
        c.stop_think_token = self.stop_think_token
        c.smoothing = self.smoothing
        c.window = self.window
        return c


NOALLOC_MAX_ROWS = 64


GEMM_WEIGHTS = ("fc", "wqkv", "wo", "wgate_up", "wdown", "head", "target_head")


def sx_tile_weight(w: torch.Tensor) -> torch.Tensor:
    """Repacks a row-major bf16 ``[N, K]`` device matrix tile by tile (``[ceil(N/128)][ceil(K/64)][128][64]``,
    zero padded), the layout a context created with ``tiled=True`` expects.  Returns a flat bf16 tensor."""
    lib = load_library()
    N, K = int(w.shape[0]), int(w.shape[1])
    if w.dtype != torch.bfloat16 or not w.is_cuda or not w.is_contiguous():
        raise SxError("sx_tile_weight wants a contiguous bf16 matrix on the device")
    out = torch.empty(int(lib.sx_tiled_weight_bytes(N, K)) // 2, dtype=torch.bfloat16, device=w.device)
    _check(lib.sx_tile_weight(w.data_ptr(), N, K, out.data_ptr(), torch.cuda.current_stream(w.device).cuda_stream),
           "sx_tile_weight")
    return out


def sx_verify_noalloc(target_head: torch.Tensor, target_hidden: torch.Tensor, cand_tok: torch.Tensor,
                      parent: Optional[torch.Tensor], out: Dict[str, torch.Tensor], status: torch.Tensor) -> None:
    """Verification without a context or a workspace, for callers that may not allocate device
    memory: every buffer, results included, is handed in by the caller (``out`` holds
    ``target_tok [B,P]``, ``accept_len [B]``, ``path [B,stride]`` and ``recover_tok [B]``, all
    int32 on the device) and the library's scratch is a fixed array inside its own image.  At most
    ``NOALLOC_MAX_ROWS`` hidden states (B * P) per call; calls on one device share the scratch,
    so keep them on one stream."""
    lib = load_library()
    B, P = cand_tok.shape
    V, H = target_head.shape
    _check(lib.sx_verify_noalloc(target_head.data_ptr(), V, H, B, P, target_hidden.data_ptr(), cand_tok.data_ptr(),
                                 _p(parent), out["target_tok"].data_ptr(), out["accept_len"].data_ptr(),
                                 out["path"].data_ptr(), int(out["path"].shape[1]), out["recover_tok"].data_ptr(),
                                 status.data_ptr(), torch.cuda.current_stream().cuda_stream), "sx_verify_noalloc")


class SpecExit:
    """One context: weights, KV cache, workspace and output buffers for a workload shape."""

    def __init__(self, shape: synth.ModelShape, weights: Dict[str, torch.Tensor], max_batch: int,
                 mode: int, K: int, topk: int = 1, max_nodes: int = 0,
                 act=(ACT_SIGMOID, ACT_SIGMOID, ACT_SIGMOID), device: str = "cuda:0",
                 max_verify_rows: int = 0, sample_drafts: bool = False, tiled: bool = False):
        self.lib = load_library()
        if not torch.cuda.is_available():
            raise SxError("a CUDA device is required (there is no CPU fallback)")
        self.dev = torch.device(device)
        torch.cuda.set_device(self.dev)
        self.shape, self.mode, self.K, self.topk, self.max_nodes = shape, mode, K, topk, max_nodes
        self.max_batch = max_batch
        self.rows = K if mode == MODE_CHAIN else 1 + topk * (K - 1)
        self.P = K + 1 if mode == MODE_CHAIN else 1 + max_nodes
        self.w = {k: (v.to(self.dev).contiguous() if v.device != self.dev else v) for k, v in weights.items()}
        if "target_head" not in self.w:
            self.w["target_head"] = self.w["head"]      # rows [0, V) of the shared head
        self.tiled = bool(tiled)
        if self.tiled:
            # every GEMM weight is repacked on the device (sx_tile_weight); the row-major copies are dropped
            done = {}
            for name in GEMM_WEIGHTS:
                src = self.w[name]
                if src.data_ptr() not in done:
                    done[src.data_ptr()] = sx_tile_weight(src)
                self.w[name] = done[src.data_ptr()]
            del done, src
            # weights must be complete before any call that reads them is enqueued (the GEMM kernels
            # fetch their first weight tiles ahead of stream order)
            torch.cuda.synchronize(self.dev)
        mc = ModelCfg(shape.H, shape.n_q, shape.n_kv, shape.d, shape.F, shape.V, shape.S, shape.eps,
                      shape.theta, shape.page, (C.c_int32 * 3)(*act), getattr(shape, "Vd", 0),
                      getattr(shape, "arch", 0), 1 if self.tiled else 0)
        d2t = self.w.get("draft_to_token")
        if d2t is not None and (d2t.dtype != torch.int32 or d2t.numel() != (shape.Vd or shape.V)):
            raise SxError("draft_to_token must be int32 with one entry per draft id")
        ws = Weights(*[self.w[n].data_ptr() for n in ("embed", "fc", "norm1", "wqkv", "wo", "norm2",
                                                       "wgate_up", "wdown", "normf", "head", "target_head")],
                     d2t.data_ptr() if d2t is not None else None,
                     self.w["norm_e"].data_ptr() if "norm_e" in self.w else None)
        dc = DraftCfg(mode, K, topk, max_nodes, 1 if sample_drafts else 0)
        h = C.c_void_p()
        _check(self.lib.sx_create(C.byref(mc), C.byref(ws), max_batch, C.byref(dc), max_verify_rows,
                                  C.byref(h)), "sx_create")
        self.h = h
        self.ws_bytes = int(self.lib.sx_workspace_bytes(h))
        self.ws = torch.empty(self.ws_bytes + 256, dtype=torch.uint8, device=self.dev)
        off = (-self.ws.data_ptr()) % 256
        self.ws_ptr = self.ws.data_ptr() + off
        self.status = torch.zeros(1, dtype=torch.int32, device=self.dev)
        self.kv = None
        self._kv_struct = None

    def close(self) -> None:
        if getattr(self, "h", None):
            self.lib.sx_destroy(self.h)
            self.h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # ---- buffers -------------------------------------------------------------------------
    def set_kv(self, kv: Dict[str, torch.Tensor]) -> None:
        d = self.dev
        self.kv = {"k_pages": kv["k_pages"].to(d), "v_pages": kv["v_pages"].to(d),
                   "page_table": kv["page_table"].to(d).contiguous(),
                   "cache_len": kv["cache_len"].to(d).contiguous()}
        B = int(self.kv["cache_len"].numel())
        self.B = B
        self._kv_struct = KV(B, self.kv["cache_len"].data_ptr(), self.kv["page_table"].data_ptr(),
                             int(self.kv["page_table"].shape[1]), int(self.kv["k_pages"].shape[0]),
                             self.kv["k_pages"].data_ptr(), self.kv["v_pages"].data_ptr())

    def new_state(self, B: int) -> Dict[str, torch.Tensor]:
        """Exit state of B sequences.  All arrays are views of one 4-byte-word buffer (``"_all"``), so
        that a caller can save or restore the whole state with a single copy."""
        S = self.shape.S
        sizes = [("x", B * S, torch.float32, (B, S)), ("n_updates", B, torch.int32, (B,)),
                 ("thinking", B, torch.int32, (B,)), ("hist", B * HIST * S, torch.float32, (B, HIST, S)),
                 ("par_sum", B * S, torch.float32, (B, S)), ("par_n", B, torch.int32, (B,))]
        words = sum(((n + 3) // 4) * 4 for _, n, _, _ in sizes)
        buf = torch.zeros(words, dtype=torch.int32, device=self.dev)
        st, at = {"_all": buf}, 0
        for name, n, dt, shape in sizes:
            st[name] = buf[at:at + n].view(dt).view(*shape)
            at += ((n + 3) // 4) * 4
        st["thinking"].fill_(1)
        return st

    def new_outputs(self, B: int) -> Dict[str, torch.Tensor]:
        d, P, S = self.dev, self.P, self.shape.S
        i32 = lambda *s: torch.full(s, -7, dtype=torch.int32, device=d)
        NC = max(1, self.topk + (self.K - 1) * self.topk * self.topk)
        return {"tree_cand_tok_d": i32(B, NC), "tree_cand_row_d": i32(B, NC),
                "tree_cand_score_d": torch.zeros(B, NC, dtype=torch.float32, device=d),
                "cand_tok_d": i32(B, P), "parent_d": i32(B, P), "depth_d": i32(B, P),
                "slot_row_d": i32(B, P), "slot_src_row_d": i32(B, P),
                "hidden_d": torch.zeros(B, self.rows, self.shape.H, dtype=torch.bfloat16, device=d),
                "slot_signal_d": torch.full((B, P, S), float("nan"), dtype=torch.float32, device=d),
                "target_tok_d": i32(B, P), "accept_len_d": i32(B), "path_d": i32(B, self.K + 1),
                "recover_tok_d": i32(B), "exit_flag_d": i32(B), "accept_len_out_d": i32(B),
                "recover_tok_out_d": i32(B),
                "smoothed_d": torch.zeros(B, S, dtype=torch.float32, device=d)}

    @staticmethod
    def _iter_struct(out: Dict[str, torch.Tensor]) -> IterOut:
        return IterOut(*[out[n].data_ptr() for n in _ITER_FIELDS])

    @staticmethod
    def _state_struct(st: Dict[str, torch.Tensor]) -> ExitState:
        return ExitState(st["x"].data_ptr(), st["n_updates"].data_ptr(), st["thinking"].data_ptr(),
                         _p(st.get("hist")), _p(st.get("par_sum")), _p(st.get("par_n")))

    def _stream(self) -> int:
        return torch.cuda.current_stream(self.dev).cuda_stream

    def check_status(self, what: str = "device") -> None:
        code = int(self.status.item())
        if code != 0:
            self.status.zero_()
            _check(code, what)

    def launch_count(self) -> int:
        return int(self.lib.sx_launch_count(self.h))

    def profile_begin(self) -> None:
        _check(self.lib.sx_profile_begin(self.h), "sx_profile_begin")

    def profile_end(self) -> Dict[str, Dict[str, float]]:
        """Call after synchronising.  Returns {class: {"ms": summed ms, "n": launches}}."""
        ms = (C.c_float * len(PROF_CLASSES))()
        n = (C.c_int32 * len(PROF_CLASSES))()
        _check(self.lib.sx_profile_end(self.h, ms, n), "sx_profile_end")
        return {name: {"ms": float(ms[i]), "n": int(n[i])} for i, name in enumerate(PROF_CLASSES) if n[i]}

    # ---- entry points (same names as the C ABI) ------------------------------------------------
    def sx_draft_step(self, round_: int, feat: torch.Tensor, tok: torch.Tensor,
                      row_mask: Optional[torch.Tensor] = None):
        R = int(tok.numel())
        T = self.topk if self.mode == MODE_TREE else 1
        hid = torch.empty(R, self.shape.H, dtype=torch.bfloat16, device=self.dev)
        tok_out = torch.empty(R, T, dtype=torch.int32, device=self.dev)
        logp = torch.empty(R, T, dtype=torch.float32, device=self.dev)
        sig = torch.empty(R, self.shape.S, dtype=torch.float32, device=self.dev)
        _check(self.lib.sx_draft_step(self.h, C.byref(self._kv_struct), round_, R, feat.data_ptr(),
                                      tok.data_ptr(), _p(row_mask), hid.data_ptr(), tok_out.data_ptr(),
                                      logp.data_ptr(), sig.data_ptr(), self.ws_ptr, self.ws_bytes,
                                      self.status.data_ptr(), self._stream()), "sx_draft_step")
        return hid, tok_out, logp, sig

    def sx_set_attention(self, kernel: int) -> None:
        """Decode-attention kernel of the draft calls that follow: ATTN_AUTO, ATTN_SPLIT or ATTN_TC."""
        _check(self.lib.sx_set_attention(self.h, int(kernel)), "sx_set_attention")

    def sx_set_sampling(self, temperature: float, seed: int = 0, offset: int = 0) -> None:
        """Stochastic acceptance for the verify calls that follow (0 = greedy)."""
        _check(self.lib.sx_set_sampling(self.h, float(temperature), int(seed), int(offset)), "sx_set_sampling")

    def sx_verify(self, target_hidden: torch.Tensor, cand_tok: torch.Tensor,
                  parent: Optional[torch.Tensor] = None, path_stride: Optional[int] = None):
        B, P = cand_tok.shape
        ps = path_stride or (self.K + 1)
        tt = torch.empty(B, P, dtype=torch.int32, device=self.dev)
        L = torch.empty(B, dtype=torch.int32, device=self.dev)
        path = torch.empty(B, ps, dtype=torch.int32, device=self.dev)
        rec = torch.empty(B, dtype=torch.int32, device=self.dev)
        _check(self.lib.sx_verify(self.h, B, P, target_hidden.data_ptr(), cand_tok.data_ptr(), _p(parent),
                                  tt.data_ptr(), L.data_ptr(), path.data_ptr(), ps, rec.data_ptr(),
                                  self.ws_ptr, self.ws_bytes, self.status.data_ptr(), self._stream()),
               "sx_verify")
        return tt, L, path, rec

    def sx_exit_update(self, params: ExitParams, state: Dict[str, torch.Tensor], slot_signal: torch.Tensor,
                       cand_tok: torch.Tensor, path: torch.Tensor, accept_len: torch.Tensor,
                       recover_tok: torch.Tensor):
        B, P = cand_tok.shape
        ef = torch.empty(B, dtype=torch.int32, device=self.dev)
        Lo = torch.empty(B, dtype=torch.int32, device=self.dev)
        ro = torch.empty(B, dtype=torch.int32, device=self.dev)
        sm = torch.empty(B, self.shape.S, dtype=torch.float32, device=self.dev)
        cfg, st = params.struct(), self._state_struct(state)
        _check(self.lib.sx_exit_update(self.h, B, P, C.byref(cfg), C.byref(st), slot_signal.data_ptr(),
                                       cand_tok.data_ptr(), path.data_ptr(), int(path.shape[1]),
                                       accept_len.data_ptr(), recover_tok.data_ptr(), ef.data_ptr(),
                                       Lo.data_ptr(), ro.data_ptr(), sm.data_ptr(), self.status.data_ptr(),
                                       self._stream()), "sx_exit_update")
        return ef, Lo, ro, sm

    def sx_commit(self, target_hidden: torch.Tensor, cand_tok: torch.Tensor, path: torch.Tensor,
                  accept_len_out: torch.Tensor, recover_tok_out: torch.Tensor):
        """Commits the verified tokens (the context's ``cache_len`` tensor is advanced in place) and
        returns the next iteration's first row ``(feat0 [B, H] bf16, tok0 [B] int32)``.  With the
        three-feature layer ``target_hidden`` is ``[B, P, 3H]`` (the target features of every verify
        slot) and ``feat0`` is ``[B, 3H]``."""
        B, P = cand_tok.shape
        feat0 = torch.empty(B, int(target_hidden.shape[-1]), dtype=torch.bfloat16, device=self.dev)
        tok0 = torch.empty(B, dtype=torch.int32, device=self.dev)
        _check(self.lib.sx_commit(self.h, C.byref(self._kv_struct), P, target_hidden.data_ptr(), cand_tok.data_ptr(),
                                  path.data_ptr(), int(path.shape[1]), accept_len_out.data_ptr(),
                                  recover_tok_out.data_ptr(), feat0.data_ptr(), tok0.data_ptr(), self.ws_ptr,
                                  self.ws_bytes, self.status.data_ptr(), self._stream()), "sx_commit")
        return feat0, tok0

    def sx_spec_exit_iter(self, params: ExitParams, state: Dict[str, torch.Tensor], feat0: torch.Tensor,
                          tok0: torch.Tensor, target_hidden: torch.Tensor, out: Dict[str, torch.Tensor]) -> None:
        cfg, st, io = params.struct(), self._state_struct(state), self._iter_struct(out)
        _check(self.lib.sx_spec_exit_iter(self.h, C.byref(self._kv_struct), C.byref(cfg), C.byref(st),
                                          feat0.data_ptr(), tok0.data_ptr(), target_hidden.data_ptr(),
                                          C.byref(io), self.ws_ptr, self.ws_bytes, self.status.data_ptr(),
                                          self._stream()), "sx_spec_exit_iter")

    def sx_spec_exit_iter_host(self, params: ExitParams, state: Dict[str, torch.Tensor], feat0_h: torch.Tensor,
                               tok0_h: torch.Tensor, target_hidden_h: torch.Tensor, stage: Dict[str, torch.Tensor],
                               out: Dict[str, torch.Tensor], res_h: Dict[str, torch.Tensor]) -> None:
        cfg, st, io = params.struct(), self._state_struct(state), self._iter_struct(out)
        _check(self.lib.sx_spec_exit_iter_host(
            self.h, C.byref(self._kv_struct), C.byref(cfg), C.byref(st), feat0_h.data_ptr(), tok0_h.data_ptr(),
            target_hidden_h.data_ptr(), stage["feat0"].data_ptr(), stage["tok0"].data_ptr(),
            stage["target_hidden"].data_ptr(), C.byref(io), res_h["accept_len"].data_ptr(),
            res_h["recover_tok"].data_ptr(), res_h["exit_flag"].data_ptr(), res_h["smoothed"].data_ptr(),
            self.ws_ptr, self.ws_bytes, self.status.data_ptr(), self._stream()), "sx_spec_exit_iter_host")
