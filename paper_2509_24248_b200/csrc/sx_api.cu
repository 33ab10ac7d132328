// Host side of the C ABI: argument checks, workspace carve-up and the launch sequence of one
// speculative-exit iteration.  Nothing here synchronises or allocates device memory.
#include <new>
#include <vector>
#include <stdio.h>
#include <string.h>

#include <stdlib.h>

#include <nvtx3/nvToolsExt.h>

#include "sx_kernels.cuh"

// Named ranges for timeline tools (the header-only NVTX v3: nothing is linked, and without a tool attached a
// range costs a function-pointer test).  Off unless the environment variable SX_NVTX is set to 1.
static bool sx_nvtx_on() {
  static const bool on = [] { const char *e = getenv("SX_NVTX"); return e && e[0] == '1'; }();
  return on;
}
struct SxRange {
  bool on;
  explicit SxRange(const char *name) : on(sx_nvtx_on()) { if (on) nvtxRangePushA(name); }
  SxRange(const char *fmt, int k) : on(sx_nvtx_on()) {
    if (on) { char buf[48]; snprintf(buf, sizeof(buf), fmt, k); nvtxRangePushA(buf); }
  }
  ~SxRange() { if (on) nvtxRangePop(); }
};

struct sx_ctx {
  SxShape sh;
  sx_weights w;
  sx_draft_cfg dc;
  int max_batch, Rmax, VR, sm_count, device;
  int rows_per_seq, P, NC;
  int64_t launches;
  int max_splits, part_N, head_G, head_rows;
  // workspace offsets (bytes)
  size_t off_u, off_x, off_n, off_q, off_o, off_a, off_m, off_g, off_part, off_attn, off_hparts, off_z,
      off_tok_rt, off_logp_rt, off_tree, off_cu, off_cn, off_cpart, off_cu2, off_ctok, off_dlogits, off_tlogits, off_spec, total;
  int commit_rows, commit_N;
  bool tiled;                    // GEMM weights are stored tile by tile (sx_tile_weight)
  int attn_kernel;               // SX_ATTN_AUTO / _SPLIT / _TC (sx_set_attention)
  SxSample smp;                  // sampled verification (sx_set_sampling); temp == 0: greedy
  // set around a draft round whose head samples its token and leaves its logits (sampled drafts)
  bool round_sampled;
  SxSample round_smp;
  SxLogitsOut round_lo;
  // tree sub-offsets relative to off_tree
  size_t t_tok, t_par, t_src, t_row, t_score, t_rmask, t_selcid, t_seltok, t_fidx, t_hidx, t_nmask, t_rsig;
  // optional per-class event timing
  bool prof_on;
  std::vector<cudaEvent_t> *prof_ev;     // pairs: start, stop
  std::vector<int> *prof_cls;
  size_t prof_used;
};

static void prof_mark(sx_ctx *c, int cls, bool start, cudaStream_t st) {
  if (!c->prof_on) return;
  if (start) {
    if (c->prof_used + 2 > c->prof_ev->size()) {
      if (c->prof_ev->size() >= 400000) { c->prof_on = false; return; }
      cudaEvent_t a, b;
      if (cudaEventCreate(&a) != cudaSuccess || cudaEventCreate(&b) != cudaSuccess) { c->prof_on = false; return; }
      c->prof_ev->push_back(a);
      c->prof_ev->push_back(b);
      c->prof_cls->push_back(cls);
    } else {
      (*c->prof_cls)[c->prof_used / 2] = cls;
    }
    cudaEventRecord((*c->prof_ev)[c->prof_used], st);
  } else {
    cudaEventRecord((*c->prof_ev)[c->prof_used + 1], st);
    c->prof_used += 2;
  }
}

extern "C" sx_status sx_profile_begin(sx_ctx *c) {
  if (!c) return SX_ERR_INVALID_ARG;
  c->prof_used = 0;
  c->prof_on = true;
  return SX_OK;
}

extern "C" sx_status sx_profile_end(sx_ctx *c, float *ms_out, int32_t *count_out) {
  if (!c || !ms_out || !count_out) return SX_ERR_INVALID_ARG;
  c->prof_on = false;
  for (int i = 0; i < SX_PROF_CLASSES; ++i) { ms_out[i] = 0.f; count_out[i] = 0; }
  for (size_t i = 0; i + 1 < c->prof_used; i += 2) {
    float ms = 0.f;
    if (cudaEventElapsedTime(&ms, (*c->prof_ev)[i], (*c->prof_ev)[i + 1]) != cudaSuccess) return SX_ERR_CUDA;
    const int cls = (*c->prof_cls)[i / 2];
    ms_out[cls] += ms;
    count_out[cls] += 1;
  }
  c->prof_used = 0;
  return SX_OK;
}

#define SX_COMMIT_MAX_SPLITS SX_GEMM_MAX_SPLITS

static size_t up256(size_t v) { return (v + 255) & ~(size_t)255; }

extern "C" const char *sx_strerror(sx_status s) {
  switch (s) {
    case SX_OK: return "ok";
    case SX_ERR_INVALID_ARG: return "invalid argument";
    case SX_ERR_UNSUPPORTED: return "shape or mode not supported";
    case SX_ERR_CAPACITY: return "page table too short or token id out of range";
    case SX_ERR_WORKSPACE: return "workspace too small or misaligned";
    case SX_ERR_CUDA: return "CUDA runtime error";
    case SX_ERR_TIMEOUT: return "a bounded device-side wait expired";
    case SX_ERR_STATIC_LIMIT: return "request exceeds the fixed built-in scratch of the no-allocation entry point";
    default: return "unknown status";
  }
}

static bool pow2(int v) { return v > 0 && (v & (v - 1)) == 0; }

extern "C" sx_status sx_create(const sx_model_cfg *m, const sx_weights *w, int32_t max_batch,
                               const sx_draft_cfg *dc, int32_t max_verify_rows, sx_ctx **out) {
  if (!m || !w || !dc || !out || max_batch < 1) return SX_ERR_INVALID_ARG;
  *out = nullptr;
  const void *ptrs[] = {w->embed_d, w->fc_d, w->norm1_d, w->wqkv_d, w->wo_d, w->norm2_d,
                        w->wgate_up_d, w->wdown_d, w->normf_d, w->head_d, w->target_head_d};
  for (const void *p : ptrs)
    if (!p || ((uintptr_t)p & 15)) return SX_ERR_INVALID_ARG;
  if (m->H < 8 || m->H % 8 || m->head_dim % 8 || m->ffn % 8 || !pow2(m->head_dim) || m->head_dim > 256 ||
      m->head_dim < 8)
    return SX_ERR_UNSUPPORTED;
  if (m->n_kv_heads < 1 || m->n_q_heads % m->n_kv_heads) return SX_ERR_UNSUPPORTED;
  const int G = m->n_q_heads / m->n_kv_heads;
  if (!(G == 1 || G == 2 || G == 4 || G == 8)) return SX_ERR_UNSUPPORTED;
  if (m->n_signals < 0 || m->n_signals > SX_MAX_SIGNALS || m->vocab < 1 || m->page_size < 1)
    return SX_ERR_UNSUPPORTED;
  if (m->H > 16384) return SX_ERR_UNSUPPORTED;
  const int Vd = m->draft_vocab ? m->draft_vocab : m->vocab;
  if (Vd < 1 || Vd > m->vocab) return SX_ERR_INVALID_ARG;
  if (Vd < m->vocab && !w->draft_to_token_d) return SX_ERR_INVALID_ARG;   // a reduced vocabulary needs its id map
  if (m->arch != SX_ARCH_CONCAT && m->arch != SX_ARCH_FUSED3) return SX_ERR_UNSUPPORTED;
  if (m->tiled_weights != 0 && m->tiled_weights != 1) return SX_ERR_INVALID_ARG;
  if (m->arch == SX_ARCH_FUSED3 && (!w->norm_e_d || ((uintptr_t)w->norm_e_d & 15))) return SX_ERR_INVALID_ARG;
  if (dc->K < 1) return SX_ERR_INVALID_ARG;
  if (dc->sample_drafts != 0 && dc->sample_drafts != 1) return SX_ERR_INVALID_ARG;
  if (dc->sample_drafts && (Vd != m->vocab || w->draft_to_token_d))
    return SX_ERR_UNSUPPORTED;        // sampled drafts: full draft vocabulary, no id map
  sx_ctx *c = new (std::nothrow) sx_ctx();
  if (!c) return SX_ERR_INVALID_ARG;
  memset(c, 0, sizeof(*c));
  c->prof_ev = new std::vector<cudaEvent_t>();
  c->prof_cls = new std::vector<int>();
  c->sh.H = m->H; c->sh.nq = m->n_q_heads; c->sh.nkv = m->n_kv_heads; c->sh.d = m->head_dim;
  c->sh.F = m->ffn; c->sh.V = m->vocab; c->sh.Vd = Vd; c->sh.arch = m->arch; c->sh.S = m->n_signals; c->sh.page = m->page_size;
  c->sh.eps = m->rms_eps; c->sh.theta = m->rope_theta;
  for (int i = 0; i < SX_MAX_SIGNALS; ++i) c->sh.act[i] = m->act[i];
  c->w = *w;
  c->dc = *dc;
  c->tiled = m->tiled_weights == 1;
  c->max_batch = max_batch;
  int T = 1;
  if (dc->mode == SX_MODE_TREE) {
    T = dc->topk;
    c->rows_per_seq = 1 + T * (dc->K - 1);
    c->P = 1 + dc->max_nodes;
    c->NC = T + (dc->K - 1) * T * T;
    if (T < 1 || T > SX_MAX_TOPK || T > Vd || c->rows_per_seq > SX_MAX_TREE_ROWS ||
        c->P > SX_MAX_VERIFY_SLOTS || dc->max_nodes < 1 || dc->max_nodes > c->NC) {
      delete c;
      return SX_ERR_UNSUPPORTED;
    }
  } else if (dc->mode == SX_MODE_CHAIN) {
    c->rows_per_seq = dc->K;
    c->P = dc->K + 1;
    if (dc->K > SX_MAX_TREE_ROWS - 1) { delete c; return SX_ERR_UNSUPPORTED; }
  } else {
    delete c;
    return SX_ERR_INVALID_ARG;
  }
  c->Rmax = max_batch * T;
  c->VR = max_verify_rows > max_batch * c->P ? max_verify_rows : max_batch * c->P;
  int dev = 0;
  cudaDeviceProp prop;
  if (cudaGetDevice(&dev) != cudaSuccess || cudaGetDeviceProperties(&prop, dev) != cudaSuccess) {
    delete c;
    return SX_ERR_CUDA;
  }
  if (!sx_attn_supported(c->sh)) {            // head_dim 16 / 32 / 64 / 128, group size * topk <= 64
    delete c;
    return SX_ERR_UNSUPPORTED;
  }
  c->device = dev;
  c->sm_count = prop.multiProcessorCount;
  if (sx_gemm_init(dev) != SX_OK || sx_attn_init(dev) != SX_OK || sx_attn_tc_init(dev) != SX_OK ||
      sx_kernels_init(dev) != SX_OK) {
    delete c;
    return SX_ERR_CUDA;
  }

  const SxShape &s = c->sh;
  const int R = c->Rmax;
  c->max_splits = SX_GEMM_MAX_SPLITS;
  c->part_N = s.H;
  if ((s.nq + 2 * s.nkv) * s.d > c->part_N) c->part_N = (s.nq + 2 * s.nkv) * s.d;
  if (2 * s.F > c->part_N) c->part_N = 2 * s.F;
  c->head_G = 2 * c->sm_count;
  c->head_rows = R > 256 ? R : 256;
  size_t o = 0;
  auto take = [&](size_t bytes) { size_t at = o; o = up256(o + bytes); return at; };
  c->off_u = take((size_t)R * 2 * s.H * 2);
  c->off_x = take((size_t)R * s.H * 2);
  c->off_n = take((size_t)R * s.H * 2);
  c->off_q = take((size_t)R * s.nq * s.d * 2);
  c->off_o = take((size_t)R * s.nq * s.d * 2);
  c->off_a = take((size_t)R * s.H * 2);
  c->off_m = take((size_t)R * s.F * 2);
  c->off_g = take((size_t)R * s.H * 2);
  c->off_part = take((size_t)c->max_splits * R * c->part_N * 4);
  {
    const size_t a = sx_attn_ws_bytes(s, max_batch, T, c->sm_count), b = sx_attn_tc_ws_bytes(s, max_batch, c->sm_count);
    c->off_attn = take(a > b ? a : b);
  }
  c->off_hparts = take((size_t)c->head_G * c->head_rows * sizeof(SxHeadPartial));
  c->off_z = take((size_t)R * SX_MAX_SIGNALS * 4);
  c->off_tok_rt = take((size_t)R * SX_MAX_TOPK * 4);
  c->off_logp_rt = take((size_t)R * SX_MAX_TOPK * 4);
  // commit: up to K catch-up rows per sequence through fc, norm and the K/V part of the projection
  c->commit_rows = max_batch * dc->K;
  c->commit_N = s.H > (s.nq + 2 * s.nkv) * s.d ? s.H : (s.nq + 2 * s.nkv) * s.d;
  c->off_cu = take((size_t)c->commit_rows * (s.arch == SX_ARCH_FUSED3 ? 3 : 2) * s.H * 2);
  c->off_cn = take((size_t)c->commit_rows * s.H * 2);
  c->off_cpart = take((size_t)SX_COMMIT_MAX_SPLITS * c->commit_rows * c->commit_N * 4);
  if (dc->sample_drafts) {
    // logits of every drafted row and of every verify slot (fp32), and the scratch of the accept / residual step
    c->off_dlogits = take((size_t)max_batch * c->rows_per_seq * s.V * 4);
    c->off_tlogits = take((size_t)max_batch * c->P * s.V * 4);
    const size_t a = sx_spec_sample_ws_bytes(max_batch * c->P), b = sx_tree_spec_ws_bytes(max_batch, s.V);
    c->off_spec = take(dc->mode == SX_MODE_TREE ? b : a);
  }
  if (s.arch == SX_ARCH_FUSED3) {
    c->off_cu2 = take((size_t)c->commit_rows * 2 * s.H * 2);
    c->off_ctok = take((size_t)c->commit_rows * 4);
  }
  c->off_tree = o;
  if (dc->mode == SX_MODE_TREE) {
    const size_t B = max_batch, NC = c->NC, rows = c->rows_per_seq;
    size_t base = o;
    c->t_tok = take(B * NC * 4) - base;
    c->t_par = take(B * NC * 4) - base;
    c->t_src = take(B * NC * 4) - base;
    c->t_row = take(B * NC * 4) - base;
    c->t_score = take(B * NC * 4) - base;
    c->t_rmask = take(B * rows * 8) - base;
    c->t_selcid = take(B * T * 4) - base;
    c->t_seltok = take(B * T * 4) - base;
    c->t_fidx = take(B * T * 4) - base;
    c->t_hidx = take(B * T * 4) - base;
    c->t_nmask = take(B * T * 8) - base;
    c->t_rsig = take(B * rows * SX_MAX_SIGNALS * 4) - base;
  }
  c->total = o;
  *out = c;
  return SX_OK;
}

extern "C" void sx_destroy(sx_ctx *c) {
  if (!c) return;
  if (c->prof_ev) {
    for (cudaEvent_t e : *c->prof_ev) cudaEventDestroy(e);
    delete c->prof_ev;
    delete c->prof_cls;
  }
  delete c;
}
extern "C" size_t sx_workspace_bytes(const sx_ctx *c) { return c ? c->total : 0; }
extern "C" int64_t sx_launch_count(const sx_ctx *c) { return c ? c->launches : 0; }

static sx_status check_ws(const sx_ctx *c, const void *ws, size_t bytes) {
  if (!ws || ((uintptr_t)ws & 255) || bytes < c->total) return SX_ERR_WORKSPACE;
  return SX_OK;
}

static sx_status check_kv(const sx_ctx *c, const sx_kv *kv) {
  if (!kv || !kv->cache_len_d || !kv->page_table_d || !kv->k_pages_d || !kv->v_pages_d) return SX_ERR_INVALID_ARG;
  if (kv->batch < 1 || kv->batch > c->max_batch || kv->max_pages < 1 || kv->num_pages < 1) return SX_ERR_INVALID_ARG;
  if (((uintptr_t)kv->k_pages_d & 15) || ((uintptr_t)kv->v_pages_d & 15)) return SX_ERR_INVALID_ARG;
  return SX_OK;
}

static SxTree tree_view(const sx_ctx *c, char *ws) {
  SxTree t;
  char *b = ws + c->off_tree;
  t.T = c->dc.topk; t.D = c->dc.K; t.rows = c->rows_per_seq; t.NC = c->NC; t.max_nodes = c->dc.max_nodes;
  t.cand_tok = (int32_t *)(b + c->t_tok); t.cand_parent = (int32_t *)(b + c->t_par);
  t.cand_src_row = (int32_t *)(b + c->t_src); t.cand_row = (int32_t *)(b + c->t_row);
  t.cand_score = (float *)(b + c->t_score); t.row_mask = (uint64_t *)(b + c->t_rmask);
  t.sel_cid = (int32_t *)(b + c->t_selcid); t.sel_tok = (int32_t *)(b + c->t_seltok);
  t.feat_idx = (int32_t *)(b + c->t_fidx); t.hid_idx = (int32_t *)(b + c->t_hidx);
  t.next_mask = (uint64_t *)(b + c->t_nmask); t.row_sig = (float *)(b + c->t_rsig);
  return t;
}

// GEMM + its split-K buffer; returns the split count used
static sx_status gemm(sx_ctx *c, int cls, const void *W, int N, int K, const bf16 *X, int R, char *ws, int *splits,
                      size_t *stride, int32_t *status, cudaStream_t st) {
  int sp = sx_gemm_pick_splits(N, K, c->sm_count);
  if (sp > c->max_splits) sp = c->max_splits;
  *splits = sp;
  *stride = (size_t)R * N;
  c->launches += 1;
  prof_mark(c, cls, true, st);
  sx_status rc = sx_launch_gemm_partial((const bf16 *)W, N, K, X, R, (float *)(ws + c->off_part), sp, *stride, c->sm_count, status, st,
                                        c->tiled);
  prof_mark(c, cls, false, st);
  return rc;
}

// head over R rows in chunks the kernel can hold; merges into tok/logp/signals
static sx_status head(sx_ctx *c, int cls, const void *W, int Ntot, int V, int S, const bf16 *X, int R, int T, int lse,
                      char *ws, int32_t *tok_out, SxIndex toi, float *logp_out, float *sig_out, SxIndex si,
                      int32_t *status, cudaStream_t st, SxNextInput nx = SxNextInput{nullptr, nullptr, nullptr, 0, 0},
                      const int32_t *map = nullptr, const SxSample *smp = nullptr,
                      SxLogitsOut lo = SxLogitsOut{nullptr, 0, SxIndex{nullptr, 1, 0}}) {
  const int cap = sx_head_max_rows(T, lse);
  SxHeadPartial *parts = (SxHeadPartial *)(ws + c->off_hparts);
  float *z = (float *)(ws + c->off_z);
  for (int r0 = 0; r0 < R; r0 += cap) {
    const int rc = (R - r0 < cap) ? R - r0 : cap;
    int G = 0;
    prof_mark(c, cls, true, st);
    SxSample sm2;
    if (smp) { sm2 = *smp; sm2.row0 = r0; }
    SxLogitsOut lo2 = lo;                           // the chunk's rows go to the rows ri(r0 + r)
    if (lo2.ri.idx) lo2.ri.idx += r0; else lo2.ri.add += r0 * lo2.ri.mul;
    SX_TRY(sx_launch_head((const bf16 *)W, Ntot, V, c->sh.H, X + (size_t)r0 * c->sh.H, rc, T, lse, parts,
                          c->head_rows, &G, z, S, c->sm_count, status, st, smp ? &sm2 : nullptr,
                          lo2, c->tiled));
    prof_mark(c, cls, false, st);
    SxIndex t2 = toi, s2 = si;
    if (t2.idx) t2.idx += r0; else t2.add += r0 * t2.mul;
    if (s2.idx) s2.idx += r0; else s2.add += r0 * s2.mul;
    SX_TRY(sx_launch_head_finalize(c->sh, rc, parts, G, c->head_rows, T, lse, z, S, tok_out, t2,
                            logp_out ? logp_out + (size_t)r0 * T : nullptr, sig_out, s2, st,
                            (R <= cap) ? nx : SxNextInput{nullptr, nullptr, nullptr, 0, 0}, map, V));
    c->launches += 2;
  }
  return SX_OK;
}

static sx_status draft_round(sx_ctx *c, const sx_kv *kv, int round, int R, const bf16 *feat, SxIndex fi,
                             const int32_t *tok, SxIndex ti, const uint64_t *row_mask, bf16 *hid_user, SxIndex ui,
                             int32_t *tok_out, SxIndex toi, float *logp_out, float *sig_out, SxIndex si, char *ws,
                             int32_t *status, cudaStream_t st, bool input_ready = false, bool prepare_next = false) {
  SxRange range("sx draft round %d", round);
  const SxShape &s = c->sh;
  bf16 *u = (bf16 *)(ws + c->off_u), *x = (bf16 *)(ws + c->off_x), *n = (bf16 *)(ws + c->off_n);
  bf16 *q = (bf16 *)(ws + c->off_q), *o = (bf16 *)(ws + c->off_o), *a = (bf16 *)(ws + c->off_a);
  bf16 *m = (bf16 *)(ws + c->off_m), *g = (bf16 *)(ws + c->off_g);
  float *part = (float *)(ws + c->off_part);
  SxRowMap rm;
  rm.mode = c->dc.mode; rm.round = round; rm.topk = c->dc.mode == SX_MODE_TREE ? c->dc.topk : 1; rm.R = R;
  rm.cache_len = kv->cache_len_d; rm.row_mask = row_mask;
  rm.valid_len = nullptr; rm.per_seq = 1;
  int sp; size_t stride;
  const bool fused3 = s.arch == SX_ARCH_FUSED3;
  if (fused3) {
    // round 1: x = fc . [three target features]; later rounds: x = the source row's hidden (y).
    // u = [norm_e(E[token]) ; norm_1(x)] feeds the q/k/v projection, x is the residual stream.
    if (round == 1) {
      if (fi.idx || fi.mul != 1 || fi.add != 0) return SX_ERR_UNSUPPORTED;      // the GEMM reads the rows in place
      SX_TRY(gemm(c, SX_PROF_GEMM_FC, c->w.fc_d, s.H, 3 * s.H, feat, R, ws, &sp, &stride, status, st));
      SX_TRY(sx_launch_fused_input(s, R, part, sp, stride, nullptr, fi, tok, ti, (const bf16 *)c->w.embed_d,
                            (const bf16 *)c->w.norm_e_d, (const bf16 *)c->w.norm1_d, x, u, status, st));
    } else {
      SX_TRY(sx_launch_fused_input(s, R, nullptr, 0, 0, feat, fi, tok, ti, (const bf16 *)c->w.embed_d,
                            (const bf16 *)c->w.norm_e_d, (const bf16 *)c->w.norm1_d, x, u, status, st));
    }
    SX_TRY(gemm(c, SX_PROF_GEMM_QKV, c->w.wqkv_d, (s.nq + 2 * s.nkv) * s.d, 2 * s.H, u, R, ws, &sp, &stride, status, st));
  } else {
    // input_ready: the previous round's merge kernel has already written u (chain drafting)
    if (!input_ready) {
      SX_TRY(sx_launch_embed_concat(s, R, feat, fi, tok, ti, (const bf16 *)c->w.embed_d, u, status, st));
      c->launches += 1;
    }
    SX_TRY(gemm(c, SX_PROF_GEMM_FC, c->w.fc_d, s.H, 2 * s.H, u, R, ws, &sp, &stride, status, st));
    SX_TRY(sx_launch_finish_norm(s, R, part, sp, stride, nullptr, (const bf16 *)c->w.norm1_d, x, n, nullptr, SxIndex{nullptr, 1, 0}, st));
    SX_TRY(gemm(c, SX_PROF_GEMM_QKV, c->w.wqkv_d, (s.nq + 2 * s.nkv) * s.d, s.H, n, R, ws, &sp, &stride, status, st));
  }
  SX_TRY(sx_launch_finish_qkv_rope(s, rm, part, sp, stride, q, *kv, status, st));
  const int B = kv->batch, nr = R / B;
  const int E = (c->dc.mode == SX_MODE_CHAIN) ? round : (round == 1 ? 1 : 1 + (round - 1) * c->dc.topk);
  // Which attention kernel: the tensor-memory one for long caches with more than four queries per (sequence,
  // KV head); below a few blocks of keys per SM its set-up outweighs its stream, and with up to four queries
  // the split kernel's three small CTAs per SM keep more bytes in flight (the host knows capacities, not lengths).
  bool tc = sx_attn_tc_supported(s, nr, *kv);
  if (c->attn_kernel == SX_ATTN_SPLIT) tc = false;
  else if (c->attn_kernel == SX_ATTN_AUTO)
    tc = tc && nr * (s.nq / s.nkv) > 4 && (long long)B * s.nkv * ((kv->max_pages * s.page + 127) / 128) >= 4ll * c->sm_count;
  else if (!tc) return SX_ERR_UNSUPPORTED;
  prof_mark(c, SX_PROF_ATTENTION, true, st);
  if (tc) {
    SX_TRY(sx_launch_attention_tc(s, rm, B, nr, E, q, *kv, (float *)(ws + c->off_attn), o, c->sm_count, status, st));
  } else {
    const int nsplit = sx_attn_splits(s, B, nr, kv->max_pages * s.page, c->sm_count);
    SX_TRY(sx_launch_attention(s, rm, B, nr, E, q, *kv, nsplit, (float *)(ws + c->off_attn), o, c->sm_count, status, st));
  }
  prof_mark(c, SX_PROF_ATTENTION, false, st);
  SX_TRY(gemm(c, SX_PROF_GEMM_O, c->w.wo_d, s.H, s.nq * s.d, o, R, ws, &sp, &stride, status, st));
  SX_TRY(sx_launch_finish_norm(s, R, part, sp, stride, x, (const bf16 *)c->w.norm2_d, a, n, nullptr, SxIndex{nullptr, 1, 0}, st));
  SX_TRY(gemm(c, SX_PROF_GEMM_GATE_UP, c->w.wgate_up_d, 2 * s.F, s.H, n, R, ws, &sp, &stride, status, st));
  SX_TRY(sx_launch_finish_swiglu(s, R, part, sp, stride, m, st));
  SX_TRY(gemm(c, SX_PROF_GEMM_DOWN, c->w.wdown_d, s.H, s.F, m, R, ws, &sp, &stride, status, st));
  // the hidden handed to the caller (and to the next round) is g, or y for the fused layer
  SX_TRY(sx_launch_finish_norm(s, R, part, sp, stride, a, (const bf16 *)c->w.normf_d, nullptr, g, hid_user, ui, st, fused3 ? 1 : 0));
  c->launches += 7;   // 3 norms, rope, attention x2, swiglu
  const int T = c->dc.mode == SX_MODE_TREE ? c->dc.topk : 1;
  SX_TRY(head(c, SX_PROF_HEAD_DRAFT, c->w.head_d, s.Vd + s.S, s.Vd, s.S, g, R, T, c->dc.mode == SX_MODE_TREE ? 1 : 0, ws, tok_out, toi, logp_out, sig_out, si,
              status, st,
              (prepare_next && !fused3) ? SxNextInput{g, (const bf16 *)c->w.embed_d, u, s.H, s.V}
                           : SxNextInput{nullptr, nullptr, nullptr, 0, 0},
              c->w.draft_to_token_d, (c->round_sampled && c->dc.mode == SX_MODE_CHAIN) ? &c->round_smp : nullptr,
              c->round_sampled ? c->round_lo : SxLogitsOut{nullptr, 0, SxIndex{nullptr, 1, 0}}));
  if (c->round_sampled && c->dc.mode == SX_MODE_TREE) {
    // sampled children: the head above left the rows' logits in memory; the children are the T best of
    // logit + temperature * Gumbel noise (a draw without replacement), with their raw log-probabilities
    SX_TRY(sx_launch_gumbel_topk(R, s.V, T, c->round_lo.out, c->round_lo.ld, c->round_lo.ri, c->round_smp,
                                 (SxHeadPartial *)(ws + c->off_hparts), (size_t)c->head_G * c->head_rows, c->sm_count,
                                 tok_out, logp_out, st));
    c->launches += 2;
  }
  return SX_OK;
}

extern "C" sx_status sx_draft_step(sx_ctx *c, const sx_kv *kv, int32_t round, int32_t R, const void *feat_d,
                                   const int32_t *tok_d, const uint64_t *row_mask_d, void *hidden_out_d,
                                   int32_t *tok_out_d, float *logp_out_d, float *signals_out_d, void *ws_d,
                                   size_t ws_bytes, int32_t *status_d, void *stream) {
  if (!c || !feat_d || !tok_d || !hidden_out_d || !tok_out_d || !signals_out_d || !status_d) return SX_ERR_INVALID_ARG;
  SX_TRY(check_kv(c, kv));
  SX_TRY(check_ws(c, ws_d, ws_bytes));
  if (((uintptr_t)feat_d & 15) || ((uintptr_t)hidden_out_d & 15)) return SX_ERR_INVALID_ARG;
  const bool tree = c->dc.mode == SX_MODE_TREE;
  if (round < 1 || round > c->dc.K) return SX_ERR_INVALID_ARG;
  const int expect = (tree && round > 1) ? kv->batch * c->dc.topk : kv->batch;
  if (R != expect) return SX_ERR_INVALID_ARG;
  if (tree && round > 1 && !row_mask_d) return SX_ERR_INVALID_ARG;
  if (tree && !logp_out_d) return SX_ERR_INVALID_ARG;
  const int T = tree ? c->dc.topk : 1;
  return draft_round(c, kv, round, R, (const bf16 *)feat_d, SxIndex{nullptr, 1, 0}, tok_d, SxIndex{nullptr, 1, 0},
                     (tree && round > 1) ? row_mask_d : nullptr, (bf16 *)hidden_out_d, SxIndex{nullptr, 1, 0},
                     tok_out_d, SxIndex{nullptr, T, 0}, logp_out_d, signals_out_d, SxIndex{nullptr, 1, 0},
                     (char *)ws_d, status_d, (cudaStream_t)stream);
}

extern "C" size_t sx_tiled_weight_bytes(int32_t N, int32_t K) {
  if (N < 1 || K < 1) return 0;
  return sx_tiled_elems(N, K) * sizeof(bf16);
}

extern "C" sx_status sx_tile_weight(const void *src_d, int32_t N, int32_t K, void *dst_d, void *stream) {
  if (!src_d || !dst_d || ((uintptr_t)src_d & 15) || ((uintptr_t)dst_d & 15)) return SX_ERR_INVALID_ARG;
  return sx_launch_tile_weight((const bf16 *)src_d, N, K, (bf16 *)dst_d, (cudaStream_t)stream);
}

extern "C" sx_status sx_selftest_bounded_wait(uint32_t limit, int32_t ctas, int32_t *status_d, int32_t *reached_d,
                                              void *stream) {
  if (!status_d || !reached_d) return SX_ERR_INVALID_ARG;
  return sx_launch_wait_selftest(limit, ctas, status_d, reached_d, (cudaStream_t)stream);
}

extern "C" sx_status sx_set_attention(sx_ctx *c, int32_t kernel) {
  if (!c || kernel < SX_ATTN_AUTO || kernel > SX_ATTN_TC) return SX_ERR_INVALID_ARG;
  c->attn_kernel = kernel;
  return SX_OK;
}

extern "C" sx_status sx_set_sampling(sx_ctx *c, float temperature, uint64_t seed, uint32_t offset) {
  if (!c || !(temperature >= 0.f) || !(temperature < INFINITY)) return SX_ERR_INVALID_ARG;
  c->smp.temp = temperature;
  c->smp.k0 = (uint32_t)(seed & 0xffffffffull);
  c->smp.k1 = (uint32_t)(seed >> 32);
  c->smp.offset = offset;
  return SX_OK;
}

extern "C" sx_status sx_verify(sx_ctx *c, int32_t batch, int32_t P, const void *target_hidden_d,
                               const int32_t *cand_tok_d, const int32_t *parent_d, int32_t *target_tok_d,
                               int32_t *accept_len_d, int32_t *path_d, int32_t path_stride, int32_t *recover_tok_d,
                               void *ws_d, size_t ws_bytes, int32_t *status_d, void *stream) {
  if (!c || !target_hidden_d || !cand_tok_d || !target_tok_d || !accept_len_d || !path_d || !recover_tok_d || !status_d)
    return SX_ERR_INVALID_ARG;
  if (batch < 1 || P < 1 || path_stride < 1 || ((uintptr_t)target_hidden_d & 15)) return SX_ERR_INVALID_ARG;
  if (parent_d && P > SX_MAX_VERIFY_SLOTS) return SX_ERR_UNSUPPORTED;
  SX_TRY(check_ws(c, ws_d, ws_bytes));
  SxRange range("sx verify");
  cudaStream_t st = (cudaStream_t)stream;
  SxSample smp = c->smp;
  smp.P = P;
  SX_TRY(head(c, SX_PROF_HEAD_VERIFY, c->w.target_head_d, c->sh.V, c->sh.V, 0, (const bf16 *)target_hidden_d, batch * P, 1, 0, (char *)ws_d,
              target_tok_d, SxIndex{nullptr, 1, 0}, nullptr, nullptr, SxIndex{nullptr, 1, 0}, status_d, st,
              SxNextInput{nullptr, nullptr, nullptr, 0, 0}, nullptr, smp.temp > 0.f ? &smp : nullptr));
  SX_TRY(sx_launch_accept(batch, P, cand_tok_d, parent_d, target_tok_d, accept_len_d, path_d, path_stride, recover_tok_d, st));
  c->launches += 1;
  return SX_OK;
}

extern "C" sx_status sx_exit_update(sx_ctx *c, int32_t batch, int32_t P, const sx_exit_cfg *cfg,
                                    const sx_exit_state *state, const float *slot_signal_d, const int32_t *cand_tok_d,
                                    const int32_t *path_d, int32_t path_stride, const int32_t *accept_len_d,
                                    const int32_t *recover_tok_d, int32_t *exit_flag_d, int32_t *accept_len_out_d,
                                    int32_t *recover_tok_out_d, float *smoothed_out_d, int32_t *status_d, void *stream) {
  if (!c || !cfg || !state || !slot_signal_d || !cand_tok_d || !path_d || !accept_len_d || !recover_tok_d ||
      !exit_flag_d || !accept_len_out_d || !recover_tok_out_d || !smoothed_out_d || !status_d)
    return SX_ERR_INVALID_ARG;
  if (!state->x_d || !state->n_updates_d || !state->thinking_d || batch < 1 || P < 1 || path_stride < 1)
    return SX_ERR_INVALID_ARG;
  if (!(cfg->alpha >= 0.f && cfg->alpha <= 1.f)) return SX_ERR_INVALID_ARG;
  if (cfg->smoothing < SX_SMOOTH_EWMA || cfg->smoothing > SX_SMOOTH_PARAGRAPH) return SX_ERR_INVALID_ARG;
  if ((cfg->smoothing == SX_SMOOTH_WINDOW || cfg->smoothing == SX_SMOOTH_MOMENTUM) &&
      (!state->hist_d || cfg->window < 2 || cfg->window >= SX_HIST))
    return SX_ERR_INVALID_ARG;
  if (cfg->smoothing == SX_SMOOTH_PARAGRAPH && (!state->par_sum_d || !state->par_n_d)) return SX_ERR_INVALID_ARG;
  SxRange range("sx exit update");
  SX_TRY(sx_launch_exit(batch, P, c->sh.S, *cfg, *state, slot_signal_d, cand_tok_d, path_d, path_stride, accept_len_d,
                 recover_tok_d, exit_flag_d, accept_len_out_d, recover_tok_out_d, smoothed_out_d, c->sh.V, status_d,
                 (cudaStream_t)stream));
  c->launches += 1;
  return SX_OK;
}

extern "C" sx_status sx_spec_exit_iter(sx_ctx *c, const sx_kv *kv, const sx_exit_cfg *cfg, const sx_exit_state *state,
                                       const void *feat0_d, const int32_t *tok0_d, const void *target_hidden_d,
                                       const sx_iter_out *o, void *ws_d, size_t ws_bytes, int32_t *status_d,
                                       void *stream) {
  if (!c || !cfg || !state || !feat0_d || !tok0_d || !target_hidden_d || !o || !status_d) return SX_ERR_INVALID_ARG;
  SX_TRY(check_kv(c, kv));
  SX_TRY(check_ws(c, ws_d, ws_bytes));
  if (!o->cand_tok_d || !o->hidden_d || !o->slot_signal_d || !o->target_tok_d || !o->accept_len_d || !o->path_d ||
      !o->recover_tok_d || !o->exit_flag_d || !o->accept_len_out_d || !o->recover_tok_out_d || !o->smoothed_d)
    return SX_ERR_INVALID_ARG;
  if (((uintptr_t)feat0_d & 15) || ((uintptr_t)o->hidden_d & 15) || ((uintptr_t)target_hidden_d & 15))
    return SX_ERR_INVALID_ARG;
  SxRange range("sx spec exit iteration");
  cudaStream_t st = (cudaStream_t)stream;
  char *ws = (char *)ws_d;
  const int B = kv->batch, K = c->dc.K, P = c->P, S = c->sh.S;
  bf16 *hid = (bf16 *)o->hidden_d;
  if (c->dc.mode == SX_MODE_CHAIN) {
    SX_TRY(sx_launch_chain_layout(B, K, S, tok0_d, *o, st));
    c->launches += 1;
    // one head launch per round: its merge can write the next input (concat layer only)
    const bool fuse = B <= sx_head_max_rows(1, 0) && c->sh.arch == SX_ARCH_CONCAT;
    // sampled drafts: every draft head draws its token and leaves its logits for the accept test
    const bool sampled = c->dc.sample_drafts && c->smp.temp > 0.f;
    float *dlogits = sampled ? (float *)(ws + c->off_dlogits) : nullptr;
    const int V = c->sh.V;
    for (int k = 1; k <= K; ++k) {
      const bf16 *feat = (k == 1) ? (const bf16 *)feat0_d : hid;
      SxIndex fi = (k == 1) ? SxIndex{nullptr, 1, 0} : SxIndex{nullptr, K, k - 2};
      if (sampled) {
        c->round_sampled = true;
        c->round_smp = c->smp;
        c->round_smp.P = 1;
        c->round_smp.slot_base = 0x40000000u + (uint32_t)(k - 1);
        c->round_lo = SxLogitsOut{dlogits + (size_t)(k - 1) * V, (size_t)K * V, SxIndex{nullptr, 1, 0}};
      }
      const sx_status rc = draft_round(c, kv, k, B, feat, fi, o->cand_tok_d, SxIndex{nullptr, P, k - 1}, nullptr, hid,
                                       SxIndex{nullptr, K, k - 1}, o->cand_tok_d, SxIndex{nullptr, P, k}, nullptr,
                                       o->slot_signal_d, SxIndex{nullptr, P, k - 1}, ws, status_d, st, k > 1 && fuse,
                                       k < K && fuse);
      c->round_sampled = false;
      SX_TRY(rc);
    }
    if (sampled) {
      // target logits of every slot, then the accept test / residual draw, then the usual walk
      float *tlogits = (float *)(ws + c->off_tlogits);
      SX_TRY(head(c, SX_PROF_HEAD_VERIFY, c->w.target_head_d, V, V, 0, (const bf16 *)target_hidden_d, B * P, 1, 0, ws,
                  o->target_tok_d, SxIndex{nullptr, 1, 0}, nullptr, nullptr, SxIndex{nullptr, 1, 0}, status_d, st,
                  SxNextInput{nullptr, nullptr, nullptr, 0, 0}, nullptr, nullptr, SxLogitsOut{tlogits, (size_t)V, SxIndex{nullptr, 1, 0}}));
      SX_TRY(sx_launch_spec_sample(B, P, V, tlogits, dlogits, o->cand_tok_d, c->smp, ws + c->off_spec, c->sm_count,
                            o->target_tok_d, status_d, st));
      SX_TRY(sx_launch_accept(B, P, o->cand_tok_d, nullptr, o->target_tok_d, o->accept_len_d, o->path_d, K + 1,
                       o->recover_tok_d, st));
      c->launches += 4;
    } else {
      SX_TRY(sx_verify(c, B, P, target_hidden_d, o->cand_tok_d, nullptr, o->target_tok_d, o->accept_len_d, o->path_d,
                       K + 1, o->recover_tok_d, ws_d, ws_bytes, status_d, stream));
    }
  } else {
    if (!o->parent_d) return SX_ERR_INVALID_ARG;
    SxTree t = tree_view(c, ws);
    if (o->tree_cand_tok_d) t.cand_tok = o->tree_cand_tok_d;
    if (o->tree_cand_score_d) t.cand_score = o->tree_cand_score_d;
    if (o->tree_cand_row_d) t.cand_row = o->tree_cand_row_d;
    const int T = t.T, rows = t.rows;
    int32_t *tok_rt = (int32_t *)(ws + c->off_tok_rt);
    float *logp_rt = (float *)(ws + c->off_logp_rt);
    // sampled children: every draft head leaves its rows' logits (row b * rows + drafted row) and the children
    // are drawn from them; the noise of the children of drafted row r is the stream 0x50000000 + r
    const bool sampled = c->dc.sample_drafts && c->smp.temp > 0.f;
    float *dlogits = sampled ? (float *)(ws + c->off_dlogits) : nullptr;
    const int V = c->sh.V;
    auto round_sampling = [&](int r) {
      if (!sampled) return;
      c->round_sampled = true;
      c->round_smp = c->smp;
      c->round_smp.row0 = 0;
      c->round_smp.P = (r == 1) ? 1 : T;
      c->round_smp.slot_base = 0x50000000u + (uint32_t)(r == 1 ? 0 : 1 + (r - 2) * T);
      SxLogitsOut lo;
      lo.out = dlogits;
      lo.ld = (size_t)V;
      lo.ri.idx = (r == 1) ? nullptr : t.hid_idx;
      lo.ri.mul = (r == 1) ? rows : 0;
      lo.ri.add = 0;
      c->round_lo = lo;
    };
    round_sampling(1);
    sx_status rc1 = draft_round(c, kv, 1, B, (const bf16 *)feat0_d, SxIndex{nullptr, 1, 0}, tok0_d, SxIndex{nullptr, 1, 0},
                                nullptr, hid, SxIndex{nullptr, rows, 0}, tok_rt, SxIndex{nullptr, T, 0}, logp_rt, t.row_sig,
                                SxIndex{nullptr, rows, 0}, ws, status_d, st);
    c->round_sampled = false;
    SX_TRY(rc1);
    SX_TRY(sx_launch_tree_expand(t, B, 1, tok_rt, logp_rt, st));
    c->launches += 1;
    for (int r = 2; r <= K; ++r) {
      round_sampling(r);
      const sx_status rcr = draft_round(c, kv, r, B * T, hid, SxIndex{t.feat_idx, 0, 0}, t.sel_tok, SxIndex{nullptr, 1, 0},
                                        t.next_mask, hid, SxIndex{t.hid_idx, 0, 0}, tok_rt, SxIndex{nullptr, T, 0}, logp_rt,
                                        t.row_sig, SxIndex{t.hid_idx, 0, 0}, ws, status_d, st);
      c->round_sampled = false;
      SX_TRY(rcr);
      SX_TRY(sx_launch_tree_expand(t, B, r, tok_rt, logp_rt, st));
      c->launches += 1;
    }
    SX_TRY(sx_launch_tree_layout(t, B, S, tok0_d, *o, st));
    c->launches += 1;
    if (sampled) {
      // target logits of every slot, then the walk with the accept tests and residual draws
      if (!o->slot_row_d) return SX_ERR_INVALID_ARG;
      float *tlogits = (float *)(ws + c->off_tlogits);
      SX_TRY(head(c, SX_PROF_HEAD_VERIFY, c->w.target_head_d, V, V, 0, (const bf16 *)target_hidden_d, B * P, 1, 0, ws,
                  o->target_tok_d, SxIndex{nullptr, 1, 0}, nullptr, nullptr, SxIndex{nullptr, 1, 0}, status_d, st,
                  SxNextInput{nullptr, nullptr, nullptr, 0, 0}, nullptr, nullptr,
                  SxLogitsOut{tlogits, (size_t)V, SxIndex{nullptr, 1, 0}}));
      SX_TRY(sx_launch_tree_spec_walk(B, P, V, rows, K + 1, tlogits, dlogits, o->cand_tok_d, o->parent_d, o->slot_row_d,
                                      c->smp, ws + c->off_spec, o->target_tok_d, o->accept_len_d, o->path_d,
                                      o->recover_tok_d, status_d, st));
      c->launches += 1;
    } else {
      SX_TRY(sx_verify(c, B, P, target_hidden_d, o->cand_tok_d, o->parent_d, o->target_tok_d, o->accept_len_d,
                       o->path_d, K + 1, o->recover_tok_d, ws_d, ws_bytes, status_d, stream));
    }
  }
  return sx_exit_update(c, B, P, cfg, state, o->slot_signal_d, o->cand_tok_d, o->path_d, K + 1, o->accept_len_d,
                        o->recover_tok_d, o->exit_flag_d, o->accept_len_out_d, o->recover_tok_out_d, o->smoothed_d,
                        status_d, stream);
}

// K/V part of the q/k/v projection for a commit: the rows behind the n_q * d query rows.  Row-major weights
// are entered at that row; tiled weights at that row tile (when the query rows end on a tile boundary,
// otherwise the whole projection is computed and the query part ignored).
static sx_status commit_kv_projection(sx_ctx *c, int Kin, const bf16 *X, int R, float *part, int *sp_out,
                                      bool *kv_only, int32_t *status, cudaStream_t st) {
  const SxShape &s = c->sh;
  const int Nq = s.nq * s.d, Nkv = 2 * s.nkv * s.d, N = Nq + Nkv;
  const bf16 *W = (const bf16 *)c->w.wqkv_d;
  *kv_only = !c->tiled || (Nq % SX_TILE_M) == 0;
  const int n = *kv_only ? Nkv : N;
  if (*kv_only) W += c->tiled ? sx_tiled_elems(Nq, Kin) : (size_t)Nq * Kin;
  int sp = sx_gemm_pick_splits(n, Kin, c->sm_count);
  if (sp > SX_COMMIT_MAX_SPLITS) sp = 1;
  *sp_out = sp;
  return sx_launch_gemm_partial(W, n, Kin, X, R, part, sp, (size_t)R * n, c->sm_count, status, st, c->tiled);
}

extern "C" sx_status sx_commit(sx_ctx *c, const sx_kv *kv, int32_t P, const void *target_hidden_d,
                               const int32_t *cand_tok_d, const int32_t *path_d, int32_t path_stride,
                               const int32_t *accept_len_out_d, const int32_t *recover_tok_out_d, void *feat0_next_d,
                               int32_t *tok0_next_d, void *ws_d, size_t ws_bytes, int32_t *status_d, void *stream) {
  if (!c || !target_hidden_d || !cand_tok_d || !path_d || !accept_len_out_d || !recover_tok_out_d || !feat0_next_d ||
      !tok0_next_d || !status_d)
    return SX_ERR_INVALID_ARG;
  SX_TRY(check_kv(c, kv));
  SX_TRY(check_ws(c, ws_d, ws_bytes));
  if (P < 1 || path_stride < 1 || path_stride - 1 > c->dc.K) return SX_ERR_INVALID_ARG;
  if (((uintptr_t)target_hidden_d & 15) || ((uintptr_t)feat0_next_d & 15)) return SX_ERR_INVALID_ARG;
  SxRange range("sx commit");
  cudaStream_t st = (cudaStream_t)stream;
  char *ws = (char *)ws_d;
  const SxShape &s = c->sh;
  const int B = kv->batch, M = path_stride - 1, R = B * M;
  bf16 *u = (bf16 *)(ws + c->off_cu), *n = (bf16 *)(ws + c->off_cn);
  float *part = (float *)(ws + c->off_cpart);
  if (s.arch == SX_ARCH_FUSED3) {
    // target_hidden_d holds the three target features of every verify slot ([batch, P, 3H]):
    // catch-up rows go through fc (3H -> H), the two input norms and the K/V part of the projection
    bf16 *u2 = (bf16 *)(ws + c->off_cu2);
    int32_t *trow = (int32_t *)(ws + c->off_ctok);
    SX_TRY(sx_launch_commit_gather(s, B, M, P, (const bf16 *)target_hidden_d, cand_tok_d, path_d, path_stride, accept_len_out_d,
                            recover_tok_out_d, (const bf16 *)c->w.embed_d, u, (bf16 *)feat0_next_d, tok0_next_d, status_d,
                            st, trow));
    c->launches += 1;
    if (R > 0) {
      int sp = sx_gemm_pick_splits(s.H, 3 * s.H, c->sm_count);
      if (sp > SX_COMMIT_MAX_SPLITS) sp = 1;
      SX_TRY(sx_launch_gemm_partial((const bf16 *)c->w.fc_d, s.H, 3 * s.H, u, R, part, sp, (size_t)R * s.H, c->sm_count,
                                    status_d, st, c->tiled));
      SX_TRY(sx_launch_fused_input(s, R, part, sp, (size_t)R * s.H, nullptr, SxIndex{nullptr, 1, 0}, trow, SxIndex{nullptr, 1, 0},
                            (const bf16 *)c->w.embed_d, (const bf16 *)c->w.norm_e_d, (const bf16 *)c->w.norm1_d, n, u2,
                            status_d, st));
      bool kv_only;
      SX_TRY(commit_kv_projection(c, 2 * s.H, u2, R, part, &sp, &kv_only, status_d, st));
      const int N = kv_only ? 2 * s.nkv * s.d : (s.nq + 2 * s.nkv) * s.d;
      SxRowMap rm;
      memset(&rm, 0, sizeof(rm));
      rm.mode = SX_MODE_COMMIT; rm.round = 1; rm.topk = 1; rm.R = R; rm.cache_len = kv->cache_len_d;
      rm.valid_len = accept_len_out_d; rm.per_seq = M;
      SX_TRY(sx_launch_finish_qkv_rope(s, rm, part, sp, (size_t)R * N, nullptr, *kv, status_d, st, kv_only));
      c->launches += 4;
    }
    SX_TRY(sx_launch_commit_advance(B, accept_len_out_d, kv->cache_len_d, st));
    c->launches += 1;
    return SX_OK;
  }
  SX_TRY(sx_launch_commit_gather(s, B, M, P, (const bf16 *)target_hidden_d, cand_tok_d, path_d, path_stride, accept_len_out_d,
                          recover_tok_out_d, (const bf16 *)c->w.embed_d, u, (bf16 *)feat0_next_d, tok0_next_d, status_d, st));
  c->launches += 1;
  if (R > 0) {
    int sp = sx_gemm_pick_splits(s.H, 2 * s.H, c->sm_count);
    if (sp > SX_COMMIT_MAX_SPLITS) sp = 1;
    SX_TRY(sx_launch_gemm_partial((const bf16 *)c->w.fc_d, s.H, 2 * s.H, u, R, part, sp, (size_t)R * s.H, c->sm_count,
                                  status_d, st, c->tiled));
    SX_TRY(sx_launch_finish_norm(s, R, part, sp, (size_t)R * s.H, nullptr, (const bf16 *)c->w.norm1_d, nullptr, n, nullptr,
                          SxIndex{nullptr, 1, 0}, st));
    bool kv_only;
    SX_TRY(commit_kv_projection(c, s.H, n, R, part, &sp, &kv_only, status_d, st));
    const int N = kv_only ? 2 * s.nkv * s.d : (s.nq + 2 * s.nkv) * s.d;
    SxRowMap rm;
    memset(&rm, 0, sizeof(rm));
    rm.mode = SX_MODE_COMMIT; rm.round = 1; rm.topk = 1; rm.R = R; rm.cache_len = kv->cache_len_d;
    rm.valid_len = accept_len_out_d; rm.per_seq = M;
    SX_TRY(sx_launch_finish_qkv_rope(s, rm, part, sp, (size_t)R * N, nullptr, *kv, status_d, st, kv_only));
    c->launches += 4;
  }
  SX_TRY(sx_launch_commit_advance(B, accept_len_out_d, kv->cache_len_d, st));
  c->launches += 1;
  return SX_OK;
}

extern "C" sx_status sx_spec_exit_iter_host(sx_ctx *c, const sx_kv *kv, const sx_exit_cfg *cfg,
                                            const sx_exit_state *state, const void *feat0_h, const int32_t *tok0_h,
                                            const void *target_hidden_h, void *stage_feat0_d, int32_t *stage_tok0_d,
                                            void *stage_target_hidden_d, const sx_iter_out *o,
                                            int32_t *accept_len_out_h, int32_t *recover_tok_out_h, int32_t *exit_flag_h,
                                            float *smoothed_h, void *ws_d, size_t ws_bytes, int32_t *status_d,
                                            void *stream) {
  if (!c || !kv || !feat0_h || !tok0_h || !target_hidden_h || !stage_feat0_d || !stage_tok0_d ||
      !stage_target_hidden_d || !o || !accept_len_out_h || !recover_tok_out_h || !exit_flag_h || !smoothed_h)
    return SX_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)stream;
  const size_t B = kv->batch, H = c->sh.H;
  if (cudaMemcpyAsync(stage_feat0_d, feat0_h, B * H * 2 * (c->sh.arch == SX_ARCH_FUSED3 ? 3 : 1), cudaMemcpyHostToDevice, st) != cudaSuccess) return SX_ERR_CUDA;
  if (cudaMemcpyAsync(stage_tok0_d, tok0_h, B * 4, cudaMemcpyHostToDevice, st) != cudaSuccess) return SX_ERR_CUDA;
  if (cudaMemcpyAsync(stage_target_hidden_d, target_hidden_h, B * c->P * H * 2, cudaMemcpyHostToDevice, st) != cudaSuccess)
    return SX_ERR_CUDA;
  SX_TRY(sx_spec_exit_iter(c, kv, cfg, state, stage_feat0_d, stage_tok0_d, stage_target_hidden_d, o, ws_d, ws_bytes,
                           status_d, stream));
  if (cudaMemcpyAsync(accept_len_out_h, o->accept_len_out_d, B * 4, cudaMemcpyDeviceToHost, st) != cudaSuccess ||
      cudaMemcpyAsync(recover_tok_out_h, o->recover_tok_out_d, B * 4, cudaMemcpyDeviceToHost, st) != cudaSuccess ||
      cudaMemcpyAsync(exit_flag_h, o->exit_flag_d, B * 4, cudaMemcpyDeviceToHost, st) != cudaSuccess ||
      cudaMemcpyAsync(smoothed_h, o->smoothed_d, B * c->sh.S * 4, cudaMemcpyDeviceToHost, st) != cudaSuccess)
    return SX_ERR_CUDA;
  if (cudaStreamSynchronize(st) != cudaSuccess) return SX_ERR_CUDA;
  return SX_OK;
}
