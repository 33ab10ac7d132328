// Launch wrappers of the non-GEMM kernels (defined in sx_kernels.cu) and of the GEMMs
// (sx_gemm_tc.cu) and of the attention (sx_attention.cu).  Host-side only.
#pragma once
#include "sx_common.cuh"

// affine-or-indirect row addressing: index(r) = idx ? idx[r] : r * mul + add
struct SxIndex {
  const int32_t *idx;
  int mul, add;
};

#define SX_MAX_H 16384           // widest hidden state the row kernels hold in shared memory
#define SX_TRY(e) do { sx_status _s = (e); if (_s != SX_OK) return _s; } while (0)
static inline sx_status sx_rc(cudaError_t e) { return e == cudaSuccess ? SX_OK : SX_ERR_CUDA; }
sx_status sx_kernels_init(int device);

struct SxShape {
  int H, nq, nkv, d, F, V, S, page;
  int arch;                    // SX_ARCH_CONCAT | SX_ARCH_FUSED3
  int Vd;                      // vocabulary rows of the draft head (== V without a reduced draft vocabulary)
  float eps, theta;
  int act[SX_MAX_SIGNALS];
};

sx_status sx_launch_embed_concat(const SxShape &sh, int R, const bf16 *feat, SxIndex fi, const int32_t *tok,
                            SxIndex ti, const bf16 *embed, bf16 *u, int32_t *status, cudaStream_t st);

// v = sum_s part[s][r][:] (+ residual); out_v = bf16(v); out_n = bf16(rmsnorm(out_v) * gamma);
// out_user (optional) receives out_n at row index ui(r).
sx_status sx_launch_finish_norm(const SxShape &sh, int R, const float *part, int splits, size_t split_stride,
                           const bf16 *residual, const bf16 *gamma, bf16 *out_v, bf16 *out_n,
                           bf16 *out_user, SxIndex ui, cudaStream_t st, int user_gets_v = 0);

// Layer with three-feature fusion: x_out[r] = bf16(sum of the fc partials) (part != nullptr) or the
// hidden of row fi(r) of `feat`; u[r] = [rmsnorm(E[token]) * gamma_e ; rmsnorm(x) * gamma_h].
sx_status sx_launch_fused_input(const SxShape &sh, int R, const float *part, int splits, size_t split_stride,
                           const bf16 *feat, SxIndex fi, const int32_t *tok, SxIndex ti, const bf16 *embed,
                           const bf16 *gamma_e, const bf16 *gamma_h, bf16 *x_out, bf16 *u, int32_t *status,
                           cudaStream_t st);

sx_status sx_launch_finish_qkv_rope(const SxShape &sh, const SxRowMap &rm, const float *part, int splits,
                               size_t split_stride, bf16 *q_out, const sx_kv &kv, int32_t *status,
                               cudaStream_t st, bool kv_only_partials = false);

sx_status sx_launch_commit_gather(const SxShape &sh, int B, int M, int P, const bf16 *th, const int32_t *cand,
                             const int32_t *path, int path_stride, const int32_t *accept_len,
                             const int32_t *recover, const bf16 *embed, bf16 *u, bf16 *feat0, int32_t *tok0,
                             int32_t *status, cudaStream_t st, int32_t *tok_rows = nullptr);
sx_status sx_launch_commit_advance(int B, const int32_t *accept_len, int32_t *cache_len, cudaStream_t st);

sx_status sx_launch_finish_swiglu(const SxShape &sh, int R, const float *part, int splits,
                             size_t split_stride, bf16 *m_out, cudaStream_t st);

// decode attention (sx_attention.cu).  B sequences with nr rows each this round, E drafted slots
// behind the cached prefix (this round's rows included).
bool sx_attn_supported(const SxShape &sh);
sx_status sx_attn_init(int device);
int sx_attn_splits(const SxShape &sh, int B, int nr, int n_cap, int sm_count);
size_t sx_attn_ws_bytes(const SxShape &sh, int max_batch, int max_nr, int sm_count);
sx_status sx_launch_attention(const SxShape &sh, const SxRowMap &rm, int B, int nr, int E, const bf16 *q,
                         const sx_kv &kv, int nsplit, float *ws, bf16 *o_out, int sm_count, int32_t *status, cudaStream_t st);

// The same attention on tcgen05 (sx_attention_tc.cu): head dimension 128, pages of a multiple of 64 slots,
// at most 32 queries per (sequence, KV head).
bool sx_attn_tc_supported(const SxShape &sh, int nr, const sx_kv &kv);
sx_status sx_attn_tc_init(int device);
size_t sx_attn_tc_ws_bytes(const SxShape &sh, int max_batch, int sm_count);
sx_status sx_launch_attention_tc(const SxShape &sh, const SxRowMap &rm, int B, int nr, int E, const bf16 *q,
                                 const sx_kv &kv, float *ws, bf16 *o_out, int sm_count, int32_t *status,
                                 cudaStream_t st);

// Optional fusion for chain drafting: the merge kernel also writes the next round's input row
// u[r] = [feat[r] ; embed[token chosen for row r]] (u == nullptr: off).
struct SxNextInput {
  const bf16 *feat, *embed;
  bf16 *u;
  int H, V;
};
sx_status sx_launch_head_finalize(const SxShape &sh, int R, const SxHeadPartial *parts, int G, int part_stride,
                             int T, int lse, const float *z, int S, int32_t *tok_out, SxIndex toi,
                             float *logp_out, float *sig_out, SxIndex si, cudaStream_t st,
                             SxNextInput nx = SxNextInput{nullptr, nullptr, nullptr, 0, 0},
                             const int32_t *map = nullptr, int Vd = 0);   // map: draft id -> token id

sx_status sx_launch_chain_layout(int B, int K, int S, const int32_t *tok0, const sx_iter_out &o, cudaStream_t st);

sx_status sx_launch_accept(int B, int P, const int32_t *cand, const int32_t *parent, const int32_t *target,
                      int32_t *accept_len, int32_t *path, int path_stride, int32_t *recover, cudaStream_t st);

sx_status sx_launch_exit(int B, int P, int S, const sx_exit_cfg &cfg, const sx_exit_state &state,
                    const float *slot_signal, const int32_t *cand, const int32_t *path, int path_stride,
                    const int32_t *accept_len, const int32_t *recover, int32_t *exit_flag,
                    int32_t *accept_out, int32_t *recover_out, float *smoothed, int V, int32_t *status,
                    cudaStream_t st);

// tree bookkeeping state (device, in the workspace), per sequence
struct SxTree {
  int T, D, rows, NC, max_nodes;
  int32_t *cand_tok, *cand_parent, *cand_src_row, *cand_row;   // [B, NC]
  float *cand_score;                                           // [B, NC]
  uint64_t *row_mask;                                          // [B, rows]
  int32_t *sel_cid;                                            // [B, T]
  int32_t *sel_tok;                                            // [B*T] next round's input tokens
  int32_t *feat_idx, *hid_idx;                                 // [B*T] next round's row addressing
  uint64_t *next_mask;                                         // [B*T]
  float *row_sig;                                              // [B, rows, S]
};
sx_status sx_launch_tree_expand(const SxTree &t, int B, int round, const int32_t *tok_rt, const float *logp_rt,
                           cudaStream_t st);
sx_status sx_launch_tree_layout(const SxTree &t, int B, int S, const int32_t *tok0, const sx_iter_out &o,
                           cudaStream_t st);

// ---- GEMMs (sx_gemm_tc.cu) ----------------------------------------------------------------
// part[s][r][n] = sum over the s-th K range of X[r][k] * W[n][k]   (fp32)
#define SX_GEMM_MAX_SPLITS 4      // sx_gemm_pick_splits never returns more
int sx_gemm_pick_splits(int N, int K, int sm_count);
sx_status sx_launch_gemm_partial(const bf16 *W, int N, int K, const bf16 *X, int R, float *part,
                                 int splits, size_t split_stride, int sm_count, int32_t *status,
                                 cudaStream_t st, bool tiled = false);
// weights tile by tile ([row tile][k-block][128][64], zero padded): elements of that layout, and the repack
size_t sx_tiled_elems(int N, int K);
sx_status sx_launch_tile_weight(const bf16 *src, int N, int K, bf16 *dst, cudaStream_t st);
sx_status sx_gemm_init(int device);
// cached 2-D tensor map of a bf16 matrix [rows, cols], box = box_rows x 64 columns, 128-byte swizzle
struct CUtensorMap_st;
bool sx_tma_map_2d(const void *ptr, long long rows, int cols, int box_rows, CUtensorMap_st *out);
// give-up path of the bounded mbarrier waits on its own (see sx_selftest_bounded_wait)
sx_status sx_launch_wait_selftest(uint32_t limit, int ctas, int32_t *status, int32_t *reached, cudaStream_t st);
// Sampled verification: with temp > 0 the plain-argmax head returns, per row, the arg max of
// logit + temp * Gumbel noise, i.e. a draw from softmax(logits / temp).  Row r of the launch is
// verify slot (row0 + r) % P of sequence (row0 + r) / P; the noise of (sequence, slot, token id)
// comes from Philox4x32-10 with key (k0, k1) and `offset` as the last counter word.
struct SxSample {
  float temp;
  uint32_t k0, k1, offset;
  int P, row0;
  uint32_t slot_base;            // added to the slot word (separates the draft stream from the verify stream)
};
// Optional copy of the head's logits: row r of the launch goes to out[ri(r) * ld + 0 .. V) (fp32).
struct SxLogitsOut {
  float *out;
  size_t ld;
  SxIndex ri;
};
// head: per-CTA partial results out[cta][row]; returns the number of CTAs used in *G
sx_status sx_launch_head(const bf16 *W, int Ntot, int V, int K, const bf16 *X, int R, int T, int lse,
                         SxHeadPartial *parts, int part_stride, int *G, float *z, int S, int sm_count,
                         int32_t *status, cudaStream_t st, const SxSample *smp = nullptr,
                         SxLogitsOut lo = SxLogitsOut{nullptr, 0, SxIndex{nullptr, 1, 0}}, bool tiled = false);

// Speculative sampling with sampled drafts: writes the kept draft token or the residual draw of every
// verify slot to target_tok [B, P].  target_logits [B * P, V], draft_logits [B, K, V] (K = P - 1), both
// fp32.  Three small launches (partition sums per slice, accept test + best residual score per slice,
// pick); parts_ws holds sx_spec_sample_ws_bytes(B * P) bytes.
#define SX_SPEC_MAX_SLICES 64
size_t sx_spec_sample_ws_bytes(int rows);
sx_status sx_launch_spec_sample(int B, int P, int V, const float *target_logits, const float *draft_logits,
                           const int32_t *cand_tok, SxSample smp, void *parts_ws, int sm_count, int32_t *target_tok,
                           int32_t *status, cudaStream_t st);
int sx_head_max_rows(int T, int lse);

// Sampled children in a tree: the T best of logit + temp * Gumbel noise per drafted row (rows of `logits` are
// addressed through li), and the speculative walk over the laid-out tree (pq_ws: sx_tree_spec_ws_bytes).
// parts: scratch for `cap` partial results (the head launch's per-CTA results are no longer needed by then).
sx_status sx_launch_gumbel_topk(int R, int V, int T, const float *logits, size_t ld, SxIndex li, SxSample smp,
                                SxHeadPartial *parts, size_t cap, int sm_count, int32_t *tok_out, float *logp_out,
                                cudaStream_t st);
size_t sx_tree_spec_ws_bytes(int B, int V);
sx_status sx_launch_tree_spec_walk(int B, int P, int V, int rows, int path_stride, const float *target_logits,
                                   const float *draft_logits, const int32_t *cand_tok, const int32_t *parent,
                                   const int32_t *slot_row, SxSample smp, void *pq_ws, int32_t *target_tok,
                                   int32_t *accept_len, int32_t *path, int32_t *recover, int32_t *status,
                                   cudaStream_t st);
