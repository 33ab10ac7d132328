/*
 * specexit.h - C ABI of the speculative-exit step on one B200 (sm_100a).
 *
 * One iteration of signal-guided speculative decoding (the body of the loop of
 * Algorithm 1, without the target model's trunk):
 *
 *   draft K positions (chain) or a top-k tree with a one-layer draft model whose LM head
 *   carries three extra rows (Eq. 1: confidence, progress, remaining length)
 *     -> verify with the target LM head, greedy acceptance (Algorithm 1, "accept tokens,
 *        accept length, recover token")
 *     -> smooth the signals (Appendix A.1, EWMA) and threshold them at step-split tokens
 *        (Section 3.3, "Stopping Conditions"); on exit the accepted length is cut at the
 *        split token and the recover token becomes the stop-think token.
 *
 * Conventions for every entry point
 *   - Pointers named *_d are DEVICE pointers, 16-byte aligned, owned by the caller, and
 *     borrowed until the enqueued work has finished.  Everything else is host memory.
 *   - All work is enqueued on the given stream; no entry point allocates or frees device
 *     memory (sx_create / sx_destroy only touch host memory), and none synchronises except
 *     sx_spec_exit_iter_host, which waits for the stream before it returns (its results are
 *     host buffers) and sx_profile_end's event queries.
 *   - Weight buffers must be completely written and visible to the device (stream-ordered
 *     work that produced them finished: an event wait or a synchronisation) BEFORE a call
 *     that reads them is enqueued: the GEMM kernels request their first weight tiles while
 *     the preceding kernel of the stream is still running.
 *   - Host-detectable problems (NULL, unsupported shape, workspace too small) return a
 *     negative sx_status and launch nothing.  Problems only the device can see (a page
 *     table too short for a write, a token id outside the vocabulary, a bounded wait that
 *     ran out) are written to *status_d (the smallest code wins); kernels then skip the
 *     offending access and never trap.  *status_d must be zeroed by the caller before the
 *     first call and may be shared by several calls; outputs are unspecified when it is
 *     non-zero.
 *   - Matrices are bf16, row-major [out, in].  Activations handed between layers are
 *     bf16; accumulation, normalisation, softmax, rotary and signal math are fp32.
 *   - One sx_ctx per stream: a context is not thread-safe.
 *   - The device entry points (all but sx_spec_exit_iter_host and the profiling calls) only enqueue
 *     kernels, so a call - a whole sx_spec_exit_iter included - may be captured into a CUDA graph and
 *     replayed; the replay reads the captured buffers, whatever they hold then.  sx_set_sampling takes
 *     effect at enqueue time: a captured call keeps the temperature, seed and offset it was captured with.
 *   - With the environment variable SX_NVTX=1 the entry points open NVTX ranges ("sx spec exit iteration",
 *     "sx draft round k", "sx verify", "sx exit update", "sx commit") for timeline tools.
 */
#ifndef SPECEXIT_H
#define SPECEXIT_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef int32_t sx_status;
enum {
  SX_OK = 0,
  SX_ERR_INVALID_ARG = -1,
  SX_ERR_UNSUPPORTED = -2,
  SX_ERR_CAPACITY = -3,    /* page table too short / token id out of range (device) */
  SX_ERR_WORKSPACE = -4,
  SX_ERR_CUDA = -5,
  SX_ERR_TIMEOUT = -6,     /* a bounded device-side wait expired */
  SX_ERR_STATIC_LIMIT = -7 /* request larger than a fixed built-in buffer (sx_verify_noalloc) */
};

enum { SX_MODE_CHAIN = 0, SX_MODE_TREE = 1 };
enum { SX_ACT_SIGMOID = 0, SX_ACT_EXPM1 = 1, SX_ACT_IDENTITY = 2 };   /* Eq. 3-5 */
enum { SX_DIR_GT = 0, SX_DIR_LT = 1 };                                 /* Appendix A.1 thresholds */
enum { SX_EMA_VERIFIED_CONTEXT = 0, SX_EMA_FIRST_ONLY = 1 };
/* Appendix A.1 smoothing rules.  EWMA: x <- alpha s + (1 - alpha) x.  NONE: x = s.  WINDOW: mean of
 * the last N samples (of those that exist).  MOMENTUM: x_t = s_{t-1} + (s_{t-1} - s_{t-N}) / (N - 1),
 * the printed sum of differences telescoped, with as many differences as exist.  PARAGRAPH: mean
 * of the samples since the last step-split token. */
enum { SX_SMOOTH_EWMA = 0, SX_SMOOTH_NONE = 1, SX_SMOOTH_WINDOW = 2, SX_SMOOTH_MOMENTUM = 3, SX_SMOOTH_PARAGRAPH = 4 };
#define SX_HIST 16

#define SX_MAX_SIGNALS 3
#define SX_MAX_TOPK 8
#define SX_MAX_TREE_ROWS 64   /* drafted rows per sequence in one iteration (ancestor mask is 64 bit) */
#define SX_MAX_VERIFY_SLOTS 64

/* Shape of the draft model: concat(feature, embedding) -> fc 2H->H -> one pre-norm decoder
 * layer (RMSNorm, grouped-query attention with rotary positions over a paged KV cache,
 * SwiGLU) -> final RMSNorm -> extended head (Eq. 1). */
typedef struct {
  int32_t H, n_q_heads, n_kv_heads, head_dim, ffn, vocab;
  int32_t n_signals;                /* rows appended to the LM head, <= SX_MAX_SIGNALS */
  float rms_eps, rope_theta;
  int32_t page_size;                /* KV slots per page */
  int32_t act[SX_MAX_SIGNALS];      /* activation of each signal row */
  int32_t draft_vocab;              /* rows of the draft head's vocabulary part; 0 = vocab.  A reduced
                                       draft vocabulary (draft_vocab < vocab) scores draft ids
                                       0..draft_vocab-1, see sx_weights.draft_to_token_d */
  int32_t arch;                     /* SX_ARCH_CONCAT (0) or SX_ARCH_FUSED3, see below */
  int32_t tiled_weights;            /* 0: the GEMM weights are row-major [out, in]; 1: they were repacked with
                                       sx_tile_weight (fc, wqkv, wo, wgate_up, wdown, head, target_head; the
                                       embedding table and the gains stay as they are) */
} sx_model_cfg;

/* Shape of the draft layer.
 * SX_ARCH_CONCAT: every round mixes [previous hidden ; token embedding] (2H) through fc (2H -> H);
 *   the hidden handed from round to round (and returned) is the final-normed output.
 * SX_ARCH_FUSED3 (the EAGLE-3-shaped layer, the recipe the paper trains its draft with): round 1
 *   takes three target features per row (low / middle / high layer, [R, 3H]) fused by fc
 *   (3H -> H) into x; the attention input is [RMSNorm_e(embedding) ; RMSNorm_1(x)] (2H, so wqkv is
 *   [.., 2H]) and the residual stream starts from x; later rounds take the layer's own output y
 *   (before the final norm) as x, without fc.  The head reads RMSNorm_f(y).  Every hidden state
 *   this library returns or takes between rounds (hidden_out_d, iteration output hidden_d) is y.
 *   sx_commit takes the three target features of every verify slot ([batch, P, 3H]) as its
 *   target_hidden_d and returns a [batch, 3H] feat0_next_d. */
enum { SX_ARCH_CONCAT = 0, SX_ARCH_FUSED3 = 1 };

typedef struct {
  const void *embed_d;        /* [vocab, H] */
  const void *fc_d;           /* [H, 2H]: columns 0..H-1 take the feature, H..2H-1 the embedding */
  const void *norm1_d;        /* [H] gain before attention */
  const void *wqkv_d;         /* [(n_q + 2 n_kv) * head_dim, H]: q rows, then k rows, then v rows */
  const void *wo_d;           /* [H, n_q * head_dim] */
  const void *norm2_d;        /* [H] gain before the MLP */
  const void *wgate_up_d;     /* [2 * ffn, H]: gate rows, then up rows */
  const void *wdown_d;        /* [H, ffn] */
  const void *normf_d;        /* [H] final gain */
  const void *head_d;         /* [draft_vocab + n_signals, H]: Eq. 1, vocabulary rows first, signal rows last */
  const void *target_head_d;  /* [vocab, H] target LM head; may alias head_d when draft_vocab == vocab */
  const int32_t *draft_to_token_d; /* [draft_vocab] token id of each draft id, distinct, each in
                                      [0, vocab); NULL = identity (needs draft_vocab == vocab).
                                      Every drafted token that leaves the library (draft_tok,
                                      candidate ids) or feeds the embedding of the next round is
                                      the mapped id; ties break toward the lower draft id. */
  const void *norm_e_d;            /* [H] gain of the embedding's RMSNorm; SX_ARCH_FUSED3 only (with that
                                      layer fc_d is [H, 3H] and wqkv_d is [.., 2H], embedding half first) */
} sx_weights;

/* Paged KV cache of the draft layer.  Slot s of sequence b lives in physical page
 * page_table_d[b * max_pages + s / page_size] at offset s % page_size.  K is stored rotated. */
typedef struct {
  int32_t batch;
  int32_t *cache_len_d;         /* [batch] valid slots per sequence; read by every call, advanced only by
                                   sx_commit */
  const int32_t *page_table_d;  /* [batch, max_pages] */
  int32_t max_pages;
  int32_t num_pages;            /* physical pages in k_pages_d / v_pages_d */
  void *k_pages_d;              /* [num_pages, n_kv, page_size, head_dim] bf16 */
  void *v_pages_d;
} sx_kv;

typedef struct {
  int32_t mode;        /* SX_MODE_CHAIN | SX_MODE_TREE */
  int32_t K;           /* chain length, or tree depth */
  int32_t topk;        /* tree: children per expanded node (<= SX_MAX_TOPK); chain: 1 */
  int32_t max_nodes;   /* tree: nodes kept for verification, root excluded (< SX_MAX_VERIFY_SLOTS) */
  int32_t sample_drafts; /* 0 or 1: reserve workspace for sampled drafts (chain) / sampled children (tree), see
                            sx_set_sampling; needs the full draft vocabulary without an id map */
} sx_draft_cfg;

/* Exit rule.  Signal i passes when smoothed_i > thr[i] (SX_DIR_GT) or < thr[i] (SX_DIR_LT),
 * both strict; the enabled signals are AND-combined ("all the signals exceed a predefined
 * threshold", case study of the appendix). */
typedef struct {
  float alpha;                       /* EWMA factor: x <- alpha * s + (1 - alpha) * x */
  float thr[SX_MAX_SIGNALS];
  int32_t dir[SX_MAX_SIGNALS];
  uint32_t enable_mask;              /* bit i: signal i takes part */
  int32_t ema_positions;             /* which accepted slots feed the EWMA */
  const uint32_t *split_bitmap_d;    /* vocab bits, bit (t % 32) of word t / 32; NULL: every token splits */
  int32_t stop_think_token;
  int32_t smoothing;                 /* SX_SMOOTH_*: Appendix A.1, "Signal Smoothing" */
  int32_t window;                    /* N of the sliding-window and momentum rules, 2 <= N < SX_HIST */
} sx_exit_cfg;

/* Per-sequence state carried across iterations (device, caller-owned). */
typedef struct {
  float *x_d;            /* [batch, n_signals] smoothed signals */
  int32_t *n_updates_d;  /* [batch] samples folded in so far; 0 -> the next sample initialises x */
  int32_t *thinking_d;   /* [batch] 1 while inside the reasoning phase */
  float *hist_d;         /* [batch, SX_HIST, n_signals] ring of the latest samples (sample i at i % SX_HIST);
                            needed by SX_SMOOTH_WINDOW and SX_SMOOTH_MOMENTUM, else may be NULL */
  float *par_sum_d;      /* [batch, n_signals] sum over the current paragraph; SX_SMOOTH_PARAGRAPH, else NULL */
  int32_t *par_n_d;      /* [batch] samples in the current paragraph; SX_SMOOTH_PARAGRAPH, else NULL */
} sx_exit_state;

/* Outputs of one iteration; P = K + 1 (chain) or 1 + max_nodes (tree); rows = K (chain) or
 * 1 + topk * (K - 1) (tree).  Slot 0 is the last accepted token. */
typedef struct {
  int32_t *cand_tok_d;         /* [B, P] tokens laid out for verification */
  int32_t *parent_d;           /* [B, P] parent slot (-1 for slot 0); chain: j - 1 */
  int32_t *depth_d;            /* [B, P] */
  int32_t *slot_row_d;         /* [B, P] drafted row that took the slot's token as input, or -1 */
  int32_t *slot_src_row_d;     /* [B, P] drafted row whose head produced the slot's token, -1 for slot 0 */
  void *hidden_d;              /* [B, rows, H] bf16 final-normed hidden of every drafted row */
  float *slot_signal_d;        /* [B, P, n_signals]; NaN where the slot was never drafted from */
  int32_t *target_tok_d;       /* [B, P] target argmax per slot */
  int32_t *accept_len_d;       /* [B] accepted draft tokens before the exit rule */
  int32_t *path_d;             /* [B, K + 1] accepted slots in order, path[0] = 0, unused = -1 */
  int32_t *recover_tok_d;      /* [B] */
  int32_t *exit_flag_d;        /* [B] */
  int32_t *accept_len_out_d;   /* [B] after truncation at the split token */
  int32_t *recover_tok_out_d;  /* [B] stop_think_token where exit_flag = 1 */
  float *smoothed_d;           /* [B, n_signals] */
  /* optional (may be NULL), tree mode: every candidate generated, in generation order
   * (depth 1: ids [0, topk); depth r >= 2: topk + (r-2) topk^2 + j topk + t for the t-th child
   * of the j-th expanded row), NC = topk + (K - 1) topk^2 per sequence */
  int32_t *tree_cand_tok_d;    /* [B, NC] */
  float *tree_cand_score_d;    /* [B, NC] sum of log-probabilities along the path (fp32) */
  int32_t *tree_cand_row_d;    /* [B, NC] drafted row that expanded the candidate, or -1 */
} sx_iter_out;

typedef struct sx_ctx sx_ctx;

/* Build a host-side plan for the given shapes.  Weight pointers are recorded, not copied.
 * Fails with SX_ERR_UNSUPPORTED for shapes the kernels do not cover: H, ffn not multiples of 8;
 * head_dim other than 16, 32, 64 or 128; a group size (n_q_heads / n_kv_heads) other than 1, 2,
 * 4 or 8; group size * topk > 64; topk, rows or slots beyond the SX_MAX_* limits. */
sx_status sx_create(const sx_model_cfg *model, const sx_weights *weights, int32_t max_batch,
                    const sx_draft_cfg *draft, int32_t max_verify_rows, sx_ctx **out);
void sx_destroy(sx_ctx *ctx);
/* Bytes of scratch (device, 256-byte aligned) every compute call needs for this plan. */
size_t sx_workspace_bytes(const sx_ctx *ctx);
const char *sx_strerror(sx_status s);
/* Kernels launched by this context since it was created (host-side counter). */
int64_t sx_launch_count(const sx_ctx *ctx);

/* One draft round for R rows (Algorithm 1, "generate candidate tokens with M_d"; Eq. 1 and
 * Eq. 3-5 for the head).  Chain mode: round k = 1..K, R = batch, row b sits at position
 * cache_len[b] + k - 1 and sees the cache plus the k - 1 rows drafted before it.  Tree mode:
 * round 1 drafts the root (R = batch); round r >= 2 drafts R = batch * topk rows, row
 * b * topk + j at position cache_len[b] + r - 1, stored in slot cache_len[b] + 1 +
 * (r - 2) * topk + j, attending to the cache plus the drafted rows whose bit is set in
 * row_mask_d[row] (bit i = drafted row i of the same sequence; the own bit included).
 * The rows' K/V are written into the cache at those slots; cache_len is not advanced.
 *   feat_d        [R, H] bf16   hidden state of the previous position (SX_ARCH_FUSED3, round 1:
 *                               [R, 3H], the three target features)
 *   tok_d         [R]           token at this position
 *   row_mask_d    [R] or NULL   tree rounds >= 2 only
 *   hidden_out_d  [R, H] bf16   final-normed hidden (feeds the head and the next round);
 *                               SX_ARCH_FUSED3: the layer output before the final norm
 *   tok_out_d     [R, topk]     chain: argmax (topk = 1); tree: the topk best ids, best first,
 *                               lower id first among equal logits
 *   logp_out_d    [R, topk]     tree: log-probabilities of those ids; may be NULL in chain mode
 *   signals_out_d [R, n_signals] activated signal values */
sx_status sx_draft_step(sx_ctx *ctx, const sx_kv *kv, int32_t round, int32_t R, const void *feat_d,
                        const int32_t *tok_d, const uint64_t *row_mask_d, void *hidden_out_d,
                        int32_t *tok_out_d, float *logp_out_d, float *signals_out_d, void *ws_d,
                        size_t ws_bytes, int32_t *status_d, void *stream);

/* Target LM head with a fused argmax over batch * P given hidden states, then greedy
 * acceptance (Algorithm 1, "accept tokens t_acpt, accept length l_acpt, recover token t_rec").
 * Chain (parent_d = NULL): the longest prefix with cand[j] = target[j - 1].  Tree: walk from
 * slot 0 to the child whose token is the target's choice at the current slot.
 *   path_d [batch, path_stride] receives the accepted slots (path[0] = 0, rest -1). */
sx_status sx_verify(sx_ctx *ctx, int32_t batch, int32_t P, const void *target_hidden_d,
                    const int32_t *cand_tok_d, const int32_t *parent_d, int32_t *target_tok_d,
                    int32_t *accept_len_d, int32_t *path_d, int32_t path_stride,
                    int32_t *recover_tok_d, void *ws_d, size_t ws_bytes, int32_t *status_d,
                    void *stream);

/* Weight layout for the GEMM kernels (a deployment choice; the paper describes no kernels).  A
 * row-major [N, K] matrix is read in boxes of 128 rows x 64 columns, 128 pieces of 128 bytes that lie
 * K * 2 bytes apart; stored tile by tile - [ceil(N / 128)][ceil(K / 64)][128][64], zero padded - the
 * same box is one contiguous 16 KB block and the weight stream runs about 4 % faster.
 * sx_tiled_weight_bytes gives the size of that layout; sx_tile_weight repacks src_d ([N, K] bf16,
 * K a multiple of 8, 16-byte aligned) into dst_d (16-byte aligned, not overlapping src_d) on `stream`.
 * A context created with sx_model_cfg.tiled_weights = 1 expects every GEMM weight in that layout. */
size_t sx_tiled_weight_bytes(int32_t N, int32_t K);
sx_status sx_tile_weight(const void *src_d, int32_t N, int32_t K, void *dst_d, void *stream);

/* Choice of the decode-attention kernel (a deployment choice; the paper describes no kernels).  Two kernels
 * compute the same attention over the paged cache: SX_ATTN_SPLIT cuts the keys into chunks, one warp per
 * (sequence, KV head, 8 queries, chunk), on the warp-level tensor-core path; SX_ATTN_TC streams 128-key
 * blocks through tcgen05 tensor memory, which is faster on long caches but needs head_dim = 128, a page
 * size that is a multiple of 64 and at most 32 queries per (sequence, KV head) (group size * rows drafted
 * per sequence in the round).  SX_ATTN_AUTO (the state of a new context) takes SX_ATTN_TC where it is
 * supported, the round has more than four queries per (sequence, KV head) and the cache capacity is at least
 * four 128-key blocks per SM, else SX_ATTN_SPLIT.  Forcing
 * SX_ATTN_TC makes a draft call return SX_ERR_UNSUPPORTED where the shape does not allow it.  Host-side
 * state, read when a call is issued. */
enum { SX_ATTN_AUTO = 0, SX_ATTN_SPLIT = 1, SX_ATTN_TC = 2 };
sx_status sx_set_attention(sx_ctx *ctx, int32_t kernel);

/* Stochastic acceptance: speculative sampling, the acceptance rule of the speculative-decoding
 * scheme the method builds on (Section 2, background on speculative decoding; Algorithm 1,
 * "accept tokens").  A draft token x is kept with probability min(1, p(x) / q(x)), else a token is
 * drawn from the normalised max(0, p - q); p is the target's softmax at `temperature`.  The drafts
 * of this library are deterministic (q is a point mass), so the rule is realised exactly by
 * drawing one token t ~ p per verify slot and keeping a draft token where it equals t: the
 * sx_verify and sx_spec_exit_iter calls that follow return that draw in target_tok_d and walk it
 * as they walk the greedy choice (chain and tree alike; the recover token is the draw at the
 * last accepted slot).  The draw is t = argmax_i (logit_i + temperature * g_i) with g_i =
 * -ln(-ln(u_i)), u_i = (k + 1/2) / 2^23 for k the top 23 bits of word (i mod 4) of the
 * Philox4x32-10 block with counter (i div 4, slot, sequence, offset) and key (seed mod 2^32,
 * seed div 2^32).  Give every iteration its own offset.  temperature = 0 (the state of a new
 * context) is greedy verification.  Host-side state, read when a call is issued; returns
 * SX_ERR_INVALID_ARG for a negative or non-finite temperature.
 *
 * Sampled drafts.  In a context created with sx_draft_cfg.sample_drafts = 1 (chain mode, full
 * draft vocabulary without an id map) a positive temperature makes sx_spec_exit_iter apply the
 * rule in its general form: draft token k of a sequence is drawn from q = softmax(draft logits /
 * temperature) (a Gumbel-max draw with slot word 0x40000000 + k - 1); at verify slot j the token
 * x proposed there is kept when u_j < min(1, p(x) / q(x)), u_j from word 0 of the block with
 * counter (0, 0x20000000 + j, sequence, offset); otherwise the slot's token is a Gumbel-max draw
 * over log max(0, p - q) with the noise of slot j; the last slot, which has no draft, draws from
 * p.  target_tok_d then holds the kept or drawn token of every slot, and acceptance walks it as
 * before.  For this the draft and target logits of the iteration are written to the workspace
 * (fp32, (batch * K + batch * (K + 1)) * vocab values) and three small kernels evaluate the rule.  The standalone sx_draft_step / sx_verify calls keep deterministic drafts.
 *
 * Sampled children.  In a TREE context created with sample_drafts = 1 a positive temperature makes
 * sx_spec_exit_iter draw the children of every drafted row instead of taking its top-k: the topk largest of
 * logit_i + temperature * g_i, best first, with the noise stream of slot word 0x50000000 + r for drafted row
 * r - a draw of topk tokens without replacement, in order, from q = softmax(draft logits / temperature).
 * Scores (for expansion and for the kept set) stay sums of log-probabilities.  Verification walks from slot 0:
 * with p the target's softmax at the current slot and q that of the row which produced the slot's children,
 * the kept children are tried in slot order; token x of child slot s is accepted when u_s < min(1, p(x) /
 * q(x)) (u_s as above, slot word 0x20000000 + s), a refusal replaces p by the normalised max(0, p - q) and
 * takes x out of q; when none is accepted the slot's token is drawn from what is left of p (Gumbel-max with
 * the noise of that slot) and becomes the recover token.  target_tok_d then holds, at every visited slot,
 * the accepted child's token or that draw, and -1 elsewhere; the iteration's out->slot_row_d must be given.
 * The token emitted at a slot follows the target's distribution exactly when no child drawn at that slot
 * was pruned from the tree (max_nodes = all candidates); a pruned child is simply not tried.  The logits of
 * every drafted row and verify slot are written to the workspace (fp32, batch * (rows + P) * vocab values). */
sx_status sx_set_sampling(sx_ctx *ctx, float temperature, uint64_t seed, uint32_t offset);

/* Exit decision (Section 3.3; Appendix A.1).  Walks path slots 0..accept_len; each slot that
 * carries a signal updates the EWMA (all of them, or only the first, per ema_positions); the
 * first slot whose token is a step-split token while the smoothed signals pass ends the
 * reasoning phase.  Sequences with thinking = 0 are passed through unchanged. */
sx_status sx_exit_update(sx_ctx *ctx, int32_t batch, int32_t P, const sx_exit_cfg *cfg,
                         const sx_exit_state *state, const float *slot_signal_d,
                         const int32_t *cand_tok_d, const int32_t *path_d, int32_t path_stride,
                         const int32_t *accept_len_d, const int32_t *recover_tok_d,
                         int32_t *exit_flag_d, int32_t *accept_len_out_d,
                         int32_t *recover_tok_out_d, float *smoothed_out_d, int32_t *status_d,
                         void *stream);

/* The whole iteration in one enqueue: all draft rounds, (tree) candidate selection and
 * layout, verification and the exit decision.  target_hidden_d [B, P, H] stands in for the
 * target trunk's output at the verify slots; it is read only after the draft has finished.
 * feat0_d is [B, H] bf16, the target feature of the last accepted token ([B, 3H] with
 * SX_ARCH_FUSED3); tok0_d [B] is that token. */
sx_status sx_spec_exit_iter(sx_ctx *ctx, const sx_kv *kv, const sx_exit_cfg *cfg,
                            const sx_exit_state *state, const void *feat0_d, const int32_t *tok0_d,
                            const void *target_hidden_d, const sx_iter_out *out, void *ws_d,
                            size_t ws_bytes, int32_t *status_d, void *stream);

/* End of an iteration: Algorithm 1, "Update KV-cache and hidden states accordingly".  Makes the
 * verified tokens part of the draft model's cached context and names the next iteration's
 * first draft row.  For sequence b with n = cache_len[b] and L = accept_len_out_d[b] (the
 * accepted length after the exit rule):
 *   - slot n (the last accepted token of the previous iteration, keyed in draft round 1 from
 *     its true feature) is kept;
 *   - the token of path slot j (j = 1..L) is re-keyed from the TARGET's hidden state of path
 *     slot j - 1, the state that predicted it: its K/V, at position n + j, overwrite the
 *     drafted ones (the drafted K/V came from draft hidden states); drafted rows that were
 *     not accepted are dropped;
 *   - cache_len[b] becomes n + L + 1 (kv->cache_len_d is WRITTEN by this call);
 *   - feat0_next_d[b] = target hidden of path slot L, tok0_next_d[b] = recover_tok_out_d[b].
 * path_d [batch, path_stride] as produced by sx_verify, path_stride - 1 <= K of the plan.  The
 * page table must cover cache_len + path_stride slots.  Work after this call sees the new
 * lengths (the call ends with a kernel that later launches cannot overtake). */
sx_status sx_commit(sx_ctx *ctx, const sx_kv *kv, int32_t P, const void *target_hidden_d,
                    const int32_t *cand_tok_d, const int32_t *path_d, int32_t path_stride,
                    const int32_t *accept_len_out_d, const int32_t *recover_tok_out_d,
                    void *feat0_next_d, int32_t *tok0_next_d, void *ws_d, size_t ws_bytes,
                    int32_t *status_d, void *stream);

/* Same iteration with HOST buffers for the per-iteration inputs (feature, token, target
 * hiddens) and the per-iteration results (accepted length, recover token, exit flag, smoothed
 * signals): copies them in, runs sx_spec_exit_iter, copies the results out and synchronises
 * the stream.  Staging buffers are the device arrays in `out` and `stage_*_d`. */
sx_status sx_spec_exit_iter_host(sx_ctx *ctx, const sx_kv *kv, const sx_exit_cfg *cfg,
                                 const sx_exit_state *state, const void *feat0_h,
                                 const int32_t *tok0_h, const void *target_hidden_h,
                                 void *stage_feat0_d, int32_t *stage_tok0_d,
                                 void *stage_target_hidden_d, const sx_iter_out *out,
                                 int32_t *accept_len_out_h, int32_t *recover_tok_out_h,
                                 int32_t *exit_flag_h, float *smoothed_h, void *ws_d,
                                 size_t ws_bytes, int32_t *status_d, void *stream);

/* Per-kernel-class device timing for the benchmark (the paper has no counterpart).  Between
 * begin and end every launch of the classes below is bracketed by CUDA events on its stream;
 * sx_profile_end - to be called after the caller has synchronised the stream - returns the
 * summed milliseconds and the number of launches per class and stops recording. */
enum {
  SX_PROF_HEAD_DRAFT = 0, SX_PROF_HEAD_VERIFY = 1, SX_PROF_GEMM_FC = 2, SX_PROF_GEMM_QKV = 3,
  SX_PROF_GEMM_O = 4, SX_PROF_GEMM_GATE_UP = 5, SX_PROF_GEMM_DOWN = 6, SX_PROF_ATTENTION = 7,
  SX_PROF_CLASSES = 8
};
sx_status sx_profile_begin(sx_ctx *ctx);
sx_status sx_profile_end(sx_ctx *ctx, float *ms_out, int32_t *count_out);

/* Diagnostic (the paper has no counterpart).  Every wait of the GEMM kernels on a shared-memory barrier is
 * bounded: after `wait_limit` polls the waiting role raises an abort flag, the CTA's other roles leave
 * at their next poll, SX_ERR_TIMEOUT goes to the status word, copies in flight are given time to land,
 * the CTA frees its tensor memory and returns - the context stays usable.  This call runs that path on
 * its own: `ctas` CTAs (1..1024) with the GEMM kernel's thread layout allocate tensor memory and wait, with
 * `limit` polls (1..2^20), on barriers nothing arrives at; no copy is issued.  Afterwards *status_d is
 * SX_ERR_TIMEOUT, reached_d[0] == 0 (no wait reported success) and reached_d[1] == ctas (every CTA
 * returned through the tear-down).  reached_d: two int32 on the device, zeroed by the caller. */
sx_status sx_selftest_bounded_wait(uint32_t limit, int32_t ctas, int32_t *status_d, int32_t *reached_d,
                                   void *stream);

/* Verification for callers that cannot allocate device memory (the paper has no counterpart;
 * this is a deployment convenience).  Some hosts of this library hold no allocator at the point
 * where a draft is verified: an inference server whose memory pool owns the whole device and
 * hands out fixed buffers only, a plugin called inside a latency-critical section where
 * cudaMalloc (which may synchronise the device) is off limits, or a process that runs under a
 * hard memory quota fixed at start-up.  Such a caller has nowhere to put the workspace that
 * sx_verify wants.  sx_verify_noalloc computes exactly what sx_verify computes - target LM head
 * with fused argmax over batch * P hidden states, then greedy acceptance - but needs neither a
 * context nor a workspace: the head kernel's per-CTA partial results live in a fixed array inside
 * the library image (SX_NOALLOC_SCRATCH_BYTES, about 0.7 MB, held by every GPU that loads the
 * library until the process exits).  The call allocates and frees no device memory.
 *   - Limit: batch * P <= SX_NOALLOC_MAX_ROWS; beyond it the call returns SX_ERR_STATIC_LIMIT and
 *     launches nothing.  Tree mode (parent_d != NULL) also needs P <= SX_MAX_VERIFY_SLOTS.
 *   - target_head_d is the [vocab, H] bf16 head, ROW-MAJOR as handed in (not a matrix repacked with
 *     sx_tile_weight: there is no context here to say so, and a tiled head would be misread); the other
 *     arguments are those of sx_verify.
 *   - The first call on a device resolves the array's device address and sets kernel attributes
 *     for that device (which must be current); make that first call outside any stream capture.
 *   - All calls on a device share the array and it keeps the previous call's contents.  Nothing
 *     in it needs clearing (every slice that is read was written by the same call), but two
 *     calls that overlap on one GPU - different streams or threads - race on it: keep them on
 *     one stream or order them yourself. */
#define SX_NOALLOC_MAX_ROWS 64
#define SX_NOALLOC_SCRATCH_BYTES (160 * SX_NOALLOC_MAX_ROWS * (8 * SX_MAX_TOPK + 8))
sx_status sx_verify_noalloc(const void *target_head_d, int32_t vocab, int32_t H, int32_t batch,
                            int32_t P, const void *target_hidden_d, const int32_t *cand_tok_d,
                            const int32_t *parent_d, int32_t *target_tok_d, int32_t *accept_len_d,
                            int32_t *path_d, int32_t path_stride, int32_t *recover_tok_d,
                            int32_t *status_d, void *stream);

#ifdef __cplusplus
}
#endif
#endif /* SPECEXIT_H */
