// Non-GEMM kernels of the speculative-exit step: input staging, split-K finishers fused with
// RMSNorm / rotary + KV append / SwiGLU, split-K decode attention over the paged cache, the
// head merge, greedy acceptance, the exit rule and the draft-tree bookkeeping.
#include <math.h>

#include "sx_kernels.cuh"
#include "sx_launch.cuh"

__device__ __forceinline__ int sx_index(const SxIndex &x, int r) { return x.idx ? x.idx[r] : r * x.mul + x.add; }

// ---------------------------------------------------------------------------------------
// u[r] = [ feature(r) ; E[token(r)] ]   (feature first: fc columns 0..H-1 take the feature)
// ---------------------------------------------------------------------------------------
__global__ void sx_embed_concat_kernel(int H, int V, const bf16 *feat, SxIndex fi, const int32_t *tok,
                                       SxIndex ti, const bf16 *embed, bf16 *u, int32_t *status) {
  sx_pdl_launch_dependents();
  sx_pdl_wait();
  const int r = blockIdx.x;
  int t = tok[sx_index(ti, r)];
  if (t < 0 || t >= V) {
    if (threadIdx.x == 0) sx_set_status(status, SX_ERR_CAPACITY);
    t = 0;
  }
  const uint4 *f = reinterpret_cast<const uint4 *>(feat + (size_t)sx_index(fi, r) * H);
  const uint4 *e = reinterpret_cast<const uint4 *>(embed + (size_t)t * H);
  uint4 *o = reinterpret_cast<uint4 *>(u + (size_t)r * 2 * H);
  const int n = H / 8;
  for (int i = threadIdx.x; i < n; i += blockDim.x) {
    const uint4 a = f[i], b = e[i];
    o[i] = a;
    o[n + i] = b;
  }
}

sx_status sx_launch_embed_concat(const SxShape &sh, int R, const bf16 *feat, SxIndex fi, const int32_t *tok,
                            SxIndex ti, const bf16 *embed, bf16 *u, int32_t *status, cudaStream_t st) {
  int threads = ((sh.H / 8 + 31) / 32) * 32;
  if (threads > 512) threads = 512;
  return sx_rc(sx_launch(sx_embed_concat_kernel, dim3(R), dim3(threads), 0, st, sh.H, sh.V, feat, fi, tok, ti, embed, u, status));
}

// ---------------------------------------------------------------------------------------
// split-K finisher + RMSNorm.  One CTA per row; a thread owns 4 consecutive elements per pass
// and issues the loads of all splits before it adds them (in split order).
// ---------------------------------------------------------------------------------------
// sum over the splits, in split order, of 4 consecutive floats; loads go out four splits at a time
__device__ __forceinline__ float4 sx_sum_splits4(const float *p, int splits, size_t split_stride) {
  float4 a = make_float4(0.f, 0.f, 0.f, 0.f);
  for (int s0 = 0; s0 < splits; s0 += 4) {
    float4 v[4];
#pragma unroll
    for (int s = 0; s < 4; ++s)
      if (s0 + s < splits) v[s] = *reinterpret_cast<const float4 *>(p + (size_t)(s0 + s) * split_stride);
#pragma unroll
    for (int s = 0; s < 4; ++s)
      if (s0 + s < splits) { a.x += v[s].x; a.y += v[s].y; a.z += v[s].z; a.w += v[s].w; }
  }
  return a;
}

__global__ void __launch_bounds__(1024)
sx_finish_norm_kernel(int H, float eps, const float *part, int splits, size_t split_stride,
                      const bf16 *residual, const bf16 *gamma, bf16 *out_v, bf16 *out_n,
                      bf16 *out_user, SxIndex ui, int user_gets_v) {
  extern __shared__ float sx_buf[];        // [H] values, then [H / 2] words of gain (bf16 pairs)
  __shared__ float red[32];
  uint2 *gam = reinterpret_cast<uint2 *>(sx_buf + H);
  sx_pdl_launch_dependents();
  // the gain is a weight: fetch it (from HBM) before waiting for the GEMM
  for (int i = threadIdx.x; i < H / 4; i += blockDim.x) gam[i] = reinterpret_cast<const uint2 *>(gamma)[i];
  sx_pdl_wait();
  const int r = blockIdx.x;
  float ss = 0.f;
  bf16 *user = out_user ? out_user + (size_t)sx_index(ui, r) * H : nullptr;
  for (int i = threadIdx.x * 4; i < H; i += blockDim.x * 4) {
    float4 v = sx_sum_splits4(part + (size_t)r * H + i, splits, split_stride);
    if (residual) {
      const uint2 ru = *reinterpret_cast<const uint2 *>(residual + (size_t)r * H + i);
      const float2 r0 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&ru.x));
      const float2 r1 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&ru.y));
      v.x += r0.x; v.y += r0.y; v.z += r1.x; v.w += r1.y;
    }
    __nv_bfloat162 b0 = __floats2bfloat162_rn(v.x, v.y), b1 = __floats2bfloat162_rn(v.z, v.w);
    if (out_v || (user && user_gets_v)) {
      uint2 w;
      w.x = *reinterpret_cast<uint32_t *>(&b0);
      w.y = *reinterpret_cast<uint32_t *>(&b1);
      if (out_v) *reinterpret_cast<uint2 *>(out_v + (size_t)r * H + i) = w;
      if (user && user_gets_v) *reinterpret_cast<uint2 *>(user + i) = w;
    }
    const float2 f0 = __bfloat1622float2(b0), f1 = __bfloat1622float2(b1);
    *reinterpret_cast<float4 *>(sx_buf + i) = make_float4(f0.x, f0.y, f1.x, f1.y);
    ss += (f0.x * f0.x + f0.y * f0.y) + (f1.x * f1.x + f1.y * f1.y);
  }
  ss = sx_warp_sum(ss);
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = ss;
  __syncthreads();
  float tot = 0.f;
  {
    const int nw = blockDim.x >> 5;
    for (int w = 0; w < nw; ++w) tot += red[w];           // same order in every thread
  }
  const float scale = rsqrtf(tot / (float)H + eps);
  if (user_gets_v) user = nullptr;
  for (int i = threadIdx.x * 4; i < H; i += blockDim.x * 4) {
    const float4 v = *reinterpret_cast<const float4 *>(sx_buf + i);
    const uint2 gu = gam[i >> 2];
    const float2 g0 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&gu.x));
    const float2 g1 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&gu.y));
    __nv_bfloat162 b0 = __floats2bfloat162_rn(v.x * scale * g0.x, v.y * scale * g0.y);
    __nv_bfloat162 b1 = __floats2bfloat162_rn(v.z * scale * g1.x, v.w * scale * g1.y);
    uint2 w;
    w.x = *reinterpret_cast<uint32_t *>(&b0);
    w.y = *reinterpret_cast<uint32_t *>(&b1);
    if (out_n) *reinterpret_cast<uint2 *>(out_n + (size_t)r * H + i) = w;
    if (user) *reinterpret_cast<uint2 *>(user + i) = w;
  }
}

sx_status sx_launch_finish_norm(const SxShape &sh, int R, const float *part, int splits, size_t split_stride,
                           const bf16 *residual, const bf16 *gamma, bf16 *out_v, bf16 *out_n,
                           bf16 *out_user, SxIndex ui, cudaStream_t st, int user_gets_v) {
  int threads = ((sh.H / 4 + 31) / 32) * 32;
  if (threads > 1024) threads = 1024;
  return sx_rc(sx_launch(sx_finish_norm_kernel, dim3(R), dim3(threads), sh.H * (sizeof(float) + sizeof(bf16)), st, sh.H, sh.eps, part,
            splits, split_stride, residual, gamma, out_v, out_n, out_user, ui, user_gets_v));
}

// ---------------------------------------------------------------------------------------
// Input of the layer with three-feature fusion: x = the fused feature (split-K sum of the fc
// GEMM, round 1) or the hidden state of the source row (later rounds); the attention input is
// u[r] = [ RMSNorm_e(E[token]) ; RMSNorm_1(x) ], the residual stream starts from x.
// One CTA per row; a thread owns 4 consecutive elements per pass.
// ---------------------------------------------------------------------------------------
__global__ void __launch_bounds__(1024)
sx_fused_input_kernel(int H, int V, float eps, const float *part, int splits, size_t split_stride, const bf16 *feat,
                      SxIndex fi, const int32_t *tok, SxIndex ti, const bf16 *embed, const bf16 *gamma_e,
                      const bf16 *gamma_h, bf16 *x_out, bf16 *u, int32_t *status) {
  extern __shared__ float sx_buf[];        // [H] x, [H] embedding
  __shared__ float red[2][32];
  sx_pdl_launch_dependents();
  sx_pdl_wait();
  const int r = blockIdx.x;
  int t = tok[sx_index(ti, r)];
  if (t < 0 || t >= V) {
    if (threadIdx.x == 0) sx_set_status(status, SX_ERR_CAPACITY);
    t = 0;
  }
  float *xs = sx_buf, *es = sx_buf + H;
  const bf16 *src = part ? nullptr : feat + (size_t)sx_index(fi, r) * H;
  const bf16 *erow = embed + (size_t)t * H;
  float sx = 0.f, se = 0.f;
  for (int i = threadIdx.x * 4; i < H; i += blockDim.x * 4) {
    uint2 xw;
    if (part) {
      const float4 v = sx_sum_splits4(part + (size_t)r * H + i, splits, split_stride);
      __nv_bfloat162 b0 = __floats2bfloat162_rn(v.x, v.y), b1 = __floats2bfloat162_rn(v.z, v.w);
      xw.x = *reinterpret_cast<uint32_t *>(&b0);
      xw.y = *reinterpret_cast<uint32_t *>(&b1);
    } else {
      xw = *reinterpret_cast<const uint2 *>(src + i);
    }
    *reinterpret_cast<uint2 *>(x_out + (size_t)r * H + i) = xw;
    const uint2 ew = *reinterpret_cast<const uint2 *>(erow + i);
    const float2 x0 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&xw.x));
    const float2 x1 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&xw.y));
    const float2 e0 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&ew.x));
    const float2 e1 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&ew.y));
    *reinterpret_cast<float4 *>(xs + i) = make_float4(x0.x, x0.y, x1.x, x1.y);
    *reinterpret_cast<float4 *>(es + i) = make_float4(e0.x, e0.y, e1.x, e1.y);
    sx += (x0.x * x0.x + x0.y * x0.y) + (x1.x * x1.x + x1.y * x1.y);
    se += (e0.x * e0.x + e0.y * e0.y) + (e1.x * e1.x + e1.y * e1.y);
  }
  sx = sx_warp_sum(sx);
  se = sx_warp_sum(se);
  if ((threadIdx.x & 31) == 0) { red[0][threadIdx.x >> 5] = sx; red[1][threadIdx.x >> 5] = se; }
  __syncthreads();
  float tx = 0.f, te = 0.f;
  {
    const int nw = blockDim.x >> 5;
    for (int w = 0; w < nw; ++w) { tx += red[0][w]; te += red[1][w]; }    // same order in every thread
  }
  const float scx = rsqrtf(tx / (float)H + eps), sce = rsqrtf(te / (float)H + eps);
  bf16 *urow = u + (size_t)r * 2 * H;
  for (int i = threadIdx.x * 4; i < H; i += blockDim.x * 4) {
    const float4 xv = *reinterpret_cast<const float4 *>(xs + i), ev = *reinterpret_cast<const float4 *>(es + i);
    const uint2 ge = *reinterpret_cast<const uint2 *>(gamma_e + i), gh = *reinterpret_cast<const uint2 *>(gamma_h + i);
    const float2 a0 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&ge.x));
    const float2 a1 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&ge.y));
    const float2 h0 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&gh.x));
    const float2 h1 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&gh.y));
    __nv_bfloat162 p0 = __floats2bfloat162_rn(ev.x * sce * a0.x, ev.y * sce * a0.y);
    __nv_bfloat162 p1 = __floats2bfloat162_rn(ev.z * sce * a1.x, ev.w * sce * a1.y);
    __nv_bfloat162 q0 = __floats2bfloat162_rn(xv.x * scx * h0.x, xv.y * scx * h0.y);
    __nv_bfloat162 q1 = __floats2bfloat162_rn(xv.z * scx * h1.x, xv.w * scx * h1.y);
    uint2 w;
    w.x = *reinterpret_cast<uint32_t *>(&p0);
    w.y = *reinterpret_cast<uint32_t *>(&p1);
    *reinterpret_cast<uint2 *>(urow + i) = w;
    w.x = *reinterpret_cast<uint32_t *>(&q0);
    w.y = *reinterpret_cast<uint32_t *>(&q1);
    *reinterpret_cast<uint2 *>(urow + H + i) = w;
  }
}

sx_status sx_launch_fused_input(const SxShape &sh, int R, const float *part, int splits, size_t split_stride,
                           const bf16 *feat, SxIndex fi, const int32_t *tok, SxIndex ti, const bf16 *embed,
                           const bf16 *gamma_e, const bf16 *gamma_h, bf16 *x_out, bf16 *u, int32_t *status,
                           cudaStream_t st) {
  int threads = ((sh.H / 4 + 31) / 32) * 32;
  if (threads > 1024) threads = 1024;
  return sx_rc(sx_launch(sx_fused_input_kernel, dim3(R), dim3(threads), (size_t)sh.H * 8, st, sh.H, sh.V, sh.eps, part, splits,
            split_stride, feat, fi, tok, ti, embed, gamma_e, gamma_h, x_out, u, status));
}

// The two row kernels above keep a row (and its gain, or the embedding row) in shared memory: opt in,
// once per device, to the size the largest supported hidden width needs.
sx_status sx_kernels_init(int device) {
  (void)device;
  if (cudaFuncSetAttribute(sx_finish_norm_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, SX_MAX_H * 6) != cudaSuccess ||
      cudaFuncSetAttribute(sx_fused_input_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, SX_MAX_H * 8) != cudaSuccess)
    return SX_ERR_CUDA;
  return SX_OK;
}

// ---------------------------------------------------------------------------------------
// split-K finisher of the QKV projection + rotary (rotate-half pairing) + KV append.
// One CTA per (head, row); thread i owns the pair (i, i + d/2).
// ---------------------------------------------------------------------------------------
__global__ void sx_finish_qkv_rope_kernel(int nq, int nkv, int d, double theta, SxRowMap rm, const float *part,
                                          int splits, size_t split_stride, bf16 *q_out, sx_kv kv, int page,
                                          int head_begin, int part_head0, int part_heads, int32_t *status) {
  sx_pdl_launch_dependents();
  const int hh = head_begin + blockIdx.x, r = blockIdx.y;
  const int i = threadIdx.x;
  const int half = d / 2;
  const bool rot = hh < nq + nkv;                 // q and k heads rotate, v heads do not
  const SxRowInfo ri = sx_row_place(rm, r);       // reads cache_len only (an input of the iteration)
  float c = 1.f, s = 0.f;
  if (rot && i < half) {
    // the angle needs more than fp32 at positions in the tens of thousands
    const double inv = exp2(-(2.0 * (double)i / (double)d) * log2(theta));
    double sn, cs;
    sincos((double)ri.pos * inv, &sn, &cs);
    c = (float)cs;
    s = (float)sn;
  }
  sx_pdl_wait();
  if (i >= half) return;
  if (rm.mode == SX_MODE_COMMIT && (ri.rel - 1) >= rm.valid_len[ri.b]) return;   // row does not exist
  // the partial sums hold heads [part_head0, part_head0 + part_heads) of the projection
  const float *row = part + ((size_t)r * part_heads + (hh - part_head0)) * d;
  float x1 = 0.f, x2 = 0.f;
  for (int sp = 0; sp < splits; ++sp) {
    x1 += row[sp * split_stride + i];
    x2 += row[sp * split_stride + i + half];
  }
  bf16 y1, y2;
  if (rot) {
    y1 = __float2bfloat16_rn(x1 * c - x2 * s);
    y2 = __float2bfloat16_rn(x2 * c + x1 * s);
  } else {
    y1 = __float2bfloat16_rn(x1);
    y2 = __float2bfloat16_rn(x2);
  }
  if (hh < nq) {
    q_out[((size_t)r * nq + hh) * d + i] = y1;
    q_out[((size_t)r * nq + hh) * d + i + half] = y2;
    return;
  }
  const int slot = ri.n + ri.rel;
  const int lp = slot / page, off = slot % page;
  int pp = -1;
  if (lp < kv.max_pages) pp = kv.page_table_d[(size_t)ri.b * kv.max_pages + lp];
  if (pp < 0 || pp >= kv.num_pages) {
    if (i == 0) sx_set_status(status, SX_ERR_CAPACITY);
    return;
  }
  const int kh = (hh < nq + nkv) ? hh - nq : hh - nq - nkv;
  bf16 *dst = reinterpret_cast<bf16 *>(hh < nq + nkv ? kv.k_pages_d : kv.v_pages_d) +
              (((size_t)pp * nkv + kh) * page + off) * d;
  dst[i] = y1;
  dst[i + half] = y2;
}

sx_status sx_launch_finish_qkv_rope(const SxShape &sh, const SxRowMap &rm, const float *part, int splits,
                               size_t split_stride, bf16 *q_out, const sx_kv &kv, int32_t *status,
                               cudaStream_t st, bool kv_only_partials) {
  int threads = ((sh.d / 2 + 31) / 32) * 32;
  // q_out == nullptr: only the K and V heads (commit); the partial sums then hold either the whole
  // projection or just its K and V rows
  const int head_begin = q_out ? 0 : sh.nq;
  const int part_head0 = kv_only_partials ? sh.nq : 0;
  const int part_heads = kv_only_partials ? 2 * sh.nkv : sh.nq + 2 * sh.nkv;
  return sx_rc(sx_launch(sx_finish_qkv_rope_kernel, dim3(sh.nq + 2 * sh.nkv - head_begin, rm.R), dim3(threads), 0, st, sh.nq, sh.nkv,
            sh.d, (double)sh.theta, rm, part, splits, split_stride, q_out, kv, sh.page, head_begin, part_head0,
            part_heads, status));
}

// ---------------------------------------------------------------------------------------
// commit (Algorithm 1, "Update KV-cache and hidden states accordingly")
// ---------------------------------------------------------------------------------------
// Blocks [0, B * M): catch-up input row (b, j) = [target hidden of path slot j ; embedding of the
// token of path slot j + 1] when j < L_b, zeros otherwise.  Blocks [B * M, B * M + B): the next
// iteration's first row: feature = target hidden of path slot L_b, token = recover token.
// FW is the width of a target feature row (H, or 3H for the layer with three-feature fusion).
// With tok_rows == nullptr a catch-up row is [feature ; embedding] (FW == H); otherwise it is the
// feature alone and the row's token goes to tok_rows.
__global__ void sx_commit_gather_kernel(int B, int M, int P, int H, int FW, int V, const bf16 *th, const int32_t *cand,
                                        const int32_t *path, int path_stride, const int32_t *accept_len,
                                        const int32_t *recover, const bf16 *embed, bf16 *u, int32_t *tok_rows,
                                        bf16 *feat0, int32_t *tok0, int32_t *status) {
  sx_pdl_launch_dependents();
  sx_pdl_wait();
  const int n8 = H / 8, f8 = FW / 8;
  if ((int)blockIdx.x >= B * M) {
    const int b = blockIdx.x - B * M;
    int L = accept_len[b];
    if (L < 0 || L >= path_stride) { if (threadIdx.x == 0) sx_set_status(status, SX_ERR_INVALID_ARG); L = 0; }
    int slot = path[(size_t)b * path_stride + L];
    if (slot < 0 || slot >= P) { if (threadIdx.x == 0) sx_set_status(status, SX_ERR_INVALID_ARG); slot = 0; }
    const uint4 *src = reinterpret_cast<const uint4 *>(th + ((size_t)b * P + slot) * FW);
    uint4 *dst = reinterpret_cast<uint4 *>(feat0 + (size_t)b * FW);
    for (int i = threadIdx.x; i < f8; i += blockDim.x) dst[i] = src[i];
    if (threadIdx.x == 0) tok0[b] = recover[b];
    return;
  }
  const int b = blockIdx.x / M, j = blockIdx.x - b * M;
  uint4 *o = reinterpret_cast<uint4 *>(u + (size_t)blockIdx.x * (tok_rows ? FW : 2 * H));
  const int L = accept_len[b];
  bool live = j < L && j + 1 < path_stride;
  int s0 = 0, s1 = 0, t = 0;
  if (live) {
    s0 = path[(size_t)b * path_stride + j];
    s1 = path[(size_t)b * path_stride + j + 1];
    if (s0 < 0 || s0 >= P || s1 < 0 || s1 >= P) { if (threadIdx.x == 0) sx_set_status(status, SX_ERR_INVALID_ARG); live = false; }
  }
  if (live) {
    t = cand[(size_t)b * P + s1];
    if (t < 0 || t >= V) { if (threadIdx.x == 0) sx_set_status(status, SX_ERR_CAPACITY); t = 0; }
  }
  const uint4 *f = reinterpret_cast<const uint4 *>(th + ((size_t)b * P + s0) * FW);
  const uint4 *e = reinterpret_cast<const uint4 *>(embed + (size_t)t * H);
  const uint4 zero = make_uint4(0, 0, 0, 0);
  if (tok_rows) {
    for (int i = threadIdx.x; i < f8; i += blockDim.x) o[i] = live ? f[i] : zero;
    if (threadIdx.x == 0) tok_rows[blockIdx.x] = t;
    return;
  }
  for (int i = threadIdx.x; i < n8; i += blockDim.x) {
    o[i] = live ? f[i] : zero;
    o[n8 + i] = live ? e[i] : zero;
  }
}

// The last kernel of a commit.  It does not release its dependents early: whatever is launched
// after it, however eagerly, starts once the new lengths are in memory.
__global__ void sx_commit_advance_kernel(int B, const int32_t *accept_len, int32_t *cache_len) {
  sx_pdl_wait();
  const int b = blockIdx.x * blockDim.x + threadIdx.x;
  if (b < B) cache_len[b] += accept_len[b] + 1;
}

sx_status sx_launch_commit_gather(const SxShape &sh, int B, int M, int P, const bf16 *th, const int32_t *cand,
                             const int32_t *path, int path_stride, const int32_t *accept_len, const int32_t *recover,
                             const bf16 *embed, bf16 *u, bf16 *feat0, int32_t *tok0, int32_t *status, cudaStream_t st,
                             int32_t *tok_rows) {
  int threads = ((sh.H / 8 + 31) / 32) * 32;
  if (threads > 512) threads = 512;
  const int FW = tok_rows ? 3 * sh.H : sh.H;
  return sx_rc(sx_launch(sx_commit_gather_kernel, dim3(B * M + B), dim3(threads), 0, st, B, M, P, sh.H, FW, sh.V, th, cand, path,
            path_stride, accept_len, recover, embed, u, tok_rows, feat0, tok0, status));
}

sx_status sx_launch_commit_advance(int B, const int32_t *accept_len, int32_t *cache_len, cudaStream_t st) {
  return sx_rc(sx_launch(sx_commit_advance_kernel, dim3((B + 127) / 128), dim3(128), 0, st, B, accept_len, cache_len));
}

// ---------------------------------------------------------------------------------------
// split-K finisher of gate/up + SwiGLU
// ---------------------------------------------------------------------------------------
__global__ void sx_finish_swiglu_kernel(int F, const float *part, int splits, size_t split_stride, bf16 *m_out) {
  sx_pdl_launch_dependents();
  sx_pdl_wait();
  const int r = blockIdx.y;
  const float *row = part + (size_t)r * 2 * F;
  const int i = (blockIdx.x * blockDim.x + threadIdx.x) * 4;
  if (i >= F) return;
  const float4 g = sx_sum_splits4(row + i, splits, split_stride);
  const float4 u = sx_sum_splits4(row + F + i, splits, split_stride);
  const float m0 = g.x / (1.0f + expf(-g.x)) * u.x, m1 = g.y / (1.0f + expf(-g.y)) * u.y;
  const float m2 = g.z / (1.0f + expf(-g.z)) * u.z, m3 = g.w / (1.0f + expf(-g.w)) * u.w;
  __nv_bfloat162 b0 = __floats2bfloat162_rn(m0, m1), b1 = __floats2bfloat162_rn(m2, m3);
  uint2 w;
  w.x = *reinterpret_cast<uint32_t *>(&b0);
  w.y = *reinterpret_cast<uint32_t *>(&b1);
  *reinterpret_cast<uint2 *>(m_out + (size_t)r * F + i) = w;
}

sx_status sx_launch_finish_swiglu(const SxShape &sh, int R, const float *part, int splits, size_t split_stride,
                             bf16 *m_out, cudaStream_t st) {
  dim3 grid((sh.F / 4 + 127) / 128, R);
  return sx_rc(sx_launch(sx_finish_swiglu_kernel, grid, dim3(128), 0, st, sh.F, part, splits, split_stride, m_out));
}

// ---------------------------------------------------------------------------------------
// merge of the per-CTA head results: top-T ids (+ log-probabilities), activated signals
// ---------------------------------------------------------------------------------------
// One CTA per token row, one thread per CTA of the head kernel (blockDim >= G).  Every per-CTA list
// is sorted, so the global top-T is a tournament over the list heads: T rounds of a block-wide
// maximum, the winner advances in its list.  Everything stays in registers.
__global__ void __launch_bounds__(1024)
sx_head_finalize_kernel(const SxHeadPartial *parts, int G, int part_stride, int T, int lse,
                        const float *z, int S, int act0, int act1, int act2, int32_t *tok_out,
                        SxIndex toi, float *logp_out, float *sig_out, SxIndex si, SxNextInput nx,
                        const int32_t *map, int Vd) {
  __shared__ unsigned long long s_best[2][32];
  __shared__ float s_red[32];
  __shared__ float s_lse;
  __shared__ int s_tok;
  sx_pdl_launch_dependents();
  sx_pdl_wait();
  const int r = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, nw = blockDim.x >> 5;
  unsigned long long v[SX_MAX_TOPK];
  float pm = -INFINITY, pl = 0.f;
#pragma unroll
  for (int k = 0; k < SX_MAX_TOPK; ++k) v[k] = 0ull;
  if (tid < G) {
    const SxHeadPartial &p = parts[(size_t)tid * part_stride + r];
#pragma unroll
    for (int k = 0; k < SX_MAX_TOPK; ++k)
      if (k < T) v[k] = p.top[k];
    pm = p.m;
    pl = p.l;
  }
  if (lse) {
    float mm = sx_warp_max(pm);
    if (lane == 0) s_red[warp] = mm;
    __syncthreads();
    mm = sx_warp_max(lane < nw ? s_red[lane] : -INFINITY);
    __syncthreads();
    float ll = sx_warp_sum(pl > 0.f ? pl * expf(pm - mm) : 0.f);
    if (lane == 0) s_red[warp] = ll;
    __syncthreads();
    ll = sx_warp_sum(lane < nw ? s_red[lane] : 0.f);
    if (tid == 0) s_lse = mm + logf(ll);
  }
  const int tbase = sx_index(toi, r);
  for (int t = 0; t < T; ++t) {
    unsigned long long best = v[0];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) best = max(best, __shfl_xor_sync(0xffffffffu, best, o));
    if (lane == 0) s_best[t & 1][warp] = best;
    __syncthreads();
    best = lane < nw ? s_best[t & 1][lane] : 0ull;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) best = max(best, __shfl_xor_sync(0xffffffffu, best, o));
    if (tid == 0) {
      int32_t id = (int32_t)sx_pack_index(best);
      if (map) id = (id >= 0 && id < Vd) ? map[id] : 0;      // draft id -> token id (reduced draft vocabulary)
      tok_out[tbase + t] = id;
      if (t == 0) s_tok = id;
      if (logp_out) logp_out[(size_t)r * T + t] = lse ? sx_pack_value(best) - s_lse : sx_pack_value(best);
    }
    if (best != 0ull && v[0] == best) {          // packed values are unique (index inside): one winner
#pragma unroll
      for (int k = 0; k + 1 < SX_MAX_TOPK; ++k) v[k] = v[k + 1];
      v[SX_MAX_TOPK - 1] = 0ull;
    }
  }
  if (sig_out && tid < S) {
    const int a = tid == 0 ? act0 : (tid == 1 ? act1 : act2);
    sig_out[(size_t)sx_index(si, r) * S + tid] = sx_activate(z[(size_t)r * S + tid], a);
  }
  if (nx.u) {
    // chain drafting: the next round's input row [hidden of this round ; embedding of the chosen token]
    __syncthreads();
    int t = s_tok;
    if (t < 0 || t >= nx.V) t = 0;
    const uint4 *f = reinterpret_cast<const uint4 *>(nx.feat + (size_t)r * nx.H);
    const uint4 *e = reinterpret_cast<const uint4 *>(nx.embed + (size_t)t * nx.H);
    uint4 *o = reinterpret_cast<uint4 *>(nx.u + (size_t)r * 2 * nx.H);
    const int n = nx.H / 8;
    for (int i = tid; i < n; i += blockDim.x) {
      const uint4 a = f[i], b = e[i];
      o[i] = a;
      o[n + i] = b;
    }
  }
}

sx_status sx_launch_head_finalize(const SxShape &sh, int R, const SxHeadPartial *parts, int G, int part_stride,
                             int T, int lse, const float *z, int S, int32_t *tok_out, SxIndex toi,
                             float *logp_out, float *sig_out, SxIndex si, cudaStream_t st, SxNextInput nx,
                             const int32_t *map, int Vd) {
  int threads = ((G + 31) / 32) * 32;              // one thread per CTA of the head kernel (G <= SM count)
  if (threads < 128) threads = 128;
  return sx_rc(sx_launch(sx_head_finalize_kernel, dim3(R), dim3(threads), 0, st, parts, G, part_stride, T, lse, z, S, sh.act[0],
            sh.act[1], sh.act[2], tok_out, toi, logp_out, sig_out, si, nx, map, Vd));
}

// ---------------------------------------------------------------------------------------
// chain layout: slot j holds the j-th draft token; the signal of slot j comes from round j+1
// ---------------------------------------------------------------------------------------
__global__ void sx_chain_layout_kernel(int B, int K, int S, const int32_t *tok0, sx_iter_out o) {
  sx_pdl_launch_dependents();
  sx_pdl_wait();
  const int P = K + 1;
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= B * P) return;
  const int b = i / P, j = i % P;
  if (j == 0) o.cand_tok_d[i] = tok0[b];
  if (o.parent_d) o.parent_d[i] = j - 1;
  if (o.depth_d) o.depth_d[i] = j;
  if (o.slot_row_d) o.slot_row_d[i] = (j < K) ? j : -1;
  if (o.slot_src_row_d) o.slot_src_row_d[i] = j - 1;
  if (j == K)
    for (int s = 0; s < S; ++s) o.slot_signal_d[(size_t)i * S + s] = __int_as_float(0x7fc00000);
}

sx_status sx_launch_chain_layout(int B, int K, int S, const int32_t *tok0, const sx_iter_out &o, cudaStream_t st) {
  const int n = B * (K + 1);
  return sx_rc(sx_launch(sx_chain_layout_kernel, dim3((n + 127) / 128), dim3(128), 0, st, B, K, S, tok0, o));
}

// ---------------------------------------------------------------------------------------
// greedy acceptance (Algorithm 1): chain prefix match, or the walk down the tree
// ---------------------------------------------------------------------------------------
// One warp per sequence; in a tree the lanes look for the accepted child together.
__global__ void sx_accept_kernel(int B, int P, const int32_t *cand, const int32_t *parent, const int32_t *target,
                                 int32_t *accept_len, int32_t *path, int path_stride, int32_t *recover) {
  sx_pdl_launch_dependents();
  sx_pdl_wait();
  const int b = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5), lane = threadIdx.x & 31;
  if (b >= B) return;
  const int32_t *c = cand + (size_t)b * P, *t = target + (size_t)b * P;
  int32_t *pa = path + (size_t)b * path_stride;
  int L = 0, cur = 0;
  if (lane == 0) pa[0] = 0;
  if (!parent) {
    // longest prefix with cand[j + 1] == target[j]: first mismatch among the lanes' positions
    for (int j0 = 0; j0 < P - 1; j0 += 32) {
      const int j = j0 + lane;
      const bool ok = j < P - 1 && c[j + 1] == t[j];
      const unsigned miss = ~__ballot_sync(0xffffffffu, ok);
      const int run = miss ? __ffs(miss) - 1 : 32;
      if (lane < run && j0 + lane + 1 < path_stride) pa[j0 + lane + 1] = j0 + lane + 1;
      L += run;
      if (run < 32) break;
    }
    cur = L;
  } else {
    const int32_t *par = parent + (size_t)b * P;
    for (;;) {
      const int want = t[cur];
      int nxt = -1;
      for (int s0 = 1; s0 < P && nxt < 0; s0 += 32) {
        const int sl = s0 + lane;
        const bool hit = sl < P && par[sl] == cur && c[sl] == want;
        const unsigned m = __ballot_sync(0xffffffffu, hit);
        if (m) nxt = s0 + __ffs(m) - 1;            // lowest slot wins, as in a serial scan
      }
      if (nxt < 0) break;
      cur = nxt;
      ++L;
      if (lane == 0 && L < path_stride) pa[L] = cur;
    }
  }
  for (int j = L + 1 + lane; j < path_stride; j += 32) pa[j] = -1;
  if (lane == 0) {
    accept_len[b] = L;
    recover[b] = t[cur];
  }
}

sx_status sx_launch_accept(int B, int P, const int32_t *cand, const int32_t *parent, const int32_t *target,
                      int32_t *accept_len, int32_t *path, int path_stride, int32_t *recover, cudaStream_t st) {
  return sx_rc(sx_launch(sx_accept_kernel, dim3((B + 3) / 4), dim3(128), 0, st, B, P, cand, parent, target, accept_len, path,
            path_stride, recover));
}

// ---------------------------------------------------------------------------------------
// exit rule (Section 3.3, Appendix A.1): EWMA over the accepted slots, AND of the enabled
// thresholds at the first accepted step-split token
// ---------------------------------------------------------------------------------------
struct SxExitParams {
  float alpha;
  float thr[SX_MAX_SIGNALS];
  int dir[SX_MAX_SIGNALS];
  uint32_t enable;
  int ema_positions;
  const uint32_t *bitmap;
  int stop_tok;
  int smoothing, window;
  float *hist, *par_sum;
  int32_t *par_n;
};

__global__ void sx_exit_kernel(int B, int P, int S, int V, SxExitParams p, float *x_state, int32_t *n_updates,
                               int32_t *thinking, const float *slot_signal, const int32_t *cand,
                               const int32_t *path, int path_stride, const int32_t *accept_len,
                               const int32_t *recover, int32_t *exit_flag, int32_t *accept_out,
                               int32_t *recover_out, float *smoothed, int32_t *status) {
  sx_pdl_launch_dependents();
  sx_pdl_wait();
  const int b = blockIdx.x * blockDim.x + threadIdx.x;
  if (b >= B) return;
  const int L = accept_len[b];
  int flag = 0, Lo = L, ro = recover[b];
  float x[SX_MAX_SIGNALS];
  for (int i = 0; i < S; ++i) x[i] = x_state[(size_t)b * S + i];
  int nu = n_updates[b];
  if (thinking[b] != 0) {
    for (int idx = 0; idx <= L && idx < path_stride; ++idx) {
      const int slot = path[(size_t)b * path_stride + idx];
      if (slot < 0 || slot >= P) { sx_set_status(status, SX_ERR_INVALID_ARG); break; }
      const float *sg = slot_signal + ((size_t)b * P + slot) * S;
      if (p.ema_positions == SX_EMA_VERIFIED_CONTEXT || idx == 0) {
        bool none = false;
        for (int i = 0; i < S; ++i) none |= isnan(sg[i]);
        if (none) break;
        for (int i = 0; i < S; ++i) {
          const float s = sg[i];
          if (p.smoothing == SX_SMOOTH_EWMA) {
            x[i] = (nu == 0) ? s : (float)((double)p.alpha * (double)s + (1.0 - (double)p.alpha) * (double)x[i]);
          } else if (p.smoothing == SX_SMOOTH_NONE) {
            x[i] = s;
          } else if (p.smoothing == SX_SMOOTH_PARAGRAPH) {
            float *ps = p.par_sum + (size_t)b * S + i;
            *ps = (float)((double)*ps + (double)s);
            x[i] = (float)((double)*ps / (double)(p.par_n[b] + 1));
          } else {
            float *h = p.hist + (size_t)b * SX_HIST * S + i;       // sample j of this signal at h[(j % SX_HIST) * S]
            h[(nu % SX_HIST) * S] = s;
            if (p.smoothing == SX_SMOOTH_WINDOW) {
              const int m = min(nu + 1, p.window);
              double acc = 0.0;
              for (int j = nu - m + 1; j <= nu; ++j) acc += (double)h[(j % SX_HIST) * S];
              x[i] = (float)(acc / (double)m);
            } else if (nu == 0) {
              x[i] = s;
            } else {
              const int k = min(p.window - 1, nu - 1);
              const double prev = (double)h[((nu - 1) % SX_HIST) * S];
              x[i] = (k == 0) ? (float)prev : (float)(prev + (prev - (double)h[((nu - 1 - k) % SX_HIST) * S]) / (double)k);
            }
          }
        }
        if (p.smoothing == SX_SMOOTH_PARAGRAPH) p.par_n[b] += 1;
        ++nu;
      }
      const int tok = cand[(size_t)b * P + slot];
      bool split = true;
      if (p.bitmap) split = (tok >= 0 && tok < V) ? ((p.bitmap[tok >> 5] >> (tok & 31)) & 1u) : false;
      bool pass = true;
      for (int i = 0; i < S; ++i) {
        if (!((p.enable >> i) & 1u)) continue;
        pass = pass && ((p.dir[i] == SX_DIR_GT) ? (x[i] > p.thr[i]) : (x[i] < p.thr[i]));
      }
      if (split && pass) {
        flag = 1; Lo = idx; ro = p.stop_tok;
        thinking[b] = 0;
        break;
      }
      if (split && p.smoothing == SX_SMOOTH_PARAGRAPH) {       // a paragraph delimiter went by
        for (int i = 0; i < S; ++i) p.par_sum[(size_t)b * S + i] = 0.f;
        p.par_n[b] = 0;
      }
    }
    for (int i = 0; i < S; ++i) x_state[(size_t)b * S + i] = x[i];
    n_updates[b] = nu;
  }
  exit_flag[b] = flag;
  accept_out[b] = Lo;
  recover_out[b] = ro;
  for (int i = 0; i < S; ++i) smoothed[(size_t)b * S + i] = x[i];
}

sx_status sx_launch_exit(int B, int P, int S, const sx_exit_cfg &cfg, const sx_exit_state &state,
                    const float *slot_signal, const int32_t *cand, const int32_t *path, int path_stride,
                    const int32_t *accept_len, const int32_t *recover, int32_t *exit_flag,
                    int32_t *accept_out, int32_t *recover_out, float *smoothed, int V, int32_t *status,
                    cudaStream_t st) {
  SxExitParams p;
  p.alpha = cfg.alpha;
  for (int i = 0; i < SX_MAX_SIGNALS; ++i) { p.thr[i] = cfg.thr[i]; p.dir[i] = cfg.dir[i]; }
  p.enable = cfg.enable_mask;
  p.ema_positions = cfg.ema_positions;
  p.bitmap = cfg.split_bitmap_d;
  p.stop_tok = cfg.stop_think_token;
  p.smoothing = cfg.smoothing; p.window = cfg.window;
  p.hist = state.hist_d; p.par_sum = state.par_sum_d; p.par_n = state.par_n_d;
  return sx_rc(sx_launch(sx_exit_kernel, dim3((B + 31) / 32), dim3(32), 0, st, B, P, S, V, p, state.x_d, state.n_updates_d,
            state.thinking_d, slot_signal, cand, path, path_stride, accept_len, recover, exit_flag, accept_out,
            recover_out, smoothed, status));
}

// ---------------------------------------------------------------------------------------
// draft tree bookkeeping.  Candidate ids follow generation order: depth 1 = [0, T); depth
// r >= 2 = T + (r-2) T^2 + j T + t for the t-th child of the j-th expanded row.  Score =
// fp32 sum of log-probabilities; better = higher score, then lower candidate id.
// ---------------------------------------------------------------------------------------
__device__ __forceinline__ bool sx_better(float sa, int ia, float sb, int ib) {
  return sa > sb || (sa == sb && ia < ib);
}

__global__ void sx_tree_expand_kernel(SxTree t, int round, const int32_t *tok_rt, const float *logp_rt) {
  sx_pdl_launch_dependents();
  sx_pdl_wait();
  const int b = blockIdx.x, tid = threadIdx.x;
  const int T = t.T;
  int32_t *ctok = t.cand_tok + (size_t)b * t.NC, *cpar = t.cand_parent + (size_t)b * t.NC;
  int32_t *csrc = t.cand_src_row + (size_t)b * t.NC, *crow = t.cand_row + (size_t)b * t.NC;
  float *csc = t.cand_score + (size_t)b * t.NC;
  uint64_t *rmask = t.row_mask + (size_t)b * t.rows;
  const int cnt = (round == 1) ? T : T * T;
  const int base = (round == 1) ? 0 : T + (round - 2) * T * T;
  if (round == 1 && tid == 0) rmask[0] = 1ull;
  for (int i = tid; i < cnt; i += blockDim.x) {
    const int j = i / T, tt = i % T;
    const int rrow = (round == 1) ? b : b * T + j;            // row of this round's launch
    float ps = 0.f;
    int pc = -1, src = 0;
    if (round > 1) {
      pc = t.sel_cid[b * T + j];
      ps = csc[pc];
      src = 1 + (round - 2) * T + j;
    }
    ctok[base + i] = tok_rt[(size_t)rrow * T + tt];
    csc[base + i] = ps + logp_rt[(size_t)rrow * T + tt];
    cpar[base + i] = pc;
    csrc[base + i] = src;
    crow[base + i] = -1;
  }
  __syncthreads();
  if (round >= t.D) return;
  // choose the T best of this depth for the next round (rank by counting)
  for (int i = tid; i < cnt; i += blockDim.x) {
    const float s = csc[base + i];
    int rank = 0;
    for (int k = 0; k < cnt; ++k) rank += sx_better(csc[base + k], k, s, i) ? 1 : 0;
    if (rank < T) {
      const int cid = base + i;
      const int rid = 1 + (round - 1) * T + rank;           // drafted row of the next round
      const int nr = b * T + rank;
      t.sel_cid[nr] = cid;
      t.sel_tok[nr] = ctok[cid];
      t.feat_idx[nr] = b * t.rows + csrc[cid];
      t.hid_idx[nr] = b * t.rows + rid;
      const uint64_t mk = rmask[csrc[cid]] | (1ull << rid);
      t.next_mask[nr] = mk;
      rmask[rid] = mk;
      crow[cid] = rid;
    }
  }
}

sx_status sx_launch_tree_expand(const SxTree &t, int B, int round, const int32_t *tok_rt, const float *logp_rt,
                           cudaStream_t st) {
  return sx_rc(sx_launch(sx_tree_expand_kernel, dim3(B), dim3(64), 0, st, t, round, tok_rt, logp_rt));
}

__global__ void sx_tree_layout_kernel(SxTree t, int S, const int32_t *tok0, sx_iter_out o) {
  sx_pdl_launch_dependents();
  sx_pdl_wait();
  extern __shared__ int sx_tl[];           // kept[NC], slot_of[NC], score[NC]
  const int b = blockIdx.x, tid = threadIdx.x;
  const int NC = t.NC, P = 1 + t.max_nodes, T = t.T;
  int *kept = sx_tl, *slot_of = sx_tl + NC;
  float *csc = reinterpret_cast<float *>(sx_tl + 2 * NC);
  const int32_t *ctok = t.cand_tok + (size_t)b * NC, *cpar = t.cand_parent + (size_t)b * NC;
  const int32_t *csrc = t.cand_src_row + (size_t)b * NC, *crow = t.cand_row + (size_t)b * NC;
  for (int i = tid; i < NC; i += blockDim.x) csc[i] = t.cand_score[(size_t)b * NC + i];
  __syncthreads();
  for (int i = tid; i < NC; i += blockDim.x) {      // rank of candidate i among all scores (shared-memory broadcast reads)
    const float s = csc[i];
    int rank = 0;
    for (int k = 0; k < NC; ++k) rank += sx_better(csc[k], k, s, i) ? 1 : 0;
    kept[i] = rank < t.max_nodes;
  }
  __syncthreads();
  for (int i = tid; i < NC; i += blockDim.x) {
    int s = 1;
    for (int k = 0; k < i; ++k) s += kept[k];
    slot_of[i] = kept[i] ? s : -1;
  }
  __syncthreads();
  const float qnan = __int_as_float(0x7fc00000);
  if (tid == 0) {
    const size_t at = (size_t)b * P;
    o.cand_tok_d[at] = tok0[b];
    if (o.parent_d) o.parent_d[at] = -1;
    if (o.depth_d) o.depth_d[at] = 0;
    if (o.slot_row_d) o.slot_row_d[at] = 0;
    if (o.slot_src_row_d) o.slot_src_row_d[at] = -1;
    for (int s = 0; s < S; ++s) o.slot_signal_d[at * S + s] = t.row_sig[((size_t)b * t.rows) * S + s];
  }
  for (int i = tid; i < NC; i += blockDim.x) {
    if (!kept[i]) continue;
    const size_t at = (size_t)b * P + slot_of[i];
    const int depth = (i < T) ? 1 : 2 + (i - T) / (T * T);
    o.cand_tok_d[at] = ctok[i];
    if (o.parent_d) o.parent_d[at] = (cpar[i] < 0) ? 0 : slot_of[cpar[i]];
    if (o.depth_d) o.depth_d[at] = depth;
    if (o.slot_row_d) o.slot_row_d[at] = crow[i];
    if (o.slot_src_row_d) o.slot_src_row_d[at] = csrc[i];
    for (int s = 0; s < S; ++s)
      o.slot_signal_d[at * S + s] = (crow[i] >= 0) ? t.row_sig[((size_t)b * t.rows + crow[i]) * S + s] : qnan;
  }
}

sx_status sx_launch_tree_layout(const SxTree &t, int B, int S, const int32_t *tok0, const sx_iter_out &o,
                           cudaStream_t st) {
  return sx_rc(sx_launch(sx_tree_layout_kernel, dim3(B), dim3(256), (size_t)3 * t.NC * sizeof(int), st, t, S, tok0, o));
}

// ---------------------------------------------------------------------------------------
// Speculative sampling with sampled drafts: accept test and residual draw of one verify slot.
// One CTA per (sequence, slot); probabilities are float64 functions of the fp32 logits.
// ---------------------------------------------------------------------------------------
__device__ __forceinline__ double sx_block_sum(double v, double *red) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  __syncthreads();
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = v;
  __syncthreads();
  double t = 0.0;
  for (int w = 0; w < (int)(blockDim.x >> 5); ++w) t += red[w];       // same order in every thread
  return t;
}
__device__ __forceinline__ float sx_block_max(float v, double *red) {
  v = sx_warp_max(v);
  __syncthreads();
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = (double)v;
  __syncthreads();
  double t = -INFINITY;
  for (int w = 0; w < (int)(blockDim.x >> 5); ++w) t = fmax(t, red[w]);
  return (float)t;
}

// Slice s of a row covers token ids [s * len, min(V, (s + 1) * len)), len a multiple of 4.
struct SxSpecPartial {
  double mp, sp, mq, sq;      // slice maxima and sums of exp((logit - max) / tau), target and draft
  double best;                // best residual score of the slice (phase 2)
  int besti, accept;
};

// Phase 1: per (row, slice) the pieces of the two log-partition sums.
__global__ void __launch_bounds__(512)
sx_spec_partials_kernel(int P, int V, int len, const float *target_logits, const float *draft_logits, float temp,
                        SxSpecPartial *parts) {
  __shared__ double red[32];
  sx_pdl_launch_dependents();
  sx_pdl_wait();
  const int row = blockIdx.x, sl = blockIdx.y, S = gridDim.y, b = row / P, j = row % P, K = P - 1, tid = threadIdx.x;
  const int i0 = sl * len, i1 = min(V, i0 + len);
  const float *lp = target_logits + (size_t)row * V;
  const float *lq = (j < K) ? draft_logits + ((size_t)b * K + j) * V : nullptr;
  // the exponentials are fp32 (their rounding is below the fp32 logits' own), the sums float64
  const float inv_tau = 1.0f / temp;
  float mp = -INFINITY, mq = -INFINITY;
  for (int i = i0 + tid; i < i1; i += blockDim.x) {
    mp = fmaxf(mp, lp[i]);
    if (lq) mq = fmaxf(mq, lq[i]);
  }
  mp = sx_block_max(mp, red);
  mq = sx_block_max(mq, red);
  double sp = 0.0, sq = 0.0;
  for (int i = i0 + tid; i < i1; i += blockDim.x) {
    sp += (double)expf((lp[i] - mp) * inv_tau);
    if (lq) sq += (double)expf((lq[i] - mq) * inv_tau);
  }
  sp = sx_block_sum(sp, red);
  sq = sx_block_sum(sq, red);
  if (tid == 0) {
    SxSpecPartial &o = parts[(size_t)row * S + sl];
    o.mp = (double)mp; o.sp = sp; o.mq = (double)mq; o.sq = sq;
  }
}

// Phase 2: every CTA of a row rebuilds the row's normalisers (slice order, so all agree), takes the
// accept test, and - for a refused or draft-less slot - leaves the best residual score of its slice.
__global__ void __launch_bounds__(512)
sx_spec_draw_kernel(int P, int V, int len, const float *target_logits, const float *draft_logits,
                    const int32_t *cand_tok, SxSample smp, SxSpecPartial *parts, int32_t *status) {
  __shared__ double red[32];
  __shared__ int red_i[32];
  sx_pdl_launch_dependents();
  sx_pdl_wait();
  const int row = blockIdx.x, sl = blockIdx.y, S = gridDim.y, b = row / P, j = row % P, K = P - 1, tid = threadIdx.x;
  const float *lp = target_logits + (size_t)row * V;
  const float *lq = (j < K) ? draft_logits + ((size_t)b * K + j) * V : nullptr;
  const double tau = (double)smp.temp;
  SxSpecPartial *pr = parts + (size_t)row * S;
  double mp = -INFINITY, mq = -INFINITY;
  for (int s = 0; s < S; ++s) {
    if (pr[s].sp > 0.0) mp = fmax(mp, pr[s].mp);
    if (pr[s].sq > 0.0) mq = fmax(mq, pr[s].mq);
  }
  double sp = 0.0, sq = 0.0;
  for (int s = 0; s < S; ++s) {
    if (pr[s].sp > 0.0) sp += pr[s].sp * exp((pr[s].mp - mp) / tau);
    if (pr[s].sq > 0.0) sq += pr[s].sq * exp((pr[s].mq - mq) / tau);
  }
  const double lsp = log(sp), lsq = lq ? log(sq) : 0.0;
  int x = -1, accept = 0;
  if (j < K) {
    x = cand_tok[(size_t)b * P + j + 1];
    if (x < 0 || x >= V) {
      if (tid == 0 && sl == 0) sx_set_status(status, SX_ERR_CAPACITY);
      x = 0;
    }
    // keep the draft token with probability min(1, p(x) / q(x)); every thread takes the same decision
    const double logpx = ((double)lp[x] - mp) / tau - lsp;
    const double logqx = ((double)lq[x] - mq) / tau - lsq;
    const double ratio = fmin(1.0, exp(logpx - logqx));
    uint32_t w[4];
    sx_philox4x32_10(0u, 0x20000000u + (uint32_t)j, (uint32_t)b, smp.offset, smp.k0, smp.k1, w);
    const double u = ((double)(w[0] >> 9) + 0.5) * (1.0 / 8388608.0);
    accept = (u < ratio) ? 1 : 0;
  }
  double best = -INFINITY;
  int besti = -1;
  if (!accept) {
    // a draw from the normalised max(0, p - q): Gumbel-max over log(p_i - q_i), lower index among equals
    const int i0 = sl * len, i1 = min(V, i0 + len);
    const float inv_tau = 1.0f / smp.temp, fmp = (float)mp, fmq = (float)mq, flsp = (float)lsp, flsq = (float)lsq;
    for (int a = i0 + tid * 4; a < i1; a += blockDim.x * 4) {
      uint32_t w[4];
      sx_philox4x32_10((uint32_t)(a >> 2), (uint32_t)j, (uint32_t)b, smp.offset, smp.k0, smp.k1, w);
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const int i = a + e;
        if (i < i1) {
          const float p = expf((lp[i] - fmp) * inv_tau - flsp);
          const float q = lq ? expf((lq[i] - fmq) * inv_tau - flsq) : 0.f;
          const float r = p - q;
          if (r > 0.f) {
            const float u = (float)((w[e] >> 9) * 2u + 1u) * 5.9604644775390625e-8f;
            const double sc = (double)(logf(r) - logf(-logf(u)));
            if (sc > best) { best = sc; besti = i; }
          }
        }
      }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      const double ob = __shfl_xor_sync(0xffffffffu, best, o);
      const int oi = __shfl_xor_sync(0xffffffffu, besti, o);
      if (oi >= 0 && (besti < 0 || ob > best || (ob == best && oi < besti))) { best = ob; besti = oi; }
    }
    if ((tid & 31) == 0) { red[tid >> 5] = best; red_i[tid >> 5] = besti; }
    __syncthreads();
    if (tid == 0) {
      best = -INFINITY;
      besti = -1;
      for (int w = 0; w < (int)(blockDim.x >> 5); ++w) {
        const double ob = red[w];
        const int oi = red_i[w];
        if (oi >= 0 && (besti < 0 || ob > best || (ob == best && oi < besti))) { best = ob; besti = oi; }
      }
    }
  }
  if (tid == 0) {
    pr[sl].best = best;
    pr[sl].besti = besti;
    pr[sl].accept = accept;
  }
}

// Phase 3: the slot's token - the kept draft token, or the best residual score over the slices.
__global__ void sx_spec_pick_kernel(int P, int V, int S, int rows, const int32_t *cand_tok, const SxSpecPartial *parts,
                                    int32_t *target_tok) {
  sx_pdl_launch_dependents();
  sx_pdl_wait();
  const int row = blockIdx.x * blockDim.x + threadIdx.x;
  if (row >= rows) return;
  const int b = row / P, j = row % P;
  const SxSpecPartial *pr = parts + (size_t)row * S;
  int x = (j < P - 1) ? cand_tok[(size_t)b * P + j + 1] : -1;
  if (j < P - 1 && (x < 0 || x >= V)) x = 0;
  if (pr[0].accept) { target_tok[row] = x; return; }
  double best = -INFINITY;
  int besti = -1;
  for (int s = 0; s < S; ++s)                       // slices in index order: a strict compare keeps the lower index
    if (pr[s].besti >= 0 && (besti < 0 || pr[s].best > best)) { best = pr[s].best; besti = pr[s].besti; }
  target_tok[row] = besti >= 0 ? besti : (x >= 0 ? x : 0);      // nothing left to draw from: p == q
}

int sx_spec_sample_slices(int rows, int V, int sm_count) {
  int S = (2 * sm_count + rows - 1) / rows;
  const int cap = (V + 2047) / 2048;
  if (S > cap) S = cap;
  if (S > SX_SPEC_MAX_SLICES) S = SX_SPEC_MAX_SLICES;
  return S < 1 ? 1 : S;
}
size_t sx_spec_sample_ws_bytes(int rows) { return (size_t)rows * SX_SPEC_MAX_SLICES * sizeof(SxSpecPartial); }

sx_status sx_launch_spec_sample(int B, int P, int V, const float *target_logits, const float *draft_logits,
                           const int32_t *cand_tok, SxSample smp, void *parts_ws, int sm_count, int32_t *target_tok,
                           int32_t *status, cudaStream_t st) {
  const int rows = B * P, S = sx_spec_sample_slices(rows, V, sm_count);
  const int len = (((V + S - 1) / S + 3) / 4) * 4;
  SxSpecPartial *parts = (SxSpecPartial *)parts_ws;
  SX_TRY(sx_rc(sx_launch(sx_spec_partials_kernel, dim3(rows, S), dim3(512), 0, st, P, V, len, target_logits, draft_logits,
                         smp.temp, parts)));
  SX_TRY(sx_rc(sx_launch(sx_spec_draw_kernel, dim3(rows, S), dim3(512), 0, st, P, V, len, target_logits, draft_logits,
                         cand_tok, smp, parts, status)));
  return sx_rc(sx_launch(sx_spec_pick_kernel, dim3((rows + 127) / 128), dim3(128), 0, st, P, V, S, rows, cand_tok, parts, target_tok));
}

// ---------------------------------------------------------------------------------------
// Sampled children in a draft tree
// ---------------------------------------------------------------------------------------
// The children of a drafted row are the T largest of logit + temp * Gumbel noise, best first: a draw of T
// tokens without replacement, in order, from softmax(logits / temp).  The row's logits (left in memory by
// the head launch) are cut into C chunks; CTA (chunk, row) keeps, per thread, the T best perturbed scores of
// its share in registers together with a running (max, sum) of the raw logits, merges the lists by a
// tournament over their heads and writes one partial result; a second kernel merges the C partial results
// of a row the same way.  Keys are packed (score, index), so every merge order gives the same children.
// Reported log-probabilities are those of the raw logits.
__global__ void __launch_bounds__(256)
sx_gumbel_topk_kernel(int V, int T, int chunk, const float *logits, size_t ld, SxIndex li, SxSample smp,
                      SxHeadPartial *parts) {
  __shared__ unsigned long long s_best[2][8];
  __shared__ float s_m[8], s_l[8];
  sx_pdl_launch_dependents();
  sx_pdl_wait();
  const int r = blockIdx.y, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const float *lg = logits + (size_t)sx_index(li, r) * ld;
  const int row = smp.row0 + r;
  const uint32_t sb = (uint32_t)(row / smp.P), sj = (uint32_t)(row % smp.P) + smp.slot_base;
  const int i0 = blockIdx.x * chunk, i1 = min(V, i0 + chunk);           // chunk is a multiple of 4
  unsigned long long v[SX_MAX_TOPK];
#pragma unroll
  for (int k = 0; k < SX_MAX_TOPK; ++k) v[k] = 0ull;
  float m = -INFINITY, l = 0.f;
  for (int a = i0 + tid * 4; a < i1; a += 256 * 4) {
    uint32_t w[4];
    sx_philox4x32_10((uint32_t)(a >> 2), sj, sb, smp.offset, smp.k0, smp.k1, w);
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const int i = a + e;
      if (i < i1) {
        const float x = lg[i];
        const float mn = fmaxf(m, x);
        l = l * expf(m - mn) + expf(x - mn);          // m = -inf at first: exp(-inf) = 0
        m = mn;
        const unsigned long long key = sx_pack(fmaf(smp.temp, sx_gumbel(w[e]), x), (uint32_t)i);
        if (key > v[SX_MAX_TOPK - 1]) {
          bool gt[SX_MAX_TOPK];
#pragma unroll
          for (int k = 0; k < SX_MAX_TOPK; ++k) gt[k] = v[k] > key;
#pragma unroll
          for (int k = SX_MAX_TOPK - 1; k >= 1; --k) v[k] = gt[k] ? v[k] : (gt[k - 1] ? key : v[k - 1]);
          if (!gt[0]) v[0] = key;
        }
      }
    }
  }
  // (max, sum) of the raw logits over the chunk
  float mm = sx_warp_max(m);
  if (lane == 0) s_m[warp] = mm;
  __syncthreads();
  mm = s_m[0];
  for (int w2 = 1; w2 < 8; ++w2) mm = fmaxf(mm, s_m[w2]);
  float ll = sx_warp_sum(l > 0.f ? l * expf(m - mm) : 0.f);
  if (lane == 0) s_l[warp] = ll;
  __syncthreads();
  float lsum = 0.f;
  for (int w2 = 0; w2 < 8; ++w2) lsum += s_l[w2];
  SxHeadPartial *out = parts + (size_t)r * gridDim.x + blockIdx.x;
  if (tid == 0) { out->m = mm; out->l = lsum; }
  // tournament over the heads of the 256 sorted lists
  for (int t = 0; t < SX_MAX_TOPK; ++t) {
    unsigned long long best = 0ull;
    if (t < T) {
      best = v[0];
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) best = max(best, __shfl_xor_sync(0xffffffffu, best, o));
      if (lane == 0) s_best[t & 1][warp] = best;
      __syncthreads();
      best = s_best[t & 1][0];
      for (int w2 = 1; w2 < 8; ++w2) best = max(best, s_best[t & 1][w2]);
      if (best != 0ull && v[0] == best) {            // packed keys are unique (index inside): one winner
#pragma unroll
        for (int k = 0; k + 1 < SX_MAX_TOPK; ++k) v[k] = v[k + 1];
        v[SX_MAX_TOPK - 1] = 0ull;
      }
    }
    if (tid == 0) out->top[t] = best;
  }
}

// merge of the C partial results of a row: one warp per row, lane c reads the lists of chunks c, c + 32, ...
__global__ void __launch_bounds__(32)
sx_gumbel_topk_merge_kernel(int V, int T, int C, const SxHeadPartial *parts, const float *logits, size_t ld, SxIndex li,
                            int32_t *tok_out, float *logp_out) {
  sx_pdl_launch_dependents();
  sx_pdl_wait();
  const int r = blockIdx.x, lane = threadIdx.x;
  const SxHeadPartial *pr = parts + (size_t)r * C;
  const float *lg = logits + (size_t)sx_index(li, r) * ld;
  // log-sum-exp of the raw logits
  float m = -INFINITY;
  for (int c = lane; c < C; c += 32) m = fmaxf(m, pr[c].m);
  m = sx_warp_max(m);
  float l = 0.f;
  for (int c = lane; c < C; c += 32) l += pr[c].l > 0.f ? pr[c].l * expf(pr[c].m - m) : 0.f;
  l = sx_warp_sum(l);
  const float lse = m + logf(l);
  // every chunk's list is sorted: a lane walks its chunks' lists with one cursor per chunk (C <= 128: four)
  int cur[4] = {0, 0, 0, 0};
  for (int t = 0; t < T; ++t) {
    unsigned long long mine = 0ull;
    int which = -1;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int c = lane + 32 * j;
      if (c < C && cur[j] < SX_MAX_TOPK) {
        const unsigned long long k = pr[c].top[cur[j]];
        if (k > mine) { mine = k; which = j; }
      }
    }
    unsigned long long best = mine;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) best = max(best, __shfl_xor_sync(0xffffffffu, best, o));
    if (best != 0ull && mine == best) {
#pragma unroll
      for (int j = 0; j < 4; ++j)
        if (j == which) ++cur[j];
    }
    if (lane == 0) {
      const int32_t id = (int32_t)sx_pack_index(best);
      const bool ok = best != 0ull && id >= 0 && id < V;
      tok_out[(size_t)r * T + t] = ok ? id : 0;
      logp_out[(size_t)r * T + t] = ok ? lg[id] - lse : -INFINITY;
    }
  }
}

// parts: room for `cap` partial results
sx_status sx_launch_gumbel_topk(int R, int V, int T, const float *logits, size_t ld, SxIndex li, SxSample smp,
                                SxHeadPartial *parts, size_t cap, int sm_count, int32_t *tok_out, float *logp_out,
                                cudaStream_t st) {
  if (R < 1 || T < 1 || T > SX_MAX_TOPK || (size_t)R > cap) return SX_ERR_UNSUPPORTED;
  int C = (4 * sm_count + R - 1) / R;                 // about four CTAs per SM in all
  if (C > 128) C = 128;
  if ((size_t)R * C > cap) C = (int)(cap / R);
  int chunk = (((V + C - 1) / C) + 1023) / 1024 * 1024;     // whole passes of the CTA: 256 threads x 4 indices
  C = (V + chunk - 1) / chunk;
  SX_TRY(sx_rc(sx_launch(sx_gumbel_topk_kernel, dim3(C, R), dim3(256), 0, st, V, T, chunk, logits, ld, li, smp, parts)));
  return sx_rc(sx_launch(sx_gumbel_topk_merge_kernel, dim3(R), dim3(32), 0, st, V, T, C, (const SxHeadPartial *)parts, logits,
                         ld, li, tok_out, logp_out));
}

// Speculative sampling down a tree with sampled children.  A cluster of SX_WALK_CTAS CTAs per sequence walks
// from the root; CTA k of the cluster owns the k-th slice of the vocabulary.  At the current slot
// p = softmax(target logits / temp) and q = softmax(logits of the drafted row that produced the slot's
// children / temp) are held as unnormalised fp32 vectors (pq: 2 V floats per sequence) with float64 sums; a
// kept child with token x is accepted when u < min(1, p(x) / q(x)), a refusal replaces p by max(0, p - q)
// (renormalised through its sum) and removes x from q; when nothing is accepted the slot's token is a
// Gumbel-max draw over what is left of p.  Sums, maxima and the draw are reduced per CTA, then over the
// cluster through distributed shared memory in rank order, so every CTA holds the same values and takes the
// same branches; the hardware cluster barrier is executed the same number of times by all of them.
#define SX_WALK_CTAS 8
__device__ __forceinline__ double sx_block_sum_d(double v, double *red) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  __syncthreads();
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = v;
  __syncthreads();
  double t = 0.0;
  for (int w = 0; w < (int)(blockDim.x >> 5); ++w) t += red[w];       // same order in every thread
  return t;
}

struct SxClusterSlot {
  double a, b;
  int i, pad;
};
__device__ __forceinline__ void sx_cluster_sync() {
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ SxClusterSlot sx_cluster_read(const SxClusterSlot *local, uint32_t rank) {
  const uint32_t la = (uint32_t)__cvta_generic_to_shared(local);
  uint32_t ra;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(ra) : "r"(la), "r"(rank));
  SxClusterSlot s;
  asm volatile("ld.shared::cluster.f64 %0, [%1];" : "=d"(s.a) : "r"(ra) : "memory");
  asm volatile("ld.shared::cluster.f64 %0, [%1];" : "=d"(s.b) : "r"(ra + 8u) : "memory");
  asm volatile("ld.shared::cluster.s32 %0, [%1];" : "=r"(s.i) : "r"(ra + 16u) : "memory");
  s.pad = 0;
  return s;
}
// Combines the CTAs' values (the same in every thread of a CTA) over the cluster, rank 0 first.
// op 0: a and b are summed; 1: maxima; 2: (a, i) is the best score and its index, larger score first, then lower index.
// slots alternate between two buffers: a CTA can only reach the write of the reduction after the next one once
// every CTA has arrived at the next one's barrier, i.e. has finished reading this one.
__device__ __forceinline__ void sx_cluster_reduce(SxClusterSlot *slots, SxClusterSlot *res, int &phase, int op, double &a,
                                                  double &b, int &i) {
  if (threadIdx.x == 0) {
    slots[phase].a = a; slots[phase].b = b; slots[phase].i = i;
  }
  sx_cluster_sync();
  if (threadIdx.x == 0) {
    SxClusterSlot acc = sx_cluster_read(&slots[phase], 0u);
    for (uint32_t r = 1; r < SX_WALK_CTAS; ++r) {
      const SxClusterSlot o = sx_cluster_read(&slots[phase], r);
      if (op == 0) { acc.a += o.a; acc.b += o.b; }
      else if (op == 1) { acc.a = fmax(acc.a, o.a); acc.b = fmax(acc.b, o.b); }
      else if (o.i >= 0 && (acc.i < 0 || o.a > acc.a || (o.a == acc.a && o.i < acc.i))) { acc.a = o.a; acc.i = o.i; }
    }
    *res = acc;
  }
  __syncthreads();
  a = res->a; b = res->b; i = res->i;
  __syncthreads();                       // res is rewritten by the next reduction
  phase ^= 1;
}

__global__ void __launch_bounds__(1024)
sx_tree_spec_walk_kernel(int P, int V, int rows, int path_stride, const float *target_logits, const float *draft_logits,
                         const int32_t *cand_tok, const int32_t *parent, const int32_t *slot_row, SxSample smp,
                         float *pq, int32_t *target_tok, int32_t *accept_len, int32_t *path, int32_t *recover,
                         int32_t *status) {
  __shared__ double red[32];
  __shared__ double s_best[32];
  __shared__ int s_besti[32];
  __shared__ SxClusterSlot slots[2], res;
  sx_pdl_launch_dependents();
  sx_pdl_wait();
  const int b = blockIdx.x / SX_WALK_CTAS, rank = blockIdx.x % SX_WALK_CTAS, tid = threadIdx.x;
  const bool lead = rank == 0 && tid == 0;
  const int len = ((V + SX_WALK_CTAS - 1) / SX_WALK_CTAS + 3) / 4 * 4;    // slices start at multiples of 4
  const int lo = min(V, rank * len), hi = min(V, lo + len);
  const float inv_tau = 1.0f / smp.temp;
  float *Pv = pq + (size_t)b * 2 * V, *Qv = Pv + V;
  const int32_t *ct = cand_tok + (size_t)b * P, *par = parent + (size_t)b * P, *srow = slot_row + (size_t)b * P;
  int32_t *tt = target_tok + (size_t)b * P, *pa = path + (size_t)b * path_stride;
  if (rank == 0)
    for (int s = tid; s < P; s += blockDim.x) tt[s] = -1;
  if (lead) pa[0] = 0;
  __syncthreads();
  int cur = 0, L = 0, phase = 0, none = -1;
  for (;;) {
    const float *lp = target_logits + ((size_t)b * P + cur) * V;
    const int row = srow[cur];
    int nkids = 0;
    for (int s = cur + 1; s < P; ++s) nkids += (par[s] == cur) ? 1 : 0;      // the same count in every thread
    const bool has_q = nkids > 0 && row >= 0 && row < rows;
    const float *lq = has_q ? draft_logits + ((size_t)b * rows + row) * V : nullptr;
    // maxima, then the unnormalised vectors and their sums
    float mpf = -INFINITY, mqf = -INFINITY;
    for (int i = lo + tid; i < hi; i += blockDim.x) {
      mpf = fmaxf(mpf, lp[i]);
      if (lq) mqf = fmaxf(mqf, lq[i]);
    }
    double mpd = (double)sx_block_max(mpf, red), mqd = (double)sx_block_max(mqf, red);
    sx_cluster_reduce(slots, &res, phase, 1, mpd, mqd, none);
    const float mp = (float)mpd, mq = (float)mqd;
    double sp = 0.0, sq = 0.0;
    for (int i = lo + tid; i < hi; i += blockDim.x) {
      const float a = expf((lp[i] - mp) * inv_tau);
      Pv[i] = a;
      sp += (double)a;
      if (lq) {
        const float c = expf((lq[i] - mq) * inv_tau);
        Qv[i] = c;
        sq += (double)c;
      }
    }
    sp = sx_block_sum_d(sp, red);
    sq = sx_block_sum_d(sq, red);
    sx_cluster_reduce(slots, &res, phase, 0, sp, sq, none);     // its barrier also publishes Pv / Qv to the cluster
    int nxt = -1;
    if (has_q) {
      int refused[SX_MAX_TOPK], nref = 0;
      for (int s = cur + 1; s < P && nxt < 0; ++s) {
        if (par[s] != cur) continue;
        int x = ct[s];
        if (x < 0 || x >= V) {
          if (lead) sx_set_status(status, SX_ERR_CAPACITY);
          x = 0;
        }
        // another CTA of the cluster may own x: read past this SM's L1.  A token refused before at this slot
        // has left q; that is taken from the list, not from memory (its owner clears Qv[x] behind the barrier
        // of the refusal, which orders nothing for the other CTAs), so that all CTAs see the same q(x).
        bool gone = false;
        for (int j = 0; j < nref; ++j) gone |= refused[j] == x;
        const double px_un = (double)__ldcg(Pv + x), qx_un = gone ? 0.0 : (double)__ldcg(Qv + x);
        const double px = px_un / sp, qx = qx_un / sq;
        const double ratio = qx > 0.0 ? fmin(1.0, px / qx) : 1.0;
        uint32_t w[4];
        sx_philox4x32_10(0u, 0x20000000u + (uint32_t)s, (uint32_t)b, smp.offset, smp.k0, smp.k1, w);
        const double u = ((double)(w[0] >> 9) + 0.5) * (1.0 / 8388608.0);
        if (u < ratio) {                                                  // every thread of the cluster takes the same decision
          nxt = s;
          break;
        }
        // refused: p <- max(0, p - q) with its new sum; x leaves q
        const float fsp = (float)(1.0 / sp), fsq = (float)(1.0 / sq);
        double nsp = 0.0, zero = 0.0;
        for (int i = lo + tid; i < hi; i += blockDim.x) {
          const float rr = fmaxf(0.f, Pv[i] * fsp - Qv[i] * fsq);
          Pv[i] = rr;
          nsp += (double)rr;
        }
        nsp = sx_block_sum_d(nsp, red);
        sx_cluster_reduce(slots, &res, phase, 0, nsp, zero, none);        // everyone has read Qv[x] by now
        if (tid == 0 && x >= lo && x < hi) Qv[x] = 0.f;
        __syncthreads();
        if (nref < SX_MAX_TOPK) refused[nref++] = x;
        sp = nsp;
        sq -= qx_un;
      }
    }
    if (nxt >= 0) {
      if (lead) {
        tt[cur] = ct[nxt];
        if (L + 1 < path_stride) pa[L + 1] = nxt;
      }
      cur = nxt;
      ++L;
      continue;
    }
    // the slot's own draw: Gumbel-max over log(what is left of p), lower index among equals
    double best = -INFINITY;
    int besti = -1;
    for (int a = lo + tid * 4; a < hi; a += blockDim.x * 4) {
      uint32_t w[4];
      sx_philox4x32_10((uint32_t)(a >> 2), (uint32_t)cur, (uint32_t)b, smp.offset, smp.k0, smp.k1, w);
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const int i = a + e;
        if (i < hi && Pv[i] > 0.f) {
          const float uu = (float)((w[e] >> 9) * 2u + 1u) * 5.9604644775390625e-8f;
          const double sc = (double)(logf(Pv[i]) - logf(-logf(uu)));
          if (sc > best) { best = sc; besti = i; }
        }
      }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      const double ob = __shfl_xor_sync(0xffffffffu, best, o);
      const int oi = __shfl_xor_sync(0xffffffffu, besti, o);
      if (oi >= 0 && (besti < 0 || ob > best || (ob == best && oi < besti))) { best = ob; besti = oi; }
    }
    if ((tid & 31) == 0) { s_best[tid >> 5] = best; s_besti[tid >> 5] = besti; }
    __syncthreads();
    best = -INFINITY;
    besti = -1;
    for (int w2 = 0; w2 < (int)(blockDim.x >> 5); ++w2) {                  // the same scan in every thread
      const double ob = s_best[w2];
      const int oi = s_besti[w2];
      if (oi >= 0 && (besti < 0 || ob > best || (ob == best && oi < besti))) { best = ob; besti = oi; }
    }
    double unused = 0.0;
    sx_cluster_reduce(slots, &res, phase, 2, best, unused, besti);
    if (lead) {
      if (besti < 0) besti = 0;
      tt[cur] = besti;
      recover[b] = besti;
      accept_len[b] = L;
      for (int j = L + 1; j < path_stride; ++j) pa[j] = -1;
    }
    break;
  }
  sx_cluster_sync();                     // no CTA leaves while another may still read its shared memory
}

size_t sx_tree_spec_ws_bytes(int B, int V) { return (size_t)B * 2 * V * sizeof(float); }

sx_status sx_launch_tree_spec_walk(int B, int P, int V, int rows, int path_stride, const float *target_logits,
                                   const float *draft_logits, const int32_t *cand_tok, const int32_t *parent,
                                   const int32_t *slot_row, SxSample smp, void *pq_ws, int32_t *target_tok,
                                   int32_t *accept_len, int32_t *path, int32_t *recover, int32_t *status,
                                   cudaStream_t st) {
  return sx_rc(sx_launch_cluster(sx_tree_spec_walk_kernel, dim3(B * SX_WALK_CTAS), dim3(1024), 0, SX_WALK_CTAS, st, P, V, rows,
                                 path_stride, target_logits, draft_logits, cand_tok, parent, slot_row, smp, (float *)pq_ws,
                                 target_tok, accept_len, path, recover, status));
}
