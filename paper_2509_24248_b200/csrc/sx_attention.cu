// Decode attention over the paged bf16 KV cache, split over the keys ("split-K").
//
// One warp owns one work item: (sequence b, KV head h, tile of 16 queries, chunk of keys).  The
// queries of an item are the G query heads of the KV head's group for every row the sequence
// drafts this round (1 row in a chain, top-k sibling rows in a tree), so each K/V byte is read
// once per sequence and round whatever the group size or the number of siblings.
//
// The products run on the warp-level tensor-core path (mma.sync m16n8k16, bf16 in, fp32 out) with
// every operand fetched straight from global memory into its fragment registers by 16-byte
// loads: the contraction index of Q.K^T (head dimension) and the column index of P.V (head
// dimension again) may be permuted freely, so each lane loads 8 consecutive elements of one key
// and uses them as the fragment entries of two k-steps (Q.K^T) or of eight column tiles (P.V).
// Every 32-byte sector that is fetched is fully used, nothing is staged in shared memory, and
// the bytes in flight are the 16 loads per lane of a 16-key step, re-issued for the next step as soon
// as the current one has consumed its registers.
//
// Softmax is the usual running (max, sum) in fp32 with exponentials in base 2; P is rounded to
// bf16 for the second product.  A warp leaves (m, l, unnormalised O) per query and chunk; the
// combine kernel merges the chunks and writes bf16.
#include <math.h>

#include "sx_kernels.cuh"
#include "sx_launch.cuh"

#define SX_ATTN_WARPS 4

__device__ __forceinline__ void sx_mma_bf16(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, "
      "{%0, %1, %2, %3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

__device__ __forceinline__ uint32_t sx_pack_bf16x2(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t *>(&v);
}

__device__ __forceinline__ uint32_t sx_word(const uint4 &u, int i) {
  return i == 0 ? u.x : (i == 1 ? u.y : (i == 2 ? u.z : u.w));
}

// storage position of head-dimension element d inside a partial-output row (the order in which
// the accumulator fragments hold it): column tile (d / 64) * 8 + d % 8, column (d % 64) / 8
__host__ __device__ __forceinline__ int sx_attn_perm(int d) { return (((d >> 6) << 3) + (d & 7)) * 8 + ((d & 63) >> 3); }

template <int D>
__global__ void __launch_bounds__(SX_ATTN_WARPS * 32, 2)
sx_attn_mma_kernel(int nq, int nkv, int G, int page, float scale_log2, SxRowMap rm, int nr, int E, int MT,
                   const bf16 *__restrict__ q, sx_kv kv, int nsplit, float2 *__restrict__ ws_ml,
                   float *__restrict__ ws_o, int32_t *status) {
  constexpr int NC = (D + 31) / 32;       // 32-element chunks of the head dimension (Q.K^T)
  constexpr int NH = (D + 63) / 64;       // 64-element halves of the head dimension (P.V)
  constexpr int DS = NH * 64;             // partial-output row length
  sx_pdl_launch_dependents();
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, t = lane & 3;
  const int wg = blockIdx.x * SX_ATTN_WARPS + warp;
  const int split = wg / MT, mt = wg - split * MT;
  if (split >= nsplit) return;
  const int b = blockIdx.z, h = blockIdx.y;
  sx_pdl_wait();
  const int n = rm.cache_len[b];
  const int total = n + E;
  int chunk = (total + nsplit - 1) / nsplit;
  chunk = (chunk + 15) & ~15;
  const int k0 = split * chunk;
  const int k1 = min(total, k0 + chunk);
  const int NQ = nr * G;

  // the two query rows of this lane
  int hq[2];
  bool qv[2];
  uint64_t vis[2];
  const bf16 *qp[2];
#pragma unroll
  for (int i = 0; i < 2; ++i) {
    const int m = mt * 16 + g + i * 8;
    qv[i] = m < NQ;
    const int j = qv[i] ? m / G : 0, gh = qv[i] ? m - (m / G) * G : 0;
    const int r = b * nr + j;
    hq[i] = r * nq + h * G + gh;
    qp[i] = q + (size_t)hq[i] * D;
    if (rm.mode == SX_MODE_TREE && rm.round > 1) vis[i] = rm.row_mask[r];
    else vis[i] = (E >= 64) ? ~0ull : ((1ull << E) - 1ull);
  }
  uint32_t qa[NC][2][4];
#pragma unroll
  for (int c = 0; c < NC; ++c) {
    uint4 u0 = make_uint4(0, 0, 0, 0), u1 = u0;
    if (c * 32 + t * 8 < D) {
      if (qv[0]) u0 = *reinterpret_cast<const uint4 *>(qp[0] + c * 32 + t * 8);
      if (qv[1]) u1 = *reinterpret_cast<const uint4 *>(qp[1] + c * 32 + t * 8);
    }
    qa[c][0][0] = u0.x; qa[c][0][1] = u1.x; qa[c][0][2] = u0.y; qa[c][0][3] = u1.y;
    qa[c][1][0] = u0.z; qa[c][1][1] = u1.z; qa[c][1][2] = u0.w; qa[c][1][3] = u1.w;
  }

  float o[NH * 8][4];
#pragma unroll
  for (int j = 0; j < NH * 8; ++j) { o[j][0] = 0.f; o[j][1] = 0.f; o[j][2] = 0.f; o[j][3] = 0.f; }
  float mrun[2] = {-INFINITY, -INFINITY}, lrun[2] = {0.f, 0.f};

  const bf16 *kp = reinterpret_cast<const bf16 *>(kv.k_pages_d);
  const bf16 *vp = reinterpret_cast<const bf16 *>(kv.v_pages_d);
  const int32_t *table = kv.page_table_d + (size_t)b * kv.max_pages;
  // page-table entries of the chunk, one per lane, when they fit
  const int lp_first = k0 / page;
  const int lp_last = (k1 > k0) ? (k1 - 1) / page : lp_first;
  const bool tbl_in_regs = (lp_last - lp_first) < 32;
  int tbl = -1;
  if (tbl_in_regs && lp_first + lane <= lp_last && lp_first + lane < kv.max_pages) tbl = table[lp_first + lane];
  bool bad = false;
  const bool one_page = (page & 15) == 0;        // chunks start on multiples of 16: a step never straddles pages

  // The K registers are refilled for step i + 1 as soon as step i's Q.K^T has consumed them, the V
  // registers as soon as its P.V has: about one step's worth of loads is in flight all the time.
  uint4 kr[2][NC], vr[4][NH];

  // offset of the K/V row of `slot` (and whether it may be read); every lane takes part in the shuffle
  auto row_offset = [&](int slot, bool &ok) -> size_t {
    const bool live = slot < k1;
    const int lp = live ? slot / page : lp_first;
    int pp;
    if (tbl_in_regs) pp = __shfl_sync(0xffffffffu, tbl, lp - lp_first);
    else pp = (lp < kv.max_pages) ? table[lp] : -1;
    ok = live && pp >= 0 && pp < kv.num_pages;
    if (live && !ok) bad = true;
    return ok ? (((size_t)pp * nkv + h) * page + (slot - lp * page)) * D : 0;
  };
  auto issue_k = [&](uint4 (&dst)[2][NC], int s0) {
    bool ok0, ok1;
    size_t o0, o1;
    if (one_page) {
      const size_t base = row_offset(s0, ok0);
      o0 = base + (size_t)g * D;
      o1 = o0 + (size_t)8 * D;
      ok1 = ok0 && (s0 + 8 + g < k1);
      ok0 = ok0 && (s0 + g < k1);
    } else {
      o0 = row_offset(s0 + g, ok0);
      o1 = row_offset(s0 + 8 + g, ok1);
    }
#pragma unroll
    for (int c = 0; c < NC; ++c) {
      dst[0][c] = make_uint4(0, 0, 0, 0);
      dst[1][c] = make_uint4(0, 0, 0, 0);
      if (c * 32 + t * 8 < D) {
        if (ok0) dst[0][c] = *reinterpret_cast<const uint4 *>(kp + o0 + c * 32 + t * 8);
        if (ok1) dst[1][c] = *reinterpret_cast<const uint4 *>(kp + o1 + c * 32 + t * 8);
      }
    }
  };
  auto issue_v = [&](uint4 (&dst)[4][NH], int s0) {
    bool ok[4];
    size_t of[4];
    if (one_page) {
      bool okb;
      const size_t base = row_offset(s0, okb);
#pragma unroll
      for (int kk = 0; kk < 4; ++kk) {
        const int key = (kk >> 1) * 8 + 2 * t + (kk & 1);
        of[kk] = base + (size_t)key * D;
        ok[kk] = okb && (s0 + key < k1);
      }
    } else {
#pragma unroll
      for (int kk = 0; kk < 4; ++kk) of[kk] = row_offset(s0 + (kk >> 1) * 8 + 2 * t + (kk & 1), ok[kk]);
    }
#pragma unroll
    for (int kk = 0; kk < 4; ++kk)
#pragma unroll
      for (int hf = 0; hf < NH; ++hf) {
        dst[kk][hf] = make_uint4(0, 0, 0, 0);
        if (ok[kk] && hf * 64 + g * 8 < D) dst[kk][hf] = *reinterpret_cast<const uint4 *>(vp + of[kk] + hf * 64 + g * 8);
      }
  };
  if (k0 < k1) {
    issue_k(kr, k0);
    issue_v(vr, k0);
  }
  for (int s0 = k0; s0 < k1; s0 += 16) {
    const bool more = s0 + 16 < k1;
    // ---- S = Q.K^T for 16 keys ----------------------------------------------------------
    float s[2][4];
#pragma unroll
    for (int nt = 0; nt < 2; ++nt) {
      s[nt][0] = 0.f; s[nt][1] = 0.f; s[nt][2] = 0.f; s[nt][3] = 0.f;
#pragma unroll
      for (int c = 0; c < NC; ++c) {
        sx_mma_bf16(s[nt], qa[c][0], kr[nt][c].x, kr[nt][c].y);
        sx_mma_bf16(s[nt], qa[c][1], kr[nt][c].z, kr[nt][c].w);
      }
    }
    if (more) issue_k(kr, s0 + 16);
    const bool edge = s0 + 16 > n;             // the step touches drafted rows or the end of the chunk
#pragma unroll
    for (int nt = 0; nt < 2; ++nt)
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        float v = s[nt][i] * scale_log2;
        if (edge) {
          const int slot = s0 + nt * 8 + 2 * t + (i & 1);
          const bool seen = slot < n || (slot < k1 && ((vis[i >> 1] >> (slot - n)) & 1ull));
          if (!seen) v = -INFINITY;
        }
        s[nt][i] = v;
      }
    // ---- running softmax ---------------------------------------------------------------------
    uint32_t pa[4];
#pragma unroll
    for (int rw = 0; rw < 2; ++rw) {
      float mx = fmaxf(fmaxf(s[0][2 * rw], s[0][2 * rw + 1]), fmaxf(s[1][2 * rw], s[1][2 * rw + 1]));
      mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
      mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
      const float mnew = fmaxf(mrun[rw], mx);
      const float msafe = (mnew == -INFINITY) ? 0.f : mnew;
      const float corr = exp2f(mrun[rw] - msafe);
      const float p00 = exp2f(s[0][2 * rw] - msafe), p01 = exp2f(s[0][2 * rw + 1] - msafe);
      const float p10 = exp2f(s[1][2 * rw] - msafe), p11 = exp2f(s[1][2 * rw + 1] - msafe);
      lrun[rw] = lrun[rw] * corr + ((p00 + p01) + (p10 + p11));
      mrun[rw] = mnew;
      pa[rw] = sx_pack_bf16x2(p00, p01);
      pa[2 + rw] = sx_pack_bf16x2(p10, p11);
      if (__any_sync(0xffffffffu, corr != 1.0f)) {
#pragma unroll
        for (int j = 0; j < NH * 8; ++j) { o[j][2 * rw] *= corr; o[j][2 * rw + 1] *= corr; }
      }
    }
    // ---- O += P.V ---------------------------------------------------------------------------------
#pragma unroll
    for (int hf = 0; hf < NH; ++hf)
#pragma unroll
      for (int e = 0; e < 8; ++e) {
        const uint32_t sel = (e & 1) ? 0x7632u : 0x5410u;
        const uint32_t b0 = __byte_perm(sx_word(vr[0][hf], e >> 1), sx_word(vr[1][hf], e >> 1), sel);
        const uint32_t b1 = __byte_perm(sx_word(vr[2][hf], e >> 1), sx_word(vr[3][hf], e >> 1), sel);
        sx_mma_bf16(o[hf * 8 + e], pa, b0, b1);
      }
    if (more) issue_v(vr, s0 + 16);
  }
  if (__any_sync(0xffffffffu, bad) && lane == 0) sx_set_status(status, SX_ERR_CAPACITY);
  // ---- leave the partial result ------------------------------------------------------------------
#pragma unroll
  for (int rw = 0; rw < 2; ++rw) {
    float l = lrun[rw];
    l += __shfl_xor_sync(0xffffffffu, l, 1);
    l += __shfl_xor_sync(0xffffffffu, l, 2);
    if (!qv[rw]) continue;
    const size_t at = (size_t)hq[rw] * nsplit + split;
    if (t == 0) ws_ml[at] = make_float2(mrun[rw], l);
    float *dst = ws_o + at * DS;
#pragma unroll
    for (int j = 0; j < NH * 8; ++j)
      *reinterpret_cast<float2 *>(dst + j * 8 + 2 * t) = make_float2(o[j][2 * rw], o[j][2 * rw + 1]);
  }
}

// o[hq][d] = sum_s O_s[d] 2^(m_s - M) / sum_s l_s 2^(m_s - M)
__global__ void sx_attn_merge_kernel(int nq, int d, int ds, int nsplit, const float2 *__restrict__ ws_ml,
                                     const float *__restrict__ ws_o, bf16 *__restrict__ o_out) {
  extern __shared__ float sx_w[];          // [nsplit] weights 2^(m_s - M)
  __shared__ float s_red[2];
  sx_pdl_launch_dependents();
  const size_t hq = (size_t)blockIdx.y * nq + blockIdx.x;
  const int tid = threadIdx.x;
  sx_pdl_wait();
  if (tid < 32) {
    float mm = -INFINITY;
    for (int s = tid; s < nsplit; s += 32) mm = fmaxf(mm, ws_ml[hq * nsplit + s].x);
    mm = sx_warp_max(mm);
    float ll = 0.f;
    for (int s = tid; s < nsplit; s += 32) {
      const float2 v = ws_ml[hq * nsplit + s];
      const float w = (v.x == -INFINITY) ? 0.f : exp2f(v.x - mm);
      sx_w[s] = w;
      ll += v.y * w;
    }
    ll = sx_warp_sum(ll);
    if (tid == 0) s_red[0] = ll;
  }
  __syncthreads();
  const float inv = 1.0f / s_red[0];
  for (int j = tid; j < d; j += blockDim.x) {
    const int at = sx_attn_perm(j);
    float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
    int s = 0;
    for (; s + 4 <= nsplit; s += 4) {
      a0 += ws_o[(hq * nsplit + s) * ds + at] * sx_w[s];
      a1 += ws_o[(hq * nsplit + s + 1) * ds + at] * sx_w[s + 1];
      a2 += ws_o[(hq * nsplit + s + 2) * ds + at] * sx_w[s + 2];
      a3 += ws_o[(hq * nsplit + s + 3) * ds + at] * sx_w[s + 3];
    }
    for (; s < nsplit; ++s) a0 += ws_o[(hq * nsplit + s) * ds + at] * sx_w[s];
    o_out[hq * d + j] = __float2bfloat16_rn(((a0 + a1) + (a2 + a3)) * inv);
  }
}

// ---- host side ------------------------------------------------------------------------------------
static int attn_ds(int d) { return ((d + 63) / 64) * 64; }

// Key chunks per (sequence, KV head, query tile): enough warps to fill the machine a few times
// over, at least 64 keys each.
int sx_attn_splits(const SxShape &sh, int B, int nr, int n_cap, int sm_count) {
  const int G = sh.nq / sh.nkv;
  const int MT = (nr * G + 15) / 16;
  const int groups = B * sh.nkv * MT;
  int want = (sm_count * 8 * 3 + groups - 1) / groups;
  int by_len = (n_cap + 63) / 64;
  int s = want < by_len ? want : by_len;
  if (s < 1) s = 1;
  if (s > 256) s = 256;
  return s;
}

size_t sx_attn_ws_bytes(const SxShape &sh, int max_batch, int max_nr, int sm_count) {
  size_t worst = 0;
  for (int B = 1; B <= max_batch; ++B)
    for (int nr = 1; nr <= max_nr; nr += (max_nr > 1 ? max_nr - 1 : 1)) {
      const size_t rows = (size_t)B * nr * sh.nq * sx_attn_splits(sh, B, nr, 1 << 30, sm_count);
      if (rows > worst) worst = rows;
    }
  return worst * (attn_ds(sh.d) + 2) * sizeof(float);
}

bool sx_attn_supported(const SxShape &sh) { return sh.d == 16 || sh.d == 32 || sh.d == 64 || sh.d == 128; }

void sx_launch_attention(const SxShape &sh, const SxRowMap &rm, int B, int nr, int E, const bf16 *q, const sx_kv &kv,
                         int nsplit, float *ws, bf16 *o_out, int32_t *status, cudaStream_t st) {
  const int R = B * nr;
  const int G = sh.nq / sh.nkv;
  const int MT = (nr * G + 15) / 16;
  const int ds = attn_ds(sh.d);
  float2 *ws_ml = reinterpret_cast<float2 *>(ws);
  float *ws_o = ws + (size_t)R * sh.nq * nsplit * 2;
  const float scale_log2 = (float)(1.4426950408889634 / sqrt((double)sh.d));
  dim3 grid((nsplit * MT + SX_ATTN_WARPS - 1) / SX_ATTN_WARPS, sh.nkv, B);
  dim3 block(SX_ATTN_WARPS * 32);
#define SX_ATTN(DD)                                                                                              \
  sx_launch(sx_attn_mma_kernel<DD>, grid, block, 0, st, sh.nq, sh.nkv, G, sh.page, scale_log2, rm, nr, E, MT, q, kv, \
            nsplit, ws_ml, ws_o, status)
  switch (sh.d) {
    case 16: SX_ATTN(16); break;
    case 32: SX_ATTN(32); break;
    case 64: SX_ATTN(64); break;
    default: SX_ATTN(128); break;
  }
#undef SX_ATTN
  sx_launch(sx_attn_merge_kernel, dim3(sh.nq, R), dim3(128), (size_t)nsplit * sizeof(float), st, sh.nq, sh.d, ds, nsplit,
            (const float2 *)ws_ml, (const float *)ws_o, o_out);
}
