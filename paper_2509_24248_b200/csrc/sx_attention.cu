// Decode attention over the paged bf16 KV cache, split over the keys ("split-K").
//
// One warp owns one work item: (sequence b, KV head h, tile of 8 queries, chunk of keys).  The
// queries of a (b, h) pair are the G query heads of the KV head's group for every row the
// sequence drafts this round (1 row in a chain, top-k sibling rows in a tree); when they need
// more than one tile, the tiles go to sibling warps that share one staged copy of the keys and
// values, so each K/V byte leaves HBM once per sequence and round whatever the group size or
// the number of siblings.
//
// Both products run on the warp-level tensor-core path (mma.sync m16n8k16, bf16 in, fp32 out)
// in transposed form, keys (then head-dimension rows) on the 16-row side and the 8 queries on
// the 8-column side:
//     S^T[key][q]  = sum_d K[key][d] Q[q][d]          A = K rows,   B = Q^T
//     O^T[d][q]   += sum_key V[key][d] P[key][q]      A = V^T,      B = P^T
// P^T is obtained from the accumulator layout of S^T with two movmatrix transposes.
//
// K and V rows are staged in a shared-memory ring by asynchronous 16-byte copies (cp.async) that
// are fully coalesced - a step's 16 rows of one page are one contiguous block and every copy
// instruction moves 512 consecutive bytes of it - and land at XOR-swizzled chunk positions, from
// which ldmatrix (plain for K, transposing for V) delivers the A fragments without bank
// conflicts or register shuffling.  Several 16-key steps are in flight while one is computed.
//
// Softmax is the usual running (max, sum) in fp32 with exponentials in base 2; P is rounded to
// bf16 for the second product.  A warp leaves (m, l, unnormalised O) per query and chunk; the
// merge kernel combines the chunks and writes bf16.
#include <math.h>

#include "sx_kernels.cuh"
#include "sx_launch.cuh"

#define SX_ATTN_MAX_STAGES 8    // 16-key steps staged per warp group: one being consumed, the rest in flight
#define SX_ATTN_SMEM_BUDGET (200 * 1024)
#define SX_ATTN_MAX_TILES 8     // query tiles (of 8) per (sequence, KV head): group size * sibling rows <= 64

__device__ __forceinline__ void sx_mma_bf16(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                            uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, "
      "{%0, %1, %2, %3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
// transpose of an 8x8 matrix of 16-bit elements held one row pair per lane
__device__ __forceinline__ uint32_t sx_movmatrix_trans(uint32_t x) {
  uint32_t y;
  asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;" : "=r"(y) : "r"(x));
  return y;
}
__device__ __forceinline__ float sx_ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ uint32_t sx_pack_bf16x2(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t *>(&v);
}
// 16-byte asynchronous copy global -> shared; reads nothing and writes zeros when !valid
// The copies go past L1 (.cg).  With .ca they allocate L1 lines on their way, and the 192 KB a full SM has in
// flight only fit when the kernel found the SM with a large L1: launched programmatically behind a GEMM the CTAs
// inherit that kernel's shared-memory carve-out (the SM never idles, so it is not reconfigured), L1 stays at its
// minimum and every CTA of a long launch ran a quarter slower (batch 32 x 2048-8192 cached tokens: 160 us against
// 126 us in plain stream order; the same 160 us in plain order with the carve-out forced to its maximum).
__device__ __forceinline__ void sx_cp_async16(uint32_t smem_dst, const void *gsrc, bool valid) {
  const uint32_t bytes = valid ? 16u : 0u;
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(smem_dst), "l"(gsrc), "r"(bytes) : "memory");
}
__device__ __forceinline__ void sx_cp_async16_full(uint32_t smem_dst, const void *gsrc) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(smem_dst), "l"(gsrc) : "memory");
}
__device__ __forceinline__ void sx_cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void sx_cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }
// waits until at most n (0..6) of this lane's copy groups are pending
__device__ __forceinline__ void sx_cp_async_wait_n(int n) {
  switch (n) {
    case 0: sx_cp_async_wait<0>(); break;
    case 1: sx_cp_async_wait<1>(); break;
    case 2: sx_cp_async_wait<2>(); break;
    case 3: sx_cp_async_wait<3>(); break;
    case 4: sx_cp_async_wait<4>(); break;
    case 5: sx_cp_async_wait<5>(); break;
    default: sx_cp_async_wait<6>(); break;
  }
}
// barrier over the `threads` threads of warp group `grp` (ids 1 and 2; a CTA holds at most two
// groups of more than one warp)
__device__ __forceinline__ void sx_group_bar(int grp, int threads) {
  if (grp == 0) asm volatile("bar.sync 1, %0;" ::"r"(threads) : "memory");
  else asm volatile("bar.sync 2, %0;" ::"r"(threads) : "memory");
}

// four 8x8 matrices of 16-bit elements from shared memory into MMA fragment registers; lane l
// gives the address of row l % 8 of matrix l / 8
__device__ __forceinline__ void sx_ldmatrix_x4(uint32_t addr, uint32_t &r0, uint32_t &r1, uint32_t &r2, uint32_t &r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
               : "r"(addr));
}
__device__ __forceinline__ void sx_ldmatrix_x4_trans(uint32_t addr, uint32_t &r0, uint32_t &r1, uint32_t &r2,
                                                     uint32_t &r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
               : "r"(addr));
}
// XOR applied to the 16-byte chunk index of a staged K/V row so that the eight rows of an
// ldmatrix phase fall into different bank groups (rows are D * 2 bytes apart)
template <int D>
__device__ __forceinline__ int sx_attn_swz(int key) {
  return D >= 64 ? (key & 7) : (D == 32 ? ((key >> 1) & 3) : ((key >> 2) & 1));
}

// A warp handles NQT tiles of 8 queries (the A fragments of K and V are fetched once per step and
// used for all of them); NT warps form a group that shares one staged copy of the keys and values
// (a warp without queries still does its share of the copies); gpc = groups per CTA.
template <int D, int NT, int NQT>
__global__ void __launch_bounds__(128, 3)
sx_attn_mma_kernel(int nq, int nkv, int G, int page, int page_shift, float scale_log2, SxRowMap rm, int nr, int E,
                   int gpc, int stages, const bf16 *__restrict__ q, sx_kv kv, int nsplit,
                   float2 *__restrict__ ws_ml, float *__restrict__ ws_o, int32_t *status) {
  constexpr int CPR = D / 8;              // 16-byte chunks per K/V row
  constexpr int NLK = D / 16;             // copies per lane for the 16 K rows of a step (as many for V)
  constexpr int NKS = D / 16;             // k-steps of the first product = 16-row tiles of the second
  constexpr int BLK = 16 * D * 2;         // bytes of the K (or V) block of a step
  constexpr bool MULTI = NT > 1;
  constexpr int CNT = (NLK + NT - 1) / NT;  // K copies (and V copies) this warp requests per step
  extern __shared__ uint4 sx_stage[];     // [groups][stages][K block | V block]
  sx_pdl_launch_dependents();
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, t = lane & 3;
  const int grp = MULTI ? warp / NT : warp, qt = MULTI ? warp - grp * NT : 0;
  const int split = blockIdx.x * gpc + grp;
  if (grp >= gpc || split >= nsplit) return;
  const int b = blockIdx.z, h = blockIdx.y;
  const uint32_t stg = (uint32_t)__cvta_generic_to_shared(sx_stage) + (uint32_t)(grp * stages * 2 * BLK);
  sx_pdl_wait();
  const int n = rm.cache_len[b];
  const int total = n + E;
  int chunk = (total + nsplit - 1) / nsplit;
  chunk = (chunk + 15) & ~15;
  const int k0 = split * chunk;
  const int k1 = min(total, k0 + chunk);
  const int NQ = nr * G;

  // B fragments of Q^T: lane (g, t) holds query g of the tile: elements 16ks + 2t, +1 and 16ks + 8 + 2t, +1
  uint32_t qb[NQT][NKS][2];
#pragma unroll
  for (int u = 0; u < NQT; ++u) {
    const int m = (qt * NQT + u) * 8 + g;
    const bool valid = m < NQ;
    const int j = valid ? m / G : 0;
    const int r = b * nr + j;
    const bf16 *qp = q + ((size_t)r * nq + h * G + (valid ? m - j * G : 0)) * D;
#pragma unroll
    for (int ks = 0; ks < NKS; ++ks) {
      qb[u][ks][0] = valid ? *reinterpret_cast<const uint32_t *>(qp + ks * 16 + 2 * t) : 0u;
      qb[u][ks][1] = valid ? *reinterpret_cast<const uint32_t *>(qp + ks * 16 + 8 + 2 * t) : 0u;
    }
  }
  // the two queries whose scores this lane holds (columns 2t and 2t + 1 of the tile)
  int hq[NQT][2];
  bool qv[NQT][2];
  uint64_t vis[NQT][2];
#pragma unroll
  for (int u = 0; u < NQT; ++u)
#pragma unroll
    for (int i = 0; i < 2; ++i) {
      const int m = (qt * NQT + u) * 8 + 2 * t + i;
      qv[u][i] = m < NQ;
      const int j = qv[u][i] ? m / G : 0;
      const int r = b * nr + j;
      hq[u][i] = r * nq + h * G + (qv[u][i] ? m - j * G : 0);
      if (rm.mode == SX_MODE_TREE && rm.round > 1) vis[u][i] = rm.row_mask[r];
      else vis[u][i] = (E >= 64) ? ~0ull : ((1ull << E) - 1ull);
    }

  float o[NQT][NKS][4], mrun[NQT][2], lrun[NQT][2];
#pragma unroll
  for (int u = 0; u < NQT; ++u) {
#pragma unroll
    for (int j = 0; j < NKS; ++j) { o[u][j][0] = 0.f; o[u][j][1] = 0.f; o[u][j][2] = 0.f; o[u][j][3] = 0.f; }
    mrun[u][0] = -INFINITY; mrun[u][1] = -INFINITY; lrun[u][0] = 0.f; lrun[u][1] = 0.f;
  }

  const bf16 *kp = reinterpret_cast<const bf16 *>(kv.k_pages_d);
  const bf16 *vp = reinterpret_cast<const bf16 *>(kv.v_pages_d);
  const int32_t *table = kv.page_table_d + (size_t)b * kv.max_pages;
  // page-table entries of the chunk, one per lane, when they fit
  const int lp_first = (page_shift >= 0) ? (k0 >> page_shift) : k0 / page;
  const int lp_last = (k1 > k0) ? ((page_shift >= 0) ? ((k1 - 1) >> page_shift) : (k1 - 1) / page) : lp_first;
  const bool tbl_in_regs = (lp_last - lp_first) < 32;
  int tbl = -1;
  if (tbl_in_regs && lp_first + lane <= lp_last && lp_first + lane < kv.max_pages) tbl = table[lp_first + lane];
  bool bad = false;
  const bool one_page = (page & 15) == 0;        // chunks start on multiples of 16: a step never straddles pages
  // ---- staging plan ---------------------------------------------------------------------------
  // A step's 16 K rows (then its 16 V rows) are one contiguous block when they share a page; lane
  // l of copy i moves the 16-byte chunk i * 32 + l of the block, i.e. every copy instruction reads
  // 512 contiguous bytes.  In shared memory chunk j of row `key` sits at key * CPR + (j ^ swz(key)).
  // The NT warps of a group take every NT-th copy each: this warp's k-th copy is copy qt + k * NT.
  uint32_t cdst[CNT];
#pragma unroll
  for (int k = 0; k < CNT; ++k) {
    const int ch = (qt + k * NT) * 32 + lane, key = ch / CPR, j = ch % CPR;
    cdst[k] = (uint32_t)((key * CPR + (j ^ sx_attn_swz<D>(key))) * 16);
  }
  // ldmatrix row addresses (relative to the stage buffer).  The XOR only touches the low three bits
  // of the chunk index, so k-step (row tile) j + 4 sits 128 bytes behind j: four addresses each.
  constexpr int NA = NKS < 4 ? NKS : 4;
  uint32_t ka[NA], va[NA];
  {
    const int keyA = (lane & 7) + ((lane >> 3) & 1) * 8, hiA = lane >> 4;
    const int keyV = (lane & 7) + (lane >> 4) * 8, hiV = (lane >> 3) & 1;
#pragma unroll
    for (int ks = 0; ks < NA; ++ks) {
      ka[ks] = (uint32_t)(keyA * 2 * D + (((2 * ks + hiA) ^ sx_attn_swz<D>(keyA)) << 4));
      va[ks] = (uint32_t)(BLK + keyV * 2 * D + (((2 * ks + hiV) ^ sx_attn_swz<D>(keyV)) << 4));
    }
  }
  // offset of the K/V row of `slot` (and whether it may be read); every lane takes part in the shuffle
  auto row_offset = [&](int slot, bool &ok) -> size_t {
    const bool live = slot < k1;
    const int lp = live ? ((page_shift >= 0) ? (slot >> page_shift) : slot / page) : lp_first;
    int pp;
    if (tbl_in_regs) pp = __shfl_sync(0xffffffffu, tbl, lp - lp_first);
    else pp = (lp < kv.max_pages) ? table[lp] : -1;
    ok = live && pp >= 0 && pp < kv.num_pages;
    if (live && !ok) bad = true;
    return ok ? (((size_t)pp * nkv + h) * page + (slot - lp * page)) * D : 0;
  };
  auto issue = [&](int buf, int s0) {
    const uint32_t dst = stg + (uint32_t)(buf * 2 * BLK);
    bool okb = false;
    size_t base = 0;
    if (one_page) base = row_offset(s0, okb);
    if (one_page && okb && s0 + 16 <= k1) {
      const bf16 *kb = kp + base + (qt * 32 + lane) * 8, *vb = vp + base + (qt * 32 + lane) * 8;
#pragma unroll
      for (int k = 0; k < CNT; ++k) {
        if (NLK % NT == 0 || qt + k * NT < NLK) {
          sx_cp_async16_full(dst + cdst[k], kb + k * NT * 256);
          sx_cp_async16_full(dst + BLK + cdst[k], vb + k * NT * 256);
        }
      }
      return;
    }
#pragma unroll
    for (int k = 0; k < CNT; ++k) {
      const int ch = (qt + k * NT) * 32 + lane, key = ch / CPR, j = ch % CPR;
      bool ok;
      size_t of;
      if (one_page) { of = base + (size_t)key * D; ok = okb && (s0 + key < k1); }
      else of = row_offset(s0 + (key < 16 ? key : 0), ok);
      if (NLK % NT == 0 || qt + k * NT < NLK) {
        sx_cp_async16(dst + cdst[k], kp + (ok ? of + j * 8 : 0), ok);
        sx_cp_async16(dst + BLK + cdst[k], vp + (ok ? of + j * 8 : 0), ok);
      }
    }
  };

  const int nsteps = (k1 > k0) ? (k1 - k0 + 15) >> 4 : 0;
  for (int i = 0; i < stages - 1; ++i) {
    if (i < nsteps) issue(i, k0 + i * 16);
    sx_cp_async_commit();
  }
  int buf = 0;
  for (int it = 0; it < nsteps; ++it) {
    const int s0 = k0 + it * 16;
    sx_cp_async_wait_n(stages - 2);                         // this lane's copies of step `it` have landed
    if (MULTI) sx_group_bar(grp, NT * 32);                  // ... and those of every other lane of the group
    else __syncwarp();
    {
      // the buffer consumed in the previous step is free now: request step it + stages - 1 into it
      const int nb = (buf == 0) ? stages - 1 : buf - 1;
      if (it + stages - 1 < nsteps) issue(nb, s0 + (stages - 1) * 16);
      sx_cp_async_commit();
    }
    const uint32_t sb = stg + (uint32_t)(buf * 2 * BLK);
    // ---- S^T = K.Q^T for 16 keys x 8 NQT queries: two accumulation chains per query tile -------
    float s[NQT][4], s2[NQT][4];
#pragma unroll
    for (int u = 0; u < NQT; ++u)
#pragma unroll
      for (int i = 0; i < 4; ++i) { s[u][i] = 0.f; s2[u][i] = 0.f; }
    uint32_t kad[NA], vad[NA];
#pragma unroll
    for (int j = 0; j < NA; ++j) { kad[j] = sb + ka[j]; vad[j] = sb + va[j]; }
#pragma unroll
    for (int ks = 0; ks < NKS; ++ks) {
      uint32_t a0, a1, a2, a3;
      sx_ldmatrix_x4(kad[ks & 3] + (ks >> 2) * 128, a0, a1, a2, a3);
#pragma unroll
      for (int u = 0; u < NQT; ++u) {
        if (ks & 1) sx_mma_bf16(s2[u], a0, a1, a2, a3, qb[u][ks][0], qb[u][ks][1]);
        else sx_mma_bf16(s[u], a0, a1, a2, a3, qb[u][ks][0], qb[u][ks][1]);
      }
    }
    // s[u][0], s[u][1]: key g, queries 2t, 2t+1 of tile u;  s[u][2], s[u][3]: key g + 8
    const bool edge = s0 + 16 > n;             // the step touches drafted rows or the end of the chunk
    uint32_t pb0[NQT], pb1[NQT];
#pragma unroll
    for (int u = 0; u < NQT; ++u) {
#pragma unroll
      for (int i = 0; i < 4; ++i) s[u][i] = (s[u][i] + s2[u][i]) * scale_log2;
      if (edge) {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const int slot = s0 + g + (i >> 1) * 8;
          const bool seen = slot < n || (slot < k1 && ((vis[u][i & 1] >> (slot - n)) & 1ull));
          if (!seen) s[u][i] = -INFINITY;
        }
      }
      // running softmax over the keys (rows): lanes with equal t hold the same two queries
      float corr[2];
#pragma unroll
      for (int i = 0; i < 2; ++i) {
        float mx = fmaxf(s[u][i], s[u][2 + i]);
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 4));
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 8));
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 16));
        // the reference maximum only moves when it is exceeded by more than 2^8: P stays below 256,
        // well inside bf16 and fp32 range, and the accumulators are rescaled rarely
        const float mnew = (mx > mrun[u][i] + 8.0f) ? mx : mrun[u][i];
        const float msafe = (mnew == -INFINITY) ? 0.f : mnew;
        corr[i] = sx_ex2(mrun[u][i] - msafe);
        s[u][i] = sx_ex2(s[u][i] - msafe);
        s[u][2 + i] = sx_ex2(s[u][2 + i] - msafe);
        lrun[u][i] = lrun[u][i] * corr[i] + (s[u][i] + s[u][2 + i]);
        mrun[u][i] = mnew;
      }
      if (__any_sync(0xffffffffu, corr[0] != 1.0f || corr[1] != 1.0f)) {
#pragma unroll
        for (int j = 0; j < NKS; ++j) {
          o[u][j][0] *= corr[0]; o[u][j][1] *= corr[1]; o[u][j][2] *= corr[0]; o[u][j][3] *= corr[1];
        }
      }
      // P^T fragments: (P[key 2t][q g], P[key 2t+1][q g]) and the same for keys 8..15
      pb0[u] = sx_movmatrix_trans(sx_pack_bf16x2(s[u][0], s[u][1]));
      pb1[u] = sx_movmatrix_trans(sx_pack_bf16x2(s[u][2], s[u][3]));
    }
    // ---- O^T += V^T.P^T: tile dt holds d = 16 dt + g (rows g) and 16 dt + 8 + g (rows g + 8) ------------
#pragma unroll
    for (int dt = 0; dt < NKS; ++dt) {
      uint32_t a0, a1, a2, a3;
      sx_ldmatrix_x4_trans(vad[dt & 3] + (dt >> 2) * 128, a0, a1, a2, a3);
#pragma unroll
      for (int u = 0; u < NQT; ++u) sx_mma_bf16(o[u][dt], a0, a1, a2, a3, pb0[u], pb1[u]);
    }
    buf = (buf + 1 == stages) ? 0 : buf + 1;
  }
  sx_cp_async_wait<0>();
  if (__any_sync(0xffffffffu, bad) && lane == 0) sx_set_status(status, SX_ERR_CAPACITY);
  // ---- leave the partial result: O[q][d] ----------------------------------------------------------------
#pragma unroll
  for (int u = 0; u < NQT; ++u)
#pragma unroll
    for (int i = 0; i < 2; ++i) {
      float l = lrun[u][i];
      l += __shfl_xor_sync(0xffffffffu, l, 4);
      l += __shfl_xor_sync(0xffffffffu, l, 8);
      l += __shfl_xor_sync(0xffffffffu, l, 16);
      if (!qv[u][i]) continue;
      const size_t at = (size_t)hq[u][i] * nsplit + split;
      if (g == 0) ws_ml[at] = make_float2(mrun[u][i], l);
      float *dst = ws_o + at * D;
#pragma unroll
      for (int dt = 0; dt < NKS; ++dt) {
        dst[dt * 16 + g] = o[u][dt][i];
        dst[dt * 16 + 8 + g] = o[u][dt][2 + i];
      }
    }
}

// o[hq][d] = sum_s O_s[d] 2^(m_s - M) / sum_s l_s 2^(m_s - M).  One CTA per query row: thread =
// (split group, float4 of the head dimension), 8 or 32 groups, so that the loads of all splits
// are in flight together; at most 256 splits.
__global__ void __launch_bounds__(1024)
sx_attn_merge_kernel(int nq, int d, int nsplit, const float2 *__restrict__ ws_ml, const float *__restrict__ ws_o,
                     bf16 *__restrict__ o_out) {
  __shared__ float s_w[256];               // weights 2^(m_s - M)
  __shared__ float s_red[32], s_sum[32];
  __shared__ float4 s_acc[32][32];
  sx_pdl_launch_dependents();
  const size_t hq = (size_t)blockIdx.y * nq + blockIdx.x;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, nw = blockDim.x >> 5;
  sx_pdl_wait();
  float2 ml = make_float2(-INFINITY, 0.f);
  if (tid < nsplit) ml = ws_ml[hq * nsplit + tid];
  float mm = sx_warp_max(ml.x);
  if (lane == 0) s_red[warp] = mm;
  __syncthreads();
  mm = s_red[0];
  for (int w = 1; w < nw && w < 8; ++w) mm = fmaxf(mm, s_red[w]);      // splits live in the first 256 threads
  const float wgt = (ml.x == -INFINITY) ? 0.f : exp2f(ml.x - mm);
  if (tid < 256) s_w[tid] = wgt;
  const float ls = sx_warp_sum(ml.y * wgt);
  if (lane == 0) s_sum[warp] = ls;
  __syncthreads();
  float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
  if (lane * 4 < d) {
    const float *src = ws_o + hq * nsplit * d + lane * 4;
    for (int sp = warp; sp < nsplit; sp += nw) {
      const float4 v = *reinterpret_cast<const float4 *>(src + (size_t)sp * d);
      const float w = s_w[sp];
      acc.x += v.x * w; acc.y += v.y * w; acc.z += v.z * w; acc.w += v.w * w;
    }
  }
  s_acc[warp][lane] = acc;
  __syncthreads();
  if (tid < d) {
    float ll = 0.f;
    for (int w = 0; w < nw && w < 8; ++w) ll += s_sum[w];
    const float *col = reinterpret_cast<const float *>(&s_acc[0][0]) + tid;
    float a = 0.f;
    for (int w = 0; w < nw; ++w) a += col[w * 128];
    o_out[hq * d + tid] = __float2bfloat16_rn(a / ll);
  }
}

// ---- host side ------------------------------------------------------------------------------------
// 8-query tiles per (sequence, KV head), rounded up to a power of two; a warp takes two of them
// when there are at least two
static int attn_qtiles(const SxShape &sh, int nr) {
  const int t = (nr * (sh.nq / sh.nkv) + 7) / 8;
  return t <= 1 ? 1 : (t <= 2 ? 2 : (t <= 4 ? 4 : 8));
}
static int attn_tiles(const SxShape &sh, int nr) {          // warps per group
  const int t = attn_qtiles(sh, nr);
  return t >= 2 ? t / 2 : 1;
}
static int attn_groups_per_cta(int NT) { return NT >= 4 ? 1 : 4 / NT; }

template <int D>
static bool attn_init_d() {
  const int smem = SX_ATTN_SMEM_BUDGET;
  const cudaFuncAttribute at = cudaFuncAttributeMaxDynamicSharedMemorySize;
  return cudaFuncSetAttribute(sx_attn_mma_kernel<D, 1, 1>, at, smem) == cudaSuccess &&
         cudaFuncSetAttribute(sx_attn_mma_kernel<D, 1, 2>, at, smem) == cudaSuccess &&
         cudaFuncSetAttribute(sx_attn_mma_kernel<D, 2, 2>, at, smem) == cudaSuccess &&
         cudaFuncSetAttribute(sx_attn_mma_kernel<D, 4, 2>, at, smem) == cudaSuccess;
}
sx_status sx_attn_init(int device) {
  (void)device;
  return (attn_init_d<16>() && attn_init_d<32>() && attn_init_d<64>() && attn_init_d<128>()) ? SX_OK : SX_ERR_CUDA;
}

// Key chunks per (sequence, KV head): enough warp groups to fill the machine a few times over,
// at least 32 keys each.
int sx_attn_splits(const SxShape &sh, int B, int nr, int n_cap, int sm_count) {
  const int NT = attn_tiles(sh, nr);
  const int groups = B * sh.nkv;
  const int warps_wanted = sm_count * 12 * 3;
  int want = (warps_wanted / NT + groups - 1) / groups;
  int by_len = (n_cap + 31) / 32;
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
  return worst * (sh.d + 2) * sizeof(float);
}

bool sx_attn_supported(const SxShape &sh) {
  return (sh.d == 16 || sh.d == 32 || sh.d == 64 || sh.d == 128) &&
         attn_qtiles(sh, SX_MAX_TOPK) <= SX_ATTN_MAX_TILES;
}

sx_status sx_launch_attention(const SxShape &sh, const SxRowMap &rm, int B, int nr, int E, const bf16 *q, const sx_kv &kv,
                         int nsplit, float *ws, bf16 *o_out, int sm_count, int32_t *status, cudaStream_t st) {
  const int R = B * nr;
  const int G = sh.nq / sh.nkv;
  const int NT = attn_tiles(sh, nr);
  const int gpc = attn_groups_per_cta(NT);
  float2 *ws_ml = reinterpret_cast<float2 *>(ws);
  float *ws_o = ws + (size_t)R * sh.nq * nsplit * 2;
  const float scale_log2 = (float)(1.4426950408889634 / sqrt((double)sh.d));
  int page_shift = -1;
  if ((sh.page & (sh.page - 1)) == 0)
    for (page_shift = 0; (1 << page_shift) < sh.page; ++page_shift) {}
  dim3 grid((nsplit + gpc - 1) / gpc, sh.nkv, B);
  dim3 block(32 * NT * gpc);
  // Stages per group: a group of NT warps shares one ring, so it gets NT times the depth of a
  // single warp's (two steps), within the shared-memory budget.
  int stages = 2 * NT;
  if (stages > SX_ATTN_MAX_STAGES) stages = SX_ATTN_MAX_STAGES;
  const size_t stage_bytes = (size_t)2 * 16 * sh.d * 2;       // 16 K rows and 16 V rows
  while (stages > 2 && gpc * stages * stage_bytes > SX_ATTN_SMEM_BUDGET) --stages;
  const size_t smem = (size_t)gpc * stages * stage_bytes;
  (void)sm_count;
  cudaError_t err = cudaSuccess;
#define SX_ATTN_NT(DD, NN, QQ)                                                                                          \
  err = sx_launch(sx_attn_mma_kernel<DD, NN, QQ>, grid, block, smem, st, sh.nq, sh.nkv, G, sh.page, page_shift, \
                      scale_log2, rm, nr, E, gpc, stages, q, kv, nsplit, ws_ml, ws_o, status)
#define SX_ATTN(DD)                                  \
  switch (attn_qtiles(sh, nr)) {                     \
    case 1: SX_ATTN_NT(DD, 1, 1); break;             \
    case 2: SX_ATTN_NT(DD, 1, 2); break;             \
    case 4: SX_ATTN_NT(DD, 2, 2); break;             \
    default: SX_ATTN_NT(DD, 4, 2); break;            \
  }
  switch (sh.d) {
    case 16: SX_ATTN(16); break;
    case 32: SX_ATTN(32); break;
    case 64: SX_ATTN(64); break;
    default: SX_ATTN(128); break;
  }
#undef SX_ATTN_NT
#undef SX_ATTN
  if (err != cudaSuccess) return SX_ERR_CUDA;
  return sx_rc(sx_launch(sx_attn_merge_kernel, dim3(sh.nq, R), dim3((nsplit > 64 && sh.nq * R <= 296) ? 1024 : 256), 0, st, sh.nq, sh.d, nsplit,
            (const float2 *)ws_ml, (const float *)ws_o, o_out));
}
