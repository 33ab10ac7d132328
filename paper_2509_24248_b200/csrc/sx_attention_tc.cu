// Decode attention over the paged bf16 KV cache on the 5th-generation tensor cores (sm_100a), for
// head dimension 128, pages of a multiple of 64 slots and up to 32 queries per (sequence, KV head) -
// the group's query heads times the rows the sequence drafts this round (1 in a chain, the sibling
// rows in a tree).
//
// Both products of a block of 128 keys run as tcgen05.mma with the 128-wide side of the data on M, so
// that no tensor-core work is spent on padding:
//     S^T[key][q] = sum_d K[key][d] Q[q][d]         A = K block (as stored: K-major), B = Q         M = keys, N = 32
//     O^T[d][q]  += sum_key V[key][d] P[key][q]     A = V block (as stored: M-major), B = P^T       M = d,    N = 32
// A softmax thread owns one TMEM lane: one key of S^T (its scores against all 32 queries), one head-dimension
// row of O^T.  The softmax of a query runs over keys, i.e. across threads; what makes that cheap is that the
// reference maximum m_q only has to keep the exponentials in range, not be the maximum: all threads hold
// the same m_q in registers and change it only when some score exceeds it by more than 2^8 - an event the
// 128 threads detect with one barrier vote per block - and the sums l_q are kept as per-thread partial sums
// (one per query) that are added up once, when the CTA leaves the (sequence, KV head) pair.  The rare
// update (always the first block of a pair) goes through shared memory: block maximum per query, rescale
// of O^T and of the partial sums.
//
// Work is cut "stream-K" style: all 128-key blocks of all (sequence, KV head) pairs form one list, CTA c
// takes the c-th run of ceil(total / CTAs) consecutive blocks, so every CTA streams the same number of
// bytes whatever the sequence lengths, and leaves one partial result per pair it touched (a pair is
// shared by the few CTAs whose runs meet inside it).  A merge kernel combines those.
//
// Warp roles (384 threads): warps 0 and 11 = TMA producers (K blocks and V blocks of 32 KB, a ring of three
// slots each), warp 1 = issuer of the first product (owns TMEM: two S^T accumulators and O^T, 32 columns each), warp 10 =
// issuer of the second product, warps 2-9 = softmax / epilogue: two warps per TMEM lane quarter, each taking half of the query columns, so that every
// scheduler has two softmax warps to interleave.  P^T is double-buffered: the softmax of a block does not
// wait for the second product of the block before it.  The kernel is compiled for 16 and for 32 query
// columns (a chain with a group of at most 16 query heads takes the narrow one).  Every mbarrier wait is
// bounded (see sx_tc_ptx.cuh).
#include <cuda.h>

#include "sx_kernels.cuh"
#include "sx_launch.cuh"
#include "sx_tc_ptx.cuh"

#define AT_D 128
#define AT_KEYS 128                         // keys per block
#define AT_SLAB 64                          // keys per TMA box (a page holds a multiple of this)
#define AT_NS 6                             // ring slots of 32 KB in all
#ifndef AT_NK
#define AT_NK 3                             // ... of them for K blocks,
#endif
#define AT_NV (AT_NS - AT_NK)               // the rest for V blocks: two rings
#define AT_BLK_BYTES (AT_KEYS * AT_D * 2)   // 32 KB
#define AT_HALF_BYTES (128 * 128)           // a 128-row tile of 64 columns (one swizzle row per matrix row)
#define AT_SLAB_BYTES (AT_SLAB * 128)
#define AT_NQ 32                            // query columns of the accumulators
#define AT_NSB 4                            // S^T accumulators: the first products run up to four blocks ahead of the softmax
#define AT_TMEM_COLS 256                    // S^T 0..3 | O^T 0 | O^T 1 (32 columns each), rounded to a power of two
#define AT_O_COL (AT_NSB * 32)
#define AT_QP_BYTES (AT_NQ * AT_D * 2)      // Q, and P^T: 32 rows of 128 elements
#define AT_SMEM_BYTES (1024 + 3 * AT_QP_BYTES + AT_NS * AT_BLK_BYTES + 256 + 512 + 256 + 128)
#define AT_EPI_THREADS 256
#define AT_MMA2_WARP 10                     // warps 0, 1: producer, first product; 2-9: softmax; 10: second product
#define AT_VPROD_WARP 11                    // producer of the V ring
#define AT_THREADS (64 + AT_EPI_THREADS + 64)

struct SxAtParams {
  int nq, nkv, G, page, nr, E, NQ, B, tree_masks;
  float scale_log2;
  const int32_t *cache_len;
  const uint64_t *row_mask;
  const int32_t *page_table;
  int max_pages, num_pages, pool_rows;
  const bf16 *q;
  float2 *ws_ml;
  float *ws_o;
  int32_t *status;
  uint32_t wait_limit;
};

__device__ __forceinline__ float sx_ex2f(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// ---- the block list --------------------------------------------------------------------------------
__device__ __forceinline__ int at_blocks(int n, int E) { return (n + E + AT_KEYS - 1) / AT_KEYS; }

struct AtCursor {
  int b, h, blk, nb;
};
// total number of blocks and the (sequence, head, block) of list position g
__device__ __forceinline__ int at_total(const SxAtParams &p) {
  int total = 0;
  for (int b = 0; b < p.B; ++b) total += p.nkv * at_blocks(p.cache_len[b], p.E);
  return total;
}
__device__ __forceinline__ AtCursor at_seek(const SxAtParams &p, int g) {
  AtCursor c{0, 0, 0, 0};
  int base = 0;
  for (int b = 0; b < p.B; ++b) {
    const int nb = at_blocks(p.cache_len[b], p.E);
    if (g < base + p.nkv * nb) {
      c.b = b; c.nb = nb; c.h = (g - base) / nb; c.blk = (g - base) - c.h * nb;
      return c;
    }
    base += p.nkv * nb;
  }
  c.b = p.B;
  return c;
}
__device__ __forceinline__ void at_next(const SxAtParams &p, AtCursor &c) {
  if (++c.blk == c.nb) {
    c.blk = 0;
    if (++c.h == p.nkv) {
      c.h = 0;
      ++c.b;
      c.nb = c.b < p.B ? at_blocks(p.cache_len[c.b], p.E) : 1;
    }
  }
}

__device__ __forceinline__ void at_bar() { asm volatile("bar.sync 1, 256;" ::: "memory"); }
// barrier over the 256 softmax threads that also ANDs a flag, so that they all take the same branch
__device__ __forceinline__ bool at_all(bool ok) {
  uint32_t out;
  asm volatile(
      "{\n\t.reg .pred pi, po;\n\t"
      "setp.ne.u32 pi, %1, 0;\n\t"
      "bar.red.and.pred po, 1, 256, pi;\n\t"
      "selp.u32 %0, 1, 0, po;\n\t}"
      : "=r"(out)
      : "r"((uint32_t)ok)
      : "memory");
  return out != 0;
}

template <int NQT>       // query columns of the accumulators: 16 or 32
__global__ void __launch_bounds__(AT_THREADS, 1)
sx_attn_tc_kernel(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV, SxAtParams p) {
  constexpr int QH = NQT / 2;                 // query columns per softmax thread
  extern __shared__ uint8_t sx_at_raw[];
  uint8_t *smem = reinterpret_cast<uint8_t *>(((uintptr_t)sx_at_raw + 1023) & ~(uintptr_t)1023);
  uint8_t *sQ = smem, *sPT = smem + AT_QP_BYTES, *ring = smem + 3 * AT_QP_BYTES;      // P^T: two buffers
  uint64_t *bars = reinterpret_cast<uint64_t *>(ring + AT_NS * AT_BLK_BYTES);
  // K ring: full[0..2] / empty[0..2]; V ring: full[3..5] / empty[3..5]
  uint64_t *full = bars, *empty = bars + AT_NS, *sfull = bars + 2 * AT_NS, *sempty = sfull + AT_NSB;
  uint64_t *pfull = sempty + AT_NSB, *pempty = pfull + 2, *qfull = pempty + 2, *ofull = qfull + 1, *oempty = ofull + 2;
  uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(oempty + 2);
  volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_slot + 1);
  float *red = reinterpret_cast<float *>(reinterpret_cast<uint8_t *>(bars) + 256);  // [4 lane quarters][32 queries]
  uint64_t *vis_sh = reinterpret_cast<uint64_t *>(red + 128);                       // [32] visibility of the drafted rows
  float *m_sh = reinterpret_cast<float *>(vis_sh + 32);                             // [32]

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  sx_pdl_launch_dependents();
  // this CTA's run of the block list (cache lengths are inputs of the iteration: no wait needed)
  const int total = at_total(p);
  int per = (total + (int)gridDim.x - 1) / (int)gridDim.x;
  if (per < 1) per = 1;
  const int g0 = min(total, (int)blockIdx.x * per), g1 = min(total, g0 + per);
  if (g0 >= g1) return;
  const int nblk = g1 - g0;

  if (threadIdx.x == 0) {
    for (int i = 0; i < AT_NS; ++i) { mbar_init(smem_u32(&full[i]), 1); mbar_init(smem_u32(&empty[i]), 1); }
    for (int i = 0; i < AT_NSB; ++i) {
      mbar_init(smem_u32(&sfull[i]), 1);
      mbar_init(smem_u32(&sempty[i]), 8);
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(smem_u32(&pempty[i]), 1);
      // one barrier per P^T buffer: a buffer is refilled only after the second product that read it has
      // completed, so its barrier can never run a whole phase ahead of the MMA issuer (a single barrier
      // for both buffers could: the softmax may be a block ahead)
      mbar_init(smem_u32(&pfull[i]), 8);
    }
    mbar_init(smem_u32(qfull), 8);
    for (int i = 0; i < 2; ++i) {            // O^T of consecutive pairs alternates between two accumulators
      mbar_init(smem_u32(&ofull[i]), 1);
      mbar_init(smem_u32(&oempty[i]), 8);
    }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    tc_alloc(smem_u32(tmem_slot), AT_TMEM_COLS);
    tc_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0 || warp == AT_VPROD_WARP) {
    // ---- producers: warp 0 streams the K blocks of the run through ring slots 0-2, warp 11 the V blocks
    // through slots 3-5.  Two rings, because the two streams are consumed at different points of a block's
    // life (K at once, V only after the scores have been through the softmax): in one ring a landed V block
    // would hold a slot the K stream could have in flight.
    const bool is_v = warp != 0;
    const int base_slot = is_v ? AT_NK : 0, nring = is_v ? AT_NV : AT_NK;
    const CUtensorMap *map = is_v ? &tmV : &tmK;
    const uint64_t pol = policy_evict_first();
    AtCursor c = at_seek(p, g0);
    bool waited = false, ok = true, bad = false;
    // first rows of the two 64-key boxes of a block (lanes 0 and 1 look them up)
    auto rows_of = [&](const AtCursor &cc) -> int {
      int row = p.pool_rows;                         // a box that starts behind the last row reads zeros
      if (lane < 2 && cc.b < p.B) {
        const int ntot = p.cache_len[cc.b] + p.E, slot0 = cc.blk * AT_KEYS + lane * AT_SLAB;
        if (slot0 < ntot) {
          const int lp = slot0 / p.page, off = slot0 - lp * p.page;
          const int pp = lp < p.max_pages ? p.page_table[(size_t)cc.b * p.max_pages + lp] : -1;
          if (pp < 0 || pp >= p.num_pages) bad = true;
          else row = (pp * p.nkv + cc.h) * p.page + off;
        }
      }
      return row;
    };
    int row_cur = rows_of(c);
    // (Asking L2 for blocks further ahead with cp.async.bulk.prefetch.tensor, to have more than the rings'
    // 64 KB per stream on its way, was tried with 6 blocks of lead: 100 -> 157 us on the tree rounds.)
    for (int li = 0; li < nblk && ok; ++li) {
      // cached keys are inputs of the iteration; the rows drafted in it come from the preceding kernel
      if (!waited && (c.blk + 1) * AT_KEYS > p.cache_len[c.b]) { sx_pdl_wait(); waited = true; }
      AtCursor nx = c;
      at_next(p, nx);
      const int row_next = (li + 1 < nblk) ? rows_of(nx) : p.pool_rows;      // looked up while this block's loads wait
      const int row0 = __shfl_sync(0xffffffffu, row_cur, 0), row1 = __shfl_sync(0xffffffffu, row_cur, 1);
      if (lane == 0) {
        const int slot = base_slot + li % nring;
        const uint32_t ph = (uint32_t)(li / nring) & 1u;
        if (li >= nring && !mbar_wait(smem_u32(&empty[slot]), ph ^ 1u, abort_flag, p.wait_limit)) ok = false;
        if (ok) {
          const uint32_t fb = smem_u32(&full[slot]);
          const uint32_t dst = smem_u32(ring + (size_t)slot * AT_BLK_BYTES);
          mbar_expect_tx(fb, AT_BLK_BYTES);
#pragma unroll
          for (int s = 0; s < 2; ++s)
#pragma unroll
            for (int hf = 0; hf < 2; ++hf)
              tma_load_2d(dst + hf * AT_HALF_BYTES + s * AT_SLAB_BYTES, map, fb, hf * 64, s ? row1 : row0, pol);
        }
      }
      ok = __shfl_sync(0xffffffffu, (int)ok, 0) != 0;
      row_cur = row_next;
      c = nx;
    }
    if (!is_v && __any_sync(0xffffffffu, bad) && lane == 0) sx_set_status(p.status, SX_ERR_CAPACITY);
  } else if (warp == 1) {
    // ---- issuer of the first product (S^T = K.Q^T); owns the TMEM allocation -----------------------------
    if (lane == 0) {
      // fp32 accumulate, bf16 A and B, both K-major, M = 128, N = NQT
      const uint32_t idesc_s = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(NQT >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
      const uint32_t q_addr = smem_u32(sQ);
      AtCursor c1 = at_seek(p, g0);
      int item1 = 0;
      for (int li = 0; li < nblk; ++li) {
        const bool first = (li == 0) || (c1.blk == 0);
        if (first && li > 0) ++item1;
        if (first && !mbar_wait(smem_u32(qfull), (uint32_t)item1 & 1u, abort_flag, p.wait_limit)) break;
        const int slot = li % AT_NK, sb = li % AT_NSB, u = li / AT_NSB;
        if (!mbar_wait(smem_u32(&full[slot]), (uint32_t)(li / AT_NK) & 1u, abort_flag, p.wait_limit)) break;
        if (u >= 1 && !mbar_wait(smem_u32(&sempty[sb]), (uint32_t)(u - 1) & 1u, abort_flag, p.wait_limit)) break;
        tc_fence_after();
        const uint32_t kb = smem_u32(ring + (size_t)slot * AT_BLK_BYTES);
#pragma unroll
        for (int k = 0; k < AT_D / 16; ++k)
          tc_mma(tmem_base + (uint32_t)sb * AT_NQ, smem_desc(kb + (uint32_t)(k >> 2) * AT_HALF_BYTES + (uint32_t)(k & 3) * 32u),
                 smem_desc(q_addr + (uint32_t)(k >> 2) * (AT_NQ * 128) + (uint32_t)(k & 3) * 32u), idesc_s, k > 0 ? 1u : 0u);
        tc_commit(smem_u32(&empty[slot]));
        tc_commit(smem_u32(&sfull[sb]));
        at_next(p, c1);
      }
    }
  } else if (warp == AT_MMA2_WARP) {
    // ---- issuer of the second product (O^T += V^T.P^T): its own thread, so that its waits (probabilities
    // written, V block landed) do not hold up the first products of the blocks behind --------------------
    if (lane == 0) {
      // the second product reads V along its rows: M-major A
      const uint32_t idesc_o = (1u << 4) | (1u << 7) | (1u << 10) | (1u << 15) | ((uint32_t)(NQT >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
      const uint32_t pt_addr = smem_u32(sPT);
      AtCursor c2 = at_seek(p, g0);
      int item2 = 0;
      for (int li = 0; li < nblk; ++li) {
        const bool first = (li == 0) || (c2.blk == 0);
        const bool last = (li == nblk - 1) || (c2.blk == c2.nb - 1);
        if (first && li > 0) ++item2;
        const int slot = AT_NK + li % AT_NV, pb = li & 1;
        if (!mbar_wait(smem_u32(&pfull[pb]), (uint32_t)(li >> 1) & 1u, abort_flag, p.wait_limit)) break;
        if (!mbar_wait(smem_u32(&full[slot]), (uint32_t)(li / AT_NV) & 1u, abort_flag, p.wait_limit)) break;
        const int ob = item2 & 1;
        // the accumulator was last used two pairs ago: its result has been read out
        if (first && item2 >= 2 && !mbar_wait(smem_u32(&oempty[ob]), (uint32_t)((item2 >> 1) - 1) & 1u, abort_flag, p.wait_limit)) break;
        tc_fence_after();
        const uint32_t vb = smem_u32(ring + (size_t)slot * AT_BLK_BYTES), pt = pt_addr + (uint32_t)pb * AT_QP_BYTES;
#pragma unroll
        for (int k = 0; k < AT_KEYS / 16; ++k)
          tc_mma(tmem_base + AT_O_COL + (uint32_t)ob * AT_NQ, smem_desc_mn(vb + (uint32_t)k * 2048u, AT_HALF_BYTES, 1024u),
                 smem_desc(pt + (uint32_t)(k >> 2) * (AT_NQ * 128) + (uint32_t)(k & 3) * 32u), idesc_o,
                 (first && k == 0) ? 0u : 1u);
        tc_commit(smem_u32(&empty[slot]));
        tc_commit(smem_u32(&pempty[pb]));
        if (last) tc_commit(smem_u32(&ofull[ob]));
        at_next(p, c2);
      }
    }
  } else {
    // ---- softmax / epilogue: thread = (TMEM lane i, half hq of the query columns).  Lane i is key i of a
    // block's S^T and row i (of the head dimension) of O^T.
    const int w = warp & 3, etid = threadIdx.x - 64, hq = (warp - 2) >> 2, i = w * 32 + lane, q0 = hq * QH;
    const uint32_t lane_base = tmem_base + ((uint32_t)(w * 32) << 16);
    // this key's column in P^T: 64-key half, 16-byte chunk (XORed with the query row's low bits), byte in the chunk
    const uint32_t pt_col = (uint32_t)((i >> 6) * (AT_NQ * 128) + (i & 7) * 2);
    const int pt_chunk = (i & 63) >> 3;
    sx_pdl_wait();
    AtCursor c = at_seek(p, g0);
    int item = 0;
    float m[QH], lsum[QH];
    // the queries of a pair into shared memory (row = query, 128-byte swizzle); rows beyond the pair's queries are zero
    auto load_q = [&](const AtCursor &cc) {
      const int q = etid >> 3, c8 = etid & 7;
      const bool valid = q < p.NQ;
      const int j = valid ? q / p.G : 0, r = cc.b * p.nr + j;
      const uint4 *src = reinterpret_cast<const uint4 *>(p.q + ((size_t)r * p.nq + cc.h * p.G + (valid ? q - j * p.G : 0)) * AT_D);
#pragma unroll
      for (int jj = 0; jj < 2; ++jj) {
        const int ch = c8 * 2 + jj;
        const uint4 v = valid ? src[ch] : make_uint4(0, 0, 0, 0);
        *reinterpret_cast<uint4 *>(sQ + (ch >> 3) * (AT_NQ * 128) + q * 128 + (((ch & 7) ^ (q & 7)) << 4)) = v;
      }
      fence_async_smem();
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(qfull));
    };
    auto pair_state = [&](const AtCursor &cc) {
      if (etid < AT_NQ) {
        const int j = etid < p.NQ ? etid / p.G : 0, r = cc.b * p.nr + j;
        vis_sh[etid] = p.tree_masks ? p.row_mask[r] : (p.E >= 64 ? ~0ull : ((1ull << p.E) - 1ull));
      }
#pragma unroll
      for (int q = 0; q < QH; ++q) { m[q] = -INFINITY; lsum[q] = 0.f; }
    };
    int pend_item = -1;
    size_t pend_ps = 0;
    auto flush_pending = [&]() -> bool {
      const int ob = pend_item & 1;
      if (!at_all(mbar_wait(smem_u32(&ofull[ob]), (uint32_t)(pend_item >> 1) & 1u, abort_flag, p.wait_limit))) return false;
      tc_fence_after();
      float v[QH];
      if (QH == 16) tc_ld16(lane_base + AT_O_COL + (uint32_t)ob * AT_NQ + q0, v);
      else tc_ld8(lane_base + AT_O_COL + (uint32_t)ob * AT_NQ + q0, v);
#pragma unroll
      for (int q = 0; q < QH; ++q)
        if (q0 + q < p.NQ) p.ws_o[(pend_ps * 32 + q0 + q) * AT_D + i] = v[q];     // a warp: 32 consecutive floats
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&oempty[ob]));
      pend_item = -1;
      return true;
    };
    load_q(c);
    pair_state(c);
    for (int li = 0; li < nblk; ++li) {
      const bool first = (li == 0) || (c.blk == 0);
      const bool last = (li == nblk - 1) || (c.blk == c.nb - 1);
      const int sb = li % AT_NSB, pb = li & 1, n = p.cache_len[c.b], ntot = n + p.E;
      if (!at_all(mbar_wait(smem_u32(&sfull[sb]), (uint32_t)(li / AT_NSB) & 1u, abort_flag, p.wait_limit))) break;
      tc_fence_after();
      float s[QH];
      if (QH == 16) tc_ld16(lane_base + (uint32_t)(sb * AT_NQ + q0), s);
      else tc_ld8(lane_base + (uint32_t)(sb * AT_NQ + q0), s);
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&sempty[sb]));
      AtCursor nx = c;
      at_next(p, nx);
      // every first product of this pair has completed: the next pair's queries may replace this pair's
      if (last && li + 1 < nblk) load_q(nx);
      // scores in base 2; a slot this thread's key may not be seen from gives -inf (a select: whatever the
      // slot holds stays out)
      const int slot = c.blk * AT_KEYS + i;
      bool exceed = false;
      if ((c.blk + 1) * AT_KEYS <= n) {
#pragma unroll
        for (int q = 0; q < QH; ++q) { s[q] *= p.scale_log2; exceed |= s[q] > m[q] + 8.0f; }
      } else {
        const bool cached = slot < n, drafted = slot >= n && slot < ntot;
#pragma unroll
        for (int q = 0; q < QH; ++q) {
          const bool seen = cached || (drafted && ((vis_sh[q0 + q] >> (slot - n)) & 1ull));
          s[q] = seen ? s[q] * p.scale_log2 : -INFINITY;
          exceed |= s[q] > m[q] + 8.0f;
        }
      }
      // the second product of the block before the previous one has completed: this P^T buffer is free again
      if (li >= 2 && !at_all(mbar_wait(smem_u32(&pempty[pb]), (uint32_t)((li >> 1) - 1) & 1u, abort_flag, p.wait_limit))) break;
      if (first || !at_all(!exceed)) {
        // ---- a reference maximum moves: block maximum per query over the 128 keys -------------------------
        // O^T must be at rest for the rescale: the second product of the previous block has completed
        if (li >= 1 && !at_all(mbar_wait(smem_u32(&pempty[pb ^ 1]), (uint32_t)((li - 1) >> 1) & 1u, abort_flag, p.wait_limit))) break;
#pragma unroll
        for (int q = 0; q < QH; ++q) {
          float bm = s[q];
#pragma unroll
          for (int o = 16; o > 0; o >>= 1) bm = fmaxf(bm, __shfl_xor_sync(0xffffffffu, bm, o));
          if (lane == 0) red[w * 32 + q0 + q] = bm;
        }
        at_bar();
        float corr[QH];
        bool any = false;
#pragma unroll
        for (int q = 0; q < QH; ++q) {
          const int qa = q0 + q;
          const float bm = fmaxf(fmaxf(red[qa], red[32 + qa]), fmaxf(red[64 + qa], red[96 + qa]));
          const float mold = m[q];
          const float mnew = (first || bm > mold + 8.0f) ? bm : mold;
          corr[q] = (first || mnew == mold) ? 1.0f : sx_ex2f(mold - mnew);      // mnew > mold is finite here
          any |= corr[q] != 1.0f;
          m[q] = mnew;
          lsum[q] = first ? 0.f : lsum[q] * corr[q];
        }
        if (__any_sync(0xffffffffu, any)) {                   // the same in every lane of the warp: same inputs
          float v[QH];
          tc_fence_after();
          const uint32_t ocol = lane_base + AT_O_COL + (uint32_t)(item & 1) * AT_NQ + q0;
          if (QH == 16) tc_ld16(ocol, v);
          else tc_ld8(ocol, v);
#pragma unroll
          for (int q = 0; q < QH; ++q) v[q] *= corr[q];
          if (QH == 16) tc_st16(ocol, v);
          else tc_st8(ocol, v);
          tc_wait_st();
          tc_fence_before();
        }
        at_bar();                                              // red may be rewritten from here on
      }
      // probabilities (below 2^8), their partial sums, and this key's column of P^T
      {
        uint8_t *col = sPT + pb * AT_QP_BYTES + pt_col;
#pragma unroll
        for (int q = 0; q < QH; ++q) {
          const int qa = q0 + q;
          const float pq = sx_ex2f(s[q] - ((m[q] == -INFINITY) ? 0.f : m[q]));
          lsum[q] += pq;
          *reinterpret_cast<__nv_bfloat16 *>(col + qa * 128 + ((pt_chunk ^ (qa & 7)) << 4)) = __float2bfloat16_rn(pq);
        }
      }
      if ((c.blk + 1) * AT_KEYS > ntot) {
        // the block runs past the last slot: what the V rows behind it hold (anything, NaN included) must not
        // meet even a zero probability - clear them once the block has landed
        const int vslot = AT_NK + li % AT_NV, nv = ntot - c.blk * AT_KEYS;
        if (!at_all(mbar_wait(smem_u32(&full[vslot]), (uint32_t)(li / AT_NV) & 1u, abort_flag, p.wait_limit))) break;
        uint8_t *vb = ring + (size_t)vslot * AT_BLK_BYTES;
        for (int e = etid; e < (AT_KEYS - nv) * 16; e += AT_EPI_THREADS) {
          const int rr = nv + (e >> 4), ch = e & 15;
          *reinterpret_cast<uint4 *>(vb + (ch >> 3) * AT_HALF_BYTES + rr * 128 + ((ch & 7) << 4)) = make_uint4(0, 0, 0, 0);
        }
      }
      fence_async_smem();
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&pfull[pb]));
      // The O^T of a pair that ended one block ago: its last second product has surely completed by now, so
      // reading it out here costs no wait, and the pair that follows it was not held up (two accumulators).
      if (pend_item >= 0 && !flush_pending()) break;
      if (last) {
        // ---- leave the pair: add up the partial sums, write (m, l) per query; O^T follows one block later ----
#pragma unroll
        for (int q = 0; q < QH; ++q) {
          float a = lsum[q];
#pragma unroll
          for (int o = 16; o > 0; o >>= 1) a += __shfl_xor_sync(0xffffffffu, a, o);
          if (lane == 0) red[w * 32 + q0 + q] = a;
          if (lane == 0 && w == 0) m_sh[q0 + q] = m[q];
        }
        at_bar();
        const size_t ps = (size_t)blockIdx.x + (size_t)(c.b * p.nkv + c.h);
        if (etid < p.NQ)
          p.ws_ml[ps * 32 + etid] = make_float2(m_sh[etid], (red[etid] + red[32 + etid]) + (red[64 + etid] + red[96 + etid]));
        pend_item = item;
        pend_ps = ps;
        at_bar();                                              // red / m_sh / vis_sh are rewritten from here on
        ++item;
        if (li + 1 < nblk) pair_state(nx);
      }
      c = nx;
    }
    if (pend_item >= 0) flush_pending();
  }
  tc_teardown(abort_flag, p.status, tmem_base, AT_TMEM_COLS);
}

// o[row, head] = sum over the partial results of the pair, weighted 2^(m - M), over the summed weights.
// One CTA per (sequence, KV head, query); a thread owns one column of the head dimension.
__global__ void __launch_bounds__(AT_D) sx_attn_tc_merge_kernel(SxAtParams p, int grid_tc, bf16 *__restrict__ o_out) {
  sx_pdl_launch_dependents();
  const int pair = blockIdx.x, q = blockIdx.y, b = pair / p.nkv, h = pair - b * p.nkv, tid = threadIdx.x;
  const int total = at_total(p);
  int per = (total + grid_tc - 1) / grid_tc;
  if (per < 1) per = 1;
  int start = 0;
  for (int bb = 0; bb < b; ++bb) start += p.nkv * at_blocks(p.cache_len[bb], p.E);
  const int nb = at_blocks(p.cache_len[b], p.E);
  start += h * nb;
  // the partial results of this pair: those of the CTAs whose runs meet in it (a handful)
  const int c_first = start / per, c_last = (start + nb - 1) / per, ns = c_last - c_first + 1;
  sx_pdl_wait();
  const float2 *ml = p.ws_ml + ((size_t)c_first + pair) * 32 + q;
  const float *po = p.ws_o + (((size_t)c_first + pair) * 32 + q) * AT_D + tid;
  float M = -INFINITY;
  for (int s = 0; s < ns; ++s) M = fmaxf(M, ml[(size_t)s * 32].x);
  float L = 0.f, acc = 0.f;
  for (int s = 0; s < ns; ++s) {
    const float2 v = ml[(size_t)s * 32];
    const float wg = (v.x == -INFINITY) ? 0.f : exp2f(v.x - M);
    L += v.y * wg;
    acc += po[(size_t)s * 32 * AT_D] * wg;
  }
  const int j = q / p.G, g = q - j * p.G;
  o_out[((size_t)(b * p.nr + j) * p.nq + h * p.G + g) * AT_D + tid] = __float2bfloat16_rn(acc / L);
}

// ---- host side ------------------------------------------------------------------------------------------
bool sx_attn_tc_supported(const SxShape &sh, int nr, const sx_kv &kv) {
  const long long rows = (long long)kv.num_pages * sh.nkv * sh.page;
  return sh.d == AT_D && sh.page >= AT_SLAB && (sh.page % AT_SLAB) == 0 && nr * (sh.nq / sh.nkv) <= 32 &&
         rows < (1ll << 31) - 256;
}

sx_status sx_attn_tc_init(int device) {
  (void)device;
  if (cudaFuncSetAttribute(sx_attn_tc_kernel<16>, cudaFuncAttributeMaxDynamicSharedMemorySize, AT_SMEM_BYTES) != cudaSuccess ||
      cudaFuncSetAttribute(sx_attn_tc_kernel<32>, cudaFuncAttributeMaxDynamicSharedMemorySize, AT_SMEM_BYTES) != cudaSuccess)
    return SX_ERR_CUDA;
  return SX_OK;
}

size_t sx_attn_tc_ws_bytes(const SxShape &sh, int max_batch, int sm_count) {
  return (size_t)(sm_count + max_batch * sh.nkv) * 32 * (AT_D + 2) * sizeof(float);
}

sx_status sx_launch_attention_tc(const SxShape &sh, const SxRowMap &rm, int B, int nr, int E, const bf16 *q,
                                 const sx_kv &kv, float *ws, bf16 *o_out, int sm_count, int32_t *status,
                                 cudaStream_t st) {
  if (!sx_attn_tc_supported(sh, nr, kv)) return SX_ERR_UNSUPPORTED;
  SxAtParams p;
  memset(&p, 0, sizeof(p));
  p.nq = sh.nq; p.nkv = sh.nkv; p.G = sh.nq / sh.nkv; p.page = sh.page; p.nr = nr; p.E = E; p.NQ = nr * p.G; p.B = B;
  p.tree_masks = (rm.mode == SX_MODE_TREE && rm.round > 1) ? 1 : 0;
  p.scale_log2 = (float)(1.4426950408889634 / sqrt((double)sh.d));
  p.cache_len = rm.cache_len;
  p.row_mask = rm.row_mask;
  p.page_table = kv.page_table_d;
  p.max_pages = kv.max_pages;
  p.num_pages = kv.num_pages;
  p.pool_rows = kv.num_pages * sh.nkv * sh.page;
  p.q = q;
  const size_t sets = (size_t)sm_count + (size_t)B * sh.nkv;
  p.ws_ml = reinterpret_cast<float2 *>(ws);
  p.ws_o = ws + sets * 32 * 2;
  p.status = status;
  p.wait_limit = SX_WAIT_LIMIT;
  CUtensorMap mk, mv;
  if (!sx_tma_map_2d(kv.k_pages_d, p.pool_rows, AT_D, AT_SLAB, &mk) || !sx_tma_map_2d(kv.v_pages_d, p.pool_rows, AT_D, AT_SLAB, &mv))
    return SX_ERR_CUDA;
  if (p.NQ <= 16) SX_TRY(sx_rc(sx_launch(sx_attn_tc_kernel<16>, dim3(sm_count), dim3(AT_THREADS), AT_SMEM_BYTES, st, mk, mv, p)));
  else SX_TRY(sx_rc(sx_launch(sx_attn_tc_kernel<32>, dim3(sm_count), dim3(AT_THREADS), AT_SMEM_BYTES, st, mk, mv, p)));
  return sx_rc(sx_launch(sx_attn_tc_merge_kernel, dim3(B * sh.nkv, p.NQ), dim3(AT_D), 0, st, p, sm_count, o_out));
}
