// Decode attention over the paged bf16 KV cache on the 5th-generation tensor cores (sm_100a), for
// head dimension 128, pages of a multiple of 64 slots and up to 32 queries per (sequence, KV head) -
// the group's query heads times the rows the sequence drafts this round (1 in a chain, the sibling
// rows in a tree).
//
// Both products of a block of 128 keys run as tcgen05.mma with the queries on the M side:
//     S[q][key]  = sum_d Q[q][d] K[key][d]       A = Q (shared memory), B = K block (as stored: K-major)
//     O[q][d]   += sum_key P[q][key] V[key][d]   A = P (shared memory), B = V block (as stored: N-major)
// M is 128: the (at most 32) queries are laid out four times, rows 32 w + q (w = 0..3), and replica w
// owns the keys 32 w .. 32 w + 31 of every block: its softmax threads read only those 32 columns of S
// and write only those 32 columns of P (the rest of a P row stays zero), so each of the 128 softmax
// threads owns one row (one TMEM lane) and one quarter of the keys, keeps a running (max, sum) of its
// own, and never exchanges anything with another thread inside the loop.  The four replicas of a query
// are four independent partial results over disjoint keys; they are merged once, when the CTA leaves
// the (sequence, KV head) pair.  The tensor pipe does four times the useful work - it has the time:
// the kernel is bound by the K/V stream.
//
// Work is cut "stream-K" style: all 128-key blocks of all (sequence, KV head) pairs form one list, CTA c
// takes the c-th run of ceil(total / CTAs) consecutive blocks, so every CTA streams the same number of
// bytes whatever the sequence lengths, and leaves one partial result per pair it touched (a pair is
// shared by the few CTAs whose runs meet inside it).  A merge kernel combines those.
//
// Warp roles (192 threads): warp 0 = TMA producer (K and V blocks of 32 KB through a ring of five),
// warp 1 = MMA issuer (owns TMEM: two S accumulators and O), warps 2-5 = softmax / epilogue.
// Every mbarrier wait is bounded (see sx_tc_ptx.cuh).
#include <cuda.h>

#include "sx_kernels.cuh"
#include "sx_launch.cuh"
#include "sx_tc_ptx.cuh"

#define AT_D 128
#define AT_KEYS 128                         // keys per block
#define AT_SLAB 64                          // keys per TMA box (a page holds a multiple of this)
#define AT_NS 5                             // ring slots, one K block or one V block each
#define AT_BLK_BYTES (AT_KEYS * AT_D * 2)   // 32 KB
#define AT_HALF_BYTES (128 * 128)           // a 128-row tile of 64 columns (one swizzle row per matrix row)
#define AT_SLAB_BYTES (AT_SLAB * 128)
#define AT_TMEM_COLS 512                    // S0 | S1 | O (128 columns each), rounded to a power of two
#define AT_O_COL 256
#define AT_SMEM_BYTES (1024 + 2 * 32768 + AT_NS * AT_BLK_BYTES + 256 + 1024)

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

// position of a block's K and V loads in the ring order K0, V0, K1, V1, ...  (requesting V one block later,
// when the MMA issuer gets to it, was tried: the second product then waits for the V block to land and the
// softmax of the next block behind it - 36 % slower)
__device__ __forceinline__ int at_k_entry(int li) { return 2 * li; }
__device__ __forceinline__ int at_v_entry(int li, int n) { (void)n; return 2 * li + 1; }

__global__ void __launch_bounds__(192, 1)
sx_attn_tc_kernel(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV, SxAtParams p) {
  extern __shared__ uint8_t sx_at_raw[];
  uint8_t *smem = reinterpret_cast<uint8_t *>(((uintptr_t)sx_at_raw + 1023) & ~(uintptr_t)1023);
  uint8_t *sQ = smem, *sP = smem + 32768, *ring = smem + 65536;
  uint64_t *bars = reinterpret_cast<uint64_t *>(ring + AT_NS * AT_BLK_BYTES);
  uint64_t *full = bars, *empty = bars + AT_NS, *sfull = bars + 2 * AT_NS, *sempty = sfull + 2;
  uint64_t *pfull = sempty + 2, *pempty = pfull + 1, *qfull = pempty + 1, *ofull = qfull + 1, *oempty = ofull + 1;
  uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(oempty + 1);
  volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_slot + 1);
  float *cm = reinterpret_cast<float *>(reinterpret_cast<uint8_t *>(bars) + 256), *cl = cm + 128;

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
    for (int i = 0; i < 2; ++i) { mbar_init(smem_u32(&sfull[i]), 1); mbar_init(smem_u32(&sempty[i]), 4); }
    mbar_init(smem_u32(pfull), 4);
    mbar_init(smem_u32(pempty), 1);
    mbar_init(smem_u32(qfull), 4);
    mbar_init(smem_u32(ofull), 1);
    mbar_init(smem_u32(oempty), 4);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  // Q and P start as zeros: the parts of a P row outside its owner's 32 keys are never written
  for (int i = threadIdx.x; i < 65536 / 16; i += blockDim.x) reinterpret_cast<uint4 *>(smem)[i] = make_uint4(0, 0, 0, 0);
  fence_async_smem();
  if (warp == 1) {
    tc_alloc(smem_u32(tmem_slot), AT_TMEM_COLS);
    tc_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    // ---- producer ------------------------------------------------------------------------------------
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
    auto load = [&](int entry, bool is_v, int row) {
      const int row0 = __shfl_sync(0xffffffffu, row, 0), row1 = __shfl_sync(0xffffffffu, row, 1);
      if (lane == 0 && ok) {
        const int slot = entry % AT_NS;
        const uint32_t ph = (uint32_t)(entry / AT_NS) & 1u;
        if (entry >= AT_NS && !mbar_wait(smem_u32(&empty[slot]), ph ^ 1u, abort_flag, p.wait_limit)) ok = false;
        if (ok) {
          const uint32_t fb = smem_u32(&full[slot]);
          const uint32_t dst = smem_u32(ring + (size_t)slot * AT_BLK_BYTES);
          const CUtensorMap *map = is_v ? &tmV : &tmK;
          mbar_expect_tx(fb, AT_BLK_BYTES);
#pragma unroll
          for (int s = 0; s < 2; ++s)
#pragma unroll
            for (int hf = 0; hf < 2; ++hf)
              tma_load_2d(dst + hf * AT_HALF_BYTES + s * AT_SLAB_BYTES, map, fb, hf * 64, s ? row1 : row0, pol);
        }
      }
      ok = __shfl_sync(0xffffffffu, (int)ok, 0) != 0;
    };
    int row_cur = rows_of(c);
    for (int li = 0; li < nblk && ok; ++li) {
      // cached keys are inputs of the iteration; the rows drafted in it come from the preceding kernel
      if (!waited && (c.blk + 1) * AT_KEYS > p.cache_len[c.b]) { sx_pdl_wait(); waited = true; }
      AtCursor nx = c;
      at_next(p, nx);
      const int row_next = (li + 1 < nblk) ? rows_of(nx) : p.pool_rows;      // looked up while this block's loads wait
      load(at_k_entry(li), false, row_cur);
      load(at_v_entry(li, nblk), true, row_cur);
      row_cur = row_next;
      c = nx;
    }
    if (__any_sync(0xffffffffu, bad) && lane == 0) sx_set_status(p.status, SX_ERR_CAPACITY);
  } else if (warp == 1) {
    // ---- MMA issuer -----------------------------------------------------------------------------------
    if (lane == 0) {
      // fp32 accumulate, bf16 A and B, M = 128, N = 128; the second product reads V along its rows (N-major B)
      const uint32_t idesc_s = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(128 >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
      const uint32_t idesc_o = idesc_s | (1u << 16);
      const uint32_t q_addr = smem_u32(sQ), p_addr = smem_u32(sP);
      AtCursor c1 = at_seek(p, g0);              // cursor of the next first product
      int li1 = 0, item1 = 0;                    // blocks whose first product has been issued; their item index
      bool ok = true;
      auto mma1 = [&]() {
        const bool first = (li1 == 0) || (c1.blk == 0);
        if (first && li1 > 0) ++item1;
        if (first && !mbar_wait(smem_u32(qfull), (uint32_t)item1 & 1u, abort_flag, p.wait_limit)) { ok = false; return; }
        const int cnt = at_k_entry(li1), slot = cnt % AT_NS, sb = li1 & 1, u = li1 >> 1;
        if (!mbar_wait(smem_u32(&full[slot]), (uint32_t)(cnt / AT_NS) & 1u, abort_flag, p.wait_limit)) { ok = false; return; }
        if (u >= 1 && !mbar_wait(smem_u32(&sempty[sb]), (uint32_t)(u - 1) & 1u, abort_flag, p.wait_limit)) { ok = false; return; }
        tc_fence_after();
        const uint32_t kb = smem_u32(ring + (size_t)slot * AT_BLK_BYTES);
#pragma unroll
        for (int k = 0; k < AT_D / 16; ++k) {
          const uint32_t o = (uint32_t)(k >> 2) * AT_HALF_BYTES + (uint32_t)(k & 3) * 32u;
          tc_mma(tmem_base + (uint32_t)sb * 128u, smem_desc(q_addr + o), smem_desc(kb + o), idesc_s, k > 0 ? 1u : 0u);
        }
        tc_commit(smem_u32(&empty[slot]));
        tc_commit(smem_u32(&sfull[sb]));
        ++li1;
        at_next(p, c1);
      };
      AtCursor c2 = at_seek(p, g0);              // cursor of the next second product
      int item2 = 0;
      mma1();
      for (int li = 0; li < nblk && ok; ++li) {
        if (li + 1 < nblk) mma1();               // keeps the tensor pipe busy while block li's softmax runs
        if (!ok) break;
        const bool first = (li == 0) || (c2.blk == 0);
        const bool last = (li == nblk - 1) || (c2.blk == c2.nb - 1);
        if (first && li > 0) ++item2;
        const int cnt = at_v_entry(li, nblk), slot = cnt % AT_NS;
        if (!mbar_wait(smem_u32(pfull), (uint32_t)li & 1u, abort_flag, p.wait_limit)) break;
        if (!mbar_wait(smem_u32(&full[slot]), (uint32_t)(cnt / AT_NS) & 1u, abort_flag, p.wait_limit)) break;
        if (first && item2 > 0 && !mbar_wait(smem_u32(oempty), (uint32_t)(item2 - 1) & 1u, abort_flag, p.wait_limit)) break;
        tc_fence_after();
        const uint32_t vb = smem_u32(ring + (size_t)slot * AT_BLK_BYTES);
#pragma unroll
        for (int k = 0; k < AT_KEYS / 16; ++k) {
          const uint32_t o = (uint32_t)(k >> 2) * AT_HALF_BYTES + (uint32_t)(k & 3) * 32u;
          tc_mma(tmem_base + AT_O_COL, smem_desc(p_addr + o), smem_desc_mn(vb + (uint32_t)k * 2048u, AT_HALF_BYTES, 1024u),
                 idesc_o, (first && k == 0) ? 0u : 1u);
        }
        tc_commit(smem_u32(&empty[slot]));
        tc_commit(smem_u32(pempty));
        if (last) tc_commit(smem_u32(ofull));
        at_next(p, c2);
      }
    }
  } else {
    // ---- softmax / epilogue: thread = (replica w, query `lane`), TMEM lane 32 w + lane ---------------------
    const int w = warp & 3, tid = threadIdx.x - 64, row = w * 32 + lane;
    const uint32_t lane_base = tmem_base + ((uint32_t)(w * 32) << 16);
    uint8_t *q_row = sQ + row * 128, *p_row = sP + (w >> 1) * AT_HALF_BYTES + row * 128;
    float *scratch = reinterpret_cast<float *>(sP);     // [64 columns][128 rows] at the end of a pair
    sx_pdl_wait();
    AtCursor c = at_seek(p, g0);
    int item = 0;
    float m = -INFINITY, l = 0.f;
    uint64_t vis = 0;
    bool ok = true;
    // the queries of a pair into shared memory, each laid out four times (rows 32 w + q)
    auto load_q = [&](const AtCursor &cc) {
      const bool valid = lane < p.NQ;
      const int j = valid ? lane / p.G : 0, r = cc.b * p.nr + j;
      const uint4 *src = reinterpret_cast<const uint4 *>(p.q + ((size_t)r * p.nq + cc.h * p.G + (valid ? lane - j * p.G : 0)) * AT_D);
#pragma unroll
      for (int ch = 0; ch < 16; ++ch) {
        const uint4 v = valid ? src[ch] : make_uint4(0, 0, 0, 0);
        *reinterpret_cast<uint4 *>(q_row + (ch >> 3) * AT_HALF_BYTES + (((ch & 7) ^ (row & 7)) << 4)) = v;
      }
      fence_async_smem();
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(qfull));
    };
    auto pair_state = [&](const AtCursor &cc) {
      const int j = lane < p.NQ ? lane / p.G : 0, r = cc.b * p.nr + j;
      vis = p.tree_masks ? p.row_mask[r] : (p.E >= 64 ? ~0ull : ((1ull << p.E) - 1ull));
      m = -INFINITY;
      l = 0.f;
    };
    load_q(c);
    pair_state(c);
    for (int li = 0; li < nblk; ++li) {
      const bool first = (li == 0) || (c.blk == 0);
      const bool last = (li == nblk - 1) || (c.blk == c.nb - 1);
      const int sb = li & 1, n = p.cache_len[c.b], ntot = n + p.E;
      if (!epi_all(mbar_wait(smem_u32(&sfull[sb]), (uint32_t)(li >> 1) & 1u, abort_flag, p.wait_limit))) { ok = false; break; }
      tc_fence_after();
      float s[32];
      tc_ld32(lane_base + (uint32_t)(sb * 128 + w * 32), s);
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&sempty[sb]));
      AtCursor nx = c;
      at_next(p, nx);
      // every first product of this pair has completed: the next pair's queries may replace this pair's
      if (last && li + 1 < nblk) load_q(nx);
      // scores in base 2, visibility, block maximum
      const int key0 = c.blk * AT_KEYS + w * 32;
      float mx = -INFINITY;
      if ((c.blk + 1) * AT_KEYS <= n) {
#pragma unroll
        for (int i = 0; i < 32; ++i) { s[i] *= p.scale_log2; mx = fmaxf(mx, s[i]); }
      } else {
#pragma unroll
        for (int i = 0; i < 32; ++i) {
          const int slot = key0 + i;
          const bool seen = slot < n || (slot < ntot && ((vis >> (slot - n)) & 1ull));
          s[i] = seen ? s[i] * p.scale_log2 : -INFINITY;      // a select: whatever an unseen slot holds stays out
          mx = fmaxf(mx, s[i]);
        }
      }
      // the reference maximum moves only when it is exceeded by more than 2^8 (P stays below 256)
      const float mnew = (mx > m + 8.0f) ? mx : m;
      const float msafe = (mnew == -INFINITY) ? 0.f : mnew;
      const float corr = (mnew == m) ? 1.0f : sx_ex2f(m - msafe);
      // the second product of the previous block has completed: P is free again and O is at rest
      if (li >= 1 && !epi_all(mbar_wait(smem_u32(pempty), (uint32_t)(li - 1) & 1u, abort_flag, p.wait_limit))) { ok = false; break; }
      if (!first && __any_sync(0xffffffffu, corr != 1.0f)) {
        tc_fence_after();
#pragma unroll 1
        for (int c0 = 0; c0 < AT_D; c0 += 16) {
          float v[16];
          tc_ld16(lane_base + AT_O_COL + c0, v);
#pragma unroll
          for (int i = 0; i < 16; ++i) v[i] *= corr;
          tc_st16(lane_base + AT_O_COL + c0, v);
        }
        tc_wait_st();
        tc_fence_before();
      }
      float sum = 0.f;
      uint32_t pk[16];
#pragma unroll
      for (int i = 0; i < 32; i += 2) {
        const float a = sx_ex2f(s[i] - msafe), b2 = sx_ex2f(s[i + 1] - msafe);
        sum += a + b2;
        __nv_bfloat162 t2 = __floats2bfloat162_rn(a, b2);
        pk[i >> 1] = *reinterpret_cast<uint32_t *>(&t2);
      }
      l = (first ? 0.f : l * corr) + sum;
      m = mnew;
#pragma unroll
      for (int ch = 0; ch < 4; ++ch)
        *reinterpret_cast<uint4 *>(p_row + ((((w & 1) * 4 + ch) ^ (row & 7)) << 4)) =
            make_uint4(pk[4 * ch], pk[4 * ch + 1], pk[4 * ch + 2], pk[4 * ch + 3]);
      if ((c.blk + 1) * AT_KEYS > ntot) {
        // the block runs past the last slot: what the V rows behind it hold (anything, NaN included) must not
        // meet even a zero probability - clear them once the block has landed
        const int cnt = at_v_entry(li, nblk), slot = cnt % AT_NS, nv = ntot - c.blk * AT_KEYS;
        if (!epi_all(mbar_wait(smem_u32(&full[slot]), (uint32_t)(cnt / AT_NS) & 1u, abort_flag, p.wait_limit))) { ok = false; break; }
        uint8_t *vb = ring + (size_t)slot * AT_BLK_BYTES;
        for (int i = tid; i < (AT_KEYS - nv) * 16; i += 128) {
          const int rr = nv + (i >> 4), ch = i & 15;
          *reinterpret_cast<uint4 *>(vb + (ch >> 3) * AT_HALF_BYTES + rr * 128 + ((ch & 7) << 4)) = make_uint4(0, 0, 0, 0);
        }
      }
      fence_async_smem();
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(pfull));
      if (last) {
        // ---- leave the pair: merge the four replicas of every query, write one partial result ------------
        if (!epi_all(mbar_wait(smem_u32(ofull), (uint32_t)item & 1u, abort_flag, p.wait_limit))) { ok = false; break; }
        tc_fence_after();
        cm[row] = m;
        cl[row] = l;
        epi_bar();
        const float M = fmaxf(fmaxf(cm[lane], cm[32 + lane]), fmaxf(cm[64 + lane], cm[96 + lane]));
        const float wgt = (m == -INFINITY) ? 0.f : sx_ex2f(m - M);
        const int qq = tid & 31, seg = tid >> 5;                   // reduction role: query qq, 16 columns of a half
        const size_t ps = (size_t)blockIdx.x + (size_t)(c.b * p.nkv + c.h);
        if (seg == 0 && qq < p.NQ) {
          float L = 0.f;
#pragma unroll
          for (int ww = 0; ww < 4; ++ww) {
            const float mw = cm[ww * 32 + qq];
            if (mw != -INFINITY) L += cl[ww * 32 + qq] * sx_ex2f(mw - M);
          }
          p.ws_ml[ps * 32 + qq] = make_float2(M, L);
        }
#pragma unroll 1
        for (int hf = 0; hf < 2; ++hf) {
#pragma unroll 1
          for (int c0 = 0; c0 < 64; c0 += 16) {
            float v[16];
            tc_ld16(lane_base + AT_O_COL + hf * 64 + c0, v);
#pragma unroll
            for (int i = 0; i < 16; ++i) scratch[(c0 + i) * 128 + row] = v[i] * wgt;
          }
          epi_bar();
          if (qq < p.NQ) {
            float *dst = p.ws_o + (ps * 32 + qq) * AT_D + hf * 64 + seg * 16;
#pragma unroll
            for (int i = 0; i < 16; i += 4) {
              float4 a;
              const float *sc = scratch + (seg * 16 + i) * 128 + qq;
              a.x = sc[0] + sc[32] + sc[64] + sc[96];
              a.y = sc[128] + sc[160] + sc[192] + sc[224];
              a.z = sc[256] + sc[288] + sc[320] + sc[352];
              a.w = sc[384] + sc[416] + sc[448] + sc[480];
              *reinterpret_cast<float4 *>(dst + i) = a;
            }
          }
          epi_bar();
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(oempty));
        // P served as scratch: back to zeros before the next block's probabilities go in
        for (int i = tid; i < 32768 / 16; i += 128) reinterpret_cast<uint4 *>(sP)[i] = make_uint4(0, 0, 0, 0);
        fence_async_smem();
        epi_bar();
        ++item;
        if (li + 1 < nblk) pair_state(nx);
      }
      c = nx;
    }
    (void)ok;
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
  return sx_rc(cudaFuncSetAttribute(sx_attn_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, AT_SMEM_BYTES));
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
  SX_TRY(sx_rc(sx_launch(sx_attn_tc_kernel, dim3(sm_count), dim3(192), AT_SMEM_BYTES, st, mk, mv, p)));
  return sx_rc(sx_launch(sx_attn_tc_merge_kernel, dim3(B * sh.nkv, p.NQ), dim3(AT_D), 0, st, p, sm_count, o_out));
}
