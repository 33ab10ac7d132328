// Skinny GEMMs on the 5th-generation tensor cores (sm_100a): weights stream through a TMA-fed
// shared-memory ring, tcgen05.mma accumulates into TMEM, the epilogue reads TMEM back.
//
//   out[r][n] = sum_k X[r][k] * W[n][k]        W: [n_rows, K] bf16 row-major (K-major)
//                                              X: [R, K]      bf16 row-major (K-major)
//
// The product is formed "swapped": a tile of 128 weight rows is the M side of the MMA, the R
// token rows (padded to a multiple of 16, at most 256) are the N side, so that a handful of
// token rows still fills the 128 TMEM lanes.  Every shape this path sees is bound by the weight
// stream from HBM; the design goal is bytes in flight (deep ring, one persistent CTA per SM),
// not MMA rate.
//
// Warp roles (192 threads): warp 0 = TMA producer (one lane), warp 1 = MMA issuer (one lane,
// owns the TMEM allocation), warps 2-5 = epilogue (one TMEM lane quarter each).  Two TMEM
// accumulators let the epilogue of one tile overlap the main loop of the next.
//
// Every wait on an mbarrier is bounded; when one runs out the CTA raises SX_ERR_TIMEOUT in the
// status word, stops issuing work, lets in-flight copies land, frees its TMEM and returns.
#include <cuda.h>
#include <cudaTypedefs.h>

#include <mutex>
#include <unordered_map>

#include "sx_kernels.cuh"
#include "sx_launch.cuh"
#include "sx_tc_ptx.cuh"

#define SX_BK 64                 // K elements per stage (128 bytes: one swizzle row)
#define SX_A_BYTES (SX_TILE_M * SX_BK * 2)
#define SX_SMEM_MAX 232448
#define SX_ARGMAX_CHUNKS 8        // 32-row chunks of token rows in the plain-argmax epilogue (<= 256 rows)
#define SX_ARGMAX_SMEM (128 * 33 * 4)
#define SX_TOPK_SMEM (4 * 64 * 18 * 4)  // merge buffer of the top-8 epilogue: 4 quarters x 64 rows x 18 words

struct SxTcParams {
  int n_rows, num_kb, R, nmma, num_tiles, splits, kb_per_split, stages, acc_cols, tmem_cols;
  float *part;
  size_t split_stride;
  int V, S, T, lse, part_stride;
  SxHeadPartial *parts;
  float *z;
  int32_t *status;
  SxSample smp;                  // temp > 0: the argmax epilogue draws a Gumbel-max sample instead
  SxLogitsOut lo;                // argmax epilogue: also leave the logits in global memory
  int w_tiled;                   // weights stored tile by tile: [row tile][k-block][128 rows][64 columns]
  uint32_t wait_limit;           // polls of an mbarrier before a wait gives up
};

__device__ __forceinline__ int sx_lo_row(const SxLogitsOut &lo, int r) { return lo.ri.idx ? lo.ri.idx[r] : r * lo.ri.mul + lo.ri.add; }

template <bool HEAD>
__global__ void __launch_bounds__(192, 1)
sx_tc_gemm_kernel(const __grid_constant__ CUtensorMap tmW, const __grid_constant__ CUtensorMap tmX, SxTcParams p) {
  extern __shared__ uint8_t sx_tc_raw[];
  uint8_t *smem = reinterpret_cast<uint8_t *>(((uintptr_t)sx_tc_raw + 1023) & ~(uintptr_t)1023);
  const uint32_t stage_bytes = SX_A_BYTES + (uint32_t)p.nmma * 128u;
  uint64_t *bars = reinterpret_cast<uint64_t *>(smem + (size_t)p.stages * stage_bytes);
  uint64_t *full = bars, *empty = bars + p.stages, *tfull = bars + 2 * p.stages, *tempty = tfull + 2;
  uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(tempty + 2);
  volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_slot + 1);
  uint8_t *epi_smem = reinterpret_cast<uint8_t *>(tmem_slot + 4);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  sx_pdl_launch_dependents();
  if (threadIdx.x == 0) {
    for (int i = 0; i < p.stages; ++i) {
      mbar_init(smem_u32(&full[i]), 1);
      mbar_init(smem_u32(&empty[i]), 1);
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(smem_u32(&tfull[i]), 1);
      mbar_init(smem_u32(&tempty[i]), 4);
    }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    tc_alloc(smem_u32(tmem_slot), (uint32_t)p.tmem_cols);
    tc_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  const int items = HEAD ? p.num_tiles : p.num_tiles * p.splits;

  if (warp == 0) {
    if (lane == 0) {
      const uint64_t pol_w = policy_evict_first(), pol_x = policy_evict_last();
      // The weight tiles depend on nothing: the first ring of them is requested before the wait on
      // the preceding kernel, the activation tiles of those stages right after it.
      //   pass 0: weights of the first `stages` k-blocks     pass 1: their activations
      //   pass 2: every later k-block, weights and activations together
      bool ok = true;
      for (int pass = 0; pass < 3 && ok; ++pass) {
        if (pass == 1) sx_pdl_wait();
        int stage = 0, cnt = 0;
        uint32_t phase = 0;
        for (int item = blockIdx.x; item < items && ok; item += gridDim.x) {
          const int tile = HEAD ? item : item / p.splits;
          const int sp = HEAD ? 0 : item % p.splits;
          const int kb0 = sp * p.kb_per_split;
          const int kb1 = min(p.num_kb, kb0 + p.kb_per_split);
          for (int kb = kb0; kb < kb1; ++kb, ++cnt) {
            if (pass < 2 && cnt >= p.stages) break;
            const uint32_t fb = smem_u32(&full[stage]);
            const uint32_t dst = smem_u32(smem + (size_t)stage * stage_bytes);
            if (pass == 0) {
              mbar_expect_tx(fb, stage_bytes);
              tma_load_2d(dst, &tmW, fb, p.w_tiled ? 0 : kb * SX_BK,
                          p.w_tiled ? (tile * p.num_kb + kb) * SX_TILE_M : tile * SX_TILE_M, pol_w);
            } else if (pass == 1) {
              tma_load_2d(dst + SX_A_BYTES, &tmX, fb, kb * SX_BK, 0, pol_x);
            } else if (cnt >= p.stages) {
              if (!mbar_wait(smem_u32(&empty[stage]), phase ^ 1u, abort_flag, p.wait_limit)) { ok = false; break; }
              mbar_expect_tx(fb, stage_bytes);
              tma_load_2d(dst, &tmW, fb, p.w_tiled ? 0 : kb * SX_BK,
                          p.w_tiled ? (tile * p.num_kb + kb) * SX_TILE_M : tile * SX_TILE_M, pol_w);
              tma_load_2d(dst + SX_A_BYTES, &tmX, fb, kb * SX_BK, 0, pol_x);
            }
            if (++stage == p.stages) { stage = 0; phase ^= 1u; }
          }
          if (pass < 2 && cnt >= p.stages) break;
        }
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      // instruction descriptor: fp32 accumulate, bf16 A and B, both K-major, N = nmma, M = 128
      const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(p.nmma >> 3) << 17) |
                             ((uint32_t)(SX_TILE_M >> 4) << 24);
      int stage = 0, acc = 0;
      uint32_t phase = 0, acc_phase = 0;
      bool ok = true;
      for (int item = blockIdx.x; item < items && ok; item += gridDim.x) {
        const int sp = HEAD ? 0 : item % p.splits;
        const int kb0 = sp * p.kb_per_split;
        const int kb1 = min(p.num_kb, kb0 + p.kb_per_split);
        if (!mbar_wait(smem_u32(&tempty[acc]), acc_phase ^ 1u, abort_flag, p.wait_limit)) break;
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + (uint32_t)(acc * p.acc_cols);
        for (int kb = kb0; kb < kb1; ++kb) {
          if (!mbar_wait(smem_u32(&full[stage]), phase, abort_flag, p.wait_limit)) { ok = false; break; }
          tc_fence_after();
          const uint32_t a = smem_u32(smem + (size_t)stage * stage_bytes);
          const uint32_t b = a + SX_A_BYTES;
#pragma unroll
          for (int k = 0; k < SX_BK / 16; ++k)
            tc_mma(d_tmem, smem_desc(a + k * 32), smem_desc(b + k * 32), idesc, (kb > kb0 || k > 0) ? 1u : 0u);
          tc_commit(smem_u32(&empty[stage]));          // frees the stage once these MMAs have read it
          if (++stage == p.stages) { stage = 0; phase ^= 1u; }
        }
        if (!ok) break;
        tc_commit(smem_u32(&tfull[acc]));              // accumulator complete
        if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
      }
    }
  } else {
    const int q = warp & 3;                            // TMEM lane quarter this warp may read
    const int et = q * 32 + lane;                      // row of the tile owned by this thread
    int acc = 0;
    uint32_t acc_phase = 0;
    sx_pdl_wait();
    if (HEAD && p.T == 1 && !p.lse) {
      // Plain argmax (chain drafting, verification).  The logits of a tile go through a small
      // shared-memory buffer, 32 token rows at a time, so that afterwards a thread owns one token
      // row (column of the tile) and a quarter of the vocabulary rows: it scans them in index
      // order with a strict compare and keeps its running best in registers for the whole
      // kernel - no reductions across lanes and no atomics in the loop.
      float *tb = reinterpret_cast<float *>(epi_smem);          // [128 rows][33]
      const int tid = threadIdx.x - 64, col = tid & 31, part = tid >> 5;
      float bestv[SX_ARGMAX_CHUNKS];
      int besti[SX_ARGMAX_CHUNKS];
#pragma unroll
      for (int ch = 0; ch < SX_ARGMAX_CHUNKS; ++ch) { bestv[ch] = -INFINITY; besti[ch] = -1; }
      for (int item = blockIdx.x; item < items; item += gridDim.x) {
        if (!epi_all(mbar_wait(smem_u32(&tfull[acc]), acc_phase, abort_flag, p.wait_limit))) break;
        tc_fence_after();
        const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(acc * p.acc_cols);
        const int n = item * SX_TILE_M + et;
        const bool in_vocab = n < p.V;
        const bool is_signal = n >= p.V && n < p.V + p.S;
#pragma unroll
        for (int ch = 0; ch < SX_ARGMAX_CHUNKS; ++ch) {
          if (ch * 32 < p.R) {
            float v[32];
            tc_ld16(taddr + ch * 32, v);
            if (ch * 32 + 16 < p.nmma) tc_ld16(taddr + ch * 32 + 16, v + 16);
            else {
#pragma unroll
              for (int j = 16; j < 32; ++j) v[j] = 0.f;
            }
            if ((ch + 1) * 32 >= p.R) {                           // last chunk: the accumulator is free again
              tc_fence_before();
              __syncwarp();
              if (lane == 0) mbar_arrive(smem_u32(&tempty[acc]));
            }
#pragma unroll
            for (int j = 0; j < 32; ++j) tb[et * 33 + j] = in_vocab ? v[j] : -INFINITY;
            if (is_signal) {
#pragma unroll
              for (int j = 0; j < 32; ++j)
                if (ch * 32 + j < p.R) p.z[(size_t)(ch * 32 + j) * p.S + (n - p.V)] = v[j];
            }
            if (p.lo.out && in_vocab) {                           // lanes hold consecutive vocabulary rows
#pragma unroll
              for (int j = 0; j < 32; ++j)
                if (ch * 32 + j < p.R) p.lo.out[(size_t)sx_lo_row(p.lo, ch * 32 + j) * p.lo.ld + n] = v[j];
            }
            epi_bar();
            if (ch * 32 + col < p.R) {
              float bv = bestv[ch];
              int bi = besti[ch];
              const float *src = tb + (part * 32) * 33 + col;
              const int base = item * SX_TILE_M + part * 32;
              if (p.smp.temp > 0.f) {
                // sampled verification: score = logit + temperature * Gumbel(sequence, slot, token id);
                // one generator block serves four consecutive token ids
                const int row = p.smp.row0 + ch * 32 + col;
                const uint32_t sb = (uint32_t)(row / p.smp.P), sj = (uint32_t)(row % p.smp.P) + p.smp.slot_base;
#pragma unroll 2
                for (int r4 = 0; r4 < 8; ++r4) {
                  uint32_t w[4];
                  sx_philox4x32_10((uint32_t)(base >> 2) + r4, sj, sb, p.smp.offset, p.smp.k0, p.smp.k1, w);
#pragma unroll
                  for (int e = 0; e < 4; ++e) {
                    const float x = fmaf(p.smp.temp, sx_gumbel(w[e]), src[(r4 * 4 + e) * 33]);
                    if (x > bv) { bv = x; bi = base + r4 * 4 + e; }
                  }
                }
              } else {
#pragma unroll
                for (int rr = 0; rr < 32; ++rr) {
                  const float x = src[rr * 33];
                  if (x > bv) { bv = x; bi = base + rr; }
                }
              }
              bestv[ch] = bv;
              besti[ch] = bi;
            }
            epi_bar();
          }
        }
        if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
      }
      // Merge the four row quarters per token row.  A quarter's best may come from any tile of this CTA,
      // so quarter order is not index order: the merge ranks (value, then lower index) through the
      // packed key.
      epi_bar();
      int *ci = reinterpret_cast<int *>(tb + 4 * 256);
#pragma unroll
      for (int ch = 0; ch < SX_ARGMAX_CHUNKS; ++ch)
        if (ch * 32 + col < p.R) { tb[part * 256 + ch * 32 + col] = bestv[ch]; ci[part * 256 + ch * 32 + col] = besti[ch]; }
      epi_bar();
      SxHeadPartial *out = p.parts + (size_t)blockIdx.x * p.part_stride;
      for (int r = tid; r < p.R; r += 128) {
        unsigned long long best = 0ull;
        for (int w = 0; w < 4; ++w) {
          const int xi = ci[w * 256 + r];
          if (xi >= 0) best = max(best, sx_pack(tb[w * 256 + r], (uint32_t)xi));
        }
        SxHeadPartial hp;
        hp.top[0] = best;
#pragma unroll
        for (int tt = 1; tt < SX_MAX_TOPK; ++tt) hp.top[tt] = 0ull;
        hp.m = -INFINITY;
        hp.l = 0.f;
        out[r] = hp;
      }
    } else if (HEAD) {
      // Top-8 (value, index) and log-sum-exp per token row (tree drafting; at most 64 token rows).
      // Same data flow as above: a thread owns one token row and a quarter of the vocabulary rows
      // of each tile, and keeps a sorted list of its 8 best and a running (max, sum) in registers.
      float *tb = reinterpret_cast<float *>(epi_smem);          // [128 rows][33]
      const int tid = threadIdx.x - 64, col = tid & 31, part = tid >> 5;
      const float LOG2E = 1.4426950408889634f;
      float tv[2][8], m2[2], ll[2];
      int ti[2][8];
#pragma unroll
      for (int ch = 0; ch < 2; ++ch) {
        m2[ch] = -INFINITY;
        ll[ch] = 0.f;
#pragma unroll
        for (int k = 0; k < 8; ++k) { tv[ch][k] = -INFINITY; ti[ch][k] = -1; }
      }
      for (int item = blockIdx.x; item < items; item += gridDim.x) {
        if (!epi_all(mbar_wait(smem_u32(&tfull[acc]), acc_phase, abort_flag, p.wait_limit))) break;
        tc_fence_after();
        const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(acc * p.acc_cols);
        const int n = item * SX_TILE_M + et;
        const bool in_vocab = n < p.V;
        const bool is_signal = n >= p.V && n < p.V + p.S;
#pragma unroll
        for (int ch = 0; ch < 2; ++ch) {
          if (ch * 32 < p.R) {
            {
              float v[32];
              tc_ld16(taddr + ch * 32, v);
              if (ch * 32 + 16 < p.nmma) tc_ld16(taddr + ch * 32 + 16, v + 16);
              else {
#pragma unroll
                for (int j = 16; j < 32; ++j) v[j] = 0.f;
              }
              if ((ch + 1) * 32 >= p.R) {                         // last chunk: the accumulator is free again
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&tempty[acc]));
              }
#pragma unroll
              for (int j = 0; j < 32; ++j) tb[et * 33 + j] = in_vocab ? v[j] : -INFINITY;
              if (is_signal) {
#pragma unroll
                for (int j = 0; j < 32; ++j)
                  if (ch * 32 + j < p.R) p.z[(size_t)(ch * 32 + j) * p.S + (n - p.V)] = v[j];
              }
              if (p.lo.out && in_vocab) {                         // lanes hold consecutive vocabulary rows
#pragma unroll
                for (int j = 0; j < 32; ++j)
                  if (ch * 32 + j < p.R) p.lo.out[(size_t)sx_lo_row(p.lo, ch * 32 + j) * p.lo.ld + n] = v[j];
              }
            }
            epi_bar();
            if (ch * 32 + col < p.R) {
              const float *src = tb + (part * 32) * 33 + col;
              const int base = item * SX_TILE_M + part * 32;
              float x[32];
#pragma unroll
              for (int rr = 0; rr < 32; ++rr) x[rr] = src[rr * 33];
              if (p.lse) {
                float mx = x[0];
#pragma unroll
                for (int rr = 1; rr < 32; ++rr) mx = fmaxf(mx, x[rr]);
                const float mnew = fmaxf(m2[ch], mx * LOG2E);
                if (mnew > -INFINITY) {
                  float a0 = 0.f, a1 = 0.f;
#pragma unroll
                  for (int rr = 0; rr < 32; rr += 2) {
                    a0 += exp2f(fmaf(x[rr], LOG2E, -mnew));
                    a1 += exp2f(fmaf(x[rr + 1], LOG2E, -mnew));
                  }
                  ll[ch] = ll[ch] * exp2f(m2[ch] - mnew) + (a0 + a1);
                  m2[ch] = mnew;
                }
              }
#pragma unroll
              for (int rr = 0; rr < 32; ++rr) {
                const float xv = x[rr];
                if (xv > tv[ch][7]) {
                  // entries >= xv stay in front of it (they have lower indices), the rest move down
                  bool ge[8];
#pragma unroll
                  for (int k = 0; k < 8; ++k) ge[k] = tv[ch][k] >= xv;
#pragma unroll
                  for (int k = 7; k >= 1; --k) {
                    tv[ch][k] = ge[k] ? tv[ch][k] : (ge[k - 1] ? xv : tv[ch][k - 1]);
                    ti[ch][k] = ge[k] ? ti[ch][k] : (ge[k - 1] ? base + rr : ti[ch][k - 1]);
                  }
                  if (!ge[0]) { tv[ch][0] = xv; ti[ch][0] = base + rr; }
                }
              }
            }
            epi_bar();
          }
        }
        if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
      }
      // Merge the four row quarters per token row.  A quarter's list may hold entries of any tile of this
      // CTA, so the lists are merged on the packed key: larger value first, then the lower index.
      epi_bar();
      int *tbi = reinterpret_cast<int *>(tb);
#pragma unroll
      for (int ch = 0; ch < 2; ++ch)
        if (ch * 32 + col < p.R) {
          const int at = (part * 64 + ch * 32 + col) * 18;
#pragma unroll
          for (int k = 0; k < 8; ++k) { tb[at + k] = tv[ch][k]; tbi[at + 8 + k] = ti[ch][k]; }
          tb[at + 16] = m2[ch];
          tb[at + 17] = ll[ch];
        }
      epi_bar();
      SxHeadPartial *out = p.parts + (size_t)blockIdx.x * p.part_stride;
      if (tid < p.R) {
        const int r = tid;
        unsigned long long bk[8];                  // 0 = empty (below every real entry)
        float M = -INFINITY;
#pragma unroll
        for (int k = 0; k < 8; ++k) bk[k] = 0ull;
        for (int w = 0; w < 4; ++w) {
          const int at = (w * 64 + r) * 18;
          M = fmaxf(M, tb[at + 16]);
          for (int e = 0; e < 8; ++e) {
            const int xi = tbi[at + 8 + e];
            if (xi < 0) break;                     // a list is filled from the front
            const unsigned long long xk = sx_pack(tb[at + e], (uint32_t)xi);
            if (xk > bk[7]) {
              bool gt[8];
#pragma unroll
              for (int k = 0; k < 8; ++k) gt[k] = bk[k] > xk;
#pragma unroll
              for (int k = 7; k >= 1; --k) bk[k] = gt[k] ? bk[k] : (gt[k - 1] ? xk : bk[k - 1]);
              if (!gt[0]) bk[0] = xk;
            }
          }
        }
        float L = 0.f;
        for (int w = 0; w < 4; ++w) {
          const int at = (w * 64 + r) * 18;
          if (tb[at + 17] > 0.f) L += tb[at + 17] * exp2f(tb[at + 16] - M);
        }
        SxHeadPartial hp;
#pragma unroll
        for (int k = 0; k < SX_MAX_TOPK; ++k)
          hp.top[k] = (k < p.T) ? bk[k] : 0ull;
        hp.m = (L > 0.f) ? M * 0.6931471805599453f : -INFINITY;
        hp.l = L;
        out[r] = hp;
      }
    } else {
      // plain GEMM: this split's partial sums to global memory
      for (int item = blockIdx.x; item < items; item += gridDim.x) {
        const int tile = item / p.splits;
        const int sp = item % p.splits;
        if (!epi_all(mbar_wait(smem_u32(&tfull[acc]), acc_phase, abort_flag, p.wait_limit))) break;
        tc_fence_after();
        const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(acc * p.acc_cols);
        const int n = tile * SX_TILE_M + et;
        for (int c0 = 0; c0 < p.nmma && c0 < p.R; c0 += 16) {
          float v[16];
          tc_ld16(taddr + c0, v);
          if (n < p.n_rows) {
            float *dst = p.part + (size_t)sp * p.split_stride + n;
#pragma unroll
            for (int j = 0; j < 16; ++j)
              if (c0 + j < p.R) dst[(size_t)(c0 + j) * p.n_rows] = v[j];
          }
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&tempty[acc]));
        if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
      }
    }
  }
  tc_teardown(abort_flag, p.status, tmem_base, (uint32_t)p.tmem_cols);
}

// Give-up path of the bounded waits, on its own: a CTA with the GEMM kernel's thread layout allocates
// TMEM, then every role waits on a barrier that nothing ever arrives at (no copy is in flight).  The
// first wait to run out raises the abort flag, the others see it at their next poll, and the CTA leaves
// through the same tear-down as the GEMM kernel: SX_ERR_TIMEOUT in the status word, TMEM freed, a
// normal return.  Used by the tests; `limit` is small there.
__global__ void __launch_bounds__(192, 1) sx_wait_selftest_kernel(uint32_t limit, int32_t *status, int32_t *reached) {
  __shared__ __align__(8) uint64_t bars[3];
  __shared__ uint32_t tmem_slot;
  __shared__ int abort_word;
  volatile int *abort_flag = &abort_word;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    for (int i = 0; i < 3; ++i) mbar_init(smem_u32(&bars[i]), 1);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    tc_alloc(smem_u32(&tmem_slot), 32u);
    tc_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = tmem_slot;
  bool ok = false;
  if (warp == 0) {
    if (lane == 0) ok = mbar_wait(smem_u32(&bars[0]), 0u, abort_flag, limit);                 // producer's wait
  } else if (warp == 1) {
    if (lane == 0) ok = mbar_wait(smem_u32(&bars[1]), 0u, abort_flag, limit * 4u);            // MMA issuer's wait
  } else {
    ok = epi_all(mbar_wait(smem_u32(&bars[2]), 0u, abort_flag, limit * 4u));                  // epilogue's wait
  }
  if (ok) atomicAdd(reached, 1);           // stays 0: no wait may report success
  tc_teardown(abort_flag, status, tmem_base, 32u);
  if (threadIdx.x == 0) atomicAdd(reached + 1, 1);      // CTAs that returned through the tear-down
}

sx_status sx_launch_wait_selftest(uint32_t limit, int ctas, int32_t *status, int32_t *reached, cudaStream_t st) {
  if (limit < 1 || limit > (1u << 20) || ctas < 1 || ctas > 1024) return SX_ERR_INVALID_ARG;
  sx_wait_selftest_kernel<<<ctas, 192, 0, st>>>(limit, status, reached);
  return sx_rc(cudaGetLastError());
}

// ---- host side ------------------------------------------------------------------------------
static PFN_cuTensorMapEncodeTiled_v12000 g_encode = nullptr;
static std::mutex g_mu;
struct MapKey {
  const void *ptr; long long rows; int cols, box_rows;
  bool operator==(const MapKey &o) const { return ptr == o.ptr && rows == o.rows && cols == o.cols && box_rows == o.box_rows; }
};
struct MapKeyHash {
  size_t operator()(const MapKey &k) const {
    return std::hash<const void *>()(k.ptr) ^ ((size_t)k.rows * 1000003u) ^ ((size_t)k.cols * 7919u) ^ ((size_t)k.box_rows << 48);
  }
};
static std::unordered_map<MapKey, CUtensorMap, MapKeyHash> g_maps;

bool sx_tma_map_2d(const void *ptr, long long rows, int cols, int box_rows, CUtensorMap *out) {
  std::lock_guard<std::mutex> lk(g_mu);
  if (!g_encode) {
    void *fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess || !fn) return false;
    g_encode = reinterpret_cast<PFN_cuTensorMapEncodeTiled_v12000>(fn);
  }
  MapKey key{ptr, rows, cols, box_rows};
  auto it = g_maps.find(key);
  if (it != g_maps.end()) { *out = it->second; return true; }
  CUtensorMap m;
  cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
  cuuint64_t strides[1] = {(cuuint64_t)cols * 2};
  cuuint32_t box[2] = {SX_BK, (cuuint32_t)box_rows};
  cuuint32_t estr[2] = {1, 1};
  CUresult rc = g_encode(&m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(ptr), dims, strides, box, estr,
                         CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                         CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (rc != CUDA_SUCCESS) return false;
  if (g_maps.size() > 4096) g_maps.clear();
  g_maps.emplace(key, m);
  *out = m;
  return true;
}

static int pow2_at_least(int v) { int p = 32; while (p < v) p <<= 1; return p; }

static bool fill_common(SxTcParams &p, int n_rows, int K, int R, size_t epi_bytes) {
  p.n_rows = n_rows;
  p.num_kb = (K + SX_BK - 1) / SX_BK;
  p.R = R;
  p.nmma = ((R + 15) / 16) * 16;
  if (p.nmma > 256) return false;
  p.num_tiles = (n_rows + SX_TILE_M - 1) / SX_TILE_M;
  p.acc_cols = p.nmma;
  p.wait_limit = SX_WAIT_LIMIT;
  p.tmem_cols = pow2_at_least(2 * p.nmma);
  const size_t stage_bytes = SX_A_BYTES + (size_t)p.nmma * 128;
  const size_t fixed = 1024 + 256 + 64 + epi_bytes + 64;
  int stages = (int)((SX_SMEM_MAX - fixed) / stage_bytes);
  if (stages > 10) stages = 10;
  if (stages < 2) return false;
  p.stages = stages;
  return true;
}

static size_t smem_bytes(const SxTcParams &p, size_t epi_bytes) {
  return 1024 + (size_t)p.stages * (SX_A_BYTES + (size_t)p.nmma * 128) + (size_t)(2 * p.stages + 4) * 8 + 16 + epi_bytes + 64;
}

sx_status sx_gemm_init(int device) {
  (void)device;
  if (cudaFuncSetAttribute(sx_tc_gemm_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, SX_SMEM_MAX) != cudaSuccess ||
      cudaFuncSetAttribute(sx_tc_gemm_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, SX_SMEM_MAX) != cudaSuccess)
    return SX_ERR_CUDA;
  return SX_OK;
}

// Choose the K split: fill the SMs in whole waves, keep at least 4 k-blocks per item, and use at
// most 4 splits: beyond that the extra partial sums (written, then read back by the finisher in
// dependent batches) cost more than the better SM coverage gains (measured on C1 and C2).
int sx_gemm_pick_splits(int N, int K, int sm_count) {
  const int tiles = (N + SX_TILE_M - 1) / SX_TILE_M;
  const int num_kb = (K + SX_BK - 1) / SX_BK;
  int best = 1;
  double best_eff = 0.0;
  for (int s = 1; s <= SX_GEMM_MAX_SPLITS; ++s) {
    const int per = (num_kb + s - 1) / s;
    if (per < 4 && s > 1) break;
    const int real = (num_kb + per - 1) / per;
    if (real != s) continue;
    const int items = tiles * s;
    const int waves = (items + sm_count - 1) / sm_count;
    const double eff = (double)items / ((double)waves * sm_count);
    if (eff > best_eff + 0.02) { best_eff = eff; best = s; }
  }
  return best;
}

// Tensor map of a weight matrix.  Row-major [N, K]: a box is 128 rows x 64 columns, i.e. 128 pieces of
// 128 bytes that lie K * 2 bytes apart.  Tiled ([row tile][k-block][128][64], zero padded): the same box
// is one contiguous 16 KB block, which keeps the DRAM pages it touches open for the whole transfer.
static bool weight_map(const bf16 *W, int N, int K, bool tiled, CUtensorMap *out) {
  if (!tiled) return sx_tma_map_2d(W, N, K, SX_TILE_M, out);
  const int tiles = (N + SX_TILE_M - 1) / SX_TILE_M, kbs = (K + SX_BK - 1) / SX_BK;
  return sx_tma_map_2d(W, tiles * kbs * SX_TILE_M, SX_BK, SX_TILE_M, out);
}

sx_status sx_launch_gemm_partial(const bf16 *W, int N, int K, const bf16 *X, int R, float *part, int splits,
                                 size_t split_stride, int sm_count, int32_t *status, cudaStream_t st, bool tiled) {
  if ((K % 8) != 0 || R < 1) return SX_ERR_UNSUPPORTED;
  for (int r0 = 0; r0 < R; r0 += 256) {
    const int rc = (R - r0 < 256) ? R - r0 : 256;
    SxTcParams p;
    memset(&p, 0, sizeof(p));
    if (!fill_common(p, N, K, rc, 0)) return SX_ERR_UNSUPPORTED;
    p.kb_per_split = (p.num_kb + splits - 1) / splits;
    p.splits = (p.num_kb + p.kb_per_split - 1) / p.kb_per_split;
    if (p.splits != splits) return SX_ERR_INVALID_ARG;
    p.part = part + (size_t)r0 * N;
    p.split_stride = split_stride;
    p.status = status;
    CUtensorMap mw, mx;
    p.w_tiled = tiled ? 1 : 0;
    if (!weight_map(W, N, K, tiled, &mw) || !sx_tma_map_2d(X + (size_t)r0 * K, rc, K, p.nmma, &mx)) return SX_ERR_CUDA;
    const int items = p.num_tiles * p.splits;
    const int per_cta = (items + sm_count - 1) / sm_count;          // the same number of items for every CTA
    const int grid = (items + per_cta - 1) / per_cta;
    if (sx_launch(sx_tc_gemm_kernel<false>, dim3(grid), dim3(192), smem_bytes(p, 0), st, mw, mx, p) != cudaSuccess)
      return SX_ERR_CUDA;
  }
  return SX_OK;
}

int sx_head_max_rows(int T, int lse) { return (T == 1 && !lse) ? 256 : 64; }

sx_status sx_launch_head(const bf16 *W, int Ntot, int V, int K, const bf16 *X, int R, int T, int lse,
                         SxHeadPartial *parts, int part_stride, int *G, float *z, int S, int sm_count, int32_t *status,
                         cudaStream_t st, const SxSample *smp, SxLogitsOut lo, bool tiled) {
  if ((K % 8) != 0 || R < 1 || R > sx_head_max_rows(T, lse)) return SX_ERR_UNSUPPORTED;
  if (smp && smp->temp > 0.f && (T != 1 || lse || smp->P < 1)) return SX_ERR_UNSUPPORTED;
  if (lo.out && smp && smp->temp > 0.f && lse) return SX_ERR_UNSUPPORTED;
  SxTcParams p;
  memset(&p, 0, sizeof(p));
  const size_t epi = (T == 1 && !lse) ? SX_ARGMAX_SMEM : SX_TOPK_SMEM;
  if (!fill_common(p, Ntot, K, R, epi)) return SX_ERR_UNSUPPORTED;
  p.splits = 1;
  p.kb_per_split = p.num_kb;
  p.V = V; p.S = S; p.T = T; p.lse = lse; p.parts = parts; p.part_stride = part_stride; p.z = z; p.status = status;
  if (smp) p.smp = *smp;
  p.lo = lo;
  CUtensorMap mw, mx;
  p.w_tiled = tiled ? 1 : 0;
  if (!weight_map(W, Ntot, K, tiled, &mw) || !sx_tma_map_2d(X, R, K, p.nmma, &mx)) return SX_ERR_CUDA;
  // every CTA gets the same number of tiles (no CTA is left alone with one more 1 MB tile at the end):
  // with w = ceil(tiles / SMs) tiles per CTA, ceil(tiles / w) CTAs cover the matrix
  const int per_cta = (p.num_tiles + sm_count - 1) / sm_count;
  const int grid = (p.num_tiles + per_cta - 1) / per_cta;
  if (sx_launch(sx_tc_gemm_kernel<true>, dim3(grid), dim3(192), smem_bytes(p, epi), st, mw, mx, p) != cudaSuccess)
    return SX_ERR_CUDA;
  *G = grid;
  return SX_OK;
}

// ---- weight tiling ------------------------------------------------------------------------
// dst[tile][kb][r][c] = src[tile * 128 + r][kb * 64 + c], zero outside the matrix.  One CTA per
// (k-block, row tile); a thread moves 16 bytes at a time.
__global__ void sx_tile_weight_kernel(const bf16 *__restrict__ src, int N, int K, bf16 *__restrict__ dst) {
  const int kb = blockIdx.x, tile = blockIdx.y, kbs = gridDim.x;
  uint4 *out = reinterpret_cast<uint4 *>(dst + ((size_t)tile * kbs + kb) * SX_TILE_M * SX_BK);
  for (int i = threadIdx.x; i < SX_TILE_M * SX_BK / 8; i += blockDim.x) {
    const int r = i / (SX_BK / 8), c8 = i % (SX_BK / 8);
    const int row = tile * SX_TILE_M + r, col = kb * SX_BK + c8 * 8;
    uint4 v = make_uint4(0, 0, 0, 0);
    if (row < N && col < K) v = *reinterpret_cast<const uint4 *>(src + (size_t)row * K + col);   // K % 8 == 0
    out[i] = v;
  }
}

size_t sx_tiled_elems(int N, int K) {
  return (size_t)((N + SX_TILE_M - 1) / SX_TILE_M) * ((K + SX_BK - 1) / SX_BK) * SX_TILE_M * SX_BK;
}

sx_status sx_launch_tile_weight(const bf16 *src, int N, int K, bf16 *dst, cudaStream_t st) {
  if (N < 1 || K < 8 || (K % 8) != 0) return SX_ERR_UNSUPPORTED;
  dim3 grid((K + SX_BK - 1) / SX_BK, (N + SX_TILE_M - 1) / SX_TILE_M);
  sx_tile_weight_kernel<<<grid, 256, 0, st>>>(src, N, K, dst);
  return cudaGetLastError() == cudaSuccess ? SX_OK : SX_ERR_CUDA;
}
