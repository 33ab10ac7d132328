// Shared device-side helpers and host/device structs of the speculative-exit kernels.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/specexit.h"

typedef __nv_bfloat16 bf16;

#define SX_WARP 32
#define SX_TILE_M 128          // weight rows per GEMM tile

// How the rows of one draft round map to sequences, positions and cache slots.
struct SxRowMap {
  int mode;                    // SX_MODE_*
  int round;                   // 1-based
  int topk;
  int R;                       // rows this round
  const int32_t *cache_len;    // [B]
  const uint64_t *row_mask;    // [R] tree rounds >= 2, else nullptr
  // commit (mode SX_MODE_COMMIT): per_seq rows per sequence, row j of sequence b sits at slot and
  // position n + 1 + j and exists only if j < valid_len[b]
  const int32_t *valid_len;
  int per_seq;
};
#define SX_MODE_COMMIT 2

struct SxRowInfo {
  int b;          // sequence
  int n;          // cached prefix length
  int pos;        // rotary position
  int rel;        // drafted-row index within the sequence (slot = n + rel)
};

// placement only (sequence, cached length, position, drafted-row index): touches nothing a kernel
// of the same iteration writes, so it may run before the wait on the preceding kernel
__device__ __forceinline__ SxRowInfo sx_row_place(const SxRowMap &m, int r) {
  SxRowInfo i;
  if (m.mode == SX_MODE_COMMIT) {
    i.b = r / m.per_seq;
    i.rel = 1 + (r - i.b * m.per_seq);
    i.n = m.cache_len[i.b];
    i.pos = i.n + i.rel;
    return i;
  }
  if (m.mode == SX_MODE_CHAIN) { i.b = r; i.rel = m.round - 1; }
  else if (m.round == 1) { i.b = r; i.rel = 0; }
  else { i.b = r / m.topk; i.rel = 1 + (m.round - 2) * m.topk + (r % m.topk); }
  i.n = m.cache_len[i.b];
  i.pos = i.n + m.round - 1;
  return i;
}

__device__ __forceinline__ void sx_set_status(int32_t *status, int32_t code) {
  if (status) atomicMin(status, code);
}

// float -> unsigned key with the same order (NaN sorts above +inf; callers never rank NaN)
__device__ __forceinline__ uint32_t sx_order_key(float f) {
  uint32_t u = __float_as_uint(f);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
__device__ __forceinline__ float sx_key_value(uint32_t k) {
  uint32_t u = (k & 0x80000000u) ? (k & 0x7fffffffu) : ~k;
  return __uint_as_float(u);
}
// (value, index) packed so that a larger value wins and, among equal values, the lower index
__device__ __forceinline__ unsigned long long sx_pack(float v, uint32_t idx) {
  return ((unsigned long long)sx_order_key(v) << 32) | (unsigned long long)(0xffffffffu - idx);
}
__device__ __forceinline__ float sx_pack_value(unsigned long long p) {
  return sx_key_value((uint32_t)(p >> 32));
}
__device__ __forceinline__ uint32_t sx_pack_index(unsigned long long p) {
  return 0xffffffffu - (uint32_t)(p & 0xffffffffu);
}

__device__ __forceinline__ float sx_warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ float sx_warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}

__device__ __forceinline__ float sx_activate(float z, int act) {
  if (act == SX_ACT_SIGMOID) return 1.0f / (1.0f + expf(-z));
  if (act == SX_ACT_EXPM1) return expm1f(z);
  return z;
}

// ----------------------------------------------------------------------------------------
// What a CTA of the head kernel leaves per token row for the merge kernel: its top-T (value,
// index) pairs and the log-sum-exp state over the vocabulary rows it has seen.
// ----------------------------------------------------------------------------------------
struct SxHeadPartial {       // what a CTA leaves behind for the merge, per row
  unsigned long long top[SX_MAX_TOPK];   // packed (value, index), best first; 0 = empty
  float m, l;                            // running max and sum of exp(v - m)
};
// ---- counter-based random numbers for sampled verification ---------------------------------
// Philox4x32 with 10 rounds (Salmon et al., SC'11), written from its definition: two 32x32->64
// multiplies per round on counter words 0 and 2, the high halves xored with words 1 and 3 and
// the round key, the key advanced by the Weyl constants between rounds.
__device__ __forceinline__ void sx_philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3, uint32_t k0,
                                                 uint32_t k1, uint32_t out[4]) {
#pragma unroll
  for (int r = 0; r < 10; ++r) {
    const uint32_t hi0 = __umulhi(0xD2511F53u, c0), lo0 = 0xD2511F53u * c0;
    const uint32_t hi1 = __umulhi(0xCD9E8D57u, c2), lo1 = 0xCD9E8D57u * c2;
    const uint32_t n0 = hi1 ^ c1 ^ k0, n2 = hi0 ^ c3 ^ k1;
    c0 = n0; c1 = lo1; c2 = n2; c3 = lo0;
    k0 += 0x9E3779B9u;
    k1 += 0xBB67AE85u;
  }
  out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}
// standard Gumbel draw from a 32-bit word: u = (top 23 bits + 1/2) / 2^23 lies strictly inside (0, 1)
__device__ __forceinline__ float sx_gumbel(uint32_t w) {
  const float u = (float)((w >> 9) * 2u + 1u) * 5.9604644775390625e-8f;      // exact: odd / 2^24
  // inner logarithm at full accuracy (u close to 1 gives the largest draws, the likely winners);
  // the outer one only needs absolute accuracy: its argument lies in [6e-8, 17]
  return -__logf(-logf(u));
}


