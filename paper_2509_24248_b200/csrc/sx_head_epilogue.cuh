// Fused epilogue of the extended LM head (Eq. 1): the logits of a 128-row vocabulary tile
// are consumed where they are produced - running top-T (value, index) per token row, an
// optional running log-sum-exp, and the raw signal rows - so they never reach HBM.
//
// Calling convention: 128 threads (4 warps) cooperate; thread t owns vocabulary row
// tile_base + t and is handed its logit for one token row ("column") at a time.
#pragma once
#include "sx_common.cuh"

struct SxHeadSmem {
  // carve-up of a caller-provided shared buffer
  unsigned long long *top;     // [Rcap][T] packed, best first (T == 1: updated with atomicMax)
  unsigned long long *thr;     // [Rcap] T-th best so far (0 while the list is not full), T > 1
  unsigned long long *pend;    // [Rcap][SX_HEAD_PEND], T > 1
  int *pend_cnt;               // [Rcap], T > 1
  float2 *ml;                  // [4][Rcap] per-warp running (max, sum exp), when lse is wanted
  int Rcap, T, lse;
};

__host__ __device__ inline size_t sx_head_smem_bytes(int Rcap, int T, int lse) {
  size_t b = (size_t)Rcap * T * 8;
  if (T > 1) b += (size_t)Rcap * 8 + (size_t)Rcap * SX_HEAD_PEND * 8 + (size_t)Rcap * 4;
  b = (b + 7) & ~(size_t)7;
  if (lse) b += (size_t)4 * Rcap * 8;
  return b;
}

__device__ inline SxHeadSmem sx_head_carve(void *buf, int Rcap, int T, int lse) {
  SxHeadSmem s;
  char *p = reinterpret_cast<char *>(buf);
  s.top = reinterpret_cast<unsigned long long *>(p);
  p += (size_t)Rcap * T * 8;
  s.thr = nullptr; s.pend = nullptr; s.pend_cnt = nullptr; s.ml = nullptr;
  if (T > 1) {
    s.thr = reinterpret_cast<unsigned long long *>(p);
    p += (size_t)Rcap * 8;
    s.pend = reinterpret_cast<unsigned long long *>(p);
    p += (size_t)Rcap * SX_HEAD_PEND * 8;
    s.pend_cnt = reinterpret_cast<int *>(p);
    p += (size_t)Rcap * 4;
  }
  p = reinterpret_cast<char *>(((uintptr_t)p + 7) & ~(uintptr_t)7);
  if (lse) s.ml = reinterpret_cast<float2 *>(p);
  s.Rcap = Rcap; s.T = T; s.lse = lse;
  return s;
}

// tid in [0,128).  Clears the state for R rows; the caller synchronises afterwards.
__device__ inline void sx_head_init(const SxHeadSmem &s, int R, int tid) {
  for (int i = tid; i < R * s.T; i += 128) s.top[i] = 0ull;
  if (s.T > 1)
    for (int i = tid; i < R; i += 128) { s.thr[i] = 0ull; s.pend_cnt[i] = 0; }
  if (s.lse)
    for (int i = tid; i < 4 * s.Rcap; i += 128) s.ml[i] = make_float2(-INFINITY, 0.f);
}

// One logit of vocabulary row `idx` for token row r.  `valid` is false for rows outside the
// vocabulary (signal rows, padding).  All 32 lanes of a warp call this together.
__device__ __forceinline__ void sx_head_column(const SxHeadSmem &s, int r, float v, uint32_t idx,
                                               bool valid, int warp, int lane) {
  const uint32_t key = valid ? sx_order_key(v) : 0u;
  const uint32_t wk = __reduce_max_sync(0xffffffffu, key);
  if (wk == 0u) return;                                   // no valid row in this warp
  if (s.T == 1) {
    const uint32_t who = __ballot_sync(0xffffffffu, key == wk);
    if (lane == __ffs(who) - 1) {
      const unsigned long long cur = *((volatile unsigned long long *)&s.top[r]);
      if (wk >= (uint32_t)(cur >> 32)) atomicMax(&s.top[r], sx_pack(v, idx));
    }
  } else {
    const unsigned long long p = sx_pack(v, idx);
    if (valid && p > s.thr[r]) {
      const int at = atomicAdd(&s.pend_cnt[r], 1);
      if (at < SX_HEAD_PEND) s.pend[(size_t)r * SX_HEAD_PEND + at] = p;
    }
  }
  if (s.lse) {
    const float wm = sx_key_value(wk);
    const float e = valid ? __expf(v - wm) : 0.f;
    const float sum = sx_warp_sum(e);
    if (lane == 0) {
      float2 st = s.ml[warp * s.Rcap + r];
      if (wm > st.x) { st.y = st.y * __expf(st.x - wm) + sum; st.x = wm; }
      else           { st.y += sum * __expf(wm - st.x); }
      s.ml[warp * s.Rcap + r] = st;
    }
  }
}

// After every column of a tile (and a barrier over the 128 threads): fold the pending
// entries into the sorted lists.  The caller puts another barrier behind it.  T > 1 only.
__device__ inline void sx_head_merge_pending(const SxHeadSmem &s, int R, int tid) {
  if (s.T == 1) return;
  for (int r = tid; r < R; r += 128) {
    int cnt = s.pend_cnt[r];
    if (cnt == 0) continue;
    if (cnt > SX_HEAD_PEND) cnt = SX_HEAD_PEND;
    unsigned long long *top = s.top + (size_t)r * s.T;
    for (int i = 0; i < cnt; ++i) {
      unsigned long long p = s.pend[(size_t)r * SX_HEAD_PEND + i];
      if (p <= top[s.T - 1]) continue;
      int j = s.T - 1;
      while (j > 0 && top[j - 1] < p) { top[j] = top[j - 1]; --j; }
      top[j] = p;
    }
    s.thr[r] = top[s.T - 1];
    s.pend_cnt[r] = 0;
  }
}

// Leave the CTA's result for the merge kernel: out[cta][r].
__device__ inline void sx_head_flush(const SxHeadSmem &s, int R, int tid, SxHeadPartial *out) {
  for (int r = tid; r < R; r += 128) {
    SxHeadPartial hp;
#pragma unroll
    for (int t = 0; t < SX_MAX_TOPK; ++t) hp.top[t] = (t < s.T) ? s.top[(size_t)r * s.T + t] : 0ull;
    float m = -INFINITY, l = 0.f;
    if (s.lse) {
      for (int w = 0; w < 4; ++w) m = fmaxf(m, s.ml[w * s.Rcap + r].x);
      for (int w = 0; w < 4; ++w) {
        float2 st = s.ml[w * s.Rcap + r];
        if (st.y > 0.f) l += st.y * __expf(st.x - m);
      }
    }
    hp.m = m; hp.l = l;
    out[r] = hp;
  }
}
