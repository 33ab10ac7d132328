// Plain CUDA-core GEMM kernels (bring-up path): one warp per weight row, 16-byte loads.
// Same interfaces and same per-tile epilogues as the tensor-core kernels.
#include "sx_head_epilogue.cuh"
#include "sx_kernels.cuh"

#define SX_REF_RC 64    // token rows per pass

// dot products of weight row n with up to 8 token rows, reduced over the warp
template <int RT>
__device__ __forceinline__ void sx_row_dots(const bf16 *w, const bf16 *X, int K, int r0, int R, int lane,
                                            float *out) {
  float acc[RT];
#pragma unroll
  for (int i = 0; i < RT; ++i) acc[i] = 0.f;
  for (int k = lane * 8; k < K; k += 256) {
    float wf[8];
    sx_unpack8(*reinterpret_cast<const uint4 *>(w + k), wf);
#pragma unroll
    for (int i = 0; i < RT; ++i) {
      if (r0 + i < R) {
        float xf[8];
        sx_unpack8(*reinterpret_cast<const uint4 *>(X + (size_t)(r0 + i) * K + k), xf);
#pragma unroll
        for (int j = 0; j < 8; ++j) acc[i] = fmaf(wf[j], xf[j], acc[i]);
      }
    }
  }
#pragma unroll
  for (int i = 0; i < RT; ++i) out[i] = sx_warp_sum(acc[i]);
}

__global__ void sx_gemm_partial_ref_kernel(const bf16 *W, int N, int K, const bf16 *X, int R, float *part) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int n = blockIdx.x * 4 + warp;
  if (n >= N) return;
  for (int r0 = 0; r0 < R; r0 += 8) {
    float o[8];
    sx_row_dots<8>(W + (size_t)n * K, X, K, r0, R, lane, o);
    if (lane == 0)
      for (int i = 0; i < 8 && r0 + i < R; ++i) part[(size_t)(r0 + i) * N + n] = o[i];
  }
}


sx_status sx_ref_gemm_partial(const bf16 *W, int N, int K, const bf16 *X, int R, float *part, int splits,
                                 size_t split_stride, int32_t *status, cudaStream_t st) {
  if (splits != 1 || (K % 8) != 0) return SX_ERR_UNSUPPORTED;
  sx_gemm_partial_ref_kernel<<<(N + 3) / 4, 128, 0, st>>>(W, N, K, X, R, part);
  return SX_OK;
}

// persistent over 128-row tiles; logits of a tile go through shared memory to the epilogue
__global__ void sx_head_ref_kernel(const bf16 *W, int Ntot, int V, int K, const bf16 *X, int R, int T, int lse,
                                   SxHeadPartial *parts, int part_stride, float *z, int S) {
  extern __shared__ __align__(16) unsigned char sx_hs[];
  float *tile = reinterpret_cast<float *>(sx_hs);                     // [128][R + 1]
  const int ld = R + 1;
  SxHeadSmem hs = sx_head_carve(sx_hs + (((size_t)128 * ld * sizeof(float) + 15) & ~(size_t)15), R, T, lse);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  sx_head_init(hs, R, tid);
  __syncthreads();
  const int ntiles = (Ntot + SX_TILE_M - 1) / SX_TILE_M;
  for (int tl = blockIdx.x; tl < ntiles; tl += gridDim.x) {
    const int n0 = tl * SX_TILE_M;
    for (int i = 0; i < 32; ++i) {
      const int row = warp * 32 + i, n = n0 + row;
      for (int r0 = 0; r0 < R; r0 += 8) {
        float o[8];
        if (n < Ntot) sx_row_dots<8>(W + (size_t)n * K, X, K, r0, R, lane, o);
        if (lane == 0)
          for (int j = 0; j < 8 && r0 + j < R; ++j) tile[row * ld + r0 + j] = (n < Ntot) ? o[j] : 0.f;
      }
    }
    __syncthreads();
    const int n = n0 + tid;
    const bool valid = n < V;
    for (int r = 0; r < R; ++r) {
      const float v = tile[tid * ld + r];
      sx_head_column(hs, r, v, (uint32_t)n, valid, warp, lane);
      if (n >= V && n < V + S) z[(size_t)r * S + (n - V)] = v;
    }
    __syncthreads();
    sx_head_merge_pending(hs, R, tid);
    __syncthreads();
  }
  sx_head_flush(hs, R, tid, parts + (size_t)blockIdx.x * part_stride);
}

int sx_ref_head_max_rows(int T) { return SX_REF_RC; }

void sx_ref_init(int device) {
  cudaFuncSetAttribute(sx_head_ref_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
}

sx_status sx_ref_head(const bf16 *W, int Ntot, int V, int K, const bf16 *X, int R, int T, int lse,
                         SxHeadPartial *parts, int part_stride, int *G, float *z, int S, int sm_count,
                         int32_t *status, cudaStream_t st) {
  if ((K % 8) != 0 || R > SX_REF_RC) return SX_ERR_UNSUPPORTED;
  const int ntiles = (Ntot + SX_TILE_M - 1) / SX_TILE_M;
  int grid = ntiles < 2 * sm_count ? ntiles : 2 * sm_count;
  const size_t smem = (size_t)128 * (R + 1) * sizeof(float) + 16 + sx_head_smem_bytes(R, T, lse);
  sx_head_ref_kernel<<<grid, 128, smem, st>>>(W, Ntot, V, K, X, R, T, lse, parts, part_stride, z, S);
  *G = grid;
  return SX_OK;
}
