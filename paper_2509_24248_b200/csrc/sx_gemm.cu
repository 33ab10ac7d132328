// GEMM dispatch: the tensor-core kernels are the product path; SX_GEMM_IMPL=ref selects the
// plain CUDA-core kernels for debugging comparisons.
#include <stdlib.h>
#include <string.h>

#include "sx_kernels.cuh"

sx_status sx_ref_gemm_partial(const bf16 *, int, int, const bf16 *, int, float *, int, size_t, int32_t *, cudaStream_t);
sx_status sx_ref_head(const bf16 *, int, int, int, const bf16 *, int, int, int, SxHeadPartial *, int, int *, float *, int,
                      int, int32_t *, cudaStream_t);
int sx_ref_head_max_rows(int);
void sx_ref_init(int);
sx_status sx_tc_gemm_partial(const bf16 *, int, int, const bf16 *, int, float *, int, size_t, int, int32_t *, cudaStream_t);
sx_status sx_tc_head(const bf16 *, int, int, int, const bf16 *, int, int, int, SxHeadPartial *, int, int *, float *, int,
                     int, int32_t *, cudaStream_t);
int sx_tc_head_max_rows(int);
int sx_tc_pick_splits(int, int, int);
void sx_tc_init(int);

static bool g_ref = false;
static int g_sm = 148;

void sx_gemm_init(int device) {
  const char *e = getenv("SX_GEMM_IMPL");
  g_ref = e && !strcmp(e, "ref");
  cudaDeviceProp prop;
  if (cudaGetDeviceProperties(&prop, device) == cudaSuccess) g_sm = prop.multiProcessorCount;
  sx_ref_init(device);
  sx_tc_init(device);
}

int sx_gemm_pick_splits(int N, int K, int sm_count) { return g_ref ? 1 : sx_tc_pick_splits(N, K, sm_count); }

sx_status sx_launch_gemm_partial(const bf16 *W, int N, int K, const bf16 *X, int R, float *part, int splits,
                                 size_t split_stride, int32_t *status, cudaStream_t st) {
  if (g_ref) return sx_ref_gemm_partial(W, N, K, X, R, part, splits, split_stride, status, st);
  return sx_tc_gemm_partial(W, N, K, X, R, part, splits, split_stride, g_sm, status, st);
}

int sx_head_max_rows(int T) { return g_ref ? sx_ref_head_max_rows(T) : sx_tc_head_max_rows(T); }

sx_status sx_launch_head(const bf16 *W, int Ntot, int V, int K, const bf16 *X, int R, int T, int lse,
                         SxHeadPartial *parts, int part_stride, int *G, float *z, int S, int sm_count, int32_t *status,
                         cudaStream_t st) {
  if (g_ref) return sx_ref_head(W, Ntot, V, K, X, R, T, lse, parts, part_stride, G, z, S, sm_count, status, st);
  return sx_tc_head(W, Ntot, V, K, X, R, T, lse, parts, part_stride, G, z, S, sm_count, status, st);
}
