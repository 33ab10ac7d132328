// Verification entry point for callers that must not allocate device memory.
//
// Some hosts of this library cannot call cudaMalloc at the point where they verify a draft: a
// serving loop whose whole device memory already belongs to another component's pool, a
// plugin that runs inside a latency-critical section where an allocation (which may
// synchronise the device) is forbidden, or firmware-like code that was given fixed buffers
// only.  sx_verify_noalloc does what sx_verify does - target LM head with fused argmax, then
// greedy acceptance - but keeps the head kernel's scratch (the per-CTA partial results that
// the merge kernel reads) in a fixed array inside the library image instead of a caller
// workspace.
//
// The array below is part of the loaded module: every GPU that loads the library holds it
// (SX_NOALLOC_SCRATCH_BYTES, about 0.7 MB) until the process exits.  All calls on a device
// share it and it keeps the last call's contents.  Nothing in it has to start at zero: every
// CTA rewrites its whole slice for the rows of the call before the merge kernel reads exactly
// those slices.  Two calls that overlap on one GPU (different streams, or different threads)
// would race on it: issue them on one stream, or order them yourself.
#include <mutex>

#include "sx_kernels.cuh"

#define SX_NOALLOC_MAX_CTAS 160     // CTAs of the head kernel that may leave a partial result
static_assert(SX_NOALLOC_SCRATCH_BYTES == SX_NOALLOC_MAX_CTAS * SX_NOALLOC_MAX_ROWS * sizeof(SxHeadPartial),
              "the header's SX_NOALLOC_SCRATCH_BYTES must match the partial-result record");

// In host code this name is only a handle for the runtime, never a device address: the address
// comes from cudaGetSymbolAddress, once per device.
static __device__ __align__(256) unsigned char sx_noalloc_scratch[SX_NOALLOC_SCRATCH_BYTES];

#define SX_NOALLOC_MAX_DEVICES 64
static std::mutex g_setup_mu;
static void *g_scratch_ptr[SX_NOALLOC_MAX_DEVICES];
static int g_sm_count[SX_NOALLOC_MAX_DEVICES];
static bool g_ready[SX_NOALLOC_MAX_DEVICES];

// First call on a device: resolve the device address of the array (with that device current),
// read the SM count, opt the kernels in to their shared-memory size.
static sx_status noalloc_setup(int dev, void **scratch, int *sm) {
  if (dev < 0 || dev >= SX_NOALLOC_MAX_DEVICES) return SX_ERR_UNSUPPORTED;
  std::lock_guard<std::mutex> lk(g_setup_mu);
  if (!g_ready[dev]) {
    void *p = nullptr;
    if (cudaGetSymbolAddress(&p, sx_noalloc_scratch) != cudaSuccess || p == nullptr) return SX_ERR_CUDA;
    int n = 0;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n < 1) return SX_ERR_CUDA;
    if (sx_gemm_init(dev) != SX_OK) return SX_ERR_CUDA;
    g_scratch_ptr[dev] = p;
    g_sm_count[dev] = n;
    g_ready[dev] = true;
  }
  *scratch = g_scratch_ptr[dev];
  *sm = g_sm_count[dev];
  return SX_OK;
}

extern "C" sx_status sx_verify_noalloc(const void *target_head_d, int32_t vocab, int32_t H, int32_t batch, int32_t P,
                                       const void *target_hidden_d, const int32_t *cand_tok_d,
                                       const int32_t *parent_d, int32_t *target_tok_d, int32_t *accept_len_d,
                                       int32_t *path_d, int32_t path_stride, int32_t *recover_tok_d,
                                       int32_t *status_d, void *stream) {
  if (!target_head_d || !target_hidden_d || !cand_tok_d || !target_tok_d || !accept_len_d || !path_d ||
      !recover_tok_d || !status_d)
    return SX_ERR_INVALID_ARG;
  if (((uintptr_t)target_head_d & 15) || ((uintptr_t)target_hidden_d & 15)) return SX_ERR_INVALID_ARG;
  if (vocab < 1 || H < 8 || (H % 8) || batch < 1 || P < 1 || path_stride < 1) return SX_ERR_INVALID_ARG;
  if (parent_d && P > SX_MAX_VERIFY_SLOTS) return SX_ERR_UNSUPPORTED;
  if ((long long)batch * P > SX_NOALLOC_MAX_ROWS) return SX_ERR_STATIC_LIMIT;
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return SX_ERR_CUDA;
  void *scratch = nullptr;
  int sm = 0;
  sx_status rc = noalloc_setup(dev, &scratch, &sm);
  if (rc != SX_OK) return rc;
  // The head kernel never uses more CTAs than the SM count it is given (a CTA takes several tiles instead),
  // and every CTA leaves one slice: capping that count here keeps the launch inside the array.
  if (sm > SX_NOALLOC_MAX_CTAS) sm = SX_NOALLOC_MAX_CTAS;
  cudaStream_t st = (cudaStream_t)stream;
  const int R = batch * P;
  SxHeadPartial *parts = reinterpret_cast<SxHeadPartial *>(scratch);
  int G = 0;
  rc = sx_launch_head((const bf16 *)target_head_d, vocab, vocab, H, (const bf16 *)target_hidden_d, R, 1, 0, parts,
                      SX_NOALLOC_MAX_ROWS, &G, nullptr, 0, sm, status_d, st);
  if (rc != SX_OK) return rc;
  SxShape sh;
  memset(&sh, 0, sizeof(sh));
  sh.H = H; sh.V = vocab;
  SX_TRY(sx_launch_head_finalize(sh, R, parts, G, SX_NOALLOC_MAX_ROWS, 1, 0, nullptr, 0, target_tok_d, SxIndex{nullptr, 1, 0},
                          nullptr, nullptr, SxIndex{nullptr, 1, 0}, st));
  SX_TRY(sx_launch_accept(batch, P, cand_tok_d, parent_d, target_tok_d, accept_len_d, path_d, path_stride, recover_tok_d, st));
  return SX_OK;
}
