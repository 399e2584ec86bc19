// pact_prune_static: the percentile split (Eq. 3-4) for callers that must not allocate.
//
// pact_prune needs a caller-provided workspace, and somebody has to cudaMalloc that workspace.
// Some hosts of this library cannot: code that runs inside another framework's stream callback or
// between the iterations of a latency-critical decode loop, plugins that are handed tensors but no
// allocator, and processes whose memory pool is already carved up and closed.  For them the scratch
// of this one stage lives in a fixed array inside the library image.  Every GPU that loads the
// library carries the array (kStaticScratchBytes, a little over 256 KiB) until the process exits.
#include <math.h>
#include <string.h>

#include <mutex>

#include "kernels.cuh"

using namespace pact;

namespace {

constexpr int kStaticMaxN = PACT_PRUNE_STATIC_MAX_N;
constexpr int kStaticCntInts = 32;
constexpr size_t kStaticScratchBytes = (size_t)kStaticMaxN * sizeof(int32_t) + kStaticCntInts * sizeof(int32_t);
constexpr int kMaxDevices = 64;

// [0, kStaticMaxN) ints: position of every token in its list; then kStaticCntInts counters.
static __device__ __align__(256) unsigned char g_prune_scratch[kStaticScratchBytes];

// Device address of g_prune_scratch per device ordinal.  In host code the array's name is only a
// handle for the runtime; the address a kernel can use comes from cudaGetSymbolAddress, asked once
// per device while that device is current.
std::mutex g_mu;
void *g_scratch_addr[kMaxDevices];

cudaError_t scratch_for_current_device(void **out) {
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
  std::lock_guard<std::mutex> lock(g_mu);
  if (!g_scratch_addr[dev]) {
    void *p = nullptr;
    e = cudaGetSymbolAddress(&p, g_prune_scratch);
    if (e != cudaSuccess) return e;
    if (!p) return cudaErrorInvalidSymbol;
    e = select_configure();
    if (e != cudaSuccess) return e;
    g_scratch_addr[dev] = p;
  }
  *out = g_scratch_addr[dev];
  return cudaSuccess;
}

}  // namespace

extern "C" pact_status pact_prune_static(const float *score, int N, const pact_params *p, uint8_t *keep,
                                         int32_t *kept_idx, int32_t *pruned_idx, int32_t *counts,
                                         void *stream) {
  if (!score || !keep || !kept_idx || !pruned_idx || !counts || !p || N < 1) return PACT_ERR_INVALID_ARG;
  if (N > kStaticMaxN) return PACT_ERR_UNSUPPORTED;          // beyond the built-in scratch
  if (!(p->lambda >= 0.0 && p->lambda <= 1.0)) return PACT_ERR_INVALID_ARG;
  void *base = nullptr;
  if (scratch_for_current_device(&base) != cudaSuccess) return PACT_ERR_CUDA;
  cudaStream_t st = (cudaStream_t)stream;
  Batch bt;
  memset(&bt, 0, sizeof(bt));
  bt.B = 1;
  ImgDesc &m = bt.img[0];
  m.N = N;
  long long mt = p->n_prune >= 0 ? (long long)p->n_prune : (long long)floor(p->lambda * (double)N + 1e-6);
  if (mt > N - 1) mt = N - 1;
  if (mt < 0) mt = 0;
  m.m_target = (int)mt;
  m.slot = reinterpret_cast<int32_t *>(base);
  m.cnt = reinterpret_cast<int32_t *>(base) + kStaticMaxN;
  m.score = const_cast<float *>(score);
  m.keep = keep;
  m.kept_idx = kept_idx;
  m.pruned_idx = pruned_idx;
  // The array keeps whatever the previous call left: start the counters from zero.
  if (cudaMemsetAsync(m.cnt, 0, kStaticCntInts * sizeof(int32_t), st) != cudaSuccess) return PACT_ERR_CUDA;
  launch_select_gather(bt, N, true, false, st);
  if (cudaGetLastError() != cudaSuccess) return PACT_ERR_CUDA;
  if (cudaMemcpyAsync(counts, m.cnt + PACT_CNT_Q, sizeof(int32_t), cudaMemcpyDeviceToDevice, st) != cudaSuccess)
    return PACT_ERR_CUDA;
  if (cudaMemcpyAsync(counts + 1, m.cnt + PACT_CNT_M, sizeof(int32_t), cudaMemcpyDeviceToDevice, st) != cudaSuccess)
    return PACT_ERR_CUDA;
  return PACT_OK;
}
