// stem_score_static: the scoring stage for callers that cannot provide (or allocate) a workspace.
// It launches the same two kernels as stem_score (pooling, then the tensor-core metric kernel); only
// the home of the pooled tensors differs: a fixed array in the library image instead of caller memory.
#include <mutex>

#include "stem_internal.h"

namespace {

// Scratch for the status words and the pooled tensors (MV, Qbar parts, Kbar parts).  One copy per GPU
// that loads the library, held until the process exits.
static __device__ __align__(256) unsigned char g_static_scratch[STEM_STATIC_SCRATCH_BYTES];

constexpr int kMaxDevices = 64;
std::mutex g_mu;
void* g_scratch_addr[kMaxDevices] = {nullptr};

size_t align256(size_t x) { return (x + 255) / 256 * 256; }

// In host code `g_static_scratch` is only a handle for the runtime, not a device address; the
// address the kernels need is looked up once per device, with that device current.
int scratch_address(int device, void** out) {
  if (device < 0 || device >= kMaxDevices) return STEM_ERR_UNSUPPORTED;
  std::lock_guard<std::mutex> lock(g_mu);
  if (!g_scratch_addr[device]) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || !p) {
      cudaGetLastError();
      return STEM_ERR_CUDA;
    }
    g_scratch_addr[device] = p;
  }
  *out = g_scratch_addr[device];
  return STEM_OK;
}

}  // namespace

namespace stem {

// The status words of the built-in scratch on `device` (the current device), for stem_check_status.
int static_scratch_status_words(int device, int32_t** out) {
  void* base = nullptr;
  const int rc = scratch_address(device, &base);
  if (rc == STEM_OK) *out = (int32_t*)base;
  return rc;
}

}  // namespace stem

extern "C" int stem_score_static(const stem_plan* plan, const void* Q, const void* K, const void* V, float* M,
                                 void* stream) {
  using namespace stem;
  if (!plan || !Q || !K || !V || !M) return STEM_ERR_INVALID_ARG;
  if (((uintptr_t)Q | (uintptr_t)K | (uintptr_t)V | (uintptr_t)M) & 15) return STEM_ERR_INVALID_ARG;
  const Plan& p = plan->p;
  if (p.kcache_blocks > 0 || p.score_mode != 0) return STEM_ERR_INVALID_ARG;

  // Size check first: nothing is touched when the problem does not fit.
  const size_t status_bytes = align256(kStatusWords * sizeof(int32_t));
  const size_t mv_bytes = align256((size_t)p.cfg.num_kv_heads * p.KB_tot * sizeof(float));
  const size_t q_bytes = align256((size_t)3 * p.H_list * p.R_tot * kHeadDim * 2);
  const size_t k_bytes = align256((size_t)3 * p.cfg.num_kv_heads * p.KB_tot * kHeadDim * 2);
  if (status_bytes + mv_bytes + q_bytes + k_bytes > (size_t)STEM_STATIC_SCRATCH_BYTES) return STEM_ERR_STATIC_SCRATCH;

  int device = -1;
  if (cudaGetDevice(&device) != cudaSuccess) { cudaGetLastError(); return STEM_ERR_CUDA; }
  if (device != p.device) return STEM_ERR_INVALID_ARG;
  void* base = nullptr;
  const int rc = scratch_address(device, &base);
  if (rc != STEM_OK) return rc;

  unsigned char* b = (unsigned char*)base;
  int32_t* status = (int32_t*)b;
  float* mv = (float*)(b + status_bytes);
  void* qsplit = b + status_bytes + mv_bytes;
  void* ksplit = b + status_bytes + mv_bytes + q_bytes;
  cudaStream_t s = (cudaStream_t)stream;
  p.last_launches = 0;
  // The array keeps what the previous call left.  The status words must start at zero, so they are
  // cleared here; the pooling kernel writes every pooled element the metric kernel's result depends on
  // (tiles that reach past a sequence's last block read rows of a neighbour or stale rows, and only
  // into entries the epilogue never stores).
  if (cudaMemsetAsync(status, 0, kStatusWords * sizeof(int32_t), s) != cudaSuccess) { cudaGetLastError(); return STEM_ERR_CUDA; }
  if (launch_pool(p, Q, K, V, mv, qsplit, ksplit, false, s) != cudaSuccess) { cudaGetLastError(); return STEM_ERR_CUDA; }
  p.last_launches++;
  if (launch_metric_gemm(p, qsplit, ksplit, mv, M, false, true, status, s) != cudaSuccess) { cudaGetLastError(); return STEM_ERR_CUDA; }
  p.last_launches++;
  return STEM_OK;
}
