// stem_score_static: the scoring stage for callers that cannot provide (or allocate) a workspace.
// It runs the same pooling and metric kernels as stem_score; only the home of the pooled tensors
// differs: a fixed array in the library image instead of caller memory.
#include <mutex>

#include "stem_internal.h"

namespace {

// Scratch for the pooled tensors (Qbar, Kbar, MV).  One copy per GPU that loads the library,
// held until the process exits.
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

extern "C" int stem_score_static(const stem_plan* plan, const void* Q, const void* K, const void* V, float* M,
                                 void* stream) {
  using namespace stem;
  if (!plan || !Q || !K || !V || !M) return STEM_ERR_INVALID_ARG;
  if (((uintptr_t)Q | (uintptr_t)K | (uintptr_t)V | (uintptr_t)M) & 15) return STEM_ERR_INVALID_ARG;
  const Plan& p = plan->p;

  // Size check first: nothing is touched when the problem does not fit.
  const size_t qbar_bytes = align256((size_t)p.cfg.num_q_heads * p.R_tot * kHeadDim * sizeof(float));
  const size_t kbar_bytes = align256((size_t)p.cfg.num_kv_heads * kHeadDim * p.kt_width * sizeof(float));
  const size_t mv_bytes = align256((size_t)p.cfg.num_kv_heads * p.R_tot * sizeof(float));
  if (qbar_bytes + kbar_bytes + mv_bytes > (size_t)STEM_STATIC_SCRATCH_BYTES) return STEM_ERR_STATIC_SCRATCH;

  int device = -1;
  if (cudaGetDevice(&device) != cudaSuccess) { cudaGetLastError(); return STEM_ERR_CUDA; }
  if (device != p.device) return STEM_ERR_INVALID_ARG;
  void* base = nullptr;
  const int rc = scratch_address(device, &base);
  if (rc != STEM_OK) return rc;

  float* qbar = (float*)base;
  float* kbar = (float*)((unsigned char*)base + qbar_bytes);
  float* mv = (float*)((unsigned char*)base + qbar_bytes + kbar_bytes);
  cudaStream_t s = (cudaStream_t)stream;
  p.last_launches = 0;
  // The pooling kernel writes every element of qbar / kbar / mv that the metric kernel reads, so
  // whatever an earlier call left in the array is never observed.
  if (launch_pool(p, Q, K, V, qbar, kbar, mv, nullptr, nullptr, s) != cudaSuccess) return STEM_ERR_CUDA;
  p.last_launches++;
  if (launch_score_select(p, kFromPooled | kWriteMetric, qbar, kbar, mv, nullptr, M, nullptr, nullptr, s) != cudaSuccess)
    return STEM_ERR_CUDA;
  p.last_launches++;
  return STEM_OK;
}
