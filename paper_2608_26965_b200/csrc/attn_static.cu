// cluster_attention_fwd_static: the attention stage for callers that cannot hand
// the library a workspace because they cannot allocate device memory at all.
//
// Who that is: code that runs inside a host framework's "execute" callback where
// allocation is forbidden, serving loops that must not take the implicit
// device-wide synchronisation of an allocation, and processes whose device
// memory has been reserved up front by another pool so that a fresh allocation
// would simply fail.  For them the scratch lives in a fixed array that is part
// of the library image on every GPU that loads it.
#include <math.h>

#include "kernels.h"

namespace {

constexpr size_t kStaticScratchBytes = 32u << 20;     // 32 MiB per GPU, held until the process exits

// Scratch of cluster_attention_fwd_static.  Host code must never use this name
// as a pointer: on the host it is only a handle; the device address is looked up
// below with cudaGetSymbolAddress.
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

constexpr int kMaxDevices = 64;
void* g_scratch_ptr[kMaxDevices] = {};                // device address of the array, per device

// One-time set-up for the current device: look up the array's device address.
int static_scratch_for_current_device(void** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return CA_ERR_CUDA;
  if (!g_scratch_ptr[dev]) {
    void* ptr = nullptr;
    if (cudaGetSymbolAddress(&ptr, g_static_scratch) != cudaSuccess || !ptr) {
      (void)cudaGetLastError();
      return CA_ERR_CUDA;
    }
    g_scratch_ptr[dev] = ptr;
  }
  *out = g_scratch_ptr[dev];
  return CA_OK;
}

}  // namespace

extern "C" {

size_t ca_static_scratch_bytes(void) { return kStaticScratchBytes; }

int cluster_attention_fwd_static(const ca_problem_t* p, const void* Qp, const void* Kp, const void* Vp,
                                 const float* ck, const float* cv, const int32_t* count_k,
                                 const int32_t* block_idx, const int32_t* perm_q, void* O, float* lse,
                                 void* stream) {
  size_t need = 0;
  const int rc = ca_workspace_bytes(p, nullptr, nullptr, &need);     // also validates the problem
  if (rc != CA_OK) return rc;
  if (need > kStaticScratchBytes) return CA_ERR_WORKSPACE;           // problem too large for the fixed array
  void* scratch = nullptr;
  const int rs = static_scratch_for_current_device(&scratch);
  if (rs != CA_OK) return rs;
  // The array keeps whatever the previous call left.  The only part that has to
  // start from zero is the status word; the callee clears it on the stream, and
  // the centroid copies (including their zero padding) are rewritten on every call.
  return cluster_attention_fwd(p, Qp, Kp, Vp, ck, cv, count_k, block_idx, perm_q, O, lse, scratch,
                               kStaticScratchBytes, stream);
}

int ca_static_last_status(void) {
  void* scratch = nullptr;
  const int rs = static_scratch_for_current_device(&scratch);
  if (rs != CA_OK) return rs;
  return ca_last_status(scratch);
}

}  // extern "C"
