// Shared host/device helpers of libclusterattn (sm_100a only).
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <atomic>

#include "../../include/cluster_attention.h"

namespace ca {

// Status block at the start of every workspace: word 0 is the status code (CA_OK or the first
// error a kernel recorded); every call clears the first kStatusClearBytes on its stream.  The last
// word is a counter that calls only add to (query clusters recomputed by the second attention pass).
constexpr size_t kStatusBytes = 256;
constexpr size_t kStatusClearBytes = 252;
constexpr int kRecomputedWord = 63;

extern std::atomic<unsigned long long> g_kernel_launches;   // kernels enqueued since the library was loaded

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }
inline int ceil_div(int a, int b) { return (a + b - 1) / b; }

#define CA_RETURN_IF_CUDA(expr)                    \
  do {                                             \
    cudaError_t _e = (expr);                       \
    if (_e != cudaSuccess) return CA_ERR_CUDA;     \
  } while (0)

// Follows every kernel launch: counts it and turns a launch error into CA_ERR_CUDA.
#define CA_LAUNCH_CHECK()                                   \
  do {                                                      \
    ++::ca::g_kernel_launches;                              \
    if (cudaPeekAtLastError() != cudaSuccess) {             \
      (void)cudaGetLastError();                             \
      return CA_ERR_CUDA;                                   \
    }                                                       \
  } while (0)

// Per-kernel-group device times (ca_profile / ca_profile_read of the public header).  A scope
// records a pair of CUDA events around the launches it encloses when profiling is on.
enum ProfGroup {
  kProfGram = 0, kProfFactor, kProfPca, kProfTransform, kProfSplitLevels, kProfSplitTail, kProfPermute,
  kProfSelect, kProfAttnPrep, kProfAttn, kProfAttnSecond, kProfGroups
};
bool prof_enabled();
void prof_mark(int group, cudaStream_t st, bool begin);
struct ProfScope {
  int group;
  cudaStream_t st;
  bool on;
  ProfScope(int g, cudaStream_t s) : group(g), st(s), on(prof_enabled()) { if (on) prof_mark(group, st, true); }
  ~ProfScope() { if (on) prof_mark(group, st, false); }
};

template <typename T>
__device__ __forceinline__ float to_f32(T x);
template <>
__device__ __forceinline__ float to_f32<float>(float x) { return x; }
template <>
__device__ __forceinline__ float to_f32<__nv_bfloat16>(__nv_bfloat16 x) { return __bfloat162float(x); }

template <typename T>
__device__ __forceinline__ T from_f32(float x);
template <>
__device__ __forceinline__ float from_f32<float>(float x) { return x; }
template <>
__device__ __forceinline__ __nv_bfloat16 from_f32<__nv_bfloat16>(float x) { return __float2bfloat16_rn(x); }

// Carves aligned sub-buffers out of a workspace (host side).
struct Carver {
  char* base;
  size_t off;
  explicit Carver(void* p) : base(static_cast<char*>(p)), off(0) {}
  template <typename T>
  T* take(size_t n) {
    off = align_up(off, 256);
    T* r = reinterpret_cast<T*>(base + off);
    off += n * sizeof(T);
    return r;
  }
  size_t used() const { return align_up(off, 256); }
};

}  // namespace ca
