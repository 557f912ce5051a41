// 8-bit storage of queries, keys and key centroids for the attention variant
// with a quantised Q K^T (Section 3.1: the paper's block-sparse kernel is a
// quantised one).  Scheme: E4M3 codes (4 exponent bits, 3 mantissa bits, largest
// finite value 448), one scale per query row, per key cluster and per run of 64
// key centroids.  A scale maps the largest magnitude of its group to 448; all of
// it in float32 with IEEE operations, so that any implementation gets the same
// codes:  amax = max |x|;  inv = 448 / amax;  s = amax / 448  (both 0 when amax
// is 0);  code = E4M3(x * inv), round to nearest even, saturating.  The logits
// are formed from the codes and multiplied by the two scales afterwards.
#include <cuda_fp8.h>

#include "kernels.h"

namespace ca {

namespace {

__device__ __forceinline__ unsigned char to_e4m3(float y) {
  return (unsigned char)__nv_cvt_float_to_fp8(y, __NV_SATFINITE, __NV_E4M3);
}

__device__ __forceinline__ float warp_max(float v) {
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}

// One group per CTA: `rows` consecutive rows of D elements (a query row: rows = 1; a key cluster:
// rows = c_k; a run of centroids: rows = 64, of which only `live` exist -- the rest is written as
// zero codes).  T = bf16 (rows of Qp / Kp) or float (centroids).
template <typename T, int D>
__global__ void __launch_bounds__(256) quantize_groups_kernel(const T* __restrict__ X, int rows, int live_total,
                                                              int groups_per_problem, int src_rows_per_problem,
                                                              unsigned char* __restrict__ codes,
                                                              float* __restrict__ scales) {
  __shared__ float part[8];
  __shared__ float s_inv;
  const int g = blockIdx.x, p = blockIdx.y;
  const int first = g * rows;                                        // first row of the group inside the problem
  const int live = min(rows, max(0, live_total - first));            // rows that exist in the source
  const T* src = X + ((size_t)p * src_rows_per_problem + first) * D;
  unsigned char* dst = codes + ((size_t)p * groups_per_problem * rows + first) * D;
  const int n_live = live * D, n_all = rows * D;
  float mx = 0.f;
  for (int e = threadIdx.x; e < n_live; e += 256) mx = fmaxf(mx, fabsf(to_f32<T>(src[e])));
  mx = warp_max(mx);
  if ((threadIdx.x & 31) == 0) part[threadIdx.x >> 5] = mx;
  __syncthreads();
  if (threadIdx.x == 0) {
    float amax = 0.f;
    for (int w = 0; w < 8; ++w) amax = fmaxf(amax, part[w]);
    s_inv = amax > 0.f ? __fdiv_rn(448.f, amax) : 0.f;
    scales[(size_t)p * groups_per_problem + g] = amax > 0.f ? __fdiv_rn(amax, 448.f) : 0.f;
  }
  __syncthreads();
  const float inv = s_inv;
  for (int e = threadIdx.x; e < n_all; e += 256)
    dst[e] = e < n_live ? to_e4m3(__fmul_rn(to_f32<T>(src[e]), inv)) : (unsigned char)0;
}

// One warp per row (queries): 8 rows per CTA.
template <int D>
__global__ void __launch_bounds__(256) quantize_rows_kernel(const __nv_bfloat16* __restrict__ X, size_t n_rows,
                                                            unsigned char* __restrict__ codes,
                                                            float* __restrict__ scales) {
  const size_t row = (size_t)blockIdx.x * 8 + (threadIdx.x >> 5);
  if (row >= n_rows) return;
  const int lane = threadIdx.x & 31;
  constexpr int PER = D / 32;
  float x[PER];
  float mx = 0.f;
#pragma unroll
  for (int i = 0; i < PER; ++i) {
    x[i] = __bfloat162float(X[row * D + lane * PER + i]);
    mx = fmaxf(mx, fabsf(x[i]));
  }
  mx = warp_max(mx);
  const float inv = mx > 0.f ? __fdiv_rn(448.f, mx) : 0.f;
  if (lane == 0) scales[row] = mx > 0.f ? __fdiv_rn(mx, 448.f) : 0.f;
#pragma unroll
  for (int i = 0; i < PER; ++i) codes[row * D + lane * PER + i] = to_e4m3(__fmul_rn(x[i], inv));
}

}  // namespace

// Qp [P * n_qc * c_q, D] -> codes + one scale per row; Kp [P, n_kc * c_k, D] -> codes + one scale per
// cluster; ck [P, n_kc, D] fp32 -> codes [P, cen_tiles * 64, D] (zero rows behind the last centroid)
// + one scale per run of 64.
int launch_quantize_qk(const void* Qp, const void* Kp, const float* ck, int P, int n_qc, int c_q, int n_kc, int c_k,
                       int cen_tiles, int D, unsigned char* q8, float* sq, unsigned char* k8, float* sk,
                       unsigned char* c8, float* sc, cudaStream_t st) {
  if (D != 128) return CA_ERR_UNSUPPORTED;
  const size_t q_rows = (size_t)P * n_qc * c_q;
  quantize_rows_kernel<128><<<(unsigned)((q_rows + 7) / 8), 256, 0, st>>>(static_cast<const __nv_bfloat16*>(Qp), q_rows, q8, sq);
  CA_LAUNCH_CHECK();
  quantize_groups_kernel<__nv_bfloat16, 128><<<dim3(n_kc, P), 256, 0, st>>>(
      static_cast<const __nv_bfloat16*>(Kp), c_k, n_kc * c_k, n_kc, n_kc * c_k, k8, sk);
  CA_LAUNCH_CHECK();
  if (ck) {
    quantize_groups_kernel<float, 128><<<dim3(cen_tiles, P), 256, 0, st>>>(ck, 64, n_kc, cen_tiles, n_kc, c8, sc);
    CA_LAUNCH_CHECK();
  }
  return CA_OK;
}

}  // namespace ca
