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

// A run of 64 key centroids (fp32) per CTA: `live` of them exist, the rest is written as zero codes.
template <int D>
__global__ void __launch_bounds__(256) quantize_centroids_kernel(const float* __restrict__ X, int n_kc, int cen_tiles,
                                                                 unsigned char* __restrict__ codes,
                                                                 float* __restrict__ scales) {
  __shared__ float part[8];
  __shared__ float s_inv;
  const int g = blockIdx.x, p = blockIdx.y;
  const int first = g * 64;
  const int live = min(64, max(0, n_kc - first));
  const float* src = X + ((size_t)p * n_kc + first) * D;
  unsigned char* dst = codes + ((size_t)p * cen_tiles * 64 + first) * D;
  const int n_live = live * D, n_all = 64 * D;
  float mx = 0.f;
  for (int e = threadIdx.x; e < n_live; e += 256) mx = fmaxf(mx, fabsf(src[e]));
  mx = warp_max(mx);
  if ((threadIdx.x & 31) == 0) part[threadIdx.x >> 5] = mx;
  __syncthreads();
  if (threadIdx.x == 0) {
    float amax = 0.f;
    for (int w = 0; w < 8; ++w) amax = fmaxf(amax, part[w]);
    s_inv = amax > 0.f ? __fdiv_rn(448.f, amax) : 0.f;
    scales[(size_t)p * cen_tiles + g] = amax > 0.f ? __fdiv_rn(amax, 448.f) : 0.f;
  }
  __syncthreads();
  const float inv = s_inv;
  for (int e = threadIdx.x; e < n_all; e += 256)
    dst[e] = e < n_live ? to_e4m3(__fmul_rn(src[e], inv)) : (unsigned char)0;
}

// eight bf16 values (16 bytes) -> floats
__device__ __forceinline__ void unpack8(const uint4& raw, float (&x)[8]) {
  const __nv_bfloat16* h = reinterpret_cast<const __nv_bfloat16*>(&raw);
#pragma unroll
  for (int i = 0; i < 8; ++i) x[i] = __bfloat162float(h[i]);
}
__device__ __forceinline__ uint2 codes8(const float (&x)[8], float inv) {
  unsigned char c[8];
#pragma unroll
  for (int i = 0; i < 8; ++i) c[i] = to_e4m3(__fmul_rn(x[i], inv));
  uint2 out;
  out.x = c[0] | (c[1] << 8) | (c[2] << 16) | ((unsigned)c[3] << 24);
  out.y = c[4] | (c[5] << 8) | (c[6] << 16) | ((unsigned)c[7] << 24);
  return out;
}

// One key cluster (c_k rows of D bf16) per CTA of 256 threads: the rows are read once with 16-byte
// loads and stay in registers between the maximum and the codes (c_k * D / 2048 vectors per thread).
template <int D, int VPT>
__global__ void __launch_bounds__(256) quantize_clusters_kernel(const __nv_bfloat16* __restrict__ X, int c_k,
                                                                unsigned char* __restrict__ codes,
                                                                float* __restrict__ scales) {
  __shared__ float part[8];
  __shared__ float s_inv;
  const size_t group = blockIdx.x;                                   // cluster index over all problems
  const uint4* src = reinterpret_cast<const uint4*>(X + group * (size_t)c_k * D);
  uint2* dst = reinterpret_cast<uint2*>(codes + group * (size_t)c_k * D);
  const int n_vec = c_k * D / 8;
  float x[VPT][8];
  float mx = 0.f;
#pragma unroll
  for (int v = 0; v < VPT; ++v) {
    const int e = threadIdx.x + v * 256;
    if (e < n_vec) {
      unpack8(src[e], x[v]);
#pragma unroll
      for (int i = 0; i < 8; ++i) mx = fmaxf(mx, fabsf(x[v][i]));
    }
  }
  mx = warp_max(mx);
  if ((threadIdx.x & 31) == 0) part[threadIdx.x >> 5] = mx;
  __syncthreads();
  if (threadIdx.x == 0) {
    float amax = 0.f;
    for (int w = 0; w < 8; ++w) amax = fmaxf(amax, part[w]);
    s_inv = amax > 0.f ? __fdiv_rn(448.f, amax) : 0.f;
    scales[group] = amax > 0.f ? __fdiv_rn(amax, 448.f) : 0.f;
  }
  __syncthreads();
  const float inv = s_inv;
#pragma unroll
  for (int v = 0; v < VPT; ++v) {
    const int e = threadIdx.x + v * 256;
    if (e < n_vec) dst[e] = codes8(x[v], inv);
  }
}

// One query row per 16 threads (each 8 values of a 128-wide row), 16 rows per CTA.
template <int D>
__global__ void __launch_bounds__(256) quantize_rows_kernel(const __nv_bfloat16* __restrict__ X, size_t n_rows,
                                                            unsigned char* __restrict__ codes,
                                                            float* __restrict__ scales) {
  static_assert(D == 128, "one 16-byte vector per thread, 16 threads per row");
  const size_t row = (size_t)blockIdx.x * 16 + (threadIdx.x >> 4);
  const int sub = threadIdx.x & 15;
  float x[8];
  float mx = 0.f;
  if (row < n_rows) {
    unpack8(reinterpret_cast<const uint4*>(X + row * D)[sub], x);
#pragma unroll
    for (int i = 0; i < 8; ++i) mx = fmaxf(mx, fabsf(x[i]));
  }
  for (int o = 8; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
  if (row >= n_rows) return;
  const float inv = mx > 0.f ? __fdiv_rn(448.f, mx) : 0.f;
  if (sub == 0) scales[row] = mx > 0.f ? __fdiv_rn(mx, 448.f) : 0.f;
  reinterpret_cast<uint2*>(codes + row * D)[sub] = codes8(x, inv);
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
  quantize_rows_kernel<128><<<(unsigned)((q_rows + 15) / 16), 256, 0, st>>>(static_cast<const __nv_bfloat16*>(Qp), q_rows, q8, sq);
  CA_LAUNCH_CHECK();
  const __nv_bfloat16* kp = static_cast<const __nv_bfloat16*>(Kp);
  const unsigned clusters = (unsigned)((size_t)P * n_kc);
  if (c_k == 64) quantize_clusters_kernel<128, 4><<<clusters, 256, 0, st>>>(kp, c_k, k8, sk);
  else if (c_k == 128) quantize_clusters_kernel<128, 8><<<clusters, 256, 0, st>>>(kp, c_k, k8, sk);
  else if (c_k == 256) quantize_clusters_kernel<128, 16><<<clusters, 256, 0, st>>>(kp, c_k, k8, sk);
  else return CA_ERR_UNSUPPORTED;
  CA_LAUNCH_CHECK();
  if (ck) {
    quantize_centroids_kernel<128><<<dim3(cen_tiles, P), 256, 0, st>>>(ck, n_kc, cen_tiles, c8, sc);
    CA_LAUNCH_CHECK();
  }
  return CA_OK;
}

}  // namespace ca
