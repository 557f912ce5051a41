// Gathers rows into cluster order and reduces the cluster centroids
// (Section 3.1: clusters of fixed size c, the short last one padded;
// Section 3.3.1 / Appendix A: centroids are means over the actual members).
#include "kernels.h"

namespace ca {

// One CTA (128 threads) per cluster.  A row is VEC 16-byte vectors; thread t owns
// vector t % VEC of rows t / VEC, t / VEC + G, ...  Row sums are combined in a
// fixed order, so the centroids are reproducible.  A second tensor gathered by the same
// permutation (the values next to the keys) rides along as blockIdx.z = 1.
template <typename T, int D>
__global__ void __launch_bounds__(128) permute_centroid_kernel(const T* __restrict__ X0, const T* __restrict__ X1,
                                                               const int32_t* __restrict__ perm, int n,
                                                               int c, int n_c, T* __restrict__ Xp0,
                                                               T* __restrict__ Xp1,
                                                               float* __restrict__ centroid0,
                                                               float* __restrict__ centroid1,
                                                               int32_t* __restrict__ count0) {
  const T* X = blockIdx.z ? X1 : X0;
  T* Xp = blockIdx.z ? Xp1 : Xp0;
  float* centroid = blockIdx.z ? centroid1 : centroid0;
  int32_t* count = blockIdx.z ? nullptr : count0;
  constexpr int EPV = 16 / sizeof(T);          // elements per 16-byte vector
  constexpr int VEC = D / EPV;                 // vectors per row
  constexpr int G = 128 / VEC;                 // rows in flight
  __shared__ float part[G][D];
  const int p = blockIdx.y, j = blockIdx.x;
  const T* Xh = X + (size_t)p * n * D;
  const int32_t* ph = perm + (size_t)p * n;
  T* out = Xp + ((size_t)p * n_c + j) * (size_t)c * D;
  const int members = min(c, n - j * c);
  const int v = threadIdx.x % VEC, g = threadIdx.x / VEC;
  float acc[EPV];
#pragma unroll
  for (int e = 0; e < EPV; ++e) acc[e] = 0.f;
  for (int r = g; r < c; r += G) {
    uint4 raw = make_uint4(0u, 0u, 0u, 0u);
    if (r < members) {
      const int row = ph[j * c + r];
      raw = *reinterpret_cast<const uint4*>(Xh + (size_t)row * D + v * EPV);
      const T* el = reinterpret_cast<const T*>(&raw);
#pragma unroll
      for (int e = 0; e < EPV; ++e) acc[e] += to_f32<T>(el[e]);
    }
    *reinterpret_cast<uint4*>(out + (size_t)r * D + v * EPV) = raw;
  }
#pragma unroll
  for (int e = 0; e < EPV; ++e) part[g][v * EPV + e] = acc[e];
  __syncthreads();
  if (threadIdx.x < D) {
    float s = 0.f;
    for (int gg = 0; gg < G; ++gg) s += part[gg][threadIdx.x];
    centroid[((size_t)p * n_c + j) * D + threadIdx.x] = s / (float)members;
  }
  if (count && threadIdx.x == 0) count[(size_t)p * n_c + j] = members;
}

template <typename T>
static int launch_t(const T* X, const T* X2, const int32_t* perm, int P, int n, int D, int c, T* Xp, T* Xp2,
                    float* cen, float* cen2, int32_t* count, cudaStream_t st) {
  const int n_c = ceil_div(n, c);
  dim3 grid(n_c, P, X2 ? 2 : 1);
  if (D == 64)
    permute_centroid_kernel<T, 64><<<grid, 128, 0, st>>>(X, X2, perm, n, c, n_c, Xp, Xp2, cen, cen2, count);
  else
    permute_centroid_kernel<T, 128><<<grid, 128, 0, st>>>(X, X2, perm, n, c, n_c, Xp, Xp2, cen, cen2, count);
  CA_LAUNCH_CHECK();
  return CA_OK;
}

int launch_permute_centroid(const void* X, int dtype, const int32_t* perm, int P, int n, int D, int c,
                            void* Xp, float* cen, int32_t* count, cudaStream_t st, const void* X2, void* Xp2,
                            float* cen2) {
  if (dtype == CA_DTYPE_BF16)
    return launch_t(static_cast<const __nv_bfloat16*>(X), static_cast<const __nv_bfloat16*>(X2), perm, P, n, D, c,
                    static_cast<__nv_bfloat16*>(Xp), static_cast<__nv_bfloat16*>(Xp2), cen, cen2, count, st);
  return launch_t(static_cast<const float*>(X), static_cast<const float*>(X2), perm, P, n, D, c,
                  static_cast<float*>(Xp), static_cast<float*>(Xp2), cen, cen2, count, st);
}

}  // namespace ca
