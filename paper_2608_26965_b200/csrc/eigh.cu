// Cholesky factors of the metric matrices (Section 3.2.2); the metric matrices themselves
// for the basic splitting variant.  (Covariances and principal components: eigh_tql.cu.)
#include "kernels.h"

namespace ca {

// ---------------------------------------------------------------------------
// Factor of a positive semi-definite matrix: lower-triangular F with F F^T = A
// (right-looking Cholesky in double, one CTA of 1024 threads per matrix).  A pivot
// that is not above 1e-12 of the largest diagonal entry marks a direction in
// which the (pseudo-)metric is zero: its column of F is set to zero, which is the
// counterpart of clamping small or negative eigenvalues (Section 3.2.2).
// Any factor of the metric matrix gives the same principal-component
// coordinates as its symmetric root, because the two differ by a rotation.
//
// The matrix is formed on load from a Gram matrix and column sums: gram * scale (the query metric
// M = Q^T Q / n_q, `sum` null) or (gram - s s^T / n) * scale (the centred scatter of the keys).
// Besides F in double and float, F^T can be written as bf16 hi + lo parts, the layout in which the
// tensor-core projection takes its weights (the query representation multiplies by F).
//
// Thread (i, q) = (warp, lane) keeps the entries (i + 32 a, q + 32 b), a, b < d / 32, in registers
// for the whole elimination: rows and columns both dealt out cyclically, so that the shrinking
// trailing block stays spread over all threads.  A step is bound by the instructions it issues,
// not by the arithmetic: with a whole row per eight threads every multiply-add came with a
// shared-memory load and three index tests, a dozen instructions per entry; a tile takes d / 32
// entries of column j for its rows and d / 32 for its columns, and the only tests left are
// uniform ones per tile row and per step (the body of a step is compiled once per position of
// column j among the tile columns, so that finished tile columns cost nothing).  Step j needs
// column j, which its owners publish to shared memory during step j - 1 (right after their last
// update of it), so a step takes one barrier; the trailing block takes
// A[r][k] -= A[r][j] A[k][j] / pivot_j with the unscaled column, and the columns are scaled by
// 1 / sqrt(pivot) at the end.  The one division of a step is made by the thread that completes
// the next pivot, also a step ahead.  A dropped pivot (reciprocal 0) leaves the trailing block
// alone and gives a zero column.  Entries above the diagonal inside a diagonal tile block take the
// same updates as their mirror images; they are never read and are written as zeros.
// ---------------------------------------------------------------------------
// One elimination step for the case that column j + 1 lies in tile column B0 (tile columns and
// tile rows below B0 are final).
template <int TB, int B0, typename T>
__device__ __forceinline__ void cholesky_step(T (&a)[TB][TB], const T* __restrict__ col, T* __restrict__ col_next,
                                              T* __restrict__ ip_next, T ip, T tol, int i, int q, int j) {
  T c[TB];
#pragma unroll
  for (int tb = B0; tb < TB; ++tb) {
    const int k = q + 32 * tb;
    c[tb] = (tb > B0 || k > j) ? col[k] : (T)0;            // columns up to j are final: they take a - f * 0
  }
#pragma unroll
  for (int ta = B0; ta < TB; ++ta) {
    const int r = i + 32 * ta;
    if (ta == B0 && r <= j) continue;                      // uniform over the warp: rows up to j are final
    const T f = col[r] * ip;
#pragma unroll
    for (int tb = B0; tb <= ta; ++tb) a[ta][tb] -= f * c[tb];
  }
  if (q == ((j + 1) & 31)) {                               // column j + 1 is complete: publish it
#pragma unroll
    for (int ta = B0; ta < TB; ++ta) {
      const int r = i + 32 * ta;
      if (r > j) {
        col_next[r] = a[ta][B0];
        if (r == j + 1) *ip_next = a[ta][B0] > tol ? (T)1 / a[ta][B0] : (T)0;
      }
    }
  }
}

template <int D, typename T>
__global__ void __launch_bounds__(1024) cholesky_factor_kernel(const double* __restrict__ gram,
                                                               const double* __restrict__ sum, double n,
                                                               double scale, double* __restrict__ out64,
                                                               float* __restrict__ out32,
                                                               __nv_bfloat16* __restrict__ wt_hi,
                                                               __nv_bfloat16* __restrict__ wt_lo) {
  constexpr int TB = D / 32;       // rows and columns of a thread's tile
  static_assert(TB >= 1 && TB <= 4, "tile of at most 4 x 4 entries per thread");
  __shared__ T colbuf[2][D];       // column j of the trailing matrix, rows >= j (two in rotation)
  __shared__ T pivots[D];          // diagonal entries; afterwards 1 / sqrt(pivot) per column
  __shared__ T s_ip[2];
  __shared__ T s_tol;
  const T kDrop = sizeof(T) == 8 ? (T)1e-12 : (T)1e-6;   // share of the largest diagonal entry below which a pivot drops out
  const int tid = threadIdx.x;
  const int i = tid >> 5, q = tid & 31;
  const double* G = gram + (size_t)blockIdx.x * D * D;
  const double* sm = sum ? sum + (size_t)blockIdx.x * D : nullptr;
  T a[TB][TB];
#pragma unroll
  for (int ta = 0; ta < TB; ++ta) {
    const int r = i + 32 * ta;
    // the centring needs double precision: the Gram matrix is n mean^2 + scatter
    const double row_term = sm ? sm[r] * (scale / n) : 0.0;
#pragma unroll
    for (int tb = 0; tb < TB; ++tb) {
      const int k = q + 32 * tb;
      a[ta][tb] = (T)0;
      if (k <= r) a[ta][tb] = (T)(sm ? fma(-row_term, sm[k], G[r * D + k] * scale) : G[r * D + k] * scale);
      if (k == r) pivots[r] = a[ta][tb];
      if (k == 0) colbuf[0][r] = a[ta][tb];
    }
  }
  __syncthreads();
  if (tid < 32) {
    T mx = (T)0;
    for (int t = tid; t < D; t += 32) mx = max(mx, pivots[t]);
    for (int o = 16; o > 0; o >>= 1) mx = max(mx, __shfl_xor_sync(0xffffffffu, mx, o));
    if (tid == 0) {
      s_tol = kDrop * mx;
      s_ip[0] = pivots[0] > kDrop * mx ? (T)1 / pivots[0] : (T)0;
    }
  }
  __syncthreads();
  const T tol = s_tol;
  for (int j = 0; j < D - 1; ++j) {
    const T* col = colbuf[j & 1];
    T* col_next = colbuf[(j + 1) & 1];
    T* ip_next = &s_ip[(j + 1) & 1];
    const T ip = s_ip[j & 1];
    switch ((j + 1) >> 5) {                                // uniform over the CTA
      case 0: cholesky_step<TB, 0>(a, col, col_next, ip_next, ip, tol, i, q, j); break;
      case 1: if constexpr (TB > 1) cholesky_step<TB, 1>(a, col, col_next, ip_next, ip, tol, i, q, j); break;
      case 2: if constexpr (TB > 2) cholesky_step<TB, 2>(a, col, col_next, ip_next, ip, tol, i, q, j); break;
      default: if constexpr (TB > 3) cholesky_step<TB, 3>(a, col, col_next, ip_next, ip, tol, i, q, j); break;
    }
    __syncthreads();
  }
  if (q == i) {
#pragma unroll
    for (int t = 0; t < TB; ++t) pivots[i + 32 * t] = a[t][t];
  }
  __syncthreads();
  if (tid < D) pivots[tid] = pivots[tid] > tol ? (T)rsqrt((double)pivots[tid]) : (T)0;
  __syncthreads();
  double* o64 = out64 + (size_t)blockIdx.x * D * D;
  float* o32 = out32 ? out32 + (size_t)blockIdx.x * D * D : nullptr;
#pragma unroll
  for (int ta = 0; ta < TB; ++ta) {
    const int r = i + 32 * ta;
#pragma unroll
    for (int tb = 0; tb < TB; ++tb) {
      const int k = q + 32 * tb;
      const double v = (k <= r) ? (double)(a[ta][tb] * pivots[k]) : 0.0;
      o64[r * D + k] = v;
      if (o32) o32[r * D + k] = (float)v;
      if (wt_hi) {                                          // F^T [out k][in r] = F[r][k] as bf16 hi + lo
        const float vf = (float)v;
        const __nv_bfloat16 h = __float2bfloat16_rn(vf);
        wt_hi[(size_t)blockIdx.x * D * D + (size_t)k * D + r] = h;
        wt_lo[(size_t)blockIdx.x * D * D + (size_t)k * D + r] = __float2bfloat16_rn(vf - __bfloat162float(h));
      }
    }
  }
}

typedef double CholT;   // arithmetic of the elimination (float32 was measured: no faster, and less exact)

int launch_cholesky_factor(const double* gram, const double* sum, double n, double scale, int count, int D,
                           double* out64, float* out32, void* wt_hi, void* wt_lo, cudaStream_t st) {
  __nv_bfloat16* hi = static_cast<__nv_bfloat16*>(wt_hi);
  __nv_bfloat16* lo = static_cast<__nv_bfloat16*>(wt_lo);
  if (D == 64) cholesky_factor_kernel<64, CholT><<<count, 1024, 0, st>>>(gram, sum, n, scale, out64, out32, hi, lo);
  else cholesky_factor_kernel<128, CholT><<<count, 1024, 0, st>>>(gram, sum, n, scale, out64, out32, hi, lo);
  CA_LAUNCH_CHECK();
  return CA_OK;
}

// ---------------------------------------------------------------------------
// d x d algebra in double (one CTA per problem unless noted).
// ---------------------------------------------------------------------------
// M = gramQ / n_q ;  C_K = gramK - sumK sumK^T / n_k   (centred scatter)
__global__ void metric_kernel(const double* __restrict__ gramQ, const double* __restrict__ gramK,
                              const double* __restrict__ sumK, int D, double n_q, double n_k,
                              double ck_scale, double* __restrict__ M, double* __restrict__ CK) {
  // either output may be left out (null): the two come from different streams in cluster_qk
  const int p = blockIdx.y;
  const int e = blockIdx.x * blockDim.x + threadIdx.x;
  if (e >= D * D) return;
  const int i = e / D, j = e % D;
  const size_t o = (size_t)p * D * D + e;
  if (M) M[o] = gramQ[o] / n_q;
  if (CK) CK[o] = (gramK[o] - sumK[(size_t)p * D + i] * sumK[(size_t)p * D + j] / n_k) * ck_scale;
}

__global__ void cast_f64_f32_kernel(const double* __restrict__ src, float* __restrict__ dst, size_t count) {
  const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i < count) dst[i] = (float)src[i];
}
int launch_cast_f64_f32(const double* src, float* dst, size_t count, cudaStream_t st) {
  cast_f64_f32_kernel<<<(unsigned)((count + 255) / 256), 256, 0, st>>>(src, dst, count);
  CA_LAUNCH_CHECK();
  return CA_OK;
}

int launch_metric(const double* gramQ, const double* gramK, const double* sumK, int P, int D, int n_q,
                  int n_k, double ck_scale, double* M, double* CK, cudaStream_t st) {
  metric_kernel<<<dim3(ceil_div(D * D, 256), P), 256, 0, st>>>(gramQ, gramK, sumK, D, (double)n_q,
                                                                (double)n_k, ck_scale, M, CK);
  CA_LAUNCH_CHECK();
  return CA_OK;
}
}  // namespace ca
