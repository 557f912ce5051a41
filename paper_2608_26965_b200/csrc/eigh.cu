// Cholesky factors of the metric matrices (Section 3.2.2); the metric matrices themselves
// for the basic splitting variant.  (Covariances and principal components: eigh_tql.cu.)
#include "kernels.h"

namespace ca {

// ---------------------------------------------------------------------------
// Factor of a positive semi-definite matrix: lower-triangular F with F F^T = A
// (right-looking Cholesky in double, one CTA per matrix).  A pivot that is not
// above 1e-12 of the largest diagonal entry marks a direction in which the
// (pseudo-)metric is zero: its column of F is set to zero, which is the
// counterpart of clamping small or negative eigenvalues (Section 3.2.2).
// Any factor of the metric matrix gives the same principal-component
// coordinates as its symmetric root, because the two differ by a rotation.
// ---------------------------------------------------------------------------
// The matrix is formed on load from a Gram matrix and column sums: gram * scale (the query metric
// M = Q^T Q / n_q, `sum` null) or (gram - s s^T / n) * scale (the centred scatter of the keys).
// Besides F in double and float, F^T can be written as bf16 hi + lo parts, the layout in which the
// tensor-core projection takes its weights (the query representation multiplies by F).
template <int D>
__global__ void __launch_bounds__(1024) cholesky_factor_kernel(const double* __restrict__ gram,
                                                               const double* __restrict__ sum, double n,
                                                               double scale, double* __restrict__ out64,
                                                               float* __restrict__ out32,
                                                               __nv_bfloat16* __restrict__ wt_hi,
                                                               __nv_bfloat16* __restrict__ wt_lo) {
  constexpr int LDA = D + 1;
  extern __shared__ __align__(16) unsigned char smem_raw[];
  double* A = reinterpret_cast<double*>(smem_raw);       // [D][LDA], lower triangle is updated in place
  __shared__ double s_tol;
  __shared__ double s_inv, s_l10, s_inv1;
  const int tid = threadIdx.x, NT = blockDim.x;
  const double* G = gram + (size_t)blockIdx.x * D * D;
  const double* sm = sum ? sum + (size_t)blockIdx.x * D : nullptr;
  for (int e = tid; e < D * D; e += NT) {
    const int i = e / D, j = e % D;
    const double centre = sm ? sm[i] * sm[j] / n : 0.0;
    A[i * LDA + j] = (0.5 * (G[i * D + j] + G[j * D + i]) - centre) * scale;
  }
  __syncthreads();
  if (tid == 0) {
    double mx = 0.0;
    for (int i = 0; i < D; ++i) mx = fmax(mx, A[i * LDA + i]);
    s_tol = 1e-12 * mx;
  }
  __syncthreads();
  // two columns per round (three barriers for the pair): thread 0 prepares both pivots -- the second
  // one after its update by the first column -- then every row scales its two entries, then the
  // trailing block takes the rank-2 update
  for (int j = 0; j < D; j += 2) {
    if (tid == 0) {
      const double piv0 = A[j * LDA + j];
      const double inv0 = (piv0 > s_tol) ? rsqrt(piv0) : 0.0;
      const double l10 = A[(j + 1) * LDA + j] * inv0;
      const double piv1 = A[(j + 1) * LDA + j + 1] - l10 * l10;
      s_inv = inv0;
      s_l10 = l10;
      s_inv1 = (piv1 > s_tol) ? rsqrt(piv1) : 0.0;
    }
    __syncthreads();
    const double inv0 = s_inv, l10 = s_l10, inv1 = s_inv1;
    // columns j and j+1 of F; a dropped pivot gives a zero column
    for (int i = j + tid; i < D; i += NT) {
      const double c0 = A[i * LDA + j] * inv0;
      A[i * LDA + j] = c0;
      if (i > j) A[i * LDA + j + 1] = (A[i * LDA + j + 1] - c0 * l10) * inv1;
    }
    __syncthreads();
    // trailing update of the lower triangle
    const int rem = D - 2 - j;
    for (int e = tid; e < rem * rem; e += NT) {
      const int i = j + 2 + e / rem, k = j + 2 + e % rem;
      if (k <= i)
        A[i * LDA + k] -= A[i * LDA + j] * A[k * LDA + j] + A[i * LDA + j + 1] * A[k * LDA + j + 1];
    }
    __syncthreads();
  }
  double* o64 = out64 + (size_t)blockIdx.x * D * D;
  float* o32 = out32 ? out32 + (size_t)blockIdx.x * D * D : nullptr;
  for (int e = tid; e < D * D; e += NT) {
    const int i = e / D, j = e % D;
    const double v = (j <= i) ? A[i * LDA + j] : 0.0;
    o64[e] = v;
    if (o32) o32[e] = (float)v;
  }
  if (wt_hi) {
    // F^T [out j][in i] = F[i][j] as bf16 hi + lo
    for (int e = tid; e < D * D; e += NT) {
      const int j = e / D, i = e % D;
      const float v = (j <= i) ? (float)A[i * LDA + j] : 0.f;
      const __nv_bfloat16 h = __float2bfloat16_rn(v);
      wt_hi[(size_t)blockIdx.x * D * D + e] = h;
      wt_lo[(size_t)blockIdx.x * D * D + e] = __float2bfloat16_rn(v - __bfloat162float(h));
    }
  }
}

int launch_cholesky_factor(const double* gram, const double* sum, double n, double scale, int count, int D,
                           double* out64, float* out32, void* wt_hi, void* wt_lo, cudaStream_t st) {
  const size_t smem = sizeof(double) * D * (D + 1);
  __nv_bfloat16* hi = static_cast<__nv_bfloat16*>(wt_hi);
  __nv_bfloat16* lo = static_cast<__nv_bfloat16*>(wt_lo);
  if (D == 64) {
    auto k = cholesky_factor_kernel<64>;
    CA_RETURN_IF_CUDA(cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    k<<<count, 512, smem, st>>>(gram, sum, n, scale, out64, out32, hi, lo);
  } else {
    auto k = cholesky_factor_kernel<128>;
    CA_RETURN_IF_CUDA(cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    k<<<count, 1024, smem, st>>>(gram, sum, n, scale, out64, out32, hi, lo);
  }
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
