// Cholesky factors of the metric matrices (Section 3.2.2) and the d x d algebra
// around the eigendecompositions (which live in eigh_tql.cu).
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
template <int D>
__global__ void __launch_bounds__(1024) cholesky_factor_kernel(const double* __restrict__ A_in,
                                                               double* __restrict__ out64,
                                                               float* __restrict__ out32) {
  constexpr int LDA = D + 1;
  extern __shared__ __align__(16) unsigned char smem_raw[];
  double* A = reinterpret_cast<double*>(smem_raw);       // [D][LDA], lower triangle is updated in place
  __shared__ double s_tol;
  __shared__ double s_inv, s_l10, s_inv1;
  const int tid = threadIdx.x, NT = blockDim.x;
  const double* Ain = A_in + (size_t)blockIdx.x * D * D;
  for (int e = tid; e < D * D; e += NT) {
    const int i = e / D, j = e % D;
    A[i * LDA + j] = 0.5 * (Ain[i * D + j] + Ain[j * D + i]);
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
}

int launch_cholesky_factor(const double* A, int count, int D, double* out64, float* out32, cudaStream_t st) {
  const size_t smem = sizeof(double) * D * (D + 1);
  if (D == 64) {
    auto k = cholesky_factor_kernel<64>;
    CA_RETURN_IF_CUDA(cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    k<<<count, 512, smem, st>>>(A, out64, out32);
  } else {
    auto k = cholesky_factor_kernel<128>;
    CA_RETURN_IF_CUDA(cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    k<<<count, 1024, smem, st>>>(A, out64, out32);
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

// Cov = gram / n - mean mean^T, mean = sum / n
__global__ void covariance_kernel(const double* __restrict__ gram, const double* __restrict__ sum,
                                  int D, double n, double* __restrict__ cov) {
  const int p = blockIdx.y;
  const int e = blockIdx.x * blockDim.x + threadIdx.x;
  if (e >= D * D) return;
  const int i = e / D, j = e % D;
  const size_t o = (size_t)p * D * D + e;
  cov[o] = gram[o] / n - (sum[(size_t)p * D + i] / n) * (sum[(size_t)p * D + j] / n);
}

// C[p] = alpha * op(A[p]) * B[p], op = transpose if trans_a; optional fp32 copy.
// Operands are double in memory; the products are formed in float (FP64 throughput of the
// CUDA cores is low on this part, and the results only feed fp32 projections).  One CTA of
// 256 threads per 64 x 64 tile of C, 4 x 4 outputs per thread, 16-deep slices in shared memory.
__global__ void __launch_bounds__(256) small_matmul_kernel(const double* __restrict__ A,
                                                           const double* __restrict__ B, int D, double alpha,
                                                           int trans_a, double* __restrict__ C,
                                                           float* __restrict__ C32) {
  constexpr int KS = 64;                // slice depth: one round of global loads per 64 columns of A
  __shared__ float As[KS][64 + 4];     // As[k][i]
  __shared__ float Bs[KS][64 + 4];     // Bs[k][j]
  const int p = blockIdx.z;
  const double* Ap = A + (size_t)p * D * D;
  const double* Bp = B + (size_t)p * D * D;
  const int i0 = blockIdx.y * 64, j0 = blockIdx.x * 64;
  const int ti = threadIdx.x / 16, tj = threadIdx.x % 16;
  float acc[4][4];
#pragma unroll
  for (int a = 0; a < 4; ++a)
#pragma unroll
    for (int b = 0; b < 4; ++b) acc[a][b] = 0.f;
  for (int k0 = 0; k0 < D; k0 += KS) {
#pragma unroll 8
    for (int e = threadIdx.x; e < KS * 64; e += 256) {
      const int k = e / 64, x = e % 64;
      // the untransposed operand is read along its rows (k fastest) and stored transposed
      if (trans_a) As[k][x] = (float)Ap[(size_t)(k0 + k) * D + i0 + x];
      else As[x][k] = (float)Ap[(size_t)(i0 + k) * D + k0 + x];
      Bs[k][x] = (float)Bp[(size_t)(k0 + k) * D + j0 + x];
    }
    __syncthreads();
#pragma unroll 16
    for (int k = 0; k < KS; ++k) {
      float a[4], b[4];
#pragma unroll
      for (int x = 0; x < 4; ++x) { a[x] = As[k][ti * 4 + x]; b[x] = Bs[k][tj * 4 + x]; }
#pragma unroll
      for (int x = 0; x < 4; ++x)
#pragma unroll
        for (int y = 0; y < 4; ++y) acc[x][y] = fmaf(a[x], b[y], acc[x][y]);
    }
    __syncthreads();
  }
#pragma unroll
  for (int x = 0; x < 4; ++x)
#pragma unroll
    for (int y = 0; y < 4; ++y) {
      const size_t o = (size_t)p * D * D + (size_t)(i0 + ti * 4 + x) * D + j0 + tj * 4 + y;
      const double v = alpha * (double)acc[x][y];
      C[o] = v;
      if (C32) C32[o] = (float)v;
    }
}

// bias[p][j] = - sum_i (sum[p][i] / n) * W[p][i][j].  Eight threads per output column, each with all of
// its loads in flight at once; partial sums combined in a fixed order.  The same CTA also lays W out
// for the tensor-core projection (W^T as bf16 hi + lo parts, [D out][D in]) when asked to.
template <int D>
__global__ void __launch_bounds__(8 * D) bias_kernel(const double* __restrict__ sum, const float* __restrict__ W,
                                                     double n, float* __restrict__ bias,
                                                     __nv_bfloat16* __restrict__ wt_hi,
                                                     __nv_bfloat16* __restrict__ wt_lo) {
  constexpr int PER = D / 8;
  __shared__ float mean[D];
  __shared__ float part[8][D];
  const int p = blockIdx.x;
  const int j = threadIdx.x % D, g = threadIdx.x / D;
  if (threadIdx.x < D) mean[threadIdx.x] = (float)(sum[(size_t)p * D + threadIdx.x] / n);
  const float* Wp = W + (size_t)p * D * D + (size_t)g * PER * D + j;
  float w[PER];
#pragma unroll
  for (int i = 0; i < PER; ++i) w[i] = Wp[(size_t)i * D];
  __syncthreads();
  float s = 0.f;
#pragma unroll
  for (int i = 0; i < PER; ++i) s = fmaf(mean[g * PER + i], w[i], s);
  part[g][j] = s;
  __syncthreads();
  if (g == 0) {
    float t = 0.f;
#pragma unroll
    for (int q = 0; q < 8; ++q) t += part[q][j];
    bias[(size_t)p * D + j] = -t;
  }
  if (wt_hi) {
    for (int e = threadIdx.x; e < D * D; e += 8 * D) {
      const int o = e / D, k = e % D;
      const float w = W[(size_t)p * D * D + k * D + o];
      const __nv_bfloat16 h = __float2bfloat16_rn(w);
      wt_hi[(size_t)p * D * D + e] = h;
      wt_lo[(size_t)p * D * D + e] = __float2bfloat16_rn(w - __bfloat162float(h));
    }
  }
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
int launch_covariance(const double* gram, const double* sum, int P, int D, int n, double* cov,
                      cudaStream_t st) {
  covariance_kernel<<<dim3(ceil_div(D * D, 256), P), 256, 0, st>>>(gram, sum, D, (double)n, cov);
  CA_LAUNCH_CHECK();
  return CA_OK;
}
int launch_small_matmul(const double* A, const double* B, int P, int D, double alpha, int trans_a,
                        double* C, float* C32, cudaStream_t st) {
  small_matmul_kernel<<<dim3(D / 64, D / 64, P), 256, 0, st>>>(A, B, D, alpha, trans_a, C, C32);
  CA_LAUNCH_CHECK();
  return CA_OK;
}
int launch_bias(const double* sum, const float* W, int P, int D, int n, float* bias, cudaStream_t st,
                void* wt_hi, void* wt_lo) {
  __nv_bfloat16* hi = static_cast<__nv_bfloat16*>(wt_hi);
  __nv_bfloat16* lo = static_cast<__nv_bfloat16*>(wt_lo);
  if (D == 64) bias_kernel<64><<<P, 512, 0, st>>>(sum, W, (double)n, bias, hi, lo);
  else bias_kernel<128><<<P, 1024, 0, st>>>(sum, W, (double)n, bias, hi, lo);
  CA_LAUNCH_CHECK();
  return CA_OK;
}

}  // namespace ca
