// Batched symmetric eigendecomposition of d x d matrices (d = 64, 128) by
// parallel cyclic Jacobi, one CTA per matrix, and the d x d algebra around it:
// roots of the metric matrices (Section 3.2.2, negative eigenvalues clamped to
// zero) and principal-component bases (Section 3.2.1).
#include "kernels.h"

namespace ca {

constexpr int kMaxSweeps = 16;

template <int D>
struct EighCfg {
  static constexpr int H = D / 2;                       // rotations per step
  static constexpr int NBLK = H * (H + 1) / 2;          // 2x2 blocks with k1 <= k2
  static constexpr int THREADS = (D == 128) ? 1024 : 512;
  static constexpr int LDA = D + 1;
};

// mode 0: out = E sqrt(max(lambda,0)) E^T      (symmetric root)
// mode 1: out = eigenvectors as columns, descending eigenvalue, each column's
//         entry of largest magnitude (lowest row on ties) made positive
template <int D, typename VT>
__global__ void __launch_bounds__(EighCfg<D>::THREADS)
eigh_kernel(const double* __restrict__ A_in, int mode, double* __restrict__ out64,
            float* __restrict__ out32, double* __restrict__ evals_out) {
  using C = EighCfg<D>;
  constexpr int H = C::H, LDA = C::LDA, NT = C::THREADS;
  extern __shared__ __align__(16) unsigned char smem_raw[];
  double* A = reinterpret_cast<double*>(smem_raw);                 // [D][LDA]
  VT* Vt = reinterpret_cast<VT*>(A + D * LDA);                     // [D][LDA]  (rows = eigenvectors)
  double* rc = reinterpret_cast<double*>(Vt + D * LDA);            // [H]
  double* rs = rc + H;                                             // [H]
  double* red = rs + H;                                            // [64]
  short* pp = reinterpret_cast<short*>(red + 64);                  // [H]
  short* qq = pp + H;                                              // [H]
  unsigned short* blk = reinterpret_cast<unsigned short*>(qq + H); // [NBLK] packed (k1<<8|k2)
  int* flag = reinterpret_cast<int*>(blk + C::NBLK + (C::NBLK & 1));

  const int tid = threadIdx.x;
  const double* Ain = A_in + (size_t)blockIdx.x * D * D;
  for (int e = tid; e < D * D; e += NT) {
    int i = e / D, j = e % D;
    // symmetrise on load
    A[i * LDA + j] = 0.5 * (Ain[i * D + j] + Ain[j * D + i]);
    Vt[i * LDA + j] = (i == j) ? (VT)1 : (VT)0;
  }
  // scale so that the largest diagonal entry is 1 (eigenvectors unchanged, eigenvalues scaled back)
  __syncthreads();
  if (tid == 0) {
    double mx = 0.0;
    for (int i = 0; i < D; ++i) mx = fmax(mx, fabs(A[i * LDA + i]));
    red[0] = mx > 0.0 ? mx : 1.0;
  }
  __syncthreads();
  const double a_scale = red[0];
  {
    const double inv = 1.0 / a_scale;
    for (int e = tid; e < D * D; e += NT) A[(e / D) * LDA + (e % D)] *= inv;
  }
  __syncthreads();
  for (int e = tid; e < H * H; e += NT) {
    int k1 = e / H, k2 = e % H;
    if (k1 <= k2) {
      int idx = k1 * H - (k1 * (k1 - 1)) / 2 + (k2 - k1);
      blk[idx] = (unsigned short)((k1 << 8) | k2);
    }
  }
  __syncthreads();

  for (int sweep = 0; sweep < kMaxSweeps; ++sweep) {
    // convergence: off-diagonal mass against the whole matrix
    double off = 0.0, tot = 0.0;
    for (int e = tid; e < D * D; e += NT) {
      int i = e / D, j = e % D;
      double v = A[i * LDA + j];
      tot += v * v;
      if (i != j) off += v * v;
    }
    for (int o = 16; o > 0; o >>= 1) {
      off += __shfl_xor_sync(0xffffffffu, off, o);
      tot += __shfl_xor_sync(0xffffffffu, tot, o);
    }
    if ((tid & 31) == 0) { red[tid >> 5] = off; red[32 + (tid >> 5)] = tot; }
    __syncthreads();
    if (tid == 0) {
      double o = 0.0, t = 0.0;
      for (int w = 0; w < NT / 32; ++w) { o += red[w]; t += red[32 + w]; }
      *flag = (o <= 1e-24 * t) ? 1 : 0;       // off-diagonal norm below 1e-12 of the matrix norm
    }
    __syncthreads();
    if (*flag) break;

    for (int round = 0; round < D - 1; ++round) {
      if (tid < H) {
        int p, q;
        if (tid == 0) { p = D - 1; q = round; }
        else { p = (round + tid) % (D - 1); q = (round - tid + (D - 1)) % (D - 1); }
        if (p > q) { int t = p; p = q; q = t; }
        const double apq = A[p * LDA + q], app = A[p * LDA + p], aqq = A[q * LDA + q];
        // tan of the rotation angle: t = sgn / (|tau| + sqrt(1 + tau^2)), tau = (aqq - app) / (2 apq),
        // rewritten as sgn |apq| / (|alpha| + hypot(alpha, apq)), alpha = (aqq - app) / 2.  t only needs
        // single precision (an inexact angle leaves a residual of 1e-7 |apq|, removed by the next
        // sweep); c = 1/sqrt(1 + t^2) and s = t c are formed in double so that the rotation is
        // orthogonal to double precision.
        double c = 1.0, s = 0.0;
        const double alpha = 0.5 * (aqq - app);
        const float fa = (float)fabs(alpha), fb = (float)fabs(apq);   // entries are scaled to at most 1
        if (fb > 0.f) {
          const float tf = fb / (fa + sqrtf(fmaf(fa, fa, fb * fb)));
          const double t = ((alpha >= 0.0) == (apq >= 0.0)) ? (double)tf : -(double)tf;
          c = rsqrt(fma(t, t, 1.0));
          s = t * c;
        }
        pp[tid] = (short)p; qq[tid] = (short)q; rc[tid] = c; rs[tid] = s;
      }
      __syncthreads();
      // A <- J^T A J on 2x2 blocks (rows of pair k1, columns of pair k2), mirrored
      for (int b = tid; b < C::NBLK; b += NT) {
        const int k1 = blk[b] >> 8, k2 = blk[b] & 255;
        const int p1 = pp[k1], q1 = qq[k1], p2 = pp[k2], q2 = qq[k2];
        const double c1 = rc[k1], s1 = rs[k1], c2 = rc[k2], s2 = rs[k2];
        double a_pp = A[p1 * LDA + p2], a_pq = A[p1 * LDA + q2];
        double a_qp = A[q1 * LDA + p2], a_qq = A[q1 * LDA + q2];
        // columns: B = blk * J2
        double b_pp = c2 * a_pp - s2 * a_pq, b_pq = s2 * a_pp + c2 * a_pq;
        double b_qp = c2 * a_qp - s2 * a_qq, b_qq = s2 * a_qp + c2 * a_qq;
        // rows: J1^T * B
        double n_pp = c1 * b_pp - s1 * b_qp, n_pq = c1 * b_pq - s1 * b_qq;
        double n_qp = s1 * b_pp + c1 * b_qp, n_qq = s1 * b_pq + c1 * b_qq;
        A[p1 * LDA + p2] = n_pp; A[p1 * LDA + q2] = n_pq;
        A[q1 * LDA + p2] = n_qp; A[q1 * LDA + q2] = n_qq;
        if (k1 != k2) {
          A[p2 * LDA + p1] = n_pp; A[q2 * LDA + p1] = n_pq;
          A[p2 * LDA + q1] = n_qp; A[q2 * LDA + q1] = n_qq;
        }
      }
      // V <- V J  (rows p, q of V^T)
      for (int e = tid; e < H * D; e += NT) {
        const int k = e / D, i = e % D;
        const int p = pp[k], q = qq[k];
        const VT c = (VT)rc[k], s = (VT)rs[k];
        VT vp = Vt[p * LDA + i], vq = Vt[q * LDA + i];
        Vt[p * LDA + i] = c * vp - s * vq;
        Vt[q * LDA + i] = s * vp + c * vq;
      }
      __syncthreads();
    }
  }

  // eigenvalues on the diagonal
  double* lam = rc;          // reuse: [D] fits in rc+rs (H+H)
  if (tid < D) lam[tid] = A[tid * LDA + tid] * a_scale;
  __syncthreads();
  double* o64 = out64 + (size_t)blockIdx.x * D * D;
  float* o32 = out32 ? out32 + (size_t)blockIdx.x * D * D : nullptr;
  if (mode == 0) {
    if (evals_out && tid < D) evals_out[(size_t)blockIdx.x * D + tid] = lam[tid];
    __syncthreads();
    if (tid < D) lam[tid] = sqrt(fmax(lam[tid], 0.0));
    __syncthreads();
    for (int e = tid; e < D * D; e += NT) {
      const int i = e / D, j = e % D;
      double s = 0.0;
      for (int k = 0; k < D; ++k) s += (double)Vt[k * LDA + i] * lam[k] * (double)Vt[k * LDA + j];
      o64[e] = s;
      if (o32) o32[e] = (float)s;
    }
  } else {
    // rank of each eigenvalue in descending order (ties: lower index first)
    if (tid < D) {
      const double mine = lam[tid];
      int rank = 0;
      for (int k = 0; k < D; ++k) {
        const double other = lam[k];
        rank += (other > mine) || (other == mine && k < tid);
      }
      // sign: entry of largest magnitude positive
      double best = -1.0; double sgn = 1.0;
      for (int i = 0; i < D; ++i) {
        double v = (double)Vt[tid * LDA + i];
        if (fabs(v) > best) { best = fabs(v); sgn = (v < 0.0) ? -1.0 : 1.0; }
      }
      // stash rank and sign: reuse A's first two rows
      A[tid] = (double)rank;
      A[LDA + tid] = sgn;
      if (evals_out) evals_out[(size_t)blockIdx.x * D + rank] = mine;
    }
    __syncthreads();
    for (int e = tid; e < D * D; e += NT) {
      const int k = e / D, i = e % D;           // eigenvector k, component i
      const int col = (int)A[k];
      const double v = A[LDA + k] * (double)Vt[k * LDA + i];
      o64[i * D + col] = v;
      if (o32) o32[i * D + col] = (float)v;
    }
  }
}

template <int D, typename VT>
static size_t eigh_smem() {
  using C = EighCfg<D>;
  return sizeof(double) * D * C::LDA + sizeof(VT) * D * C::LDA + sizeof(double) * (2 * C::H + 64) +
         sizeof(short) * 2 * C::H + sizeof(unsigned short) * (C::NBLK + 1) + 16;
}

int launch_eigh(const double* A, int count, int D, int mode, double* out64, float* out32,
                double* evals, cudaStream_t st) {
  if (D == 64) {
    auto k = eigh_kernel<64, double>;
    size_t smem = eigh_smem<64, double>();
    CA_RETURN_IF_CUDA(cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    k<<<count, EighCfg<64>::THREADS, smem, st>>>(A, mode, out64, out32, evals);
  } else {
    auto k = eigh_kernel<128, float>;
    size_t smem = eigh_smem<128, float>();
    CA_RETURN_IF_CUDA(cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    k<<<count, EighCfg<128>::THREADS, smem, st>>>(A, mode, out64, out32, evals);
  }
  CA_LAUNCH_CHECK();
  return CA_OK;
}


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
  __shared__ double s_inv;
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
  for (int j = 0; j < D; ++j) {
    if (tid == 0) {
      const double piv = A[j * LDA + j];
      s_inv = (piv > s_tol) ? rsqrt(piv) : 0.0;
    }
    __syncthreads();
    const double inv = s_inv;
    // column j of F (rows j..D-1); a dropped pivot gives a zero column
    for (int i = j + tid; i < D; i += NT) A[i * LDA + j] *= inv;
    __syncthreads();
    // trailing update of the lower triangle
    const int rem = D - 1 - j;
    for (int e = tid; e < rem * rem; e += NT) {
      const int i = j + 1 + e / rem, k = j + 1 + e % rem;
      if (k <= i) A[i * LDA + k] -= A[i * LDA + j] * A[k * LDA + j];
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
                              double* __restrict__ M, double* __restrict__ CK) {
  const int p = blockIdx.y;
  const int e = blockIdx.x * blockDim.x + threadIdx.x;
  if (e >= D * D) return;
  const int i = e / D, j = e % D;
  const size_t o = (size_t)p * D * D + e;
  M[o] = gramQ[o] / n_q;
  CK[o] = gramK[o] - sumK[(size_t)p * D + i] * sumK[(size_t)p * D + j] / n_k;
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
__global__ void small_matmul_kernel(const double* __restrict__ A, const double* __restrict__ B, int D,
                                    double alpha, int trans_a, double* __restrict__ C,
                                    float* __restrict__ C32) {
  const int p = blockIdx.y;
  const double* Ap = A + (size_t)p * D * D;
  const double* Bp = B + (size_t)p * D * D;
  const int e = blockIdx.x * blockDim.x + threadIdx.x;
  if (e >= D * D) return;
  const int i = e / D, j = e % D;
  double s = 0.0;
  if (trans_a) for (int k = 0; k < D; ++k) s += Ap[k * D + i] * Bp[k * D + j];
  else for (int k = 0; k < D; ++k) s += Ap[i * D + k] * Bp[k * D + j];
  s *= alpha;
  C[(size_t)p * D * D + e] = s;
  if (C32) C32[(size_t)p * D * D + e] = (float)s;
}

// bias[p][j] = - sum_i (sum[p][i] / n) * W[p][i][j]
__global__ void bias_kernel(const double* __restrict__ sum, const double* __restrict__ W, int D, double n,
                            float* __restrict__ bias) {
  const int p = blockIdx.x;
  const int j = threadIdx.x;
  if (j >= D) return;
  double s = 0.0;
  for (int i = 0; i < D; ++i) s += (sum[(size_t)p * D + i] / n) * W[(size_t)p * D * D + i * D + j];
  bias[(size_t)p * D + j] = (float)(-s);
}

int launch_metric(const double* gramQ, const double* gramK, const double* sumK, int P, int D, int n_q,
                  int n_k, double* M, double* CK, cudaStream_t st) {
  metric_kernel<<<dim3(ceil_div(D * D, 256), P), 256, 0, st>>>(gramQ, gramK, sumK, D, (double)n_q,
                                                                (double)n_k, M, CK);
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
  small_matmul_kernel<<<dim3(ceil_div(D * D, 256), P), 256, 0, st>>>(A, B, D, alpha, trans_a, C, C32);
  CA_LAUNCH_CHECK();
  return CA_OK;
}
int launch_bias(const double* sum, const double* W, int P, int D, int n, float* bias, cudaStream_t st) {
  bias_kernel<<<P, 128, 0, st>>>(sum, W, D, (double)n, bias);
  CA_LAUNCH_CHECK();
  return CA_OK;
}

}  // namespace ca
