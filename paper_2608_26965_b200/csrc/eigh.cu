// Batched symmetric eigendecomposition of d x d matrices (d = 64, 128) by
// parallel cyclic Jacobi, one CTA per matrix (principal-component bases,
// Section 3.2.1), Cholesky factors of the metric matrices (Section 3.2.2), and
// the d x d algebra around them.
#include "kernels.h"

namespace ca {

constexpr int kMaxSweeps = 12;
constexpr int kEighThreads = 1024;

template <int D>
struct EighCfg {
  static constexpr int H = D / 2;                                   // rotations per step
  static constexpr int NB = (H * H) / kEighThreads > 0 ? (H * H) / kEighThreads : 1;   // 2x2 blocks per thread
  static constexpr int NV = (H * D / 4) / kEighThreads > 0 ? (H * D / 4) / kEighThreads : 1;
  static constexpr int LDA = D + 4;                                 // 16-byte aligned rows, staggered banks
};

// Position permutation applied after every step (round-robin tournament): the
// rows/columns sitting at positions (2k, 2k+1) are the pair rotated next.
template <int D>
__device__ __forceinline__ int next_position(int i) {
  if (i == 0) return 0;
  if (i & 1) return i == 1 ? 2 : i - 2;
  return i == D - 2 ? D - 1 : i + 2;
}

template <typename T> struct Vec2;
template <> struct Vec2<float> { using type = float2; };
template <> struct Vec2<double> { using type = double2; };
template <typename T> struct __align__(16) Vec4 { T x, y, z, w; };

// Eigenvectors of symmetric d x d matrices by parallel cyclic Jacobi, one CTA per
// matrix.  The matrix lives in shared memory in "position space": each step
// rotates the d/2 adjacent pairs (2k, 2k+1) at once -- every thread transforms
// 2x2 blocks J1^T B J2 read with vector loads from one copy of the matrix --
// and stores the result into a second copy at the positions of the next
// pairing, so pairs are always adjacent and a step needs two barriers.  The
// rows of V^T follow the same permutation (their stores are deferred past the
// barrier instead of being double-buffered).  AT is the working precision of
// the matrix and of V (float for d = 128, where two double copies would not fit
// in shared memory; the split coordinates are fp32 anyway).  Output:
// eigenvectors as columns, descending eigenvalue, each column's entry of largest
// magnitude (lowest row on ties) made positive.
template <int D, typename AT>
__global__ void __launch_bounds__(kEighThreads)
eigh_kernel(const double* __restrict__ A_in, double* __restrict__ out64, float* __restrict__ out32,
            double* __restrict__ evals_out) {
  using C = EighCfg<D>;
  using V2 = typename Vec2<AT>::type;
  constexpr int H = C::H, LDA = C::LDA, NT = kEighThreads;
  extern __shared__ __align__(16) unsigned char smem_raw[];
  AT* Abuf0 = reinterpret_cast<AT*>(smem_raw);                     // [D][LDA]
  AT* Abuf1 = Abuf0 + D * LDA;                                     // [D][LDA]
  AT* Vt = Abuf1 + D * LDA;                                        // [D][D]  (rows = eigenvectors)
  AT* rc = Vt + D * D;                                             // [H]
  AT* rs = rc + H;                                                 // [H]
  double* red = reinterpret_cast<double*>(rs + H);                 // [64 + D]
  int* flag = reinterpret_cast<int*>(red + 64 + D);

  const int tid = threadIdx.x;
  const double* Ain = A_in + (size_t)blockIdx.x * D * D;
  // scale so that the largest diagonal entry is 1 (eigenvectors unchanged, eigenvalues scaled back)
  if (tid < 32) {
    double mx = 0.0;
    for (int i = tid; i < D; i += 32) mx = fmax(mx, fabs(Ain[i * D + i]));
    for (int o = 16; o > 0; o >>= 1) mx = fmax(mx, __shfl_xor_sync(0xffffffffu, mx, o));
    if (tid == 0) red[0] = mx > 0.0 ? mx : 1.0;
  }
  __syncthreads();
  const double a_scale = red[0];
  {
    const double inv = 1.0 / a_scale;
    for (int e = tid; e < D * D; e += NT) {
      const int i = e / D, j = e % D;
      Abuf0[i * LDA + j] = (AT)(0.5 * (Ain[i * D + j] + Ain[j * D + i]) * inv);   // symmetrise on load
      Vt[e] = (i == j) ? (AT)1 : (AT)0;
    }
  }
  __syncthreads();

  // fixed work assignment in position space
  int rd[C::NB], w00[C::NB], w01[C::NB], w10[C::NB], w11[C::NB], bk1[C::NB], bk2[C::NB];
#pragma unroll
  for (int u = 0; u < C::NB; ++u) {
    const int b = tid + u * NT;
    const int k1 = (b / H) % H, k2 = b % H;
    bk1[u] = k1; bk2[u] = k2;
    rd[u] = (2 * k1) * LDA + 2 * k2;
    const int p1 = next_position<D>(2 * k1) * LDA, q1 = next_position<D>(2 * k1 + 1) * LDA;
    const int p2 = next_position<D>(2 * k2), q2 = next_position<D>(2 * k2 + 1);
    w00[u] = p1 + p2; w01[u] = p1 + q2; w10[u] = q1 + p2; w11[u] = q1 + q2;
  }
  int vk[C::NV], vrd[C::NV], vw0[C::NV], vw1[C::NV];
#pragma unroll
  for (int u = 0; u < C::NV; ++u) {
    const int e = tid + u * NT;
    const int k = (e / (D / 4)) % H, i4 = e % (D / 4);
    vk[u] = k;
    vrd[u] = (2 * k) * D + 4 * i4;
    vw0[u] = next_position<D>(2 * k) * D + 4 * i4;
    vw1[u] = next_position<D>(2 * k + 1) * D + 4 * i4;
  }
  const bool blk_live = tid < H * H, v_live = tid < H * D / 4;      // only d = 64 leaves threads idle

  AT* Acur = Abuf0;
  AT* Anext = Abuf1;
  Vec4<AT> nv0[C::NV], nv1[C::NV];
  bool v_pending = false;
  // Stop when the squared off-diagonal norm is below `tol` of the matrix norm, or when a sweep no
  // longer reduces it fourfold (the rounding floor of the working precision has been reached).
  const double tol = sizeof(AT) == 4 ? 1e-11 : 1e-24;
  double prev_off = 1e300;       // used by thread 0 only
  for (int sweep = 0; sweep < kMaxSweeps; ++sweep) {
    // convergence: off-diagonal mass against the whole matrix
    double off = 0.0, tot = 0.0;
    for (int e = tid; e < D * D; e += NT) {
      const int i = e / D, j = e % D;
      const double v = (double)Acur[i * LDA + j];
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
      *flag = (o <= tol * t || (sweep >= 3 && o > 0.25 * prev_off)) ? 1 : 0;
      prev_off = o;
    }
    __syncthreads();
    if (*flag) break;

    for (int step = 0; step < D - 1; ++step) {
      // rotation of each adjacent pair; deferred stores of the previous step's V rows
      if (tid < H) {
        const int p = 2 * tid, q = p + 1;
        const float apq = (float)Acur[p * LDA + q];
        const float alpha = 0.5f * ((float)Acur[q * LDA + q] - (float)Acur[p * LDA + p]);
        // t = tan(angle) = sgn |apq| / (|alpha| + hypot(alpha, apq)); c = 1/sqrt(1 + t^2), s = t c.
        // An inexact t only leaves a small residual in a_pq that the next sweep removes;
        // c and s are formed in the working precision so that c^2 + s^2 = 1 to rounding.
        AT c = (AT)1, s = (AT)0;
        const float fa = fabsf(alpha), fb = fabsf(apq);
        if (fb > 0.f) {
          const float tf = fb / (fa + sqrtf(fmaf(fa, fa, fb * fb)));
          const AT t = ((alpha >= 0.f) == (apq >= 0.f)) ? (AT)tf : -(AT)tf;
          if (sizeof(AT) == 4) c = (AT)rsqrtf((float)(t * t + (AT)1)); else c = (AT)rsqrt((double)(t * t + (AT)1));
          s = t * c;
        }
        rc[tid] = c; rs[tid] = s;
      }
      if (v_pending && v_live) {
#pragma unroll
        for (int u = 0; u < C::NV; ++u) {
          *reinterpret_cast<Vec4<AT>*>(&Vt[vw0[u]]) = nv0[u];
          *reinterpret_cast<Vec4<AT>*>(&Vt[vw1[u]]) = nv1[u];
        }
      }
      __syncthreads();
      if (blk_live) {
#pragma unroll
        for (int u = 0; u < C::NB; ++u) {
          const AT c1 = rc[bk1[u]], s1 = rs[bk1[u]], c2 = rc[bk2[u]], s2 = rs[bk2[u]];
          const V2 r0 = *reinterpret_cast<const V2*>(&Acur[rd[u]]);
          const V2 r1 = *reinterpret_cast<const V2*>(&Acur[rd[u] + LDA]);
          // columns: B = blk * J2 ; rows: J1^T * B
          const AT b_pp = c2 * r0.x - s2 * r0.y, b_pq = s2 * r0.x + c2 * r0.y;
          const AT b_qp = c2 * r1.x - s2 * r1.y, b_qq = s2 * r1.x + c2 * r1.y;
          Anext[w00[u]] = c1 * b_pp - s1 * b_qp; Anext[w01[u]] = c1 * b_pq - s1 * b_qq;
          Anext[w10[u]] = s1 * b_pp + c1 * b_qp; Anext[w11[u]] = s1 * b_pq + c1 * b_qq;
        }
      }
      if (v_live) {
#pragma unroll
        for (int u = 0; u < C::NV; ++u) {
          const AT c = rc[vk[u]], s = rs[vk[u]];
          const Vec4<AT> vp = *reinterpret_cast<const Vec4<AT>*>(&Vt[vrd[u]]);
          const Vec4<AT> vq = *reinterpret_cast<const Vec4<AT>*>(&Vt[vrd[u] + D]);
          nv0[u].x = c * vp.x - s * vq.x; nv0[u].y = c * vp.y - s * vq.y;
          nv0[u].z = c * vp.z - s * vq.z; nv0[u].w = c * vp.w - s * vq.w;
          nv1[u].x = s * vp.x + c * vq.x; nv1[u].y = s * vp.y + c * vq.y;
          nv1[u].z = s * vp.z + c * vq.z; nv1[u].w = s * vp.w + c * vq.w;
        }
      }
      v_pending = true;
      __syncthreads();
      AT* t = Acur; Acur = Anext; Anext = t;
    }
  }
  if (v_pending && v_live) {
#pragma unroll
    for (int u = 0; u < C::NV; ++u) {
      *reinterpret_cast<Vec4<AT>*>(&Vt[vw0[u]]) = nv0[u];
      *reinterpret_cast<Vec4<AT>*>(&Vt[vw1[u]]) = nv1[u];
    }
  }
  __syncthreads();

  // eigenvalues on the diagonal
  double* lam = red + 64;
  if (tid < D) lam[tid] = (double)Acur[tid * LDA + tid] * a_scale;
  __syncthreads();
  double* o64 = out64 + (size_t)blockIdx.x * D * D;
  float* o32 = out32 ? out32 + (size_t)blockIdx.x * D * D : nullptr;
  // rank of each eigenvalue in descending order (ties: lower position first)
  int* rank_of = reinterpret_cast<int*>(Anext);
  float* sign_of = reinterpret_cast<float*>(rank_of + D);
  if (tid < D) {
    const double mine = lam[tid];
    int rank = 0;
    for (int k = 0; k < D; ++k) {
      const double other = lam[k];
      rank += (other > mine) || (other == mine && k < tid);
    }
    // sign: entry of largest magnitude positive
    double best = -1.0; float sgn = 1.f;
    for (int i = 0; i < D; ++i) {
      const double v = (double)Vt[tid * D + i];
      if (fabs(v) > best) { best = fabs(v); sgn = (v < 0.0) ? -1.f : 1.f; }
    }
    rank_of[tid] = rank;
    sign_of[tid] = sgn;
    if (evals_out) evals_out[(size_t)blockIdx.x * D + rank] = mine;
  }
  __syncthreads();
  for (int e = tid; e < D * D; e += NT) {
    const int k = e / D, i = e % D;           // eigenvector k, component i
    const double v = (double)sign_of[k] * (double)Vt[k * D + i];
    o64[i * D + rank_of[k]] = v;
    if (o32) o32[i * D + rank_of[k]] = (float)v;
  }
}

template <int D, typename AT>
static size_t eigh_smem() {
  using C = EighCfg<D>;
  return sizeof(AT) * (2 * D * C::LDA + D * D + 2 * C::H) + sizeof(double) * (64 + D) + 16;
}

int launch_eigh(const double* A, int count, int D, double* out64, float* out32, double* evals,
                cudaStream_t st) {
  if (D == 64) {
    auto k = eigh_kernel<64, float>;
    size_t smem = eigh_smem<64, float>();
    CA_RETURN_IF_CUDA(cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    k<<<count, kEighThreads, smem, st>>>(A, out64, out32, evals);
  } else {
    auto k = eigh_kernel<128, float>;
    size_t smem = eigh_smem<128, float>();
    CA_RETURN_IF_CUDA(cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    k<<<count, kEighThreads, smem, st>>>(A, out64, out32, evals);
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
                              double ck_scale, double* __restrict__ M, double* __restrict__ CK) {
  const int p = blockIdx.y;
  const int e = blockIdx.x * blockDim.x + threadIdx.x;
  if (e >= D * D) return;
  const int i = e / D, j = e % D;
  const size_t o = (size_t)p * D * D + e;
  M[o] = gramQ[o] / n_q;
  CK[o] = (gramK[o] - sumK[(size_t)p * D + i] * sumK[(size_t)p * D + j] / n_k) * ck_scale;
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
  __shared__ float As[16][64 + 4];     // As[k][i]
  __shared__ float Bs[16][64 + 4];     // Bs[k][j]
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
  for (int k0 = 0; k0 < D; k0 += 16) {
    for (int e = threadIdx.x; e < 16 * 64; e += 256) {
      const int k = e / 64, x = e % 64;
      As[k][x] = (float)(trans_a ? Ap[(size_t)(k0 + k) * D + i0 + x] : Ap[(size_t)(i0 + x) * D + k0 + k]);
      Bs[k][x] = (float)Bp[(size_t)(k0 + k) * D + j0 + x];
    }
    __syncthreads();
#pragma unroll
    for (int k = 0; k < 16; ++k) {
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

// bias[p][j] = - sum_i (sum[p][i] / n) * W[p][i][j]   (float accumulation, four independent chains)
__global__ void bias_kernel(const double* __restrict__ sum, const double* __restrict__ W, int D, double n,
                            float* __restrict__ bias) {
  const int p = blockIdx.x;
  const int j = threadIdx.x;
  if (j >= D) return;
  const float inv_n = (float)(1.0 / n);
  float s0 = 0.f, s1 = 0.f, s2 = 0.f, s3 = 0.f;
  const double* Wp = W + (size_t)p * D * D + j;
  const double* sp = sum + (size_t)p * D;
  for (int i = 0; i < D; i += 4) {
    s0 = fmaf((float)sp[i] * inv_n, (float)Wp[(size_t)i * D], s0);
    s1 = fmaf((float)sp[i + 1] * inv_n, (float)Wp[(size_t)(i + 1) * D], s1);
    s2 = fmaf((float)sp[i + 2] * inv_n, (float)Wp[(size_t)(i + 2) * D], s2);
    s3 = fmaf((float)sp[i + 3] * inv_n, (float)Wp[(size_t)(i + 3) * D], s3);
  }
  bias[(size_t)p * D + j] = -((s0 + s1) + (s2 + s3));
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
int launch_bias(const double* sum, const double* W, int P, int D, int n, float* bias, cudaStream_t st) {
  bias_kernel<<<P, 128, 0, st>>>(sum, W, D, (double)n, bias);
  CA_LAUNCH_CHECK();
  return CA_OK;
}

}  // namespace ca
