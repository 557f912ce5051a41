// Second moments of row sets and row transforms (Section 3.2.2: metric matrices
// Q^T Q and K_c^T K_c; Section 3.2.1: covariance for the global principal
// components; projection of the rows).
#include "kernels.h"

namespace ca {

// ---------------------------------------------------------------------------
// Gram matrix and column sums of a chunk of rows.  One CTA per (chunk, problem),
// 256 threads; thread (ti, tj) owns a TM x TM tile of the D x D result.
// partial[(p * n_chunks + chunk) * (D*D + D)] : D*D Gram (row-major) then D sums.
// ---------------------------------------------------------------------------
template <typename T, int D>
__global__ void __launch_bounds__(256) gram_chunk_kernel(const T* __restrict__ X, int n_rows,
                                                         int chunk_rows, int n_chunks,
                                                         float* __restrict__ partial) {
  constexpr int TR = 32;            // rows staged per step
  constexpr int TM = D / 16;        // 4 (D=64) or 8 (D=128)
  __shared__ float xs[TR][D + 4];
  const int p = blockIdx.y, chunk = blockIdx.x;
  const T* Xp = X + (size_t)p * n_rows * D;
  const int r_begin = chunk * chunk_rows;
  const int r_end = min(n_rows, r_begin + chunk_rows);
  const int ti = threadIdx.x / 16, tj = threadIdx.x % 16;
  float acc[TM][TM];
#pragma unroll
  for (int i = 0; i < TM; ++i)
#pragma unroll
    for (int j = 0; j < TM; ++j) acc[i][j] = 0.f;
  float colsum = 0.f;
  for (int r0 = r_begin; r0 < r_end; r0 += TR) {
    const int nr = min(TR, r_end - r0);
    for (int e = threadIdx.x; e < TR * D; e += 256) {
      int r = e / D, col = e % D;
      xs[r][col] = (r < nr) ? to_f32<T>(Xp[(size_t)(r0 + r) * D + col]) : 0.f;
    }
    __syncthreads();
#pragma unroll 4
    for (int r = 0; r < TR; ++r) {
      float a[TM], b[TM];
#pragma unroll
      for (int i = 0; i < TM; ++i) a[i] = xs[r][ti * TM + i];
#pragma unroll
      for (int j = 0; j < TM; ++j) b[j] = xs[r][tj * TM + j];
#pragma unroll
      for (int i = 0; i < TM; ++i)
#pragma unroll
        for (int j = 0; j < TM; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
    }
    if (threadIdx.x < D) {
      for (int r = 0; r < TR; ++r) colsum += xs[r][threadIdx.x];
    }
    __syncthreads();
  }
  float* out = partial + ((size_t)p * n_chunks + chunk) * (D * D + D);
#pragma unroll
  for (int i = 0; i < TM; ++i)
#pragma unroll
    for (int j = 0; j < TM; ++j) out[(ti * TM + i) * D + tj * TM + j] = acc[i][j];
  if (threadIdx.x < D) out[D * D + threadIdx.x] = colsum;
}

// Sums the chunk partials in a fixed order, in double.
__global__ void gram_finalize_kernel(const float* __restrict__ partial, int n_chunks, int elems,
                                     double* __restrict__ gram, double* __restrict__ colsum,
                                     int dd) {
  const int p = blockIdx.y;
  const int e = blockIdx.x * blockDim.x + threadIdx.x;
  if (e >= elems) return;
  const float* src = partial + (size_t)p * n_chunks * elems + e;
  double s = 0.0;
  for (int c = 0; c < n_chunks; ++c) s += (double)src[(size_t)c * elems];
  if (e < dd) gram[(size_t)p * dd + e] = s;
  else colsum[(size_t)p * (elems - dd) + (e - dd)] = s;
}

int moments_chunking(int n_rows, int problems, int* chunk_rows, int* n_chunks) {
  long long target = ((long long)n_rows * problems + 1183) / 1184;   // ~8 CTAs per SM
  int cr = (int)((target + 63) / 64 * 64);
  if (cr < 256) cr = 256;
  if (cr > 8192) cr = 8192;
  *chunk_rows = cr;
  *n_chunks = ceil_div(n_rows, cr);
  return 0;
}

int launch_gram_finalize(const float* partial, int problems, int n_chunks, int D, double* gram,
                         double* colsum, cudaStream_t st) {
  const int elems = D * D + D;
  gram_finalize_kernel<<<dim3(ceil_div(elems, 256), problems), 256, 0, st>>>(partial, n_chunks, elems, gram,
                                                                              colsum, D * D);
  CA_LAUNCH_CHECK();
  return CA_OK;
}

template <typename T>
static int launch_moments_t(const T* X, int problems, int n_rows, int D, float* partial,
                            double* gram, double* colsum, cudaStream_t st) {
  int chunk_rows, n_chunks;
  moments_chunking(n_rows, problems, &chunk_rows, &n_chunks);
  dim3 grid(n_chunks, problems);
  if (D == 64) gram_chunk_kernel<T, 64><<<grid, 256, 0, st>>>(X, n_rows, chunk_rows, n_chunks, partial);
  else gram_chunk_kernel<T, 128><<<grid, 256, 0, st>>>(X, n_rows, chunk_rows, n_chunks, partial);
  CA_LAUNCH_CHECK();
  return launch_gram_finalize(partial, problems, n_chunks, D, gram, colsum, st);
}

int launch_moments(const void* X, int dtype, int problems, int n_rows, int D, float* partial,
                   double* gram, double* colsum, cudaStream_t st) {
  if (dtype == CA_DTYPE_BF16)
    return launch_moments_t(static_cast<const __nv_bfloat16*>(X), problems, n_rows, D, partial, gram, colsum, st);
  return launch_moments_t(static_cast<const float*>(X), problems, n_rows, D, partial, gram, colsum, st);
}

// ---------------------------------------------------------------------------
// Row transform: out[r,:] = g(X[r,:] W + b), W [D,D] row-major fp32, b [D] (may
// be null).  g = identity, or division by the row's Euclidean norm (rows whose
// norm is below 1e-30 map to zero).  Output fp32.  One CTA per 64 rows.
// ---------------------------------------------------------------------------
template <typename T, int D>
__global__ void __launch_bounds__(256) transform_rows_kernel(const T* __restrict__ X, int n_rows,
                                                             const float* __restrict__ W,
                                                             const float* __restrict__ bias,
                                                             int normalize, float* __restrict__ out) {
  constexpr int TR = 64;
  constexpr int CN = D / 16;     // columns per thread (4 or 8), rows per thread = 4
  extern __shared__ float smem[];
  float* Ws = smem;                       // [D][D]
  float* xs = Ws + D * D;                 // [TR][D+1]
  float* ys = xs + TR * (D + 1);          // [TR][D+1]
  __shared__ float inv_norm[TR];
  const int p = blockIdx.y;
  const int r0 = blockIdx.x * TR;
  const int nr = min(TR, n_rows - r0);
  const T* Xp = X + (size_t)p * n_rows * D;
  const float* Wp = W + (size_t)p * D * D;
  for (int e = threadIdx.x; e < D * D; e += 256) Ws[e] = Wp[e];
  for (int e = threadIdx.x; e < TR * D; e += 256) {
    int r = e / D, col = e % D;
    xs[r * (D + 1) + col] = (r < nr) ? to_f32<T>(Xp[(size_t)(r0 + r) * D + col]) : 0.f;
  }
  __syncthreads();
  const int tr = threadIdx.x / 16;        // 16 row groups of 4 rows
  const int tc = threadIdx.x % 16;        // 16 column groups of CN columns (interleaved by 16)
  float acc[4][CN];
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < CN; ++j) acc[i][j] = 0.f;
#pragma unroll 4
  for (int k = 0; k < D; ++k) {
    float a[4], b[CN];
#pragma unroll
    for (int i = 0; i < 4; ++i) a[i] = xs[(tr * 4 + i) * (D + 1) + k];
#pragma unroll
    for (int j = 0; j < CN; ++j) b[j] = Ws[k * D + tc + 16 * j];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
      for (int j = 0; j < CN; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
  }
  const float* bp = bias ? bias + (size_t)p * D : nullptr;
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < CN; ++j) {
      float v = acc[i][j] + (bp ? bp[tc + 16 * j] : 0.f);
      ys[(tr * 4 + i) * (D + 1) + tc + 16 * j] = v;
    }
  __syncthreads();
  if (normalize) {
    // 4 threads per row, fixed summation order
    const int r = threadIdx.x / 4, q = threadIdx.x % 4;
    float s = 0.f;
    for (int col = q; col < D; col += 4) { float v = ys[r * (D + 1) + col]; s = fmaf(v, v, s); }
    s += __shfl_xor_sync(0xffffffffu, s, 1);
    s += __shfl_xor_sync(0xffffffffu, s, 2);
    if (q == 0) { float n = sqrtf(s); inv_norm[r] = (n >= 1e-30f) ? 1.f / n : 0.f; }
    __syncthreads();
  }
  float* op = out + ((size_t)p * n_rows + r0) * D;
  for (int e = threadIdx.x; e < nr * D; e += 256) {
    int r = e / D, col = e % D;
    float v = ys[r * (D + 1) + col];
    if (normalize) v *= inv_norm[r];
    op[(size_t)r * D + col] = v;
  }
}

template <typename T>
static int launch_transform_t(const T* X, int problems, int n_rows, int D, const float* W,
                              const float* bias, int normalize, float* out, cudaStream_t st) {
  dim3 grid(ceil_div(n_rows, 64), problems);
  size_t smem = (size_t)(D * D + 2 * 64 * (D + 1)) * sizeof(float);
  if (D == 64) {
    auto k = transform_rows_kernel<T, 64>;
    CA_RETURN_IF_CUDA(cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    k<<<grid, 256, smem, st>>>(X, n_rows, W, bias, normalize, out);
  } else {
    auto k = transform_rows_kernel<T, 128>;
    CA_RETURN_IF_CUDA(cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    k<<<grid, 256, smem, st>>>(X, n_rows, W, bias, normalize, out);
  }
  CA_LAUNCH_CHECK();
  return CA_OK;
}

int launch_transform_rows(const void* X, int dtype, int problems, int n_rows, int D, const float* W,
                          const float* bias, int normalize, float* out, cudaStream_t st) {
  if (dtype == CA_DTYPE_BF16)
    return launch_transform_t(static_cast<const __nv_bfloat16*>(X), problems, n_rows, D, W, bias, normalize, out, st);
  return launch_transform_t(static_cast<const float*>(X), problems, n_rows, D, W, bias, normalize, out, st);
}

}  // namespace ca
