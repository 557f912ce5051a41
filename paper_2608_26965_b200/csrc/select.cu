// Assignment (Section 3.3): centroid-centroid scores and exact top-k selection.
// score(i, j) = cq_i . ck_j in float32 with a fixed operation order (terms added
// for k = 0, 1, ..., product and sum rounded separately, no fused multiply-add),
// so the scores -- and with them the selection -- are reproducible bit for bit;
// the k best per query cluster by (score descending, index ascending), written
// in ascending index order.  With fewer than 128 key clusters one kernel scores
// and selects; otherwise the scores are computed in tiles first (score_tile_kernel).
// The second half of the file is the adaptive (mass-recall) selection.
#include "kernels.h"

namespace ca {

constexpr int kSelectThreads = 256;
constexpr int kSelectQT = 4;          // query clusters per CTA (key centroids are read once for all)
// From this many key clusters on the scores are computed in tiles first: measured faster from 128
// clusters up (0.041 -> 0.030 ms at 512 x 128 clusters of 16 heads, 0.75 -> 0.56 ms at 1024 x 1024).
constexpr int kSelectTiledMinClusters = 128;

__device__ __forceinline__ uint32_t score_key(float s) {
  if (s == 0.0f) s = 0.0f;                        // -0 and +0 compare equal
  const uint32_t u = __float_as_uint(s);
  return (u >> 31) ? ~u : (u | 0x80000000u);
}

// QT query clusters per CTA: 4 when the CTA computes the scores itself (the key centroids are read
// once for the four), 1 when the scores come from memory (less shared memory, more CTAs per SM).
template <int D, int QT>
__global__ void __launch_bounds__(kSelectThreads)
score_select_kernel(const float* __restrict__ cq, const float* __restrict__ ck, int n_qc, int n_kc,
                    int keep, int32_t* __restrict__ block_idx, const float* __restrict__ scores, int row0,
                    int chunk_rows) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  uint32_t* keys = reinterpret_cast<uint32_t*>(smem_raw);                       // [QT][n_kc]
  float* qs = reinterpret_cast<float*>(keys + (size_t)QT * n_kc);        // [QT][D]
  __shared__ int s_hist[QT][256];
  __shared__ int s_warp[QT][64];
  __shared__ int s_scalar[QT][4];
  const int p = blockIdx.y;
  const int q0 = row0 + blockIdx.x * QT;
  const int nq = min(QT, min(n_qc, row0 + chunk_rows) - q0);
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const float* cqp = cq + ((size_t)p * n_qc + q0) * D;
  const float* ckp = ck + (size_t)p * n_kc * D;
  if (scores) {
    // the scores of this chunk of rows were computed by score_tile_kernel (same operation order)
    for (int t = 0; t < nq; ++t) {
      const float* srow = scores + ((size_t)p * chunk_rows + (q0 - row0 + t)) * n_kc;
      for (int j = tid; j < n_kc; j += kSelectThreads) keys[(size_t)t * n_kc + j] = score_key(__ldg(srow + j));
    }
  } else {
  for (int e = tid; e < QT * D; e += kSelectThreads) qs[e] = (e < nq * D) ? cqp[e] : 0.f;
  __syncthreads();

  for (int j = tid; j < n_kc; j += kSelectThreads) {
    float acc[QT];
#pragma unroll
    for (int t = 0; t < QT; ++t) acc[t] = 0.f;
    const float4* row = reinterpret_cast<const float4*>(ckp + (size_t)j * D);
    for (int k4 = 0; k4 < D / 4; ++k4) {
      const float4 kv = __ldg(row + k4);
#pragma unroll
      for (int t = 0; t < QT; ++t) {
        const float* q = qs + t * D + k4 * 4;
        acc[t] = __fadd_rn(acc[t], __fmul_rn(q[0], kv.x));
        acc[t] = __fadd_rn(acc[t], __fmul_rn(q[1], kv.y));
        acc[t] = __fadd_rn(acc[t], __fmul_rn(q[2], kv.z));
        acc[t] = __fadd_rn(acc[t], __fmul_rn(q[3], kv.w));
      }
    }
#pragma unroll
    for (int t = 0; t < QT; ++t) keys[(size_t)t * n_kc + j] = score_key(acc[t]);
  }
  }
  __syncthreads();

  // ---- radix selection of the keep-th largest key, the QT rows side by side (one set of barriers
  // for all of them: a row on its own is bound by the barriers of its passes, not by work)
  uint32_t prefix[QT], mask = 0;
  int remaining[QT];
#pragma unroll
  for (int t = 0; t < QT; ++t) { prefix[t] = 0; remaining[t] = keep; }
  for (int shift = 24; shift >= 0; shift -= 8) {
#pragma unroll
    for (int t = 0; t < QT; ++t) s_hist[t][tid] = 0;                 // kSelectThreads == 256 bins
    __syncthreads();
    for (int j0 = 0; j0 < n_kc; j0 += kSelectThreads) {
      const int j = j0 + tid;
      const bool ok = j < n_kc;
#pragma unroll
      for (int t = 0; t < QT; ++t) {
        if (t >= nq) break;
        const uint32_t k = ok ? keys[(size_t)t * n_kc + j] : 0u;
        // one atomic per candidate, also for the leading digit (a warp match per position to merge
        // equal digits measured three times as slow as the atomics it saves)
        if (ok && ((k & mask) == prefix[t])) atomicAdd(&s_hist[t][(k >> shift) & 255u], 1);
      }
    }
    __syncthreads();
    if (warp < nq) {
      // warp t scans row t's bins from the top: lane 0 owns bins 255..248
      int local[8]; int sum = 0;
#pragma unroll
      for (int b = 0; b < 8; ++b) { local[b] = s_hist[warp][255 - (lane * 8 + b)]; sum += local[b]; }
      int incl = sum;
      for (int o = 1; o < 32; o <<= 1) {
        const int v = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += v;
      }
      int before = incl - sum;
      int rem = 0;
#pragma unroll
      for (int t = 0; t < QT; ++t) if (t == warp) rem = remaining[t];
#pragma unroll
      for (int b = 0; b < 8; ++b) {
        if (before < rem && rem <= before + local[b]) {
          s_scalar[warp][0] = 255 - (lane * 8 + b);
          s_scalar[warp][1] = rem - before;
        }
        before += local[b];
      }
    }
    __syncthreads();
#pragma unroll
    for (int t = 0; t < QT; ++t) {
      if (t < nq) {
        prefix[t] |= (uint32_t)s_scalar[t][0] << shift;
        remaining[t] = s_scalar[t][1];
      }
    }
    mask |= 255u << shift;
    // the next pass's first barrier (after the bins are cleared) orders these reads before the
    // next writes of s_scalar
  }

  // ---- output, ascending index: keys above the threshold, then threshold-valued ones, lowest
  // indices first, until the list is full; again all rows per barrier
  int gt_before[QT], eq_before[QT];
#pragma unroll
  for (int t = 0; t < QT; ++t) { gt_before[t] = 0; eq_before[t] = 0; }
  for (int j0 = 0; j0 < n_kc; j0 += kSelectThreads) {
    const int j = j0 + tid;
    const bool ok = j < n_kc;
    int packed[QT], incl[QT];
#pragma unroll
    for (int t = 0; t < QT; ++t) {
      const uint32_t k = (ok && t < nq) ? keys[(size_t)t * n_kc + j] : 0u;
      const int is_gt = (ok && t < nq && k > prefix[t]) ? 1 : 0;
      const int is_eq = (ok && t < nq && k == prefix[t]) ? 1 : 0;
      packed[t] = is_gt | (is_eq << 16);
      int v = packed[t];
      for (int o = 1; o < 32; o <<= 1) {
        const int u = __shfl_up_sync(0xffffffffu, v, o);
        if (lane >= o) v += u;
      }
      incl[t] = v;
      if (lane == 31) s_warp[t][warp] = v;
    }
    __syncthreads();
    if (warp < QT) {
      const int w = (lane < kSelectThreads / 32) ? s_warp[warp][lane] : 0;
      int wi = w;
      for (int o = 1; o < 32; o <<= 1) {
        const int v = __shfl_up_sync(0xffffffffu, wi, o);
        if (lane >= o) wi += v;
      }
      s_warp[warp][32 + lane] = wi - w;
      if (lane == 31) s_scalar[warp][2] = wi;
    }
    __syncthreads();
#pragma unroll
    for (int t = 0; t < QT; ++t) {
      if (t >= nq) break;
      const int excl = incl[t] - packed[t] + s_warp[t][32 + warp];
      const int gt_here = gt_before[t] + (excl & 0xffff);
      const int eq_here = eq_before[t] + (excl >> 16);
      const int eq_take = remaining[t];    // threshold-valued clusters taken, lowest indices first
      const bool is_gt = (packed[t] & 1) != 0, is_eq = (packed[t] >> 16) != 0;
      int32_t* out = block_idx + ((size_t)p * n_qc + q0 + t) * keep;
      if (is_gt || (is_eq && eq_here < eq_take)) out[gt_here + min(eq_here, eq_take)] = j;
      const int total = s_scalar[t][2];
      gt_before[t] += total & 0xffff;
      eq_before[t] += total >> 16;
    }
    __syncthreads();
  }
}

size_t select_smem_bytes(int n_kc, int D, int qt) {
  return (size_t)qt * n_kc * sizeof(uint32_t) + (size_t)qt * D * sizeof(float);
}

// ---------------------------------------------------------------------------
// Scores of a chunk of query clusters against every key cluster, 64 x 64 tiles.
// Used when there are many key clusters: the fused kernels re-read all key
// centroids for every few query clusters, which is bound by L2 traffic.  Every
// score is accumulated for k = 0, 1, ... with separately rounded product and sum,
// exactly as in the fused kernels, so both paths give the same bits.
//   scores [P][chunk_rows][n_kc]
// ---------------------------------------------------------------------------
template <int D>
__global__ void __launch_bounds__(256)
score_tile_kernel(const float* __restrict__ cq, const float* __restrict__ ck, int n_qc, int n_kc, int row0,
                  int chunk_rows, float* __restrict__ scores) {
  extern __shared__ __align__(16) float tile_smem[];
  float* As = tile_smem;                 // [D][64]  As[k][i]
  float* Bs = tile_smem + D * 64;        // [D][64]  Bs[k][j]
  const int p = blockIdx.z;
  const int i0 = row0 + blockIdx.y * 64, j0 = blockIdx.x * 64;
  const int row_end = min(n_qc, row0 + chunk_rows);
  const int tid = threadIdx.x;
  const float* cqp = cq + (size_t)p * n_qc * D;
  const float* ckp = ck + (size_t)p * n_kc * D;
  // lanes take consecutive rows of one 16-byte column group: the transposing stores below then fall
  // in consecutive banks (with consecutive column groups per lane they all hit one bank)
  for (int e = tid; e < 64 * (D / 4); e += 256) {
    const int r = e % 64, k4 = e / 64;
    float4 a = make_float4(0.f, 0.f, 0.f, 0.f), b = a;
    if (i0 + r < row_end) a = __ldg(reinterpret_cast<const float4*>(cqp + (size_t)(i0 + r) * D) + k4);
    if (j0 + r < n_kc) b = __ldg(reinterpret_cast<const float4*>(ckp + (size_t)(j0 + r) * D) + k4);
    As[(k4 * 4 + 0) * 64 + r] = a.x; As[(k4 * 4 + 1) * 64 + r] = a.y;
    As[(k4 * 4 + 2) * 64 + r] = a.z; As[(k4 * 4 + 3) * 64 + r] = a.w;
    Bs[(k4 * 4 + 0) * 64 + r] = b.x; Bs[(k4 * 4 + 1) * 64 + r] = b.y;
    Bs[(k4 * 4 + 2) * 64 + r] = b.z; Bs[(k4 * 4 + 3) * 64 + r] = b.w;
  }
  __syncthreads();
  const int ti = tid / 16, tj = tid % 16;
  float acc[4][4];
#pragma unroll
  for (int x = 0; x < 4; ++x)
#pragma unroll
    for (int y = 0; y < 4; ++y) acc[x][y] = 0.f;
#pragma unroll 4
  for (int k = 0; k < D; ++k) {
    const float4 a = *reinterpret_cast<const float4*>(&As[k * 64 + ti * 4]);
    const float4 b = *reinterpret_cast<const float4*>(&Bs[k * 64 + tj * 4]);
    const float av[4] = {a.x, a.y, a.z, a.w}, bv[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
    for (int x = 0; x < 4; ++x)
#pragma unroll
      for (int y = 0; y < 4; ++y) acc[x][y] = __fadd_rn(acc[x][y], __fmul_rn(av[x], bv[y]));
  }
#pragma unroll
  for (int x = 0; x < 4; ++x) {
    const int i = i0 + ti * 4 + x;
    if (i >= row_end) continue;
    float* out = scores + ((size_t)p * chunk_rows + (i - row0)) * n_kc + j0 + tj * 4;
    if (j0 + tj * 4 + 3 < n_kc && (n_kc & 3) == 0) {
      *reinterpret_cast<float4*>(out) = make_float4(acc[x][0], acc[x][1], acc[x][2], acc[x][3]);
    } else {
#pragma unroll
      for (int y = 0; y < 4; ++y)
        if (j0 + tj * 4 + y < n_kc) out[y] = acc[x][y];
    }
  }
}

// rows of scores that fit the workspace (a multiple of 64), or 0: use the fused kernels
int select_chunk_rows(int P, int n_qc, int n_kc, size_t score_floats) {
  if (n_kc < kSelectTiledMinClusters || score_floats == 0) return 0;
  size_t rows = score_floats / ((size_t)P * n_kc);
  if (rows >= (size_t)n_qc) return n_qc;
  rows = rows / 64 * 64;
  return (int)rows;
}

size_t select_score_floats(int P, int n_qc, int n_kc) {
  if (n_kc < kSelectTiledMinClusters) return 0;
  const size_t all = (size_t)P * n_qc * n_kc;
  const size_t budget = (size_t)64 << 20;            // 256 MB of scores at a time
  const size_t least = (size_t)P * 64 * n_kc;        // at least one 64-row chunk
  size_t take = all < budget ? all : budget;
  if (take < least) take = least;
  return (take + 63) / 64 * 64;
}

template <int D>
static int launch_score_tiles(const float* cq, const float* ck, int P, int n_qc, int n_kc, int row0, int chunk_rows,
                              float* scores, cudaStream_t st) {
  auto k = score_tile_kernel<D>;
  const size_t smem = (size_t)2 * D * 64 * sizeof(float);
  CA_RETURN_IF_CUDA(cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  const int rows = min(chunk_rows, n_qc - row0);
  k<<<dim3(ceil_div(n_kc, 64), ceil_div(rows, 64), P), 256, smem, st>>>(cq, ck, n_qc, n_kc, row0, chunk_rows, scores);
  CA_LAUNCH_CHECK();
  return CA_OK;
}

int launch_score_select(const float* cq, const float* ck, int P, int n_qc, int n_kc, int D, int keep,
                        int32_t* block_idx, float* score_ws, size_t score_floats, cudaStream_t st) {
  const int chunk = select_chunk_rows(P, n_qc, n_kc, score_ws ? score_floats : 0);
  if (chunk == 0) {
    const size_t smem = select_smem_bytes(n_kc, D, kSelectQT);
    if (smem > 200 * 1024) return CA_ERR_UNSUPPORTED;
    dim3 grid(ceil_div(n_qc, kSelectQT), P);
    if (D == 64) {
      auto k = score_select_kernel<64, kSelectQT>;
      CA_RETURN_IF_CUDA(cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
      k<<<grid, kSelectThreads, smem, st>>>(cq, ck, n_qc, n_kc, keep, block_idx, nullptr, 0, n_qc);
    } else {
      auto k = score_select_kernel<128, kSelectQT>;
      CA_RETURN_IF_CUDA(cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
      k<<<grid, kSelectThreads, smem, st>>>(cq, ck, n_qc, n_kc, keep, block_idx, nullptr, 0, n_qc);
    }
    CA_LAUNCH_CHECK();
    return CA_OK;
  }
  const size_t smem = select_smem_bytes(n_kc, D, 1);
  if (smem > 200 * 1024) return CA_ERR_UNSUPPORTED;
  auto k64 = score_select_kernel<64, 1>;
  auto k128 = score_select_kernel<128, 1>;
  CA_RETURN_IF_CUDA(cudaFuncSetAttribute(k64, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  CA_RETURN_IF_CUDA(cudaFuncSetAttribute(k128, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  for (int row0 = 0; row0 < n_qc; row0 += chunk) {
    const int rows = min(chunk, n_qc - row0);
    if (D == 64) { int rc = launch_score_tiles<64>(cq, ck, P, n_qc, n_kc, row0, chunk, score_ws, st); if (rc != CA_OK) return rc; }
    else { int rc = launch_score_tiles<128>(cq, ck, P, n_qc, n_kc, row0, chunk, score_ws, st); if (rc != CA_OK) return rc; }
    dim3 grid(rows, P);
    if (D == 64) k64<<<grid, kSelectThreads, smem, st>>>(cq, ck, n_qc, n_kc, keep, block_idx, score_ws, row0, chunk);
    else k128<<<grid, kSelectThreads, smem, st>>>(cq, ck, n_qc, n_kc, keep, block_idx, score_ws, row0, chunk);
    CA_LAUNCH_CHECK();
  }
  return CA_OK;
}

}  // namespace ca

namespace ca {

// ---------------------------------------------------------------------------
// Adaptive selection (Section 3.3.2): the most massive key clusters, by the
// centroid estimate |c_j| exp(qbar_i . kbar_j / sqrt(d)), until their share of
// the estimated mass reaches the recall threshold; never fewer than min_count.
// Every floating-point step is float32 with separately rounded operations in a
// stated order, so the decision is reproducible bit for bit:
//   score as in score_select_kernel; x = (s - max_j s) * c, c = scale * log2(e);
//   2^x: clamp to [-100, 100], n = (x + 1.5*2^23) - 1.5*2^23, f = x - n,
//        ((c3 f + c2) f + c1) f + c0 by Horner's rule, scaled by 2^n;
//   mass = 2^x * |c_j|; clusters ordered by (mass descending, index ascending);
//   running sum in that order; shortest prefix with sum >= recall * total.
// One CTA (256 threads) per query cluster.
// ---------------------------------------------------------------------------
__device__ __forceinline__ float exp2_recipe(float x) {
  x = fminf(fmaxf(x, -100.0f), 100.0f);
  const float n = __fsub_rn(__fadd_rn(x, 12582912.0f), 12582912.0f);
  const float f = __fsub_rn(x, n);
  float p = __fadd_rn(__fmul_rn(0.05517165f, f), 0.24261113f);
  p = __fadd_rn(__fmul_rn(p, f), 0.69326097f);
  p = __fadd_rn(__fmul_rn(p, f), 0.99992806f);
  return ldexpf(p, (int)n);
}

template <int D>
__global__ void __launch_bounds__(256)
select_adaptive_kernel(const float* __restrict__ cq, const float* __restrict__ ck,
                       const int32_t* __restrict__ count_k, int n_qc, int n_kc, int n_pad, float c_log2,
                       float recall, int min_count, int32_t* __restrict__ block_idx,
                       int32_t* __restrict__ keep_count, const float* __restrict__ scores, int row0,
                       int chunk_rows) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  unsigned long long* keys = reinterpret_cast<unsigned long long*>(smem_raw);   // [n_pad] (mass, ~index)
  float* score = reinterpret_cast<float*>(keys + n_pad);                         // [n_kc]
  float* qs = score + n_kc;                                                      // [D]
  __shared__ float s_red[8];
  __shared__ int s_warp[64];
  __shared__ int s_need;
  const int p = blockIdx.y, i = row0 + blockIdx.x;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const float* ckp = ck + (size_t)p * n_kc * D;
  const int32_t* cnt = count_k + (size_t)p * n_kc;
  for (int e = tid; e < D; e += 256) qs[e] = cq[((size_t)p * n_qc + i) * D + e];
  __syncthreads();
  float mx = -INFINITY;
  if (scores) {
    const float* srow = scores + ((size_t)p * chunk_rows + (i - row0)) * n_kc;
    for (int j = tid; j < n_kc; j += 256) {
      const float v = __ldg(srow + j);
      score[j] = v;
      mx = fmaxf(mx, v);
    }
  } else
  for (int j = tid; j < n_kc; j += 256) {
    float acc = 0.f;
    const float4* row = reinterpret_cast<const float4*>(ckp + (size_t)j * D);
    for (int k4 = 0; k4 < D / 4; ++k4) {
      const float4 kv = __ldg(row + k4);
      const float* q = qs + k4 * 4;
      acc = __fadd_rn(acc, __fmul_rn(q[0], kv.x));
      acc = __fadd_rn(acc, __fmul_rn(q[1], kv.y));
      acc = __fadd_rn(acc, __fmul_rn(q[2], kv.z));
      acc = __fadd_rn(acc, __fmul_rn(q[3], kv.w));
    }
    score[j] = acc;
    mx = fmaxf(mx, acc);
  }
  for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
  if (lane == 0) s_red[warp] = mx;
  __syncthreads();
  mx = s_red[0];
  for (int w = 1; w < 8; ++w) mx = fmaxf(mx, s_red[w]);
  // sort keys: mass bits (non-negative floats order like unsigned integers) above the complemented index
  for (int j = tid; j < n_pad; j += 256) {
    unsigned long long key = 0ull;                         // padding sorts last
    if (j < n_kc) {
      const float mass = __fmul_rn(exp2_recipe(__fmul_rn(__fsub_rn(score[j], mx), c_log2)), (float)cnt[j]);
      key = ((unsigned long long)__float_as_uint(mass) << 32) | (unsigned)(0x7fffffff - j);
      key |= 1ull << 63;                                   // real entries above the padding even when mass = 0
    }
    keys[j] = key;
  }
  __syncthreads();
  // bitonic sort, descending
  for (int k = 2; k <= n_pad; k <<= 1) {
    for (int jj = k >> 1; jj > 0; jj >>= 1) {
      for (int t = tid; t < n_pad; t += 256) {
        const int partner = t ^ jj;
        if (partner > t) {
          const unsigned long long a = keys[t], b = keys[partner];
          const bool desc = (t & k) == 0;
          if (desc ? (a < b) : (a > b)) { keys[t] = b; keys[partner] = a; }
        }
      }
      __syncthreads();
    }
  }
  // running sum in sorted order (one thread: the order of the additions is part of the definition)
  if (tid == 0) {
    float total = 0.f;
    for (int r = 0; r < n_kc; ++r) total = __fadd_rn(total, __uint_as_float((unsigned)((keys[r] >> 32) & 0x7fffffffu)));
    const float target = __fmul_rn(recall, total);
    int need = n_kc;
    float run = 0.f;
    for (int r = 0; r < n_kc; ++r) {
      run = __fadd_rn(run, __uint_as_float((unsigned)((keys[r] >> 32) & 0x7fffffffu)));
      if (run >= target) { need = r + 1; break; }
    }
    if (recall >= 1.0f) need = n_kc;
    need = max(need, min_count);
    need = min(need, n_kc);
    s_need = need;
  }
  __syncthreads();
  const int need = s_need;
  // mark the selected clusters (reuse `score` as flags), then write them in ascending index order
  for (int j = tid; j < n_kc; j += 256) score[j] = 0.f;
  __syncthreads();
  for (int r = tid; r < need; r += 256) score[0x7fffffff - (int)(keys[r] & 0x7fffffffu)] = 1.f;
  __syncthreads();
  int32_t* out = block_idx + ((size_t)p * n_qc + i) * n_kc;
  int before = 0;
  for (int j0 = 0; j0 < n_kc; j0 += 256) {
    const int j = j0 + tid;
    const int flag = (j < n_kc && score[j] != 0.f) ? 1 : 0;
    int incl = flag;
    for (int o = 1; o < 32; o <<= 1) {
      const int v = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += v;
    }
    if (lane == 31) s_warp[warp] = incl;
    __syncthreads();
    int wbase = 0, total = 0;
    for (int w = 0; w < 8; ++w) { const int v = s_warp[w]; if (w < warp) wbase += v; total += v; }
    if (flag) out[before + wbase + incl - 1] = j;
    before += total;
    __syncthreads();
  }
  for (int r = need + tid; r < n_kc; r += 256) out[r] = -1;
  if (tid == 0) keep_count[(size_t)p * n_qc + i] = need;
}

int launch_select_adaptive(const float* cq, const float* ck, const int32_t* count_k, int P, int n_qc, int n_kc,
                           int D, float scale, float recall, int min_count, int32_t* block_idx,
                           int32_t* keep_count, float* score_ws, size_t score_floats, cudaStream_t st) {
  int n_pad = 1;
  while (n_pad < n_kc) n_pad <<= 1;
  const size_t smem = (size_t)n_pad * 8 + (size_t)n_kc * 4 + (size_t)D * 4;
  if (smem > 200 * 1024) return CA_ERR_UNSUPPORTED;
  const float c_log2 = scale * 1.4426950408889634f;      // one float32 product, as in the definition
  auto k64 = select_adaptive_kernel<64>;
  auto k128 = select_adaptive_kernel<128>;
  CA_RETURN_IF_CUDA(cudaFuncSetAttribute(k64, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  CA_RETURN_IF_CUDA(cudaFuncSetAttribute(k128, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  const int chunk = select_chunk_rows(P, n_qc, n_kc, score_ws ? score_floats : 0);
  const int step = chunk == 0 ? n_qc : chunk;
  for (int row0 = 0; row0 < n_qc; row0 += step) {
    const int rows = min(step, n_qc - row0);
    const float* scores = nullptr;
    if (chunk != 0) {
      int rc = D == 64 ? launch_score_tiles<64>(cq, ck, P, n_qc, n_kc, row0, chunk, score_ws, st)
                       : launch_score_tiles<128>(cq, ck, P, n_qc, n_kc, row0, chunk, score_ws, st);
      if (rc != CA_OK) return rc;
      scores = score_ws;
    }
    dim3 grid(rows, P);
    if (D == 64)
      k64<<<grid, 256, smem, st>>>(cq, ck, count_k, n_qc, n_kc, n_pad, c_log2, recall, min_count, block_idx,
                                   keep_count, scores, row0, step);
    else
      k128<<<grid, 256, smem, st>>>(cq, ck, count_k, n_qc, n_kc, n_pad, c_log2, recall, min_count, block_idx,
                                    keep_count, scores, row0, step);
    CA_LAUNCH_CHECK();
  }
  return CA_OK;
}

}  // namespace ca
