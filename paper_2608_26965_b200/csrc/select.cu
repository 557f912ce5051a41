// Assignment (Section 3.3): centroid-centroid scores and exact top-k selection.
// score(i, j) = cq_i . ck_j in float32 with a fixed operation order (terms added
// for k = 0, 1, ..., product and sum rounded separately, no fused multiply-add),
// so the scores -- and with them the selection -- are reproducible bit for bit;
// the k best per query cluster by (score descending, index ascending), written
// in ascending index order.
#include "kernels.h"

namespace ca {

constexpr int kSelectThreads = 256;
constexpr int kSelectQT = 4;          // query clusters per CTA (key centroids are read once for all)

__device__ __forceinline__ uint32_t score_key(float s) {
  if (s == 0.0f) s = 0.0f;                        // -0 and +0 compare equal
  const uint32_t u = __float_as_uint(s);
  return (u >> 31) ? ~u : (u | 0x80000000u);
}

template <int D>
__global__ void __launch_bounds__(kSelectThreads)
score_select_kernel(const float* __restrict__ cq, const float* __restrict__ ck, int n_qc, int n_kc,
                    int keep, int32_t* __restrict__ block_idx) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  uint32_t* keys = reinterpret_cast<uint32_t*>(smem_raw);                       // [QT][n_kc]
  float* qs = reinterpret_cast<float*>(keys + (size_t)kSelectQT * n_kc);        // [QT][D]
  __shared__ int s_hist[256];
  __shared__ int s_warp[64];
  __shared__ int s_scalar[4];
  const int p = blockIdx.y;
  const int q0 = blockIdx.x * kSelectQT;
  const int nq = min(kSelectQT, n_qc - q0);
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const float* cqp = cq + ((size_t)p * n_qc + q0) * D;
  const float* ckp = ck + (size_t)p * n_kc * D;
  for (int e = tid; e < kSelectQT * D; e += kSelectThreads) qs[e] = (e < nq * D) ? cqp[e] : 0.f;
  __syncthreads();

  for (int j = tid; j < n_kc; j += kSelectThreads) {
    float acc[kSelectQT];
#pragma unroll
    for (int t = 0; t < kSelectQT; ++t) acc[t] = 0.f;
    const float4* row = reinterpret_cast<const float4*>(ckp + (size_t)j * D);
    for (int k4 = 0; k4 < D / 4; ++k4) {
      const float4 kv = __ldg(row + k4);
#pragma unroll
      for (int t = 0; t < kSelectQT; ++t) {
        const float* q = qs + t * D + k4 * 4;
        acc[t] = __fadd_rn(acc[t], __fmul_rn(q[0], kv.x));
        acc[t] = __fadd_rn(acc[t], __fmul_rn(q[1], kv.y));
        acc[t] = __fadd_rn(acc[t], __fmul_rn(q[2], kv.z));
        acc[t] = __fadd_rn(acc[t], __fmul_rn(q[3], kv.w));
      }
    }
#pragma unroll
    for (int t = 0; t < kSelectQT; ++t) keys[(size_t)t * n_kc + j] = score_key(acc[t]);
  }
  __syncthreads();

  for (int t = 0; t < nq; ++t) {
    const uint32_t* kt = keys + (size_t)t * n_kc;
    // radix selection of the keep-th largest key
    uint32_t prefix = 0, mask = 0;
    int remaining = keep;
    for (int shift = 24; shift >= 0; shift -= 8) {
      s_hist[tid] = 0;                             // kSelectThreads == 256 bins
      __syncthreads();
      for (int j0 = 0; j0 < n_kc; j0 += kSelectThreads) {
        const int j = j0 + tid;
        const bool ok = j < n_kc;
        const uint32_t k = ok ? kt[j] : 0u;
        const bool cand = ok && ((k & mask) == prefix);
        const int bin = cand ? (int)((k >> shift) & 255u) : -1;
        const unsigned peers = __match_any_sync(0xffffffffu, bin);
        if (cand && lane == (__ffs(peers) - 1)) atomicAdd(&s_hist[bin], __popc(peers));
      }
      __syncthreads();
      if (warp == 0) {
        // bins from the top: lane 0 owns bins 255..248
        int local[8]; int sum = 0;
#pragma unroll
        for (int b = 0; b < 8; ++b) { local[b] = s_hist[255 - (lane * 8 + b)]; sum += local[b]; }
        int incl = sum;
        for (int o = 1; o < 32; o <<= 1) {
          const int v = __shfl_up_sync(0xffffffffu, incl, o);
          if (lane >= o) incl += v;
        }
        int before = incl - sum;
#pragma unroll
        for (int b = 0; b < 8; ++b) {
          if (before < remaining && remaining <= before + local[b]) {
            s_scalar[0] = 255 - (lane * 8 + b);
            s_scalar[1] = remaining - before;
          }
          before += local[b];
        }
      }
      __syncthreads();
      prefix |= (uint32_t)s_scalar[0] << shift;
      mask |= 255u << shift;
      remaining = s_scalar[1];
      __syncthreads();
    }
    const uint32_t thr = prefix;
    const int eq_take = remaining;         // threshold-valued clusters taken, lowest indices first

    int32_t* out = block_idx + ((size_t)p * n_qc + q0 + t) * keep;
    int gt_before = 0, eq_before = 0;
    for (int j0 = 0; j0 < n_kc; j0 += kSelectThreads) {
      const int j = j0 + tid;
      const bool ok = j < n_kc;
      const uint32_t k = ok ? kt[j] : 0u;
      const int is_gt = (ok && k > thr) ? 1 : 0;
      const int is_eq = (ok && k == thr) ? 1 : 0;
      const int packed = is_gt | (is_eq << 16);
      int incl = packed;
      for (int o = 1; o < 32; o <<= 1) {
        const int v = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += v;
      }
      if (lane == 31) s_warp[warp] = incl;
      __syncthreads();
      if (warp == 0) {
        const int w = (lane < kSelectThreads / 32) ? s_warp[lane] : 0;
        int wi = w;
        for (int o = 1; o < 32; o <<= 1) {
          const int v = __shfl_up_sync(0xffffffffu, wi, o);
          if (lane >= o) wi += v;
        }
        s_warp[32 + lane] = wi - w;
        if (lane == 31) s_scalar[2] = wi;
      }
      __syncthreads();
      const int excl = incl - packed + s_warp[32 + warp];
      const int gt_here = gt_before + (excl & 0xffff);
      const int eq_here = eq_before + (excl >> 16);
      if (ok && (is_gt || (is_eq && eq_here < eq_take))) out[gt_here + min(eq_here, eq_take)] = j;
      const int total = s_scalar[2];
      gt_before += total & 0xffff;
      eq_before += total >> 16;
      __syncthreads();
    }
  }
}

size_t select_smem_bytes(int n_kc, int D) {
  return (size_t)kSelectQT * n_kc * sizeof(uint32_t) + (size_t)kSelectQT * D * sizeof(float);
}

int launch_score_select(const float* cq, const float* ck, int P, int n_qc, int n_kc, int D, int keep,
                        int32_t* block_idx, cudaStream_t st) {
  const size_t smem = select_smem_bytes(n_kc, D);
  if (smem > 200 * 1024) return CA_ERR_UNSUPPORTED;
  dim3 grid(ceil_div(n_qc, kSelectQT), P);
  if (D == 64) {
    auto k = score_select_kernel<64>;
    CA_RETURN_IF_CUDA(cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    k<<<grid, kSelectThreads, smem, st>>>(cq, ck, n_qc, n_kc, keep, block_idx);
  } else {
    auto k = score_select_kernel<128>;
    CA_RETURN_IF_CUDA(cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    k<<<grid, kSelectThreads, smem, st>>>(cq, ck, n_qc, n_kc, keep, block_idx);
  }
  CA_LAUNCH_CHECK();
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
                       int32_t* __restrict__ keep_count) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  unsigned long long* keys = reinterpret_cast<unsigned long long*>(smem_raw);   // [n_pad] (mass, ~index)
  float* score = reinterpret_cast<float*>(keys + n_pad);                         // [n_kc]
  float* qs = score + n_kc;                                                      // [D]
  __shared__ float s_red[8];
  __shared__ int s_warp[64];
  __shared__ int s_need;
  const int p = blockIdx.y, i = blockIdx.x;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const float* ckp = ck + (size_t)p * n_kc * D;
  const int32_t* cnt = count_k + (size_t)p * n_kc;
  for (int e = tid; e < D; e += 256) qs[e] = cq[((size_t)p * n_qc + i) * D + e];
  __syncthreads();
  float mx = -INFINITY;
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
                           int32_t* keep_count, cudaStream_t st) {
  int n_pad = 1;
  while (n_pad < n_kc) n_pad <<= 1;
  const size_t smem = (size_t)n_pad * 8 + (size_t)n_kc * 4 + (size_t)D * 4;
  if (smem > 200 * 1024) return CA_ERR_UNSUPPORTED;
  const float c_log2 = scale * 1.4426950408889634f;      // one float32 product, as in the definition
  dim3 grid(n_qc, P);
  if (D == 64) {
    auto k = select_adaptive_kernel<64>;
    CA_RETURN_IF_CUDA(cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    k<<<grid, 256, smem, st>>>(cq, ck, count_k, n_qc, n_kc, n_pad, c_log2, recall, min_count, block_idx, keep_count);
  } else {
    auto k = select_adaptive_kernel<128>;
    CA_RETURN_IF_CUDA(cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    k<<<grid, 256, smem, st>>>(cq, ck, count_k, n_qc, n_kc, n_pad, c_log2, recall, min_count, block_idx, keep_count);
  }
  CA_LAUNCH_CHECK();
  return CA_OK;
}

}  // namespace ca
