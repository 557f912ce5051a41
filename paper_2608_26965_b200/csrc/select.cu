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
