// FP32 CUDA-core kernel for block-sparse attention with striped
// mean-compensation (eq. 2 over the selected clusters; Appendix A: an excluded
// cluster enters through its centroid key and value with weight
// |c| exp(q . kbar / sqrt(d)), in numerator and denominator).
// Serves fp32 storage, unusual cluster sizes, and as an on-device cross-check of
// the tensor-core kernel.  Flash-style online softmax, fp32 throughout.
#include "kernels.h"

namespace ca {

constexpr int kRefQR = 16;       // query rows per CTA
constexpr int kRefKT = 32;       // keys per staged tile
constexpr int kRefThreads = 128;

template <typename T, int D>
__global__ void __launch_bounds__(kRefThreads)
attn_ref_kernel(const T* __restrict__ Qp, const T* __restrict__ Kp, const T* __restrict__ Vp,
                const float* __restrict__ ck, const float* __restrict__ cv,
                const int32_t* __restrict__ count_k, const int32_t* __restrict__ block_idx,
                const int32_t* __restrict__ keep_count, int list_stride,
                const int32_t* __restrict__ perm_q, int n_q, int n_k, int c_q, int c_k, int keep_all,
                int compensate, float scale, T* __restrict__ O, float* __restrict__ lse,
                int* __restrict__ status, const int32_t* __restrict__ redo, int redo_tiles,
                int* __restrict__ redo_count) {
  constexpr int LD = D + 1;
  constexpr int NC = D / 8;              // output columns per thread
  extern __shared__ float smem[];
  float* qs = smem;                      // [QR][LD]
  float* ks = qs + kRefQR * LD;          // [KT][LD]
  float* vs = ks + kRefKT * LD;          // [KT][LD]
  float* ps = vs + kRefKT * LD;          // [QR][KT+1]
  float* bias = ps + kRefQR * (kRefKT + 1);   // [KT] per-key additive term (ln|c| or -inf)
  unsigned* selected = reinterpret_cast<unsigned*>(bias + kRefKT);   // bitmap over key clusters

  const int n_qc = (n_q + c_q - 1) / c_q, n_kc = (n_k + c_k - 1) / c_k;
  const int tiles_per_cluster = (c_q + kRefQR - 1) / kRefQR;
  const int p = blockIdx.y;
  // first pass of a problem: one CTA per tile of 16 query rows.  Second pass behind the
  // tensor-core kernel (`redo` given): one CTA per query cluster, which returns at once unless the
  // cluster is marked ([B*H, n_qc, 2]) and otherwise walks over the tiles of the cluster.
  const int qc = redo ? blockIdx.x : blockIdx.x / tiles_per_cluster;
  const int r0_first = redo ? 0 : (blockIdx.x % tiles_per_cluster) * kRefQR;
  const int r0_end = redo ? c_q : r0_first + kRefQR;
  const int tid = threadIdx.x;
  const int row = tid / 8, sub = tid % 8;
  if (redo) {
    bool marked = false;
    for (int t = 0; t < redo_tiles; ++t) marked |= redo[((size_t)p * n_qc + qc) * 2 + t] != 0;
    if (!marked) return;
    if (threadIdx.x == 0 && redo_count) atomicAdd(redo_count, 1);   // statistics: clusters recomputed
  }
  const size_t q_base = ((size_t)p * n_qc + qc) * (size_t)c_q;
  const T* Kh = Kp + (size_t)p * n_kc * (size_t)c_k * D;
  const T* Vh = Vp + (size_t)p * n_kc * (size_t)c_k * D;
  const int32_t* sel = block_idx + ((size_t)p * n_qc + qc) * list_stride;
  int keep = keep_count ? keep_count[(size_t)p * n_qc + qc] : keep_all;   // ragged lists carry their length
  // indices from the caller are range-checked before use: a bad one sets CA_ERR_BAD_INDEX (6) in the
  // status word and is skipped (a list length is clamped to its row, a cluster that does not exist
  // is left out, a row of O that does not exist is not written)
  if (keep < 0 || keep > list_stride) {
    if (tid == 0) atomicCAS(status, 0, 6);
    keep = keep < 0 ? 0 : list_stride;
  }
  const int32_t* cnt = count_k + (size_t)p * n_kc;

  const int words = (n_kc + 31) / 32;
  for (int w = tid; w < words; w += kRefThreads) selected[w] = 0u;
  __syncthreads();
  for (int t = tid; t < keep; t += kRefThreads) {
    const int j = sel[t];
    if (j < 0 || j >= n_kc) atomicCAS(status, 0, 6);
    else atomicOr(&selected[j >> 5], 1u << (j & 31));
  }

  for (int r0 = r0_first; r0 < r0_end; r0 += kRefQR) {
    __syncthreads();                       // the previous tile's readers are done with the staged rows
    for (int e = tid; e < kRefQR * D; e += kRefThreads) {
      const int r = e / D, col = e % D;
      const int pos = qc * c_q + r0 + r;
      qs[r * LD + col] = (r0 + r < c_q && pos < n_q) ? to_f32<T>(Qp[(q_base + r0 + r) * D + col]) : 0.f;
    }
    __syncthreads();

    float m_run = -INFINITY, l_run = 0.f;
    float acc[NC];
#pragma unroll
    for (int i = 0; i < NC; ++i) acc[i] = 0.f;

    auto process_tile = [&]() {
      // logits of this thread's 4 keys
      float s[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) s[i] = 0.f;
      for (int k = 0; k < D; ++k) {
        const float q = qs[row * LD + k];
#pragma unroll
        for (int i = 0; i < 4; ++i) s[i] = fmaf(q, ks[(sub + 8 * i) * LD + k], s[i]);
      }
      float tmax = -INFINITY;
#pragma unroll
      for (int i = 0; i < 4; ++i) { s[i] = s[i] * scale + bias[sub + 8 * i]; tmax = fmaxf(tmax, s[i]); }
      tmax = fmaxf(tmax, __shfl_xor_sync(0xffffffffu, tmax, 1));
      tmax = fmaxf(tmax, __shfl_xor_sync(0xffffffffu, tmax, 2));
      tmax = fmaxf(tmax, __shfl_xor_sync(0xffffffffu, tmax, 4));
      const float m_new = fmaxf(m_run, tmax);
      float alpha = 1.f, psum = 0.f;
      if (m_new > -INFINITY) {
        alpha = expf(m_run - m_new);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const float pv = expf(s[i] - m_new);
          ps[row * (kRefKT + 1) + sub + 8 * i] = pv;
          psum += pv;
        }
      } else {
#pragma unroll
        for (int i = 0; i < 4; ++i) ps[row * (kRefKT + 1) + sub + 8 * i] = 0.f;
      }
      psum += __shfl_xor_sync(0xffffffffu, psum, 1);
      psum += __shfl_xor_sync(0xffffffffu, psum, 2);
      psum += __shfl_xor_sync(0xffffffffu, psum, 4);
      l_run = l_run * alpha + psum;
      m_run = m_new;
      __syncwarp();
#pragma unroll
      for (int i = 0; i < NC; ++i) acc[i] *= alpha;
      for (int key = 0; key < kRefKT; ++key) {
        const float pv = ps[row * (kRefKT + 1) + key];
#pragma unroll
        for (int i = 0; i < NC; ++i) acc[i] = fmaf(pv, vs[key * LD + sub + 8 * i], acc[i]);
      }
    };

    // selected clusters: every member key
    for (int t = 0; t < keep; ++t) {
      const int j = sel[t];
      if (j < 0 || j >= n_kc) continue;                  // flagged above
      const int members = min(max(cnt[j], 0), c_k);
      for (int t0 = 0; t0 < members; t0 += kRefKT) {
        __syncthreads();
        for (int e = tid; e < kRefKT * D; e += kRefThreads) {
          const int r = e / D, col = e % D;
          const bool ok = t0 + r < members;
          const size_t g = ((size_t)j * c_k + t0 + r) * D + col;
          ks[r * LD + col] = ok ? to_f32<T>(Kh[g]) : 0.f;
          vs[r * LD + col] = ok ? to_f32<T>(Vh[g]) : 0.f;
        }
        if (tid < kRefKT) bias[tid] = (t0 + tid < members) ? 0.f : -INFINITY;
        __syncthreads();
        process_tile();
      }
    }
    // excluded clusters through their centroids
    if (compensate) {
      const float* ckh = ck + (size_t)p * n_kc * D;
      const float* cvh = cv + (size_t)p * n_kc * D;
      for (int j0 = 0; j0 < n_kc; j0 += kRefKT) {
        __syncthreads();
        for (int e = tid; e < kRefKT * D; e += kRefThreads) {
          const int r = e / D, col = e % D;
          const bool ok = j0 + r < n_kc;
          ks[r * LD + col] = ok ? ckh[(size_t)(j0 + r) * D + col] : 0.f;
          vs[r * LD + col] = ok ? cvh[(size_t)(j0 + r) * D + col] : 0.f;
        }
        if (tid < kRefKT) {
          const int j = j0 + tid;
          const bool use = j < n_kc && !((selected[j >> 5] >> (j & 31)) & 1u);
          bias[tid] = use ? logf((float)cnt[j]) : -INFINITY;
        }
        __syncthreads();
        process_tile();
      }
    }

    const int pos = qc * c_q + r0 + row;
    if (r0 + row < c_q && pos < n_q) {
      const int orig = perm_q[(size_t)p * n_q + pos];
      if (orig < 0 || orig >= n_q) {
        atomicCAS(status, 0, 6);
      } else {
        // a row without a single live entry (an empty list without compensation): zeros, lse = -inf
        const bool empty = !(l_run > 0.f);
        const float inv = empty ? 0.f : 1.f / l_run;
        T* out = O + ((size_t)p * n_q + orig) * D;
#pragma unroll
        for (int i = 0; i < NC; ++i) out[sub + 8 * i] = from_f32<T>(acc[i] * inv);
        if (lse && sub == 0) lse[(size_t)p * n_q + orig] = empty ? -INFINITY : m_run + logf(l_run);
      }
    }
  }   // tiles of the cluster
}

template <typename T>
static int launch_t(const ca_problem_t& pr, const T* Qp, const T* Kp, const T* Vp, const float* ck,
                    const float* cv, const int32_t* count_k, const int32_t* block_idx,
                    const int32_t* keep_count, int list_stride, const int32_t* perm_q, float scale, T* O,
                    float* lse, int* status, cudaStream_t st, const int32_t* redo, int redo_tiles,
                    int* redo_count) {
  const int P = pr.batch * pr.heads, D = pr.head_dim;
  const int n_qc = ceil_div(pr.n_q, pr.cluster_q), n_kc = ceil_div(pr.n_k, pr.cluster_k);
  const int tiles = ceil_div(pr.cluster_q, kRefQR);
  const size_t smem = sizeof(float) * ((size_t)(kRefQR + 2 * kRefKT) * (D + 1) + kRefQR * (kRefKT + 1) + kRefKT) +
                      sizeof(unsigned) * ((n_kc + 31) / 32);
  dim3 grid(redo ? n_qc : n_qc * tiles, P);
  if (D == 64) {
    auto k = attn_ref_kernel<T, 64>;
    CA_RETURN_IF_CUDA(cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    k<<<grid, kRefThreads, smem, st>>>(Qp, Kp, Vp, ck, cv, count_k, block_idx, keep_count, list_stride, perm_q,
                                        pr.n_q, pr.n_k,
                                        pr.cluster_q, pr.cluster_k, pr.keep, pr.compensate, scale, O, lse, status, redo, redo_tiles, redo_count);
  } else {
    auto k = attn_ref_kernel<T, 128>;
    CA_RETURN_IF_CUDA(cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    k<<<grid, kRefThreads, smem, st>>>(Qp, Kp, Vp, ck, cv, count_k, block_idx, keep_count, list_stride, perm_q,
                                        pr.n_q, pr.n_k,
                                        pr.cluster_q, pr.cluster_k, pr.keep, pr.compensate, scale, O, lse, status, redo, redo_tiles, redo_count);
  }
  CA_LAUNCH_CHECK();
  return CA_OK;
}

int launch_attn_ref(const ca_problem_t& pr, const void* Qp, const void* Kp, const void* Vp,
                    const float* ck, const float* cv, const int32_t* count_k, const int32_t* block_idx,
                    const int32_t* keep_count, int list_stride, const int32_t* perm_q, float scale, void* O,
                    float* lse, int* status, cudaStream_t st, const int32_t* redo, int redo_tiles,
                    int* redo_count) {
  if (pr.dtype == CA_DTYPE_BF16)
    return launch_t(pr, static_cast<const __nv_bfloat16*>(Qp), static_cast<const __nv_bfloat16*>(Kp),
                    static_cast<const __nv_bfloat16*>(Vp), ck, cv, count_k, block_idx, keep_count, list_stride,
                    perm_q, scale,
                    static_cast<__nv_bfloat16*>(O), lse, status, st, redo, redo_tiles, redo_count);
  return launch_t(pr, static_cast<const float*>(Qp), static_cast<const float*>(Kp),
                  static_cast<const float*>(Vp), ck, cv, count_k, block_idx, keep_count, list_stride, perm_q, scale,
                  static_cast<float*>(O), lse, status, st, redo, redo_tiles, redo_count);
}

}  // namespace ca
