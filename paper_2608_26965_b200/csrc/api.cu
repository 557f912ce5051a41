// C entry points of libclusterattn: argument checks, workspace carving and the
// order in which the kernels of each stage are enqueued.
#include <math.h>

#include <atomic>
#include <mutex>

#include "kernels.h"

using namespace ca;

namespace ca {
std::atomic<unsigned long long> g_kernel_launches{0};

// ---- per-kernel-group timers (off unless ca_profile(1) was called) ------------------------------
namespace {
constexpr int kProfPairs = 512;
struct Profiler {
  bool on = false;
  int used = 0;
  cudaEvent_t begin[kProfPairs], end[kProfPairs];
  int group[kProfPairs];
  int open_pair[kProfGroups];
  int created = 0;
} g_prof;
const char* const kProfNames[kProfGroups] = {
    "gram", "cholesky_factor", "principal_components", "transform", "split_levels", "split_tail",
    "permute_centroid", "score_select", "centroid_prep", "attn_tc", "attn_second_pass"};
}  // namespace
bool prof_enabled() { return g_prof.on; }
void prof_mark(int group, cudaStream_t st, bool begin) {
  if (!g_prof.on) return;
  if (begin) {
    if (g_prof.used >= g_prof.created) return;            // out of pairs: the scope is not timed
    const int i = g_prof.used++;
    g_prof.group[i] = group;
    g_prof.open_pair[group] = i;
    cudaEventRecord(g_prof.begin[i], st);
  } else {
    const int i = g_prof.open_pair[group];
    if (i >= 0) cudaEventRecord(g_prof.end[i], st);
    g_prof.open_pair[group] = -1;
  }
}
}  // namespace ca

namespace {

bool pow2(int x) { return x > 0 && (x & (x - 1)) == 0; }
bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

int check_problem(const ca_problem_t* p) {
  if (!p) return CA_ERR_INVALID_ARG;
  if (p->batch < 1 || p->heads < 1 || p->n_q < 1 || p->n_k < 1) return CA_ERR_INVALID_ARG;
  if (p->head_dim != 64 && p->head_dim != 128) return CA_ERR_UNSUPPORTED;
  if (p->dtype != CA_DTYPE_FP32 && p->dtype != CA_DTYPE_BF16) return CA_ERR_UNSUPPORTED;
  if (!pow2(p->cluster_q) || !pow2(p->cluster_k)) return CA_ERR_INVALID_ARG;
  if (p->cluster_q < 16 || p->cluster_q > 256 || p->cluster_k < 16 || p->cluster_k > 256)
    return CA_ERR_UNSUPPORTED;
  const int n_kc = ceil_div(p->n_k, p->cluster_k);
  if (p->keep < 1 || p->keep > n_kc) return CA_ERR_INVALID_ARG;
  if ((long long)p->batch * p->heads > 65535) return CA_ERR_UNSUPPORTED;
  if (!(p->softmax_scale >= 0.f)) return CA_ERR_INVALID_ARG;
  return CA_OK;
}

struct ClusterWs {
  int* status;
  float *partial, *partial2;           // chunk sums of the Gram kernels, one buffer per stream
  double *gramQ, *sumQ, *gramK, *sumK, *roots, *gramQp, *sumQp;
  float *roots32, *basis32, *WK32, *biasK, *biasQ;
  float *Qprime, *Yq, *Yk, *Ytq, *Ytk;
  __nv_bfloat16 *wt_hi, *wt_lo, *wt2_hi, *wt2_lo;
  int32_t *perm_q_tmp, *perm_k_tmp;
  uint32_t *keybuf_q, *keybuf_k;
  size_t bytes;
};

// A level of the splitter reads one coordinate of every row of a set, rows scattered: from the
// row-major coordinates that costs a 128-byte DRAM line per row and level.  A coordinate-major copy
// makes it a 4-byte read inside an L2-resident column, at the price of writing the coordinates a
// second time (4 d bytes per row): worth it when levels x 128 > 1.5 x 4 d (long sequences, d = 64).
static bool use_yt(const ca_problem_t* p, int n, int c) {
  const bool tc = p->dtype == CA_DTYPE_BF16 && (p->head_dim == 64 || p->head_dim == 128);
  return tc && !(p->flags & CA_Y_IN) && split_top_levels_for(n, c) * 128 >= 6 * p->head_dim;
}

ClusterWs carve_cluster(const ca_problem_t* p, void* base, bool need_yq, bool need_yk) {
  ClusterWs w{};
  Carver c(base);
  const size_t P = (size_t)p->batch * p->heads, D = p->head_dim, DD = D * D;
  w.status = c.take<int>(kStatusBytes / sizeof(int));
  const bool transforms = !(p->flags & CA_Y_IN);
  if (transforms) {
    int cr, ncq, nck;
    moments_chunking(p->n_q, (int)P, &cr, &ncq);
    moments_chunking(p->n_k, (int)P, &cr, &nck);
    const size_t nchunks = (size_t)(ncq > nck ? ncq : nck);
    w.partial = c.take<float>(P * nchunks * (DD + D));
    w.partial2 = c.take<float>(P * nchunks * (DD + D));
    w.gramQ = c.take<double>(P * DD);  w.sumQ = c.take<double>(P * D);
    w.gramK = c.take<double>(P * DD);  w.sumK = c.take<double>(P * D);
    w.roots = c.take<double>(2 * P * DD);
    w.gramQp = c.take<double>(P * DD); w.sumQp = c.take<double>(P * D);
    w.roots32 = c.take<float>(2 * P * DD);
    w.basis32 = c.take<float>(2 * P * DD);
    w.WK32 = c.take<float>(P * DD);
    w.biasK = c.take<float>(P * D);
    w.biasQ = c.take<float>(P * D);
    w.Qprime = c.take<float>(P * (size_t)p->n_q * D);
    w.wt_hi = c.take<__nv_bfloat16>(P * DD);
    w.wt_lo = c.take<__nv_bfloat16>(P * DD);
    w.wt2_hi = c.take<__nv_bfloat16>(P * DD);
    w.wt2_lo = c.take<__nv_bfloat16>(P * DD);
    if (need_yq) w.Yq = c.take<float>(P * (size_t)p->n_q * D);
    if (need_yk) w.Yk = c.take<float>(P * (size_t)p->n_k * D);
    // coordinate-major copies of the split coordinates, where they pay (use_yt)
    if (use_yt(p, p->n_q, p->cluster_q)) w.Ytq = c.take<float>(P * (size_t)p->n_q * D);
    if (use_yt(p, p->n_k, p->cluster_k)) w.Ytk = c.take<float>(P * (size_t)p->n_k * D);
  }
  w.perm_q_tmp = c.take<int32_t>(P * (size_t)p->n_q);
  w.perm_k_tmp = c.take<int32_t>(P * (size_t)p->n_k);
  w.keybuf_q = c.take<uint32_t>(P * (size_t)p->n_q);
  w.keybuf_k = c.take<uint32_t>(P * (size_t)p->n_k);
  w.bytes = c.used();
  return w;
}

// The query side and the key side of cluster_qk are independent once the two factors exist.  The
// query side runs on a second stream that forks from the caller's stream and joins it again
// before the call returns (events only: nothing waits on the host, and a stream capture of the
// caller's stream picks the side stream up as a parallel branch).  A pool of four side streams, each
// with three events (fork, Gram matrix of K ready, join), per device, created at the first call on
// that device; calls take them in turn, so that up to four calls in flight on different caller
// streams (from one or several host threads) do not share a side stream.
struct SideStream {
  cudaStream_t stream = nullptr;
  cudaEvent_t fork = nullptr, mid = nullptr, join = nullptr;
};
constexpr int kSidePool = 4;
SideStream* side_stream() {
  static SideStream table[64][kSidePool];
  static bool ready[64] = {};
  static unsigned next[64] = {};
  static std::mutex guard;
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
  std::lock_guard<std::mutex> lock(guard);
  if (!ready[dev]) {
    for (SideStream& s : table[dev]) {
      if (cudaStreamCreateWithFlags(&s.stream, cudaStreamNonBlocking) != cudaSuccess) return nullptr;
      if (cudaEventCreateWithFlags(&s.fork, cudaEventDisableTiming) != cudaSuccess) return nullptr;
      if (cudaEventCreateWithFlags(&s.mid, cudaEventDisableTiming) != cudaSuccess) return nullptr;
      if (cudaEventCreateWithFlags(&s.join, cudaEventDisableTiming) != cudaSuccess) return nullptr;
    }
    ready[dev] = true;
  }
  return &table[dev][next[dev]++ % kSidePool];
}

#define CA_TRY(expr)               \
  do {                             \
    int _rc = (expr);              \
    if (_rc != CA_OK) return _rc;  \
  } while (0)

}  // namespace

extern "C" {

const char* ca_version(void) { return "libclusterattn 0.1 (sm_100a)"; }

unsigned long long ca_kernel_launches(void) { return g_kernel_launches.load(); }

int ca_profile(int enable) {
  if (enable) {
    while (g_prof.created < kProfPairs) {
      if (cudaEventCreate(&g_prof.begin[g_prof.created]) != cudaSuccess) return CA_ERR_CUDA;
      if (cudaEventCreate(&g_prof.end[g_prof.created]) != cudaSuccess) return CA_ERR_CUDA;
      ++g_prof.created;
    }
    g_prof.used = 0;
    for (int g = 0; g < kProfGroups; ++g) g_prof.open_pair[g] = -1;
  }
  g_prof.on = enable != 0;
  return CA_OK;
}

int ca_profile_read(int max_groups, const char** names, float* ms, int* scopes) {
  if (cudaDeviceSynchronize() != cudaSuccess) return -CA_ERR_CUDA;
  float total[kProfGroups] = {};
  int count[kProfGroups] = {};
  for (int i = 0; i < g_prof.used; ++i) {
    float t = 0.f;
    if (cudaEventElapsedTime(&t, g_prof.begin[i], g_prof.end[i]) != cudaSuccess) { (void)cudaGetLastError(); continue; }
    total[g_prof.group[i]] += t;
    ++count[g_prof.group[i]];
  }
  g_prof.used = 0;
  int n = 0;
  for (int g = 0; g < kProfGroups && n < max_groups; ++g) {
    if (names) names[n] = kProfNames[g];
    if (ms) ms[n] = total[g];
    if (scopes) scopes[n] = count[g];
    ++n;
  }
  return n;
}

int ca_workspace_bytes(const ca_problem_t* p, size_t* cluster_ws, size_t* select_ws, size_t* attn_ws) {
  CA_TRY(check_problem(p));
  if (cluster_ws) *cluster_ws = carve_cluster(p, nullptr, true, true).bytes;
  if (select_ws)
    *select_ws = kStatusBytes + sizeof(float) * select_score_floats(p->batch * p->heads, ceil_div(p->n_q, p->cluster_q),
                                                                    ceil_div(p->n_k, p->cluster_k));
  if (attn_ws) *attn_ws = attn_tc_supported(*p) ? attn_tc_workspace_bytes(*p) : kStatusBytes;
  return CA_OK;
}

int cluster_qk(const ca_problem_t* p, const void* Q, const void* K, const void* V, int32_t* perm_q,
               int32_t* perm_k, void* Qp, void* Kp, void* Vp, float* cq, float* ck, float* cv,
               int32_t* count_q, int32_t* count_k, float* Yq, float* Yk, void* ws, size_t ws_bytes,
               void* stream) {
  CA_TRY(check_problem(p));
  const void* ptrs[] = {Q, K, V, perm_q, perm_k, Qp, Kp, Vp, cq, ck, cv, count_q, count_k};
  for (const void* x : ptrs)
    if (!x || !aligned16(x)) return CA_ERR_INVALID_ARG;
  const bool y_in = (p->flags & CA_Y_IN) != 0;
  if (y_in && (!Yq || !Yk)) return CA_ERR_INVALID_ARG;
  if ((Yq && !aligned16(Yq)) || (Yk && !aligned16(Yk))) return CA_ERR_INVALID_ARG;
  if (!ws || !aligned16(ws)) return CA_ERR_WORKSPACE;
  ClusterWs w = carve_cluster(p, ws, Yq == nullptr, Yk == nullptr);
  if (ws_bytes < w.bytes) return CA_ERR_WORKSPACE;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const int P = p->batch * p->heads, D = p->head_dim, DD = D * D;
  CA_RETURN_IF_CUDA(cudaMemsetAsync(w.status, 0, kStatusBytes, st));

  const float* yq = Yq;
  const float* yk = Yk;
  if (!y_in) {
    float* yq_out = Yq ? Yq : w.Yq;
    float* yk_out = Yk ? Yk : w.Yk;
    // bf16 storage runs the O(n d^2) passes on the tensor cores; fp32 storage on the CUDA cores
    const bool tc = p->dtype == CA_DTYPE_BF16;
    __nv_bfloat16* qp_hi = reinterpret_cast<__nv_bfloat16*>(w.Qprime);          // r(q) as bf16 hi + lo parts
    __nv_bfloat16* qp_lo = qp_hi + (size_t)P * p->n_q * D;
    // Factors F_q F_q^T = M = Q^T Q / n_q and F_k F_k^T = C_K (Section 3.2.2; they stand in for the
    // symmetric roots: any factor yields the same principal-component coordinates).  The
    // un-normalised query representation (Appendix B.1) takes the root of K_c^T K_c / n_k, the
    // normalised one is indifferent to the scale and keeps the scatter matrix as it is.
    // F_q comes from Q on the caller's stream and leads into the key side; F_k comes from K on the
    // side stream and leads into the query side: the fork is at the very start, and the key side
    // only waits for the Gram matrix and column sums of K (event `mid`), from which its
    // principal-component kernel forms C_K itself.
    const bool unnormalized = (p->flags & CA_QUERY_UNNORMALIZED) != 0;
    const double ck_scale = unnormalized ? 1.0 / (double)p->n_k : 1.0;
    double* Fq = w.roots;
    double* Fk = w.roots + (size_t)P * DD;
    const float* Fk32 = w.roots32 + (size_t)P * DD;
    SideStream* side = side_stream();
    if (!side) return CA_ERR_CUDA;
    // while the per-kernel timers are on, both sides run on the caller's stream, one kernel after
    // the other, so that every kernel group is timed alone
    const bool serial = prof_enabled();
    cudaStream_t sq = serial ? st : side->stream;
    if (!serial) {
      CA_RETURN_IF_CUDA(cudaEventRecord(side->fork, st));
      CA_RETURN_IF_CUDA(cudaStreamWaitEvent(sq, side->fork, 0));
    }
    {
      ProfScope ps(kProfGram, st);
      if (tc) {
        CA_TRY(launch_gram_tc(Q, nullptr, P, p->n_q, D, w.partial, w.gramQ, w.sumQ, w.status, st));
        CA_TRY(launch_gram_tc(K, nullptr, P, p->n_k, D, w.partial2, w.gramK, w.sumK, w.status, sq));
      } else {
        CA_TRY(launch_moments(Q, p->dtype, P, p->n_q, D, w.partial, w.gramQ, w.sumQ, st));
        CA_TRY(launch_moments(K, p->dtype, P, p->n_k, D, w.partial2, w.gramK, w.sumK, sq));
      }
    }
    if (!serial) CA_RETURN_IF_CUDA(cudaEventRecord(side->mid, sq));
    {
      ProfScope ps(kProfFactor, st);
      CA_TRY(launch_cholesky_factor(w.gramQ, nullptr, 1.0, 1.0 / (double)p->n_q, P, D, Fq, w.roots32, nullptr, nullptr, st));
      CA_TRY(launch_cholesky_factor(w.gramK, w.sumK, (double)p->n_k, ck_scale, P, D, Fk, w.roots32 + (size_t)P * DD,
                                    tc ? w.wt2_hi : nullptr, tc ? w.wt2_lo : nullptr, sq));
    }
    // ---- query side (side stream)
    // query representation r(q) = F_k^T q / |F_k^T q|, its covariance and principal components E_Q
    // (one kernel), the coordinates Y = (r(q) - mean) E_Q
    float* EQ32 = w.basis32 + (size_t)P * DD;
    {
      ProfScope ps(kProfTransform, sq);
      if (tc) {
        CA_TRY(launch_transform_tc(Q, nullptr, P, p->n_q, D, Fk32, nullptr, unnormalized ? 0 : 1, nullptr, qp_hi, qp_lo,
                                   w.wt2_hi, w.wt2_lo, w.status, sq, nullptr, true));
      } else {
        CA_TRY(launch_transform_rows(Q, p->dtype, P, p->n_q, D, Fk32, nullptr, unnormalized ? 0 : 1, w.Qprime, sq));
      }
    }
    {
      ProfScope ps(kProfGram, sq);
      if (tc) {
        CA_TRY(launch_gram_tc(qp_hi, qp_lo, P, p->n_q, D, w.partial2, w.gramQp, w.sumQp, w.status, sq));
      } else {
        CA_TRY(launch_moments(w.Qprime, CA_DTYPE_FP32, P, p->n_q, D, w.partial2, w.gramQp, w.sumQp, sq));
      }
    }
    {
      ProfScope ps(kProfPca, sq);
      PcaArgs a{};
      a.mode = kPcaQueries;
      a.gram = w.gramQp; a.sum = w.sumQp; a.n = (double)p->n_q;
      a.lift = Fk; a.out_lifted = 0;
      a.mean_sum = w.sumQp; a.mean_n = (double)p->n_q;
      a.W32 = EQ32; a.bias = w.biasQ;
      a.wt_hi = tc ? w.wt2_hi : nullptr; a.wt_lo = tc ? w.wt2_lo : nullptr;
      CA_TRY(launch_pca(a, P, D, sq));
    }
    {
      ProfScope ps(kProfTransform, sq);
      if (tc) {
        CA_TRY(launch_transform_tc(qp_hi, qp_lo, P, p->n_q, D, EQ32, w.biasQ, 0, yq_out, nullptr, nullptr, w.wt2_hi,
                                   w.wt2_lo, w.status, sq, w.Ytq, true));
      } else {
        CA_TRY(launch_transform_rows(w.Qprime, CA_DTYPE_FP32, P, p->n_q, D, EQ32, w.biasQ, 0, yq_out, sq));
      }
    }
    CA_TRY(launch_split(yq_out, nullptr, P, D, p->n_q, p->n_k, p->cluster_q, p->cluster_k, perm_q, w.perm_q_tmp,
                        perm_k, w.perm_k_tmp, w.keybuf_q, w.keybuf_k, 1, sq, w.Ytq, nullptr));
    {
      ProfScope ps(kProfPermute, sq);
      CA_TRY(launch_permute_centroid(Q, p->dtype, perm_q, P, p->n_q, D, p->cluster_q, Qp, cq, count_q, sq));
    }
    if (!serial) CA_RETURN_IF_CUDA(cudaEventRecord(side->join, sq));
    // ---- key side on the caller's stream: covariance of the transformed keys K F_q
    // (F_q^T C_K F_q / n_k, d x d algebra), its principal components E_K and the projection
    // W = F_q E_K with its bias in one kernel; Y = (K - kbar) W
    if (!serial) CA_RETURN_IF_CUDA(cudaStreamWaitEvent(st, side->mid, 0));
    {
      ProfScope ps(kProfPca, st);
      PcaArgs a{};
      a.mode = kPcaKeys;
      a.gram = w.gramK; a.sum = w.sumK; a.n = (double)p->n_k; a.c_scale = ck_scale;
      a.alpha = unnormalized ? 1.0 : 1.0 / (double)p->n_k;
      a.lift = Fq; a.out_lifted = 1;
      a.mean_sum = w.sumK; a.mean_n = (double)p->n_k;
      a.W32 = w.WK32; a.bias = w.biasK;
      a.wt_hi = tc ? w.wt_hi : nullptr; a.wt_lo = tc ? w.wt_lo : nullptr;
      CA_TRY(launch_pca(a, P, D, st));
    }
    {
      ProfScope ps(kProfTransform, st);
      if (tc) {
        CA_TRY(launch_transform_tc(K, nullptr, P, p->n_k, D, w.WK32, w.biasK, 0, yk_out, nullptr, nullptr, w.wt_hi,
                                   w.wt_lo, w.status, st, w.Ytk, true));
      } else {
        CA_TRY(launch_transform_rows(K, p->dtype, P, p->n_k, D, w.WK32, w.biasK, 0, yk_out, st));
      }
    }
    CA_TRY(launch_split(nullptr, yk_out, P, D, p->n_q, p->n_k, p->cluster_q, p->cluster_k, perm_q, w.perm_q_tmp,
                        perm_k, w.perm_k_tmp, w.keybuf_q, w.keybuf_k, 2, st, nullptr, w.Ytk));
    {
      ProfScope ps(kProfPermute, st);
      CA_TRY(launch_permute_centroid(K, p->dtype, perm_k, P, p->n_k, D, p->cluster_k, Kp, ck, count_k, st, V, Vp, cv));
    }
    // ---- join
    if (!serial) CA_RETURN_IF_CUDA(cudaStreamWaitEvent(st, side->join, 0));
    return CA_OK;
  }
  // coordinates given by the caller: split and gather only
  CA_TRY(launch_split(yq, yk, P, D, p->n_q, p->n_k, p->cluster_q, p->cluster_k, perm_q, w.perm_q_tmp,
                      perm_k, w.perm_k_tmp, w.keybuf_q, w.keybuf_k, 3, st));
  ProfScope ps(kProfPermute, st);
  CA_TRY(launch_permute_centroid(Q, p->dtype, perm_q, P, p->n_q, D, p->cluster_q, Qp, cq, count_q, st));
  CA_TRY(launch_permute_centroid(K, p->dtype, perm_k, P, p->n_k, D, p->cluster_k, Kp, ck, count_k, st, V, Vp, cv));
  return CA_OK;
}

int select_blocks(const ca_problem_t* p, const float* cq, const float* ck, int32_t* block_idx, void* ws,
                  size_t ws_bytes, void* stream) {
  CA_TRY(check_problem(p));
  if (!cq || !ck || !block_idx || !aligned16(cq) || !aligned16(ck) || !aligned16(block_idx))
    return CA_ERR_INVALID_ARG;
  if (!ws || ws_bytes < kStatusBytes) return CA_ERR_WORKSPACE;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  CA_RETURN_IF_CUDA(cudaMemsetAsync(ws, 0, kStatusBytes, st));
  const int P = p->batch * p->heads;
  // room behind the status block holds tiles of scores when there are many key clusters
  float* score_ws = reinterpret_cast<float*>(static_cast<char*>(ws) + kStatusBytes);
  const size_t score_floats = aligned16(ws) ? (ws_bytes - kStatusBytes) / sizeof(float) : 0;
  ProfScope ps(kProfSelect, st);
  return launch_score_select(cq, ck, P, ceil_div(p->n_q, p->cluster_q), ceil_div(p->n_k, p->cluster_k),
                             p->head_dim, p->keep, block_idx, score_ws, score_floats, st);
}

int cluster_attention_fwd(const ca_problem_t* p, const void* Qp, const void* Kp, const void* Vp,
                          const float* ck, const float* cv, const int32_t* count_k,
                          const int32_t* block_idx, const int32_t* perm_q, void* O, float* lse, void* ws,
                          size_t ws_bytes, void* stream) {
  CA_TRY(check_problem(p));
  const void* ptrs[] = {Qp, Kp, Vp, ck, cv, count_k, block_idx, perm_q, O};
  for (const void* x : ptrs)
    if (!x || !aligned16(x)) return CA_ERR_INVALID_ARG;
  if ((p->flags & CA_ATTN_FP8_QK) && !attn_tc_fp8_supported(*p)) return CA_ERR_UNSUPPORTED;
  const bool tensor_cores = attn_tc_supported(*p);
  const size_t need = tensor_cores ? attn_tc_workspace_bytes(*p) : kStatusBytes;
  if (!ws || !aligned16(ws) || ws_bytes < need) return CA_ERR_WORKSPACE;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  CA_RETURN_IF_CUDA(cudaMemsetAsync(ws, 0, kStatusClearBytes, st));
  const float scale = p->softmax_scale > 0.f ? p->softmax_scale : 1.0f / sqrtf((float)p->head_dim);
  if (tensor_cores)
    return launch_attn_tc(*p, Qp, Kp, Vp, ck, cv, count_k, block_idx, nullptr, p->keep, perm_q, scale, O, lse,
                          ws, st);
  return launch_attn_ref(*p, Qp, Kp, Vp, ck, cv, count_k, block_idx, nullptr, p->keep, perm_q, scale, O, lse,
                         static_cast<int*>(ws), st);
}

int select_blocks_adaptive(const ca_problem_t* p, const float* cq, const float* ck, const int32_t* count_k,
                           float recall, int32_t min_count, int32_t* block_idx, int32_t* keep_count,
                           void* ws, size_t ws_bytes, void* stream) {
  CA_TRY(check_problem(p));
  const void* ptrs[] = {cq, ck, count_k, block_idx, keep_count};
  for (const void* x : ptrs)
    if (!x || !aligned16(x)) return CA_ERR_INVALID_ARG;
  if (!(recall > 0.f) || min_count < 1) return CA_ERR_INVALID_ARG;
  if (!ws || ws_bytes < kStatusBytes) return CA_ERR_WORKSPACE;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  CA_RETURN_IF_CUDA(cudaMemsetAsync(ws, 0, kStatusBytes, st));
  const float scale = p->softmax_scale > 0.f ? p->softmax_scale : 1.0f / sqrtf((float)p->head_dim);
  float* score_ws = reinterpret_cast<float*>(static_cast<char*>(ws) + kStatusBytes);
  const size_t score_floats = aligned16(ws) ? (ws_bytes - kStatusBytes) / sizeof(float) : 0;
  ProfScope ps(kProfSelect, st);
  return launch_select_adaptive(cq, ck, count_k, p->batch * p->heads, ceil_div(p->n_q, p->cluster_q),
                                ceil_div(p->n_k, p->cluster_k), p->head_dim, scale, recall, min_count,
                                block_idx, keep_count, score_ws, score_floats, st);
}

int cluster_attention_fwd_ragged(const ca_problem_t* p, const void* Qp, const void* Kp, const void* Vp,
                                 const float* ck, const float* cv, const int32_t* count_k,
                                 const int32_t* block_idx, const int32_t* keep_count, int32_t list_stride,
                                 const int32_t* perm_q, void* O, float* lse, void* ws, size_t ws_bytes,
                                 void* stream) {
  CA_TRY(check_problem(p));
  const void* ptrs[] = {Qp, Kp, Vp, ck, cv, count_k, block_idx, keep_count, perm_q, O};
  for (const void* x : ptrs)
    if (!x || !aligned16(x)) return CA_ERR_INVALID_ARG;
  if (list_stride < 1) return CA_ERR_INVALID_ARG;
  if ((p->flags & CA_ATTN_FP8_QK) && !attn_tc_fp8_supported(*p)) return CA_ERR_UNSUPPORTED;
  const bool tensor_cores = attn_tc_supported(*p);
  const size_t need = tensor_cores ? attn_tc_workspace_bytes(*p) : kStatusBytes;
  if (!ws || !aligned16(ws) || ws_bytes < need) return CA_ERR_WORKSPACE;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  CA_RETURN_IF_CUDA(cudaMemsetAsync(ws, 0, kStatusClearBytes, st));
  const float scale = p->softmax_scale > 0.f ? p->softmax_scale : 1.0f / sqrtf((float)p->head_dim);
  if (tensor_cores)
    return launch_attn_tc(*p, Qp, Kp, Vp, ck, cv, count_k, block_idx, keep_count, list_stride, perm_q, scale,
                          O, lse, ws, st);
  return launch_attn_ref(*p, Qp, Kp, Vp, ck, cv, count_k, block_idx, keep_count, list_stride, perm_q, scale, O,
                         lse, static_cast<int*>(ws), st);
}

namespace {
struct BasicWs {
  int* status;
  float* partial;
  double *gramQ, *sumQ, *gramK, *sumK, *metric;
  float *dirs_q, *dirs_k;
  int32_t *perm_q_tmp, *perm_k_tmp;
  uint32_t *keybuf_q, *keybuf_k;
  int nodes_q, nodes_k;
  size_t bytes;
};
BasicWs carve_basic(const ca_problem_t* p, void* base) {
  BasicWs w{};
  Carver c(base);
  const size_t P = (size_t)p->batch * p->heads, D = p->head_dim, DD = D * D;
  w.status = c.take<int>(kStatusBytes / sizeof(int));
  int cr, ncq, nck;
  moments_chunking(p->n_q, (int)P, &cr, &ncq);
  moments_chunking(p->n_k, (int)P, &cr, &nck);
  w.partial = c.take<float>(P * (size_t)(ncq > nck ? ncq : nck) * (DD + D));
  w.gramQ = c.take<double>(P * DD);  w.sumQ = c.take<double>(P * D);
  w.gramK = c.take<double>(P * DD);  w.sumK = c.take<double>(P * D);
  w.metric = c.take<double>(2 * P * DD);
  const int lq = split_levels_for(p->n_q, p->cluster_q), lk = split_levels_for(p->n_k, p->cluster_k);
  w.nodes_q = (1 << (lq > 0 ? lq : 1)) - 1;
  w.nodes_k = (1 << (lk > 0 ? lk : 1)) - 1;
  w.dirs_q = c.take<float>(P * (size_t)w.nodes_q * D);
  w.dirs_k = c.take<float>(P * (size_t)w.nodes_k * D);
  w.perm_q_tmp = c.take<int32_t>(P * (size_t)p->n_q);
  w.perm_k_tmp = c.take<int32_t>(P * (size_t)p->n_k);
  w.keybuf_q = c.take<uint32_t>(P * (size_t)p->n_q);
  w.keybuf_k = c.take<uint32_t>(P * (size_t)p->n_k);
  w.bytes = c.used();
  return w;
}
}  // namespace

int ca_basic_workspace_bytes(const ca_problem_t* p, size_t* bytes, int32_t* noise_rows_q, int32_t* noise_rows_k) {
  CA_TRY(check_problem(p));
  const BasicWs w = carve_basic(p, nullptr);
  if (bytes) *bytes = w.bytes;
  if (noise_rows_q) *noise_rows_q = w.nodes_q;
  if (noise_rows_k) *noise_rows_k = w.nodes_k;
  return CA_OK;
}

int cluster_qk_basic(const ca_problem_t* p, const void* Q, const void* K, const void* V, const float* noise_q,
                     const float* noise_k, int32_t iterations, float* A_q, float* A_k, int32_t* perm_q,
                     int32_t* perm_k, void* Qp, void* Kp, void* Vp, float* cq, float* ck, float* cv,
                     int32_t* count_q, int32_t* count_k, void* ws, size_t ws_bytes, void* stream) {
  CA_TRY(check_problem(p));
  const void* ptrs[] = {Q, K, V, noise_q, noise_k, A_q, A_k, perm_q, perm_k, Qp, Kp, Vp, cq, ck, cv, count_q, count_k};
  for (const void* x : ptrs)
    if (!x || !aligned16(x)) return CA_ERR_INVALID_ARG;
  if (iterations < 0 || iterations > 64) return CA_ERR_INVALID_ARG;
  if (!ws || !aligned16(ws)) return CA_ERR_WORKSPACE;
  const BasicWs w = carve_basic(p, ws);
  if (ws_bytes < w.bytes) return CA_ERR_WORKSPACE;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const int P = p->batch * p->heads, D = p->head_dim;
  const size_t DD = (size_t)D * D;
  CA_RETURN_IF_CUDA(cudaMemsetAsync(w.status, 0, kStatusBytes, st));
  if (!(p->flags & CA_METRIC_IN)) {
    // keys are compared in the query metric Q^T Q / n_q, queries in K_c^T K_c / n_k (Section 3.2.2)
    if (p->dtype == CA_DTYPE_BF16) {
      CA_TRY(launch_gram_tc(Q, nullptr, P, p->n_q, D, w.partial, w.gramQ, w.sumQ, w.status, st));
      CA_TRY(launch_gram_tc(K, nullptr, P, p->n_k, D, w.partial, w.gramK, w.sumK, w.status, st));
    } else {
      CA_TRY(launch_moments(Q, p->dtype, P, p->n_q, D, w.partial, w.gramQ, w.sumQ, st));
      CA_TRY(launch_moments(K, p->dtype, P, p->n_k, D, w.partial, w.gramK, w.sumK, st));
    }
    double* M = w.metric;
    double* CK = w.metric + (size_t)P * DD;
    CA_TRY(launch_metric(w.gramQ, w.gramK, w.sumK, P, D, p->n_q, p->n_k, 1.0 / (double)p->n_k, M, CK, st));
    CA_TRY(launch_cast_f64_f32(M, A_k, (size_t)P * DD, st));
    CA_TRY(launch_cast_f64_f32(CK, A_q, (size_t)P * DD, st));
  }
  CA_TRY(launch_split_basic(Q, K, p->dtype, A_q, A_k, noise_q, noise_k, w.dirs_q, w.dirs_k, iterations, P, D, p->n_q,
                            p->n_k, p->cluster_q, p->cluster_k, perm_q, w.perm_q_tmp, perm_k, w.perm_k_tmp,
                            w.keybuf_q, w.keybuf_k, st));
  CA_TRY(launch_permute_centroid(Q, p->dtype, perm_q, P, p->n_q, D, p->cluster_q, Qp, cq, count_q, st));
  CA_TRY(launch_permute_centroid(K, p->dtype, perm_k, P, p->n_k, D, p->cluster_k, Kp, ck, count_k, st, V, Vp, cv));
  return CA_OK;
}

int ca_attn_recomputed(const void* ws) {
  if (!ws) return -CA_ERR_INVALID_ARG;
  int count = 0;
  if (cudaDeviceSynchronize() != cudaSuccess) return -CA_ERR_CUDA;
  if (cudaMemcpy(&count, static_cast<const int*>(ws) + kRecomputedWord, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess)
    return -CA_ERR_CUDA;
  return count;
}

void ca_debug_attn_wait(long long wait_limit_cycles, int skip_key_load) {
  attn_tc_set_debug(wait_limit_cycles, skip_key_load);
}

int ca_debug_eigh(const double* A, int count, int d, float* W, double* evals, void* stream) {
  if (!A || !W || !aligned16(A) || !aligned16(W) || count < 1) return CA_ERR_INVALID_ARG;
  if (d != 64 && d != 128) return CA_ERR_UNSUPPORTED;
  PcaArgs a{};
  a.mode = kPcaMatrix;
  a.A_in = A;
  a.W32 = W;
  a.evals = evals;
  return launch_pca(a, count, d, static_cast<cudaStream_t>(stream));
}

int ca_last_status(const void* ws) {
  if (!ws) return CA_ERR_INVALID_ARG;
  int status = 0;
  if (cudaDeviceSynchronize() != cudaSuccess) return CA_ERR_CUDA;
  if (cudaMemcpy(&status, ws, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess) return CA_ERR_CUDA;
  return status;
}

}  // extern "C"
