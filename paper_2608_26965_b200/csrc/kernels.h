// Host-side launchers of the library's kernels (internal; the public boundary
// is include/cluster_attention.h).  Every launcher enqueues on `st` and returns
// a CA_* code.
#pragma once
#include "common.cuh"

namespace ca {

// moments.cu
int moments_chunking(int n_rows, int problems, int* chunk_rows, int* n_chunks);
int launch_moments(const void* X, int dtype, int problems, int n_rows, int D, float* partial,
                   double* gram, double* colsum, cudaStream_t st);
int launch_transform_rows(const void* X, int dtype, int problems, int n_rows, int D, const float* W,
                          const float* bias, int normalize, float* out, cudaStream_t st);

int launch_gram_finalize(const float* partial, int problems, int n_chunks, int D, double* gram,
                         double* colsum, cudaStream_t st);

// tc_linear.cu (bf16 storage: tensor-core versions of the two kernels above)
int launch_gram_tc(const void* X_hi, const void* X_lo, int problems, int n_rows, int D, float* partial,
                   double* gram, double* colsum, int* status, cudaStream_t st);
int launch_transform_tc(const void* X_hi, const void* X_lo, int problems, int n_rows, int D, const float* W,
                        const float* bias, int normalize, float* out, void* out_hi, void* out_lo,
                        void* wt_hi, void* wt_lo, int* status, cudaStream_t st, float* out_t = nullptr,
                        bool weights_ready = false);

// eigh_tql.cu: covariance + principal components + projection matrix of one side, one CTA per head
enum { kPcaMatrix = 0, kPcaKeys = 1, kPcaQueries = 2 };
struct PcaArgs {
  int mode;                 // what is decomposed:
                            //   kPcaMatrix   A_in as given
                            //   kPcaKeys     alpha F^T C F,  C = (gram - s s^T / n) c_scale,  F = lift
                            //   kPcaQueries  gram / n - (s / n)(s / n)^T
  const double* A_in;       // [P][D][D]
  const double* gram;       // [P][D][D]
  const double* sum;        // [P][D]
  double n, c_scale, alpha;
  const double* lift;       // [P][D][D] factor F of the metric the rows were transformed with (sign rule:
                            // column t of F E); null: the sign rule applies to E itself
  int out_lifted;           // 1: the projection written is F E (rows are projected from the original
                            // space); 0: E (rows are already transformed)
  const double* mean_sum;   // [P][D] column sums of the rows that will be projected, and their count:
  double mean_n;            //   bias = -(mean_sum / mean_n) . projection   (null: zero bias)
  float* W32;               // [P][D in][D out] projection matrix
  float* bias;              // [P][D] or null
  __nv_bfloat16* wt_hi;     // [P][D out][D in] transposed projection as bf16 hi + lo parts, or null
  __nv_bfloat16* wt_lo;
  double* evals;            // [P][D] eigenvalues in descending order, or null
};
int launch_pca(const PcaArgs& args, int count, int D, cudaStream_t st);

// eigh.cu
int launch_metric(const double* gramQ, const double* gramK, const double* sumK, int P, int D, int n_q,
                  int n_k, double ck_scale, double* M, double* CK, cudaStream_t st);
// factor of gram * scale (sum null) or of (gram - s s^T / n) * scale
int launch_cholesky_factor(const double* gram, const double* sum, double n, double scale, int count, int D,
                           double* out64, float* out32, void* wt_hi, void* wt_lo, cudaStream_t st);

// split.cu
int split_levels_for(int n, int c);
// levels that run as per-level launches over whole sets (the rest is finished per subtree)
int split_top_levels_for(int n, int c);
int launch_split(const float* Yq, const float* Yk, int problems, int D, int n_q, int n_k, int c_q,
                 int c_k, int32_t* perm_q_out, int32_t* perm_q_tmp, int32_t* perm_k_out,
                 int32_t* perm_k_tmp, uint32_t* keybuf_q, uint32_t* keybuf_k, int sides, cudaStream_t st,
                 const float* Ytq = nullptr, const float* Ytk = nullptr);

// permute.cu
int launch_split_basic(const void* Q, const void* K, int dtype, const float* A_q, const float* A_k,
                       const float* noise_q, const float* noise_k, float* dirs_q, float* dirs_k, int iterations,
                       int problems, int D, int n_q, int n_k, int c_q, int c_k, int32_t* perm_q_out,
                       int32_t* perm_q_tmp, int32_t* perm_k_out, int32_t* perm_k_tmp, uint32_t* keybuf_q,
                       uint32_t* keybuf_k, cudaStream_t st);
int split_levels_for(int n, int c);
int launch_cast_f64_f32(const double* src, float* dst, size_t count, cudaStream_t st);
int launch_permute_centroid(const void* X, int dtype, const int32_t* perm, int P, int n, int D, int c,
                            void* Xp, float* cen, int32_t* count, cudaStream_t st, const void* X2 = nullptr,
                            void* Xp2 = nullptr, float* cen2 = nullptr);

// select.cu
size_t select_smem_bytes(int n_kc, int D, int qt);
int launch_select_adaptive(const float* cq, const float* ck, const int32_t* count_k, int P, int n_qc, int n_kc,
                           int D, float scale, float recall, int min_count, int32_t* block_idx,
                           int32_t* keep_count, float* score_ws, size_t score_floats, cudaStream_t st);
size_t select_score_floats(int P, int n_qc, int n_kc);
int launch_score_select(const float* cq, const float* ck, int P, int n_qc, int n_kc, int D, int keep,
                        int32_t* block_idx, float* score_ws, size_t score_floats, cudaStream_t st);

// attn_ref.cu
int launch_attn_ref(const ca_problem_t& pr, const void* Qp, const void* Kp, const void* Vp,
                    const float* ck, const float* cv, const int32_t* count_k, const int32_t* block_idx,
                    const int32_t* keep_count, int list_stride, const int32_t* perm_q, float scale, void* O,
                    float* lse, int* status, cudaStream_t st, const int32_t* redo = nullptr, int redo_tiles = 0,
                    int* redo_count = nullptr);

// attn_tc.cu
bool attn_tc_supported(const ca_problem_t& pr);
bool attn_tc_fp8_supported(const ca_problem_t& pr);
// quantize.cu: E4M3 codes and scales of the cluster-ordered queries, keys and the key centroids
int launch_quantize_qk(const void* Qp, const void* Kp, const float* ck, int P, int n_qc, int c_q, int n_kc, int c_k,
                       int cen_tiles, int D, unsigned char* q8, float* sq, unsigned char* k8, float* sk,
                       unsigned char* c8, float* sc, cudaStream_t st);
size_t attn_tc_workspace_bytes(const ca_problem_t& pr);
int launch_attn_tc(const ca_problem_t& pr, const void* Qp, const void* Kp, const void* Vp, const float* ck,
                   const float* cv, const int32_t* count_k, const int32_t* block_idx, const int32_t* keep_count,
                   int list_stride, const int32_t* perm_q, float scale, void* O, float* lse, void* ws,
                   cudaStream_t st);
// diagnostic hook of the attention kernel (see ca_debug_attn_wait in the public header)
void attn_tc_set_debug(long long wait_limit_cycles, int skip_key_load);

}  // namespace ca
