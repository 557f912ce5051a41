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

// eigh.cu
int launch_eigh(const double* A, int count, int D, double* out64, float* out32, double* evals,
                cudaStream_t st);
int launch_metric(const double* gramQ, const double* gramK, const double* sumK, int P, int D, int n_q,
                  int n_k, double ck_scale, double* M, double* CK, cudaStream_t st);
int launch_covariance(const double* gram, const double* sum, int P, int D, int n, double* cov,
                      cudaStream_t st);
int launch_small_matmul(const double* A, const double* B, int P, int D, double alpha, int trans_a,
                        double* C, float* C32, cudaStream_t st);
int launch_cholesky_factor(const double* A, int count, int D, double* out64, float* out32, cudaStream_t st);
int launch_bias(const double* sum, const float* W, int P, int D, int n, float* bias, cudaStream_t st,
                void* wt_hi = nullptr, void* wt_lo = nullptr);

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
                    float* lse, cudaStream_t st, const int32_t* redo = nullptr, int redo_tiles = 0,
                    int* redo_count = nullptr);

// attn_tc.cu
bool attn_tc_supported(const ca_problem_t& pr);
size_t attn_tc_workspace_bytes(const ca_problem_t& pr);
int launch_attn_tc(const ca_problem_t& pr, const void* Qp, const void* Kp, const void* Vp, const float* ck,
                   const float* cv, const int32_t* count_k, const int32_t* block_idx, const int32_t* keep_count,
                   int list_stride, const int32_t* perm_q, float scale, void* O, float* lse, void* ws,
                   cudaStream_t st);

}  // namespace ca
