/*
 * libclusterattn — C ABI of the ClusterAttention hot path on one B200 (sm_100a).
 *
 * Three stages, one entry point each (the method's "clustering", "assignment"
 * and "attention" parts, Section 3.1):
 *   cluster_qk             transforms + diagonalized recursive splitting + centroids
 *   select_blocks          centroid scoring + top-k key clusters per query cluster
 *   cluster_attention_fwd  block-sparse attention over the selected cluster pairs
 *                          with striped mean-compensation of the excluded clusters
 *
 * Conventions for every call
 *   - All data pointers are DEVICE pointers owned by the caller, 16-byte aligned,
 *     dense row-major.  Inputs are never modified.  The library allocates no
 *     device memory: scratch is a caller-provided workspace whose size
 *     ca_workspace_bytes reports.
 *   - Work is enqueued on `stream` (a cudaStream_t passed as void*; NULL is the
 *     default stream).  Calls do not synchronise.
 *   - Tensors are [batch, heads, rows, head_dim]; batch*heads independent problems.
 *   - Return value: CA_OK or an error code; nothing is enqueued on error except
 *     for CA_ERR_CUDA (a launch failed part-way).
 *   - The first 256 bytes of a workspace hold a status word that kernels set when
 *     a bounded wait expires (CA_ERR_TIMEOUT) or an index supplied by the caller
 *     is out of range (CA_ERR_BAD_INDEX); ca_last_status reads it.  Every call
 *     clears it on its stream before its kernels run.
 */
#ifndef CLUSTER_ATTENTION_H_
#define CLUSTER_ATTENTION_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

enum {
  CA_OK = 0,
  CA_ERR_INVALID_ARG = 1,  /* null pointer, bad size, keep out of range, misaligned pointer */
  CA_ERR_UNSUPPORTED = 2,  /* dtype / head_dim / cluster size outside the supported set      */
  CA_ERR_WORKSPACE = 3,    /* workspace null or smaller than ca_workspace_bytes reports      */
  CA_ERR_CUDA = 4,         /* a CUDA runtime call or kernel launch failed                    */
  CA_ERR_TIMEOUT = 5,      /* (status word only) a bounded device-side wait gave up          */
  CA_ERR_BAD_INDEX = 6     /* (status word only) a block list entry, a list length or a perm_q
                              entry was out of range; the access was skipped                  */
};

enum { CA_DTYPE_FP32 = 0, CA_DTYPE_BF16 = 1 };

/* cluster_qk flags */
enum {
  CA_Y_IN = 1,      /* Yq/Yk hold the split coordinates: skip the transforms (used by tests
                       to feed the splitter the very same fp32 coordinates as the oracle)   */
  CA_ATTN_FP32 = 2, /* cluster_attention_fwd: force the FP32 CUDA-core kernel for bf16 data  */
  CA_METRIC_IN = 8, /* cluster_qk_basic: A_q / A_k hold the metric matrices (used by tests to feed
                       both sides the same float32 matrices)                                */
  CA_ATTN_FP8_QK = 16, /* cluster_attention_fwd: Q K^T on 8-bit floating point operands (see there) */
  CA_QUERY_UNNORMALIZED = 4 /* cluster_qk: queries are represented by R_k q with
                       R_k = sqrt(K_c^T K_c / n_k), without the division by the norm: the
                       form that goes with adaptive selection (Section 3.2.2, Appendix B.1) */
};

typedef struct {
  int32_t batch, heads;
  int32_t n_q, n_k;        /* query rows, key/value rows per head                            */
  int32_t head_dim;        /* d (values have the same width); 64 or 128                      */
  int32_t dtype;           /* CA_DTYPE_*: storage type of Q, K, V, Qp, Kp, Vp, O             */
  int32_t cluster_q;       /* query cluster size c_q, a power of two in [16, 256]            */
  int32_t cluster_k;       /* key cluster size c_k, a power of two in [16, 256]              */
  int32_t keep;            /* kept key clusters per query cluster, 1 .. ceil(n_k/c_k)        */
  int32_t compensate;      /* 0/1: striped mean-compensation off/on                          */
  float softmax_scale;     /* 0 selects 1/sqrt(head_dim)                                     */
  int32_t flags;           /* CA_Y_IN | CA_ATTN_FP32 | CA_QUERY_UNNORMALIZED | CA_METRIC_IN | CA_ATTN_FP8_QK */
} ca_problem_t;

/* Bytes of workspace each stage needs for this problem (any pointer may be NULL). */
int ca_workspace_bytes(const ca_problem_t* p, size_t* cluster_ws, size_t* select_ws,
                       size_t* attn_ws);

/*
 * Clustering (Section 3.2).  Per head, queries and keys separately:
 *   M = Q^T Q / n_q, keys -> K R_q with R_q a root of M; R_k a root of K_c^T K_c
 *   with K_c the centred keys, queries -> r(q) = R_k q / |R_k q| (Section 3.2.2);
 *   both sets are projected on their global principal components (Section 3.2.1,
 *   diagonalized variant).  The roots are Cholesky factors F F^T = M (a pivot at
 *   or below 1e-12 of the largest diagonal entry gives a zero column: the
 *   counterpart of clamping non-positive eigenvalues): the principal-component
 *   coordinates are the same for every root of the same matrix.  Component t is
 *   oriented so that the entry of largest magnitude of column t of the map from
 *   the original space to the coordinates (F E, E the principal directions) is
 *   positive, which does not depend on the root either.
 *   The rows are split recursively: at each split the coordinate of highest
 *   variance over min(d, |set|) evenly spaced rows of the set is chosen and the
 *   set is cut so that the lower side holds the multiple of c closest to half
 *   (ties in value go to the lower row index; half-way sizes go to the lower
 *   side); every set keeps its rows in ascending original order.
 * Outputs
 *   perm_q [B,H,n_q], perm_k [B,H,n_k]  position -> original row; cluster j is
 *        positions [j*c, min((j+1)*c, n)); only the last cluster can be short.
 *   Qp,Kp,Vp [B,H,n_c*c,d]  rows gathered in cluster order (V follows the key
 *        permutation); the short cluster is zero-padded to c rows.
 *   cq,ck,cv [B,H,n_c,d] fp32  centroids: means over the actual members in the
 *        original space (Section 3.3.1; Appendix A).
 *   count_q,count_k [B,H,n_c]  member counts |c|.
 *   Yq [B,H,n_q,d], Yk [B,H,n_k,d] fp32 split coordinates: input when
 *        p->flags has CA_Y_IN, otherwise output (may be NULL: kept in ws).
 * The chain from Q to the key side (metric, its factor, key projection, key split)
 * and the chain from K to the query side need each other only through C_K: the
 * second one is enqueued on a side stream of the library (a pool of four per
 * device, taken in turn, created together with their events at the first call on
 * that device) that forks from `stream` at the start of the call and joins it
 * again before the call returns.  Nothing waits on the host; a capture of `stream`
 * records the side stream as a parallel branch (make the first call on a device
 * before capturing).  The calls of this library may be issued from several host
 * threads; ca_profile, ca_debug_attn_wait and the workspaces themselves are not
 * synchronised (one workspace serves one call at a time).
 */
int cluster_qk(const ca_problem_t* p, const void* Q, const void* K, const void* V,
               int32_t* perm_q, int32_t* perm_k, void* Qp, void* Kp, void* Vp,
               float* cq, float* ck, float* cv, int32_t* count_q, int32_t* count_k,
               float* Yq, float* Yk, void* ws, size_t ws_bytes, void* stream);

/*
 * Clustering by basic recursive splitting (Section 3.2.1, the variant of principal
 * direction divisive partitioning) with the metric injected into the power
 * iteration (Section 5.2): no eigendecomposition and no transformed copy of the
 * rows.  Rows x compared in a metric A = R R have the transformed rows x R, whose
 * first principal direction w obeys w ~ (R C R) w, C the covariance of the
 * rows; with u = R w that is u <- A C u, and a row projects to x . u.  Keys use
 * A_k = Q^T Q / n_q, queries A_q = K_c^T K_c / n_k (the un-normalised
 * representation, Appendix B.1).  Per set of s > c rows, all in float32 with
 * sequential sums (each product and sum rounded on its own; the projections
 * decide the partition, so the order of operations is part of the definition):
 *   subsample: the min(d, s) rows at positions floor(j s / m) of the set;
 *   mu_k = (sum_i x_ik) / m;  z = x - mu;
 *   start vector: g / |g| at the root, (u_parent + g / |g|) / 2 elsewhere, g the
 *   node's row of `noise` (normal deviates drawn by the caller);
 *   `iterations` times: v_i = sum_k z_ik u_k; w_k = sum_i z_ik v_i;
 *   y_j = sum_k A_jk w_k; u = y / |y| (kept when |y| is zero or not finite);
 *   key of a row: t = sum_k x_k u_k; the set is split as in cluster_qk: the
 *   L = c floor((s + c) / (2c)) smallest (t, row) go down, both sides keep their
 *   rows in ascending order.
 * Nodes are numbered 2^level - 1 + slot, the bits of slot (most significant
 * first) being the path from the root, 0 = lower side.
 *   noise_q [B,H,rows_q,d], noise_k [B,H,rows_k,d] fp32, rows as reported by
 *        ca_basic_workspace_bytes (2^levels - 1).
 *   A_q, A_k [B,H,d,d] fp32: output, or input when p->flags has CA_METRIC_IN.
 *   iterations in 0 .. 64.  Other arguments and outputs as in cluster_qk.
 */
int ca_basic_workspace_bytes(const ca_problem_t* p, size_t* bytes, int32_t* noise_rows_q,
                             int32_t* noise_rows_k);
int cluster_qk_basic(const ca_problem_t* p, const void* Q, const void* K, const void* V,
                     const float* noise_q, const float* noise_k, int32_t iterations,
                     float* A_q, float* A_k, int32_t* perm_q, int32_t* perm_k, void* Qp,
                     void* Kp, void* Vp, float* cq, float* ck, float* cv, int32_t* count_q,
                     int32_t* count_k, void* ws, size_t ws_bytes, void* stream);

/*
 * Assignment (Section 3.3).  score(i,j) = cq_i . ck_j (the mean logit of the two
 * clusters); for each query cluster the `keep` best key clusters, ties to the
 * lower index, written in ascending index order.
 *   block_idx [B,H,n_qc,keep] int32.
 * With 2048 key clusters or more and a workspace as large as ca_workspace_bytes
 * reports, the scores are first computed in tiles into the workspace (same
 * operation order, same bits); a workspace of 256 bytes selects the fused kernel.
 */
int select_blocks(const ca_problem_t* p, const float* cq, const float* ck,
                  int32_t* block_idx, void* ws, size_t ws_bytes, void* stream);

/*
 * Attention (eq. 2 over the selected clusters; Appendix A for compensation).
 * For query row r of query cluster i, with s = softmax_scale:
 *   entries  (s q_r.k_t, v_t)                 for every member t of a selected cluster
 *   and, if p->compensate,
 *            (s q_r.kbar_j + ln|c_j|, vbar_j) for every cluster j NOT selected;
 *   O_r = softmax-weighted mean of the entry values; lse_r = log-sum-exp of the
 *   entry logits.  Padding rows of the short cluster are masked.
 * Accepts any valid permutation and block list (block_idx rows must be strictly
 * ascending), so the stage can be driven by another clustering.
 *   Qp,Kp,Vp, ck, cv, count_k, perm_q: as written by cluster_qk.
 *   O [B,H,n_q,d] in ORIGINAL row order, storage dtype; lse [B,H,n_q] fp32 or NULL.
 * bf16 storage runs on tcgen05 tensor cores with fp32 accumulation (head_dim
 * 64/128, c_q in {64, 128, 256}, c_k in 16..256); fp32 storage, other sizes, or
 * CA_ATTN_FP32 run the FP32 CUDA-core kernel.
 *
 * CA_ATTN_FP8_QK (off by default; bf16 storage, head_dim 128, c_k >= 64, else
 * CA_ERR_UNSUPPORTED): the variant with a quantised Q K^T (Section 3.1: the kernel
 * the paper runs is a quantised one; Section 5.1).  Queries, keys and the key
 * centroids of the compensation are turned into E4M3 codes (4 exponent bits, 3
 * mantissa bits, largest value 448) inside the call: one scale per query row, per
 * key cluster and per run of 64 key centroids, scale = (largest magnitude of the
 * group) / 448, code = E4M3(x * (448 / largest magnitude)) rounded to nearest even,
 * all in float32.  The logits are (code_q . code_k) * scale_q * scale_k * s; the
 * probabilities, the values and the value centroids are not quantised.  The
 * workspace is larger (ca_workspace_bytes with the flag set).  Query tiles that the
 * second pass recomputes (see ca_attn_recomputed) are recomputed unquantised.
 */
int cluster_attention_fwd(const ca_problem_t* p, const void* Qp, const void* Kp,
                          const void* Vp, const float* ck, const float* cv,
                          const int32_t* count_k, const int32_t* block_idx,
                          const int32_t* perm_q, void* O, float* lse, void* ws,
                          size_t ws_bytes, void* stream);

/*
 * Adaptive assignment (Section 3.3.2): instead of a fixed count, each query
 * cluster takes the key clusters of largest estimated attention mass until
 * their share of the estimate reaches `recall`.  The estimate for the pair
 * (i, j) is |c_j| exp(s cq_i . ck_j), s = softmax_scale.  All of it is float32
 * with every product and sum rounded separately, in this order:
 *   score = sum over k ascending of cq_ik ck_jk (as in select_blocks);
 *   x = (score - max_j score) * (s * log2 e);   mass = 2^x * |c_j| with 2^x from
 *   a cubic in the fractional part (x clamped to [-100, 100], nearest-integer
 *   split, Horner's rule, coefficients 0.99992806, 0.69326097, 0.24261113,
 *   0.05517165);  clusters in order of decreasing mass, ties to the lower index;
 *   running sum in that order; the shortest prefix whose sum is >= recall * total
 *   (total = the full running sum); recall >= 1 takes every cluster; never fewer
 *   than min(min_count, n_kc).
 *   block_idx [B,H,n_qc,n_kc] int32: row i holds keep_count[i] ascending cluster
 *        indices, the rest of the row is -1.   keep_count [B,H,n_qc] int32.
 * p->keep is not used (it must still be valid).  recall > 0, min_count >= 1.
 */
int select_blocks_adaptive(const ca_problem_t* p, const float* cq, const float* ck,
                           const int32_t* count_k, float recall, int32_t min_count,
                           int32_t* block_idx, int32_t* keep_count, void* ws,
                           size_t ws_bytes, void* stream);

/*
 * cluster_attention_fwd over lists of different lengths: query cluster i attends
 * the first keep_count[i] entries of row i of block_idx, whose rows are
 * list_stride entries apart (n_kc for the output of select_blocks_adaptive).
 * Everything else as in cluster_attention_fwd; p->keep is not used.
 */
int cluster_attention_fwd_ragged(const ca_problem_t* p, const void* Qp, const void* Kp,
                                 const void* Vp, const float* ck, const float* cv,
                                 const int32_t* count_k, const int32_t* block_idx,
                                 const int32_t* keep_count, int32_t list_stride,
                                 const int32_t* perm_q, void* O, float* lse, void* ws,
                                 size_t ws_bytes, void* stream);

/*
 * The attention stage without a caller-provided workspace.  (The paper has no
 * counterpart for this entry point; it exists for deployment reasons only.)
 *
 * Meant for callers that cannot allocate device memory and therefore cannot
 * supply a workspace: code inside a host framework's execute callback where
 * allocation is not allowed, serving loops that must avoid the device-wide
 * synchronisation an allocation implies, and processes whose device memory is
 * already reserved by another pool.  Same computation, arguments and results
 * as cluster_attention_fwd (inputs and outputs are still the caller's), but the
 * scratch is a fixed array of ca_static_scratch_bytes() = 32 MiB that is part
 * of the library image: every GPU that loads the library holds it until the
 * process exits.  After the set-up described below a call allocates and frees
 * nothing.
 *   - Limit: returns CA_ERR_WORKSPACE, enqueuing nothing, if the attention
 *     workspace that ca_workspace_bytes reports for `p` exceeds the array.
 *   - Set-up: the first call on each device looks up the array's device address
 *     (with that device current).  Under CUDA's lazy module loading that lookup
 *     is also what loads the library's device code on that GPU and reserves the
 *     32 MiB, so the first call can take longer, may synchronise the device, and
 *     returns CA_ERR_CUDA if the memory cannot be had.  Make that first call
 *     before any stream capture is started.
 *   - Sharing: every call on a device uses the same array, which keeps the
 *     previous call's contents; the call itself clears the status word and
 *     rewrites the centroid copies it needs (the counter that
 *     ca_attn_recomputed reports keeps adding up over the life of the process).  Two calls whose kernels overlap on
 *     the GPU (different streams) race on the array: serialise them.
 * ca_static_last_status reads the array's status word (synchronises the device).
 */
size_t ca_static_scratch_bytes(void);
int cluster_attention_fwd_static(const ca_problem_t* p, const void* Qp, const void* Kp,
                                 const void* Vp, const float* ck, const float* cv,
                                 const int32_t* count_k, const int32_t* block_idx,
                                 const int32_t* perm_q, void* O, float* lse, void* stream);
int ca_static_last_status(void);

/* Reads the status word of a workspace as the last call on it left it (synchronises the device). */
int ca_last_status(const void* ws);

/* Statistics of an attention workspace (synchronises the device): how many query clusters the
 * second pass of the attention calls on this workspace has recomputed with the fp32 kernel, summed
 * over all calls since the caller zero-filled the workspace (the calls only add to the counter,
 * the last word of the 256-byte status block).  The tensor-core kernel keeps the reference of its
 * online softmax (Section 3.1: exact softmax over the kept blocks) one half-step behind; a query
 * cluster whose scores climb by more than 2^96 within 64 keys leaves its range and is recomputed.
 * Returns the count (>= 0), or minus an error code. */
int ca_attn_recomputed(const void* ws);

/* Diagnostic hook for tests of the failure path (process-wide, not thread-safe; affects the
 * attention calls issued after it).  wait_limit_cycles: SM cycles after which a device-side wait
 * of the tensor-core attention kernel gives up (<= 0 restores the default of about two seconds).
 * skip_key_load: the loader leaves out the key rows of this half-step (64 keys) of every query
 * tile, so that the waits for them run out: the kernel records CA_ERR_TIMEOUT, releases its tensor
 * memory and returns, and the output of the call is undefined; -1 restores normal operation. */
void ca_debug_attn_wait(long long wait_limit_cycles, int skip_key_load);

/* Diagnostic: the symmetric eigen-decomposition that cluster_qk uses for the principal components
 * (Section 3.2.1, diagonalized variant), on matrices of the caller's.  A: `count` symmetric d x d
 * matrices in double precision, row-major (device, read only); d = 64 or 128.  Written (device):
 * W [count][d][d] float32, eigenvector t in column t, eigenvalues in descending order, each column
 * oriented so that its entry of largest magnitude is positive; evals [count][d] double, or NULL.
 * The arithmetic is float32 (the components only feed float32 coordinates).  Enqueued on `stream`;
 * returns CA_ERR_UNSUPPORTED for another d, CA_ERR_INVALID_ARG for null or misaligned pointers. */
int ca_debug_eigh(const double* A, int count, int d, float* W, double* evals, void* stream);

/*
 * Per-kernel-group device times (a measuring aid; process-wide, not thread-safe).
 * ca_profile(1) switches the timers on: every call issued afterwards records CUDA events around
 * its kernel groups, and cluster_qk runs its two sides one after the other on the caller's stream
 * (instead of side by side on two streams) so that every group is timed alone.  ca_profile(0)
 * switches them off.  The first ca_profile(1) creates the events (make it before a stream capture).
 * ca_profile_read synchronises the device, returns the number of groups and, for group g, its
 * name (static string), the summed device time in ms and the number of timed scopes since the
 * timers were switched on or last read; then it starts counting afresh.  Groups: gram,
 * cholesky_factor, principal_components, transform, split_levels, split_tail, permute_centroid,
 * score_select, centroid_prep, attn_tc, attn_second_pass.  Any output pointer may be NULL.
 */
int ca_profile(int enable);
int ca_profile_read(int max_groups, const char** names, float* ms, int* scopes);

/* Library version and the compute capability the kernels were built for. */
const char* ca_version(void);

/* Diagnostic: number of kernels this library has enqueued since it was loaded
 * (host-side atomic counter). */
unsigned long long ca_kernel_launches(void);

#ifdef __cplusplus
}
#endif
#endif /* CLUSTER_ATTENTION_H_ */
