// Diagonalized recursive splitting (Section 3.2.1) on fp32 principal-component
// coordinates.  One launch per tree level; one CTA per set of that level.
//
// A set [lo, lo+s) keeps its rows in ascending original order.  A split
//   1. takes m = min(d, s) rows at positions floor(j*s/m), sums each coordinate
//      over them row after row in double (mean, then squared deviations) and
//      picks the coordinate of largest variance, lowest index on exact ties;
//   2. finds, by radix selection on order-preserving 32-bit keys, the L-th
//      smallest (value, row) along it, L = c * floor((s + c) / (2c));
//   3. moves the L smallest rows to [lo, lo+L) and the others to [lo+L, lo+s),
//      both sides keeping their order (stable partition by prefix sums).
// Nothing here depends on floating-point rounding except step 1, whose
// operation order is fixed, so the permutation is reproducible bit for bit.
#include "kernels.h"

namespace ca {

constexpr int kMaxSplitThreads = 1024;

struct SegmentRef { int lo, size, active; };

// Walks from the root to slot `slot` of `level` (most significant bit first).
// A set of at most c rows is final; its slot at deeper levels is the all-zero
// continuation (it only has to be copied to the output buffer).
__device__ __forceinline__ SegmentRef locate_segment(int n, int c, int level, int slot) {
  SegmentRef r{0, n, 1};
  for (int b = level - 1; b >= 0; --b) {
    const int bit = (slot >> b) & 1;
    if (r.size <= c) {
      if (slot & ((2 << b) - 1)) r.active = 0;   // some remaining bit is set
      return r;
    }
    const int L = c * ((r.size + c) / (2 * c));
    if (bit) { r.lo += L; r.size -= L; } else { r.size = L; }
  }
  return r;
}

__device__ __forceinline__ uint32_t order_key(float x) {
  if (x == 0.0f) x = 0.0f;                       // -0 and +0 compare equal
  uint32_t u = __float_as_uint(x);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

struct SplitSide {
  const float* Y;          // [P][n][D]
  const int32_t* perm_in;  // [P][n] or null (identity)
  int32_t* perm_out;       // [P][n]
  uint32_t* keybuf;        // [P][n] staging for sets larger than the shared-memory window
  int n, c, levels;
};

struct SplitParams {
  SplitSide side[2];
  int D, level, problems, smem_rows;
};

__global__ void __launch_bounds__(kMaxSplitThreads) split_level_kernel(const SplitParams prm) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  uint32_t* s_keys = reinterpret_cast<uint32_t*>(smem_raw);       // [smem_rows]
  int32_t* s_rows = reinterpret_cast<int32_t*>(s_keys + prm.smem_rows);   // [smem_rows]
  __shared__ int s_hist[256];
  __shared__ double s_var[128];
  __shared__ int s_sub[128];
  __shared__ int s_warp[2 * 32];
  __shared__ int s_scalar[4];      // 0: coordinate, 1: digit, 2: remaining rank

  const int which = blockIdx.y / prm.problems;
  const int p = blockIdx.y % prm.problems;
  const SplitSide sd = prm.side[which];
  if (prm.level >= sd.levels) return;
  const SegmentRef seg = locate_segment(sd.n, sd.c, prm.level, blockIdx.x);
  if (!seg.active) return;
  const int tid = threadIdx.x, nt = blockDim.x, lane = tid & 31, warp = tid >> 5;
  const int D = prm.D;
  const float* Y = sd.Y + (size_t)p * sd.n * D;
  const int32_t* pin = sd.perm_in ? sd.perm_in + (size_t)p * sd.n : nullptr;
  int32_t* pout = sd.perm_out + (size_t)p * sd.n;
  const int lo = seg.lo, s = seg.size;

  if (s <= sd.c) {                                   // final set: carry over
    for (int i = tid; i < s; i += nt) pout[lo + i] = pin ? pin[lo + i] : lo + i;
    return;
  }

  // ---- 1. coordinate of largest subsample variance
  const int m = min(D, s);
  if (tid < m) {
    const int pos = lo + (int)(((long long)tid * s) / m);
    s_sub[tid] = pin ? pin[pos] : pos;
  }
  __syncthreads();
  if (tid < D) {
    double sum = 0.0;
    for (int j = 0; j < m; ++j) sum = __dadd_rn(sum, (double)__ldg(Y + (size_t)s_sub[j] * D + tid));
    const double mean = sum / (double)m;
    double acc = 0.0;
    for (int j = 0; j < m; ++j) {
      const double dev = __dsub_rn((double)__ldg(Y + (size_t)s_sub[j] * D + tid), mean);
      acc = __dadd_rn(acc, __dmul_rn(dev, dev));
    }
    s_var[tid] = acc / (double)m;
  }
  __syncthreads();
  if (warp == 0) {
    double best = -1.0; int arg = 0;
    for (int t = lane; t < D; t += 32) {
      const double v = s_var[t];
      if (v > best) { best = v; arg = t; }
    }
    for (int o = 16; o > 0; o >>= 1) {
      const double ob = __shfl_xor_sync(0xffffffffu, best, o);
      const int oa = __shfl_xor_sync(0xffffffffu, arg, o);
      if (ob > best || (ob == best && oa < arg)) { best = ob; arg = oa; }
    }
    if (lane == 0) s_scalar[0] = arg;
  }
  __syncthreads();
  const int coord = s_scalar[0];

  // ---- 2. keys
  const bool in_smem = s <= prm.smem_rows;
  uint32_t* keys = in_smem ? s_keys : sd.keybuf + (size_t)p * sd.n + lo;
  for (int i = tid; i < s; i += nt) {
    const int row = pin ? pin[lo + i] : lo + i;
    keys[i] = order_key(__ldg(Y + (size_t)row * D + coord));
    if (in_smem) s_rows[i] = row;
  }
  __syncthreads();

  // ---- radix selection of the L-th smallest key (8 bits per pass)
  const int L = sd.c * ((s + sd.c) / (2 * sd.c));
  uint32_t prefix = 0, mask = 0;
  int remaining = L;                                // 1-based rank among the candidates
  for (int shift = 24; shift >= 0; shift -= 8) {
    for (int b = tid; b < 256; b += nt) s_hist[b] = 0;
    __syncthreads();
    for (int i0 = 0; i0 < s; i0 += nt) {
      const int i = i0 + tid;
      const bool ok = i < s;
      const uint32_t k = ok ? keys[i] : 0u;
      const bool cand = ok && ((k & mask) == prefix);
      const int bin = cand ? (int)((k >> shift) & 255u) : -1;
      // one atomic per distinct bin in the warp
      const unsigned peers = __match_any_sync(0xffffffffu, bin);
      if (cand && lane == (__ffs(peers) - 1)) atomicAdd(&s_hist[bin], __popc(peers));
    }
    __syncthreads();
    if (warp == 0) {
      int local[8]; int sum = 0;
#pragma unroll
      for (int j = 0; j < 8; ++j) { local[j] = s_hist[lane * 8 + j]; sum += local[j]; }
      int incl = sum;
      for (int o = 1; o < 32; o <<= 1) {
        const int v = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += v;
      }
      int before = incl - sum;
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        if (before < remaining && remaining <= before + local[j]) {
          s_scalar[1] = lane * 8 + j;
          s_scalar[2] = remaining - before;
        }
        before += local[j];
      }
    }
    __syncthreads();
    prefix |= (uint32_t)s_scalar[1] << shift;
    mask |= 255u << shift;
    remaining = s_scalar[2];
    __syncthreads();
  }
  const uint32_t thr = prefix;
  const int eq_left = remaining;        // how many rows equal to the threshold go down

  // ---- 3. stable two-sided partition
  int less_before = 0, eq_before = 0;   // running totals over earlier positions
  for (int i0 = 0; i0 < s; i0 += nt) {
    const int i = i0 + tid;
    const bool ok = i < s;
    const uint32_t k = ok ? keys[i] : 0xffffffffu;
    const int is_less = (ok && k < thr) ? 1 : 0;
    const int is_eq = (ok && k == thr) ? 1 : 0;
    int packed = is_less | (is_eq << 16);
    int incl = packed;
    for (int o = 1; o < 32; o <<= 1) {
      const int v = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += v;
    }
    if (lane == 31) s_warp[warp] = incl;
    __syncthreads();
    if (warp == 0) {
      int w = (lane < (nt >> 5)) ? s_warp[lane] : 0;
      int wi = w;
      for (int o = 1; o < 32; o <<= 1) {
        const int v = __shfl_up_sync(0xffffffffu, wi, o);
        if (lane >= o) wi += v;
      }
      s_warp[32 + lane] = wi - w;                  // exclusive offset of each warp
      if (lane == 31) s_scalar[3] = wi;            // chunk total
    }
    __syncthreads();
    const int excl = incl - packed + s_warp[32 + warp];
    const int less_here = less_before + (excl & 0xffff);
    const int eq_here = eq_before + (excl >> 16);
    if (ok) {
      const bool down = is_less || (is_eq && eq_here < eq_left);
      const int down_before = less_here + min(eq_here, eq_left);
      const int row = in_smem ? s_rows[i] : (pin ? pin[lo + i] : lo + i);
      const int dst = down ? lo + down_before : lo + L + (i - down_before);
      pout[dst] = row;
    }
    const int total = s_scalar[3];
    less_before += total & 0xffff;
    eq_before += total >> 16;
    __syncthreads();
  }
}

int split_levels_for(int n, int c) {
  int levels = 0;
  // the largest set of each level follows the larger child
  int big = n;
  while (big > c) {
    const int L = c * ((big + c) / (2 * c));
    big = (L > big - L) ? L : big - L;
    ++levels;
  }
  return levels;
}

static int max_segment_at_level(int n, int c, int level) {
  int big = n;
  for (int l = 0; l < level && big > c; ++l) {
    const int L = c * ((big + c) / (2 * c));
    big = (L > big - L) ? L : big - L;
  }
  return big;
}

// Runs all levels for both sides.  perm_a / perm_b are ping-pong buffers per
// side; the final permutation lands in perm_final (which must be one of them,
// chosen by the caller through split_final_buffer).
int launch_split(const float* Yq, const float* Yk, int problems, int D, int n_q, int n_k, int c_q,
                 int c_k, int32_t* perm_q_out, int32_t* perm_q_tmp, int32_t* perm_k_out,
                 int32_t* perm_k_tmp, uint32_t* keybuf_q, uint32_t* keybuf_k, cudaStream_t st) {
  const int lev_q = split_levels_for(n_q, c_q), lev_k = split_levels_for(n_k, c_k);
  const int levels = lev_q > lev_k ? lev_q : lev_k;
  constexpr int kSmemRowsMax = 24576;                 // 192 KB of keys + rows
  CA_RETURN_IF_CUDA(cudaFuncSetAttribute(split_level_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         kSmemRowsMax * 8));
  // with no split to do (n <= c) one level still runs: it writes the identity
  const int run_levels = levels > 0 ? levels : 1;
  for (int level = 0; level < run_levels; ++level) {
    SplitParams prm;
    prm.D = D; prm.level = level; prm.problems = problems;
    int max_seg = 1;
    for (int w = 0; w < 2; ++w) {
      SplitSide& sd = prm.side[w];
      const int n = w == 0 ? n_q : n_k, c = w == 0 ? c_q : c_k;
      const int lev = w == 0 ? lev_q : lev_k;
      int32_t* out = w == 0 ? perm_q_out : perm_k_out;
      int32_t* tmp = w == 0 ? perm_q_tmp : perm_k_tmp;
      const int side_levels = lev > 0 ? lev : 1;
      // the last level of this side writes `out`; earlier levels alternate
      const bool to_out = ((side_levels - 1 - level) % 2) == 0;
      sd.Y = w == 0 ? Yq : Yk;
      sd.perm_out = to_out ? out : tmp;
      sd.perm_in = level == 0 ? nullptr : (to_out ? tmp : out);
      sd.keybuf = w == 0 ? keybuf_q : keybuf_k;
      sd.n = n; sd.c = c; sd.levels = side_levels;
      if (level < side_levels) {
        const int ms = max_segment_at_level(n, c, level);
        if (ms > max_seg) max_seg = ms;
      }
    }
    prm.smem_rows = max_seg < kSmemRowsMax ? max_seg : kSmemRowsMax;
    const int threads = max_seg >= 8192 ? 1024 : (max_seg >= 2048 ? 512 : 256);
    dim3 grid(1u << level, 2 * problems);
    split_level_kernel<<<grid, threads, (size_t)prm.smem_rows * 8, st>>>(prm);
    CA_LAUNCH_CHECK();
  }
  return CA_OK;
}

}  // namespace ca
