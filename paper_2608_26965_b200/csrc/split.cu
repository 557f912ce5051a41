// Diagonalized recursive splitting (Section 3.2.1) on fp32 principal-component
// coordinates.
//
// A set [lo, lo+s) keeps its rows in ascending original order.  A split
//   1. takes m = min(d, s) rows at positions floor(j*s/m), estimates the variance
//      of each coordinate over them in float32 with a fixed operation order and
//      picks the coordinate of largest variance, lowest index on exact ties;
//   2. finds, by radix selection on order-preserving 32-bit keys, the L-th
//      smallest (value, row) along it, L = c * floor((s + c) / (2c));
//   3. moves the L smallest rows to [lo, lo+L) and the others to [lo+L, lo+s),
//      both sides keeping their order (stable partition by prefix sums).
// Nothing depends on floating-point rounding except step 1, whose operation
// order is fixed, so the permutation is reproducible bit for bit.
//
// Two kernels.  Large sets: one launch per tree level, a thread-block cluster of
// up to 8 CTAs per set; each CTA keeps its slice of keys and rows in shared
// memory, histograms and partition offsets are combined through distributed
// shared memory (hardware cluster barriers, no spin waits).  Sets of at most
// kTailRows rows: one CTA finishes the whole subtree in shared memory, all
// subsets of a level side by side, and writes the permutation once.
//
// The basic variant of the splitting (a power iteration per set instead of a
// coordinate choice, at the end of this file) computes its keys in kernels of
// its own and reuses the per-level kernel for selection and partition.
#include <climits>
#include <cooperative_groups.h>

#include "kernels.h"

namespace ca {

namespace cg = cooperative_groups;

constexpr int kSplitThreads = 1024;
constexpr int kSmemRowsMax = 24576;      // rows a CTA stages (8 bytes each)
constexpr int kMaxCluster = 8;
constexpr int kLevelListMax = 1024;      // candidates that the level kernel ranks from a list after two digits
constexpr int kTailRowsMax = 4096;
constexpr int kTailSegs = 32;            // subsets a tail CTA splits side by side

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

// Variances of all coordinates over subsamples staged in shared memory, `ng` tiles of
// tile[j*D + t], j < m_g.  The estimate only feeds an argmax, so it is taken in float32 with
// a fixed operation order (reproducible bit for bit; every operation rounded on its own, no
// fused multiply-add): eight partial sums over the rows j = r, r+8, ... taken row after row,
// combined as ((p0+p1)+(p2+p3)) + ((p4+p5)+(p6+p7)); first the mean, then the squared
// deviations.  part: [ng][8][D] floats, out: [ng][D] floats.  Called by all threads of the CTA.
template <int D, typename RowsOf>
__device__ __forceinline__ void staged_variances(const float* tiles, int ng, RowsOf rows_of,
                                                 float* part, float* out, int tid, int nt) {
  for (int pass = 0; pass < 2; ++pass) {
    for (int task = tid; task < ng * 8 * D; task += nt) {
      const int gi = task / (8 * D), r = (task / D) % 8, t = task % D;
      const int m = rows_of(gi);
      const float* tile = tiles + gi * D * D;
      float acc = 0.f;
      if (pass == 0) {
        for (int j = r; j < m; j += 8) acc = __fadd_rn(acc, tile[j * D + t]);
      } else {
        const float mean = out[gi * D + t];
        for (int j = r; j < m; j += 8) {
          const float dev = __fsub_rn(tile[j * D + t], mean);
          acc = __fadd_rn(acc, __fmul_rn(dev, dev));
        }
      }
      part[(gi * 8 + r) * D + t] = acc;
    }
    __syncthreads();
    for (int task = tid; task < ng * D; task += nt) {
      const int gi = task / D, t = task % D;
      const float* p = part + gi * 8 * D + t;
      const float tot = __fadd_rn(__fadd_rn(__fadd_rn(p[0], p[D]), __fadd_rn(p[2 * D], p[3 * D])),
                                  __fadd_rn(__fadd_rn(p[4 * D], p[5 * D]), __fadd_rn(p[6 * D], p[7 * D])));
      const int m = rows_of(gi);
      out[task] = m > 0 ? __fdiv_rn(tot, (float)m) : -1.0f;
    }
    __syncthreads();
  }
}

// Two fp32 values in one 64-bit register and the instructions that work on both halves at once
// (each half rounded to nearest on its own: the same bits as two scalar operations).
typedef unsigned long long pair2;
__device__ __forceinline__ pair2 pair(float lo, float hi) {
  pair2 d;
  asm("mov.b64 %0, {%1, %2};" : "=l"(d) : "f"(lo), "f"(hi));
  return d;
}
__device__ __forceinline__ void unpair(pair2 v, float& lo, float& hi) {
  asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ pair2 add_pair(pair2 a, pair2 b) {
  pair2 d;
  asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}

// The same estimate for `ng` subsets at once, the sample rows read straight from the coordinates
// in global memory.  `sub` holds the sample rows residue-major: sub[gi * D + r * (D / 8) + k] is
// the row of sample r + 8 k of subset gi, -1 beyond its m rows.  Same operations in the same order
// as staged_variances, hence the same bits; what differs is the parallelism: every (subset,
// residue, coordinate) is a thread's task, so a round of many small subsets keeps all warps busy
// between two barriers, and a task's loads (one per sample row of its residue) are in flight four
// at a time.  The stage is bound by the instructions it issues, so a subset with all D sample rows
// (every subset that still splits when the cluster size is at least D) runs without a test per
// row; a missing row otherwise reads as 0 in the pass of the sums and as the mean in the pass of
// the squares, which adds an exact zero.
template <int D, typename RowsOf>
__device__ __forceinline__ void gathered_variances(const float* __restrict__ Y, const int* sub, int ng, RowsOf rows_of,
                                                   float* part, float* out, int tid, int nt) {
  constexpr int PER = D / 8;                       // sample rows of a residue
  constexpr int Q4 = D / 4;                        // 16-byte vectors of a row
  constexpr int B = 4;                             // loads in flight per task
  for (int pass = 0; pass < 2; ++pass) {
    for (int task = tid; task < ng * 8 * Q4; task += nt) {
      const int gi = task / (8 * Q4), r = (task / Q4) % 8, t4 = task % Q4;
      const int m = rows_of(gi);
      float4 mean = make_float4(0.f, 0.f, 0.f, 0.f);
      if (pass == 1) mean = *reinterpret_cast<const float4*>(out + gi * D + 4 * t4);
      pair2 acc_a = pair(0.f, 0.f), acc_b = acc_a;
      float4 sq = make_float4(0.f, 0.f, 0.f, 0.f);
      const pair2 nmean_a = pair(-mean.x, -mean.y), nmean_b = pair(-mean.z, -mean.w);
      const int4* idx = reinterpret_cast<const int4*>(sub + gi * D + r * PER);
      const float4* Yv = reinterpret_cast<const float4*>(Y) + t4;
      const bool full = m == D;                    // all PER rows of the residue are there
#pragma unroll
      for (int k0 = 0; k0 < PER; k0 += B) {
        const int4 ri = idx[k0 / B];
        const int row[B] = {ri.x, ri.y, ri.z, ri.w};
        float4 x[B];
        if (full) {
#pragma unroll
          for (int k = 0; k < B; ++k) x[k] = __ldg(Yv + (size_t)row[k] * Q4);
        } else {
#pragma unroll
          for (int k = 0; k < B; ++k) x[k] = row[k] >= 0 ? __ldg(Yv + (size_t)row[k] * Q4) : mean;
        }
        // Sums and differences two values per instruction (each half rounded on its own: the bits
        // of two scalar additions).  The squares and their sums stay scalar operations that are
        // never contracted: a two-value multiply followed by a two-value add is merged into one
        // fused multiply-add by the assembler, which rounds once where the definition rounds twice.
#pragma unroll
        for (int k = 0; k < B; ++k) {
          const pair2 xa = pair(x[k].x, x[k].y), xb = pair(x[k].z, x[k].w);
          if (pass == 0) {
            acc_a = add_pair(acc_a, xa);
            acc_b = add_pair(acc_b, xb);
          } else {
            float dx, dy, dz, dw;
            unpair(add_pair(xa, nmean_a), dx, dy);                                // x - mean
            unpair(add_pair(xb, nmean_b), dz, dw);
            sq.x = __fadd_rn(sq.x, __fmul_rn(dx, dx)); sq.y = __fadd_rn(sq.y, __fmul_rn(dy, dy));
            sq.z = __fadd_rn(sq.z, __fmul_rn(dz, dz)); sq.w = __fadd_rn(sq.w, __fmul_rn(dw, dw));
          }
        }
      }
      float4 acc = sq;
      if (pass == 0) {
        unpair(acc_a, acc.x, acc.y);
        unpair(acc_b, acc.z, acc.w);
      }
      *reinterpret_cast<float4*>(part + (gi * 8 + r) * D + 4 * t4) = acc;
    }
    __syncthreads();
    for (int task = tid; task < ng * D; task += nt) {
      const int gi = task / D, t = task % D;
      const float* p = part + gi * 8 * D + t;
      const float tot = __fadd_rn(__fadd_rn(__fadd_rn(p[0], p[D]), __fadd_rn(p[2 * D], p[3 * D])),
                                  __fadd_rn(__fadd_rn(p[4 * D], p[5 * D]), __fadd_rn(p[6 * D], p[7 * D])));
      const int m = rows_of(gi);
      out[task] = m > 0 ? __fdiv_rn(tot, (float)m) : -1.0f;
    }
    __syncthreads();
  }
}

// 16-byte asynchronous copy global -> shared (no registers held while in flight)
__device__ __forceinline__ void cp_async16(void* smem_dst, const void* gmem_src) {
  const uint32_t d = static_cast<uint32_t>(__cvta_generic_to_shared(smem_dst));
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(d), "l"(gmem_src) : "memory");
}
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_all;" ::: "memory"); }

struct SplitSide {
  const float* Y;          // [P][n][D]
  const float* Yt;         // [P][D][n] the same coordinates, coordinate-major, or null
  const int32_t* perm_in;  // [P][n] or null (identity)
  int32_t* perm_out;       // [P][n]
  uint32_t* keybuf;        // [P][n] staging for sets larger than the shared-memory windows
  int n, c, levels, tail_level;
  int active;              // 0: this launch leaves the side alone (the two sides can run on different streams)
};

struct SplitParams {
  SplitSide side[2];
  int D, level, problems, smem_rows;
  int keys_in;             // the keys of this level are already in keybuf (basic variant): no coordinate choice, no gather
};

// ---------------------------------------------------------------------------
// One level of the large sets.  grid.x = slots * cluster size.
// ---------------------------------------------------------------------------
template <int D>
__global__ void __launch_bounds__(kSplitThreads) split_level_kernel(const SplitParams prm) {
  cg::cluster_group cluster = cg::this_cluster();
  const int csize = (int)cluster.num_blocks();
  const int crank = (int)cluster.block_rank();
  extern __shared__ __align__(16) unsigned char smem_raw[];
  uint32_t* s_keys = reinterpret_cast<uint32_t*>(smem_raw);                  // [smem_rows]
  int32_t* s_rows = reinterpret_cast<int32_t*>(s_keys + prm.smem_rows);      // [smem_rows]
  __shared__ int s_hist2[2][256];  // digit counts of this slice, two in rotation over the passes
  __shared__ int s_total[256];
  __shared__ float s_var[128];
  __shared__ float s_part[8 * 128];
  __shared__ int s_sub[128];
  __shared__ int s_warp[2 * 32];
  __shared__ int s_scalar[4];      // 0: coordinate, 1: digit, 2: remaining rank, 3: chunk total
  __shared__ int s_counts[2];      // this CTA's (less, equal) totals
  __shared__ uint32_t s_list[kLevelListMax];   // the keys that share the first two digits with the threshold
  __shared__ int s_list_n;         // entries of the list (counted in the cluster's first CTA)
  __shared__ int s_ncand;          // keys in the digit that the last pass chose
  int* const s_hist = s_hist2[1];  // scratch of the partition (the last pass counts in the other array)

  const int which = blockIdx.y / prm.problems;
  const int p = blockIdx.y % prm.problems;
  const SplitSide sd = prm.side[which];
  if (!sd.active || prm.level >= sd.tail_level) return;   // uniform over the cluster
  const SegmentRef seg = locate_segment(sd.n, sd.c, prm.level, blockIdx.x / csize);
  if (!seg.active) return;
  const int tid = threadIdx.x, nt = blockDim.x, lane = tid & 31, warp = tid >> 5;
  const float* Y = sd.Y + (size_t)p * sd.n * D;
  const float* Yt = sd.Yt ? sd.Yt + (size_t)p * sd.n * D : nullptr;
  const int32_t* pin = sd.perm_in ? sd.perm_in + (size_t)p * sd.n : nullptr;
  int32_t* pout = sd.perm_out + (size_t)p * sd.n;
  const int lo = seg.lo, s = seg.size;

  if (s <= sd.c) {                                   // final set: carry over
    if (crank == 0)
      for (int i = tid; i < s; i += nt) pout[lo + i] = pin ? pin[lo + i] : lo + i;
    return;
  }

  // ---- 1. coordinate of largest subsample variance (every CTA of the cluster computes it)
  const int m = min(D, s);
  int coord = 0;
  if (!prm.keys_in) {
  if (tid < m) {
    const int pos = lo + (int)(((long long)tid * s) / m);
    s_sub[tid] = pin ? pin[pos] : pos;
  }
  __syncthreads();
  {
    // the subsample rows are staged by all threads (16-byte loads in flight together)
    float4* stage4 = reinterpret_cast<float4*>(smem_raw);
    constexpr int q = D / 4;
    for (int e = tid; e < m * q; e += nt)
      cp_async16(stage4 + e, reinterpret_cast<const float4*>(Y + (size_t)s_sub[e / q] * D) + (e % q));
    cp_async_wait_all();
  }
  __syncthreads();
  staged_variances<D>(reinterpret_cast<const float*>(smem_raw), 1, [&](int) { return m; }, s_part, s_var, tid, nt);
  if (warp == 0) {
    float best = -1.0f; int arg = 0;
    for (int t = lane; t < D; t += 32) {
      const float v = s_var[t];
      if (v > best) { best = v; arg = t; }
    }
    for (int o = 16; o > 0; o >>= 1) {
      const float ob = __shfl_xor_sync(0xffffffffu, best, o);
      const int oa = __shfl_xor_sync(0xffffffffu, arg, o);
      if (ob > best || (ob == best && oa < arg)) { best = ob; arg = oa; }
    }
    if (lane == 0) s_scalar[0] = arg;
  }
  __syncthreads();
  coord = s_scalar[0];
  }

  // ---- 2. keys of this CTA's slice [c0, c1) of the set
  const int chunk = (s + csize - 1) / csize;
  const int c0 = min(s, crank * chunk), c1 = min(s, c0 + chunk);
  const int cs = c1 - c0;
  const bool in_smem = cs <= prm.smem_rows;
  uint32_t* keys = in_smem ? s_keys : sd.keybuf + (size_t)p * sd.n + lo + c0;
  if (prm.keys_in) {
    // the projections of this level were turned into keys by another kernel, position by position
    if (in_smem) {
      const uint32_t* kin = sd.keybuf + (size_t)p * sd.n + lo + c0;
      for (int i = tid; i < cs; i += nt) {
        s_keys[i] = kin[i];
        s_rows[i] = pin ? pin[lo + c0 + i] : lo + c0 + i;
      }
    }
  } else {
  // gathers in batches of eight: the row indices first, then the coordinates, so that the
  // memory latencies of a batch overlap
  for (int i0 = tid; i0 < cs; i0 += 8 * nt) {
    int row[8];
    float val[8];
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      const int i = i0 + u * nt;
      row[u] = (i < cs) ? (pin ? __ldg(pin + lo + c0 + i) : lo + c0 + i) : 0;
    }
#pragma unroll
    for (int u = 0; u < 8; ++u) val[u] = Yt ? __ldg(Yt + (size_t)coord * sd.n + row[u]) : __ldg(Y + (size_t)row[u] * D + coord);
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      const int i = i0 + u * nt;
      if (i < cs) {
        keys[i] = order_key(val[u]);
        if (in_smem) s_rows[i] = row[u];
      }
    }
  }
  }
  for (int b = tid; b < 256; b += nt) s_hist2[1][b] = 0;      // the first pass (shift 24) counts here
  if (tid == 0) s_list_n = 0;
  __syncthreads();

  // ---- radix selection of the L-th smallest key of the whole set (8 bits per pass).  The slices'
  // counts alternate between two arrays: a peer may still be adding up one pass's counts while
  // this CTA counts the next pass, and an array is cleared only after the cluster barrier of the
  // pass after the one that used it, when every peer has finished reading it.
  // After two digits the keys that share them with the threshold are usually few: if they fit the
  // list, every slice appends its candidates to the list of the cluster's first CTA (one more
  // cluster barrier), every CTA takes a copy, and the last two digits are counted over that list
  // alone, with no sweep over the slice, no cluster barrier and no sums over the peers.
  const int L = sd.c * ((s + sd.c) / (2 * sd.c));
  uint32_t prefix = 0, mask = 0;
  int remaining = L;                                // 1-based rank among the candidates
  bool listed = false;
  int n_list = 0;
  for (int shift = 24; shift >= 0; shift -= 8) {
    int* const hist = s_hist2[(shift >> 3) & 1];
    int* const hist_next = s_hist2[((shift >> 3) & 1) ^ 1];
    if (shift == 8 && s_ncand <= kLevelListMax) {   // uniform over the cluster: every CTA holds the same totals
      listed = true;
      n_list = s_ncand;
      uint32_t* const list0 = csize > 1 ? cluster.map_shared_rank(s_list, 0) : s_list;
      int* const count0 = csize > 1 ? cluster.map_shared_rank(&s_list_n, 0) : &s_list_n;
      for (int i = tid; i < cs; i += nt) {
        const uint32_t k = keys[i];
        if ((k & mask) == prefix) list0[atomicAdd(count0, 1)] = k;   // n_list such keys in the whole set
      }
      if (csize > 1) {
        cluster.sync();                              // the list is complete (and every peer is past the second pass)
        if (crank != 0)
          for (int i = tid; i < n_list; i += nt) s_list[i] = list0[i];
      }
      __syncthreads();
    }
    if (!listed) {
      for (int i0 = 0; i0 < cs; i0 += nt) {
        const int i = i0 + tid;
        const bool ok = i < cs;
        const uint32_t k = ok ? keys[i] : 0u;
        // one atomic per candidate key, also for the leading digit with its few distinct values:
        // a sweep of plain atomics costs the same whatever the digit's spread, and a warp match per
        // position to merge equal digits costs three times as much
        if (ok && ((k & mask) == prefix)) atomicAdd(&hist[(k >> shift) & 255u], 1);
      }
      if (csize > 1) {
        cluster.sync();                              // every slice has counted
        for (int b = tid; b < 256; b += nt) {
          int sum = 0;
          for (int r = 0; r < csize; ++r) sum += cluster.map_shared_rank(hist, r)[b];
          s_total[b] = sum;
        }
      } else {
        __syncthreads();
        for (int b = tid; b < 256; b += nt) s_total[b] = hist[b];
      }
    } else {
      for (int i = tid; i < n_list; i += nt) {
        const uint32_t k = s_list[i];
        if ((k & mask) == prefix) atomicAdd(&hist[(k >> shift) & 255u], 1);
      }
      __syncthreads();
      for (int b = tid; b < 256; b += nt) s_total[b] = hist[b];
    }
    for (int b = tid; b < 256; b += nt) hist_next[b] = 0;
    __syncthreads();
    if (warp == 0) {
      int local[8]; int sum = 0;
#pragma unroll
      for (int j = 0; j < 8; ++j) { local[j] = s_total[lane * 8 + j]; sum += local[j]; }
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
          s_ncand = local[j];
        }
        before += local[j];
      }
    }
    __syncthreads();
    prefix |= (uint32_t)s_scalar[1] << shift;
    mask |= 255u << shift;
    remaining = s_scalar[2];
    // (s_scalar is written again only after the next pass's barriers)
  }
  const uint32_t thr = prefix;
  const int eq_left = remaining;        // how many rows equal to the threshold go down

  // ---- 3. stable two-sided partition.  Every warp owns a contiguous run of the slice and walks
  // it 32 positions at a time with ballots; offsets = totals of the earlier slices and warps.
  const int nwarps = nt >> 5;
  const int run = ((cs + nwarps - 1) / nwarps + 31) & ~31;       // positions per warp (multiple of 32)
  const int w0 = min(cs, warp * run), w1 = min(cs, w0 + run);
  int nl = 0, ne = 0;
  for (int i0 = w0; i0 < w1; i0 += 32) {
    const int i = i0 + lane;
    const uint32_t k = (i < w1) ? keys[i] : 0xffffffffu;
    nl += __popc(__ballot_sync(0xffffffffu, i < w1 && k < thr));
    ne += __popc(__ballot_sync(0xffffffffu, i < w1 && k == thr));
  }
  if (lane == 0) s_warp[warp] = nl | (ne << 16);       // a warp run holds fewer than 65536 positions
  __syncthreads();
  if (warp == 0) {
    const int v = (lane < nwarps) ? s_warp[lane] : 0;
    int vl = v & 0xffff, ve = v >> 16;
    int il = vl, ie = ve;
    for (int o = 1; o < 32; o <<= 1) {
      const int a = __shfl_up_sync(0xffffffffu, il, o), b = __shfl_up_sync(0xffffffffu, ie, o);
      if (lane >= o) { il += a; ie += b; }
    }
    s_hist[lane] = il - vl;                            // exclusive offsets per warp (s_hist is free now)
    s_hist[32 + lane] = ie - ve;
    if (lane == 31) { s_counts[0] = il; s_counts[1] = ie; }
  }
  if (csize > 1) cluster.sync(); else __syncthreads();
  int less_before = s_hist[warp], eq_before = s_hist[32 + warp];
  for (int r = 0; r < crank; ++r) {                     // totals of the earlier slices of the cluster
    const int* rc = cluster.map_shared_rank(s_counts, r);
    less_before += rc[0];
    eq_before += rc[1];
  }
  const unsigned lt_mask = (1u << lane) - 1u;
  for (int i0 = w0; i0 < w1; i0 += 32) {
    const int i = i0 + lane;
    const bool ok = i < w1;
    const uint32_t k = ok ? keys[i] : 0xffffffffu;
    const bool is_less = ok && k < thr, is_eq = ok && k == thr;
    const unsigned bl = __ballot_sync(0xffffffffu, is_less), be = __ballot_sync(0xffffffffu, is_eq);
    if (ok) {
      const int less_here = less_before + __popc(bl & lt_mask);
      const int eq_here = eq_before + __popc(be & lt_mask);
      const bool down = is_less || (is_eq && eq_here < eq_left);
      const int down_before = less_here + min(eq_here, eq_left);
      const int row = in_smem ? s_rows[i] : (pin ? pin[lo + c0 + i] : lo + c0 + i);
      const int dst = down ? lo + down_before : lo + L + (c0 + i - down_before);
      pout[dst] = row;
    }
    less_before += __popc(bl);
    eq_before += __popc(be);
  }
  if (csize > 1) cluster.sync();                     // keep shared memory alive for the peers' reads
}

// ---------------------------------------------------------------------------
// Subtree of a set of at most kTailRowsMax rows, finished by one CTA.
// ---------------------------------------------------------------------------
struct TailSmem {
  int32_t rows[2][kTailRowsMax];
  uint32_t keys[kTailRowsMax];
  uint32_t scan[kTailRowsMax];            // inclusive (less | equal << 16) counts over positions
  int hist[kTailSegs][256];
  int seg_lo[2][2 * kTailSegs + 2];       // start of each subset (relative), +1 sentinel
  int seg_coord[kTailSegs], seg_digit[kTailSegs], seg_rem[kTailSegs], seg_L[kTailSegs];
  int seg_cand[kTailSegs];                // candidates left after the first two digits; -1: threshold found
  int overflow;                           // some subset has more candidates than a warp takes
  uint32_t seg_prefix[kTailSegs];
  float vpart[4 * 8 * 64];                // partial sums of the variance stage ([ng][8][D])
  float vout[4 * 64];
  int sub_rows[4 * 64];                    // subsample rows of the subsets being staged                     // means / variances ([ng][D])
  float best[kTailSegs][4];
  int arg[kTailSegs][4];
  int warp_tot[32];
  int nseg[2];
  int more;
};

// Selection and partition of one level of a subtree, all of its subsets side by side: radix
// selection of every subset's threshold key (seg_L, seg_rem, seg_prefix set up by the caller), then
// the stable partition into rows_next.  A thread owns the four consecutive positions 4 tid .. 4 tid + 3
// (my_seg: subset of a position, -1 - g in a final subset, INT_MIN past the end; my_key: its key).
template <typename Smem>
__device__ __forceinline__ void tail_select_partition(Smem& sm, const int (&my_seg)[kTailRowsMax / kSplitThreads],
                                                      const uint32_t (&my_key)[kTailRowsMax / kSplitThreads],
                                                      int nseg, const int* slo, const int32_t* rows,
                                                      int32_t* rows_next, int tid, int* hist, uint32_t* scan) {
  constexpr int nt = kSplitThreads;
  constexpr int PT = kTailRowsMax / kSplitThreads;
  const int lane = tid & 31, warp = tid >> 5;
  // ---- radix selection, all subsets side by side: two digits of eight bits by counting; then the
  // keys that share those sixteen bits with the threshold are few (a handful per subset unless keys
  // repeat), and a warp ranks them directly.  A subset with more than 32 of them goes on with the two
  // remaining digits.  (The digit counts are cleared once per level: the warp that picks a subset's
  // digit clears the counts it has read, ready for the next pass.)
  uint32_t mask = 0;
  for (int e = tid; e < nseg * 256; e += nt) hist[e] = 0;
  if (tid < nseg) sm.seg_cand[tid] = 0;
  if (tid == 0) sm.overflow = 0;
  __syncthreads();
  for (int shift = 24; shift >= 0; shift -= 8) {
    uint32_t pre[PT];                               // read ahead of the atomics, which order memory accesses
#pragma unroll
    for (int u = 0; u < PT; ++u) pre[u] = sm.seg_prefix[my_seg[u] >= 0 ? my_seg[u] : 0];
    if (shift == 8) {
      // candidates of every subset into its list (the scan array is free until the partition)
#pragma unroll
      for (int u = 0; u < PT; ++u) {
        const int g = my_seg[u];
        if (g >= 0 && (my_key[u] & mask) == pre[u]) {
          const int slot = atomicAdd(&sm.seg_cand[g], 1);
          if (slot < 32) scan[g * 32 + slot] = my_key[u];
        }
      }
      __syncthreads();
      for (int g = warp; g < nseg; g += nt / 32) {
        if (sm.seg_L[g] == 0) continue;             // warp-uniform
        const int n = sm.seg_cand[g];
        if (n > 32) {
          if (lane == 0) sm.overflow = 1;
          continue;
        }
        const int remaining = sm.seg_rem[g];        // 1 <= remaining <= n
        const uint32_t key = lane < n ? scan[g * 32 + lane] : 0xffffffffu;
        int less = 0, eq_before = 0;
        for (int j = 0; j < n; ++j) {
          const uint32_t kj = __shfl_sync(0xffffffffu, key, j);
          less += kj < key ? 1 : 0;
          eq_before += (kj == key && j < lane) ? 1 : 0;
        }
        if (lane < n && less + eq_before == remaining - 1) {   // exactly one lane
          sm.seg_prefix[g] = key;
          sm.seg_rem[g] = remaining - less;          // how many of the keys equal to the threshold go down
          sm.seg_cand[g] = -1;
        }
      }
      __syncthreads();
      if (!sm.overflow) break;                      // uniform: every threshold is found
#pragma unroll
      for (int u = 0; u < PT; ++u) pre[u] = sm.seg_prefix[my_seg[u] >= 0 ? my_seg[u] : 0];
    }
#pragma unroll
    for (int u = 0; u < PT; ++u) {
      const int g = my_seg[u];
      const bool live = g >= 0;
      const uint32_t k = my_key[u];
      if (live && ((k & mask) == pre[u])) atomicAdd(&hist[(g << 8) | (int)((k >> shift) & 255u)], 1);
    }
    __syncthreads();
    for (int g = warp; g < nseg; g += nt / 32) {
      const int remaining = sm.seg_rem[g];
      if (sm.seg_L[g] == 0) continue;               // warp-uniform
      int local[8]; int sum = 0;
      {
        int4* h4 = reinterpret_cast<int4*>(&hist[g * 256 + lane * 8]);
        const int4 h0 = h4[0], h1 = h4[1];
        h4[0] = make_int4(0, 0, 0, 0);
        h4[1] = make_int4(0, 0, 0, 0);
        local[0] = h0.x; local[1] = h0.y; local[2] = h0.z; local[3] = h0.w;
        local[4] = h1.x; local[5] = h1.y; local[6] = h1.z; local[7] = h1.w;
      }
      if (sm.seg_cand[g] < 0) continue;             // found by the direct ranking (its keys were still counted)
#pragma unroll
      for (int j = 0; j < 8; ++j) sum += local[j];
      int incl = sum;
      for (int o = 1; o < 32; o <<= 1) {
        const int v = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += v;
      }
      int before = incl - sum;
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        if (before < remaining && remaining <= before + local[j]) {
          sm.seg_digit[g] = lane * 8 + j;
          sm.seg_rem[g] = remaining - before;
        }
        before += local[j];
      }
      __syncwarp();
      if (lane == 0) sm.seg_prefix[g] |= (uint32_t)sm.seg_digit[g] << shift;
    }
    mask |= 255u << shift;
    __syncthreads();
  }

  // ---- 3. stable partition of every subset: one scan of (less | equal << 16) over all positions
  // (a thread's four, then the warp, then the warps' totals by warp 0)
  uint32_t my_scan[PT];
  {
    int run = 0;
#pragma unroll
    for (int u = 0; u < PT; ++u) {
      if (my_seg[u] >= 0) {
        const uint32_t k = my_key[u], thr = sm.seg_prefix[my_seg[u]];
        run += (k < thr ? 1 : 0) | (k == thr ? 1 << 16 : 0);
      }
      my_scan[u] = (uint32_t)run;
    }
    int incl = run;
    for (int o = 1; o < 32; o <<= 1) {
      const int v = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += v;
    }
    if (lane == 31) sm.warp_tot[warp] = incl;
    __syncthreads();
    if (warp == 0) {
      const int v = sm.warp_tot[lane];                 // nt / 32 == 32 warps
      int wi = v;
      for (int o = 1; o < 32; o <<= 1) {
        const int x = __shfl_up_sync(0xffffffffu, wi, o);
        if (lane >= o) wi += x;
      }
      sm.warp_tot[lane] = wi - v;                      // totals of the warps before this one
    }
    __syncthreads();
    const uint32_t before = (uint32_t)(sm.warp_tot[warp] + incl - run);
#pragma unroll
    for (int u = 0; u < PT; ++u) my_scan[u] += before;
    *reinterpret_cast<uint4*>(&scan[PT * tid]) = make_uint4(my_scan[0], my_scan[1], my_scan[2], my_scan[3]);
    __syncthreads();
  }
#pragma unroll
  for (int u = 0; u < PT; ++u) {
    const int i = PT * tid + u;
    const int g = my_seg[u];
    if (g == INT_MIN) continue;
    if (g < 0) { rows_next[i] = rows[i]; continue; }
    const int a = slo[g];
    const uint32_t base = a > 0 ? scan[a - 1] : 0u;
    const uint32_t k = my_key[u], thr = sm.seg_prefix[g];
    const int is_less = k < thr, is_eq = k == thr;
    const uint32_t excl = my_scan[u] - base - (uint32_t)(is_less | (is_eq << 16));
    const int less_here = (int)(excl & 0xffffu), eq_here = (int)(excl >> 16);
    const int eq_left = sm.seg_rem[g], L = sm.seg_L[g];
    const bool down = is_less || (is_eq && eq_here < eq_left);
    const int down_before = less_here + min(eq_here, eq_left);
    const int dst = down ? a + down_before : a + L + (i - a - down_before);
    rows_next[dst] = rows[i];
  }
}

template <int D>
__global__ void __launch_bounds__(kSplitThreads) split_tail_kernel(const SplitParams prm) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  TailSmem& sm = *reinterpret_cast<TailSmem*>(smem_raw);
  const int which = blockIdx.y / prm.problems;
  const int p = blockIdx.y % prm.problems;
  const SplitSide sd = prm.side[which];
  const int level = sd.tail_level;
  if (!sd.active || (int)blockIdx.x >= (1 << level)) return;
  const SegmentRef root = locate_segment(sd.n, sd.c, level, blockIdx.x);
  if (!root.active) return;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  constexpr int nt = kSplitThreads;
  const int c = sd.c;
  const float* Y = sd.Y + (size_t)p * sd.n * D;
  const float* Yt = sd.Yt ? sd.Yt + (size_t)p * sd.n * D : nullptr;
  const int32_t* pin = sd.perm_in ? sd.perm_in + (size_t)p * sd.n : nullptr;
  int32_t* pout = sd.perm_out + (size_t)p * sd.n;
  const int lo = root.lo, s0 = root.size;

  for (int i = tid; i < s0; i += nt) sm.rows[0][i] = pin ? pin[lo + i] : lo + i;
  if (tid == 0) { sm.seg_lo[0][0] = 0; sm.seg_lo[0][1] = s0; sm.nseg[0] = 1; sm.more = s0 > c; }
  __syncthreads();

  int cur = 0;
  constexpr int wps = D / 32;                            // warps per (subset, all coordinates)
  while (sm.more) {
    const int nseg = sm.nseg[cur];
    const int* slo = sm.seg_lo[cur];
    const int32_t* rows = sm.rows[cur];
    int32_t* rows_next = sm.rows[cur ^ 1];

    // ---- 1. coordinate of largest subsample variance for every subset that still splits.
    // Rounds of up to 1024 / D subsets: their sample rows are located (one division per row), then
    // every (subset, residue, coordinate) is a thread's task that reads its sample values straight
    // from the coordinates; partial sums, means and variances live in the 64 KB that keys, scan and
    // hist occupy later in the level.
    {
      float* part = reinterpret_cast<float*>(sm.keys);                 // [G][8][D]
      constexpr int G = 1024 / D;
      float* vout = part + G * 8 * D;                                  // [G][D] means, then variances
      int* sub_rows = reinterpret_cast<int*>(vout + G * D);            // [G][D]
      for (int g0 = 0; g0 < nseg; g0 += G) {
        const int ng = min(G, nseg - g0);
        for (int e = tid; e < ng * D; e += nt) {
          const int gi = e / D, j = e % D;
          const int a = slo[g0 + gi], sz = slo[g0 + gi + 1] - a;
          const int m = min(D, sz);
          // residue-major: sample j sits at (j % 8) * (D / 8) + j / 8 of its subset's D entries
          sub_rows[gi * D + (j & 7) * (D / 8) + (j >> 3)] =
              (sz > c && j < m) ? rows[a + (int)(((unsigned)j * (unsigned)sz) / (unsigned)m)] : -1;
        }
        __syncthreads();
        gathered_variances<D>(Y, sub_rows, ng,
                              [&](int gi) { const int sz = slo[g0 + gi + 1] - slo[g0 + gi]; return sz > c ? min(D, sz) : 0; },
                              part, vout, tid, nt);
        for (int task = tid; task < ng * D; task += nt) {
          const int gi = task / D, t = task % D, g = g0 + gi;
          float v = vout[task];                        // -1 for a subset that is already final
          // argmax inside the warp (32 consecutive coordinates), lowest coordinate on ties
          int at = t;
          for (int o = 16; o > 0; o >>= 1) {
            const float ov = __shfl_xor_sync(0xffffffffu, v, o);
            const int oa = __shfl_xor_sync(0xffffffffu, at, o);
            if (ov > v || (ov == v && oa < at)) { v = ov; at = oa; }
          }
          if (lane == 0) { sm.best[g][(t / 32)] = v; sm.arg[g][(t / 32)] = at; }
        }
        __syncthreads();
      }
    }
    if (tid < nseg) {
      const int a = slo[tid], sz = slo[tid + 1] - a;
      float v = sm.best[tid][0]; int at = sm.arg[tid][0];
      for (int w = 1; w < wps; ++w)
        if (sm.best[tid][w] > v) { v = sm.best[tid][w]; at = sm.arg[tid][w]; }   // later warps hold higher coordinates
      sm.seg_coord[tid] = at;
      sm.seg_L[tid] = sz > c ? c * ((sz + c) / (2 * c)) : 0;
      sm.seg_prefix[tid] = 0u;
      sm.seg_rem[tid] = sm.seg_L[tid];
    }
    __syncthreads();

    // ---- 2. keys.  A thread owns four consecutive positions for the rest of the level (their
    // keys stay in registers); the first finds its subset by bisection of the start offsets, the
    // others walk on from there.
    constexpr int PT = kTailRowsMax / kSplitThreads;     // positions per thread
    static_assert(PT == 4 && kSplitThreads == 1024, "the scan below stores four counts per thread and scans 32 warp totals");
    int my_seg[PT];
    uint32_t my_key[PT];
    {
      const int i0 = PT * tid;
      int g = 0;
      if (i0 < s0) {
        int hi = nseg;                                  // slo[g] <= i0 < slo[g+1]
        while (hi - g > 1) { const int mid = (g + hi) >> 1; if (slo[mid] <= i0) g = mid; else hi = mid; }
      }
#pragma unroll
      for (int u = 0; u < PT; ++u) {
        const int i = i0 + u;
        my_key[u] = 0u;
        if (i < s0) {
          while (slo[g + 1] <= i) ++g;
          const bool splits = slo[g + 1] - slo[g] > c;
          if (splits) my_key[u] = order_key(Yt ? __ldg(Yt + (size_t)sm.seg_coord[g] * sd.n + rows[i])
                                               : __ldg(Y + (size_t)rows[i] * D + sm.seg_coord[g]));
          my_seg[u] = splits ? g : -1 - g;              // final subset: carried over unchanged
        } else {
          my_seg[u] = INT_MIN;
        }
      }
    }

    tail_select_partition(sm, my_seg, my_key, nseg, slo, rows, rows_next, tid, &sm.hist[0][0], sm.scan);
    // ---- next level's subsets
    if (tid == 0) {
      int* nlo = sm.seg_lo[cur ^ 1];
      int n2 = 0, more = 0;
      for (int g = 0; g < nseg; ++g) {
        const int a = slo[g], sz = slo[g + 1] - a;
        nlo[n2++] = a;
        if (sz > c) {
          const int L = sm.seg_L[g];
          nlo[n2++] = a + L;
          more |= (L > c) | (sz - L > c);
        }
      }
      nlo[n2] = s0;
      sm.nseg[cur ^ 1] = n2;
      sm.more = more;
    }
    __syncthreads();
    cur ^= 1;
  }
  for (int i = tid; i < s0; i += nt) pout[lo + i] = sm.rows[cur][i];
}

// ---------------------------------------------------------------------------
// host side
// ---------------------------------------------------------------------------
static int next_size(int big, int c) {
  const int L = c * ((big + c) / (2 * c));
  return (L > big - L) ? L : big - L;
}

int split_levels_for(int n, int c) {
  int levels = 0;
  for (int big = n; big > c; big = next_size(big, c)) ++levels;   // the largest set follows the larger child
  return levels;
}

static int max_segment_at_level(int n, int c, int level) {
  int big = n;
  for (int l = 0; l < level && big > c; ++l) big = next_size(big, c);
  return big;
}

static int tail_rows_for(int c) {
  const int r = kTailSegs * c;
  return r < kTailRowsMax ? r : kTailRowsMax;
}

// Levels [0, tail_level) run as per-level launches; the tail kernel finishes the rest.
static int tail_level_for(int n, int c) {
  int level = 0;
  for (int big = n; big > tail_rows_for(c); big = next_size(big, c)) ++level;
  return level;
}

int split_top_levels_for(int n, int c) { return tail_level_for(n, c); }

int launch_split(const float* Yq, const float* Yk, int problems, int D, int n_q, int n_k, int c_q,
                 int c_k, int32_t* perm_q_out, int32_t* perm_q_tmp, int32_t* perm_k_out,
                 int32_t* perm_k_tmp, uint32_t* keybuf_q, uint32_t* keybuf_k, int sides, cudaStream_t st,
                 const float* Ytq, const float* Ytk) {
  // sides: bit 0 = queries, bit 1 = keys
  auto level_kernel = D == 64 ? split_level_kernel<64> : split_level_kernel<128>;
  auto tail_kernel = D == 64 ? split_tail_kernel<64> : split_tail_kernel<128>;
  CA_RETURN_IF_CUDA(cudaFuncSetAttribute(level_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemRowsMax * 8));
  CA_RETURN_IF_CUDA(cudaFuncSetAttribute(tail_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         (int)sizeof(TailSmem)));
  const bool do_q = (sides & 1) != 0, do_k = (sides & 2) != 0;
  const int tail_q = tail_level_for(n_q, c_q), tail_k = tail_level_for(n_k, c_k);
  const int top_q = do_q ? tail_q : 0, top_k = do_k ? tail_k : 0;
  const int top_levels = top_q > top_k ? top_q : top_k;
  SplitParams prm;
  prm.D = D; prm.problems = problems; prm.keys_in = 0;
  // per-level launches write alternately to tmp/out so that the tail kernel, which runs last,
  // reads the buffer that is not the output
  auto fill = [&](int level) {
    for (int w = 0; w < 2; ++w) {
      SplitSide& sd = prm.side[w];
      int32_t* out = w == 0 ? perm_q_out : perm_k_out;
      int32_t* tmp = w == 0 ? perm_q_tmp : perm_k_tmp;
      const int tail = w == 0 ? tail_q : tail_k;
      sd.Y = w == 0 ? Yq : Yk;
      sd.Yt = w == 0 ? Ytq : Ytk;
      sd.keybuf = w == 0 ? keybuf_q : keybuf_k;
      sd.n = w == 0 ? n_q : n_k; sd.c = w == 0 ? c_q : c_k;
      sd.levels = split_levels_for(sd.n, sd.c);
      sd.tail_level = tail;
      sd.active = (w == 0 ? do_q : do_k) ? 1 : 0;
      // level l of this side (l < tail) writes tmp if (tail - 1 - l) is even, else out;
      // the tail kernel (level == tail) reads what level tail-1 wrote and writes out
      const bool to_tmp = ((tail - 1 - level) % 2) == 0;
      if (level < tail) {
        sd.perm_out = to_tmp ? tmp : out;
        sd.perm_in = level == 0 ? nullptr : (to_tmp ? out : tmp);
      } else {
        sd.perm_out = out;
        sd.perm_in = tail == 0 ? nullptr : tmp;
      }
    }
  };
  if (top_levels > 0 && prof_enabled()) prof_mark(kProfSplitLevels, st, true);
  for (int level = 0; level < top_levels; ++level) {
    fill(level);
    prm.level = level;
    int max_seg = 1;
    if (level < top_q) max_seg = max_segment_at_level(n_q, c_q, level);
    if (level < top_k) { const int ms = max_segment_at_level(n_k, c_k, level); if (ms > max_seg) max_seg = ms; }
    int csize = 1;
    while (csize < kMaxCluster && max_seg > csize * 16384) csize *= 2;
    const int per_cta = (max_seg + csize - 1) / csize;
    prm.smem_rows = per_cta < kSmemRowsMax ? per_cta : kSmemRowsMax;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((1u << level) * csize, 2 * problems);
    cfg.blockDim = dim3(kSplitThreads);
    // keys + rows of the slice; the same space first stages the d x d subsample tile
    cfg.dynamicSmemBytes = (size_t)prm.smem_rows * 8 > (size_t)D * D * 4 ? (size_t)prm.smem_rows * 8 : (size_t)D * D * 4;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = csize; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    CA_RETURN_IF_CUDA(cudaLaunchKernelEx(&cfg, level_kernel, prm));
    CA_LAUNCH_CHECK();
  }
  if (top_levels > 0 && prof_enabled()) prof_mark(kProfSplitLevels, st, false);
  ProfScope ps(kProfSplitTail, st);
  fill(top_levels);       // any level >= both tails selects the tail buffers
  prm.level = top_levels;
  prm.smem_rows = 0;
  const int slots = 1 << ((do_q ? tail_q : 0) > (do_k ? tail_k : 0) ? (do_q ? tail_q : 0) : (do_k ? tail_k : 0));
  tail_kernel<<<dim3(slots, 2 * problems), kSplitThreads, sizeof(TailSmem), st>>>(prm);
  CA_LAUNCH_CHECK();
  return CA_OK;
}

// ---------------------------------------------------------------------------
// Basic recursive splitting (Section 3.2.1) with the metric injected into the
// power iteration (Section 5.2): per set, the first principal direction of a
// subsample in the metric A, in the dual form u <- A C u, then the projection
// x . u of every row of the set as the key of the same select-and-partition step.
// Every floating-point step is float32 with sequential sums (each product and
// sum rounded on its own), because the projections decide the partition:
//   subsample m = min(d, s) rows at positions floor(j s / m); mu_k = (sum_i x_ik) / m;
//   z = x - mu; start g / |g| (root) or (u_parent + g / |g|) / 2, g the node's noise row;
//   iteration: v_i = sum_k z_ik u_k; w_k = sum_i z_ik v_i; y_j = sum_k A_jk w_k; u = y / |y|.
// Nodes are numbered 2^level - 1 + slot.
// ---------------------------------------------------------------------------
struct BasicSide {
  const void* X;           // [P][n][D] rows in the storage type
  const float* A;          // [P][D][D] metric
  const float* noise;      // [P][nodes][D]
  float* dirs;             // [P][nodes][D] directions of every node (output, read by the children)
  const int32_t* perm_in;  // [P][n] or null (identity)
  uint32_t* keybuf;        // [P][n]
  int n, c, levels, nodes;
};
struct BasicParams {
  BasicSide side[2];
  int level, problems, iterations;
};

__device__ __forceinline__ float seq_norm(const float* v, int d) {
  // d is a multiple of 8; the squares are formed eight at a time and added in order
  float s = 0.f;
#pragma unroll 1
  for (int j0 = 0; j0 < d; j0 += 8) {
    float sq[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) sq[j] = __fmul_rn(v[j0 + j], v[j0 + j]);
#pragma unroll
    for (int j = 0; j < 8; ++j) s = __fadd_rn(s, sq[j]);
  }
  return __fsqrt_rn(s);
}

// One CTA of D threads per (slot, side, head).
template <typename T, int D>
__global__ void __launch_bounds__(D) basic_direction_kernel(const BasicParams prm) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  float* z = reinterpret_cast<float*>(smem_raw);       // [m][D + 1]
  __shared__ float u[D], v[D], w[D], y[D], g[D];
  constexpr int LD = D + 1;
  const int which = blockIdx.y / prm.problems, p = blockIdx.y % prm.problems;
  const BasicSide sd = prm.side[which];
  if (prm.level >= sd.levels) return;
  const SegmentRef seg = locate_segment(sd.n, sd.c, prm.level, blockIdx.x);
  if (!seg.active || seg.size <= sd.c) return;
  const int tid = threadIdx.x;
  const int s = seg.size, lo = seg.lo, m = min(D, s);
  const T* X = static_cast<const T*>(sd.X) + (size_t)p * sd.n * D;
  const int32_t* pin = sd.perm_in ? sd.perm_in + (size_t)p * sd.n : nullptr;
  const int node = (1 << prm.level) - 1 + (int)blockIdx.x;
  // subsample rows, one row per thread, then centred column by column
  if (tid < m) {
    const int pos = lo + (int)(((long long)tid * s) / m);
    const int row = pin ? pin[pos] : pos;
    const T* xr = X + (size_t)row * D;
    if (sizeof(T) == 2) {                                // 16-byte loads, all in flight together
      uint4 q[D / 8];
#pragma unroll
      for (int k8 = 0; k8 < D / 8; ++k8) q[k8] = __ldg(reinterpret_cast<const uint4*>(xr) + k8);
#pragma unroll
      for (int k8 = 0; k8 < D / 8; ++k8) {
        const uint32_t wds[4] = {q[k8].x, q[k8].y, q[k8].z, q[k8].w};
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          z[tid * LD + k8 * 8 + 2 * e] = __uint_as_float(wds[e] << 16);
          z[tid * LD + k8 * 8 + 2 * e + 1] = __uint_as_float(wds[e] & 0xffff0000u);
        }
      }
    } else {
#pragma unroll 8
      for (int k4 = 0; k4 < D / 4; ++k4) {
        const float4 q = __ldg(reinterpret_cast<const float4*>(xr) + k4);
        z[tid * LD + k4 * 4] = q.x; z[tid * LD + k4 * 4 + 1] = q.y;
        z[tid * LD + k4 * 4 + 2] = q.z; z[tid * LD + k4 * 4 + 3] = q.w;
      }
    }
  }
  g[tid] = sd.noise[((size_t)p * sd.nodes + node) * D + tid];
  __syncthreads();
  {
    float mu = 0.f;                                      // thread k: column k, rows in order
    for (int i = 0; i < m; ++i) mu = __fadd_rn(mu, z[i * LD + tid]);
    mu = __fdiv_rn(mu, (float)m);
    for (int i = 0; i < m; ++i) z[i * LD + tid] = __fsub_rn(z[i * LD + tid], mu);
    const float gn = __fdiv_rn(g[tid], seq_norm(g, D));
    float start = gn;
    if (prm.level > 0) {
      const int parent = (1 << (prm.level - 1)) - 1 + ((int)blockIdx.x >> 1);
      start = __fmul_rn(__fadd_rn(sd.dirs[((size_t)p * sd.nodes + parent) * D + tid], gn), 0.5f);
    }
    u[tid] = start;
  }
  __syncthreads();
  for (int it = 0; it < prm.iterations; ++it) {
    if (tid < m) {
      float acc = 0.f;
      for (int k = 0; k < D; ++k) acc = __fadd_rn(acc, __fmul_rn(z[tid * LD + k], u[k]));
      v[tid] = acc;
    }
    __syncthreads();
    {
      float acc = 0.f;
      for (int i = 0; i < m; ++i) acc = __fadd_rn(acc, __fmul_rn(z[i * LD + tid], v[i]));
      w[tid] = acc;
    }
    __syncthreads();
    {
      const float* Ar = sd.A + ((size_t)p * D + tid) * D;
      float acc = 0.f;
      for (int k = 0; k < D; ++k) acc = __fadd_rn(acc, __fmul_rn(Ar[k], w[k]));
      y[tid] = acc;
    }
    __syncthreads();
    const float nrm = seq_norm(y, D);                    // every thread takes the same sequential sum
    if (nrm > 0.f && isfinite(nrm)) u[tid] = __fdiv_rn(y[tid], nrm);
    __syncthreads();
  }
  sd.dirs[((size_t)p * sd.nodes + node) * D + tid] = u[tid];
}

// Keys of one level: one thread per position; the set of a position follows from the size rule.
template <typename T, int D>
__global__ void __launch_bounds__(256) basic_keys_kernel(const BasicParams prm) {
  const int which = blockIdx.y / prm.problems, p = blockIdx.y % prm.problems;
  const BasicSide sd = prm.side[which];
  if (prm.level >= sd.levels) return;
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= sd.n) return;
  int lo = 0, size = sd.n, slot = 0;
  for (int l = 0; l < prm.level; ++l) {
    if (size <= sd.c) return;                           // a final set: nothing to split at this level
    const int L = sd.c * ((size + sd.c) / (2 * sd.c));
    if (i < lo + L) { size = L; slot = 2 * slot; } else { lo += L; size -= L; slot = 2 * slot + 1; }
  }
  if (size <= sd.c) return;
  const int node = (1 << prm.level) - 1 + slot;
  const float* u = sd.dirs + ((size_t)p * sd.nodes + node) * D;
  const int row = sd.perm_in ? sd.perm_in[(size_t)p * sd.n + i] : i;
  const T* xr = static_cast<const T*>(sd.X) + ((size_t)p * sd.n + row) * D;
  float t = 0.f;
  if (sizeof(T) == 2) {
    const uint4* x4 = reinterpret_cast<const uint4*>(xr);
    for (int k8 = 0; k8 < D / 8; ++k8) {
      const uint4 q = __ldg(x4 + k8);
      const uint32_t wds[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const float a = __uint_as_float(wds[e] << 16), b = __uint_as_float(wds[e] & 0xffff0000u);
        t = __fadd_rn(t, __fmul_rn(a, __ldg(u + k8 * 8 + 2 * e)));
        t = __fadd_rn(t, __fmul_rn(b, __ldg(u + k8 * 8 + 2 * e + 1)));
      }
    }
  } else {
    const float4* x4 = reinterpret_cast<const float4*>(xr);
    for (int k4 = 0; k4 < D / 4; ++k4) {
      const float4 q = __ldg(x4 + k4);
      t = __fadd_rn(t, __fmul_rn(q.x, __ldg(u + k4 * 4)));
      t = __fadd_rn(t, __fmul_rn(q.y, __ldg(u + k4 * 4 + 1)));
      t = __fadd_rn(t, __fmul_rn(q.z, __ldg(u + k4 * 4 + 2)));
      t = __fadd_rn(t, __fmul_rn(q.w, __ldg(u + k4 * 4 + 3)));
    }
  }
  sd.keybuf[(size_t)p * sd.n + i] = order_key(t);
}

// ---------------------------------------------------------------------------
// Subtree of the basic variant: a set of at most kTailRowsMax rows finished by one CTA, so that
// the deepest levels are one launch instead of three per level.  Per level: the directions of all
// subsets that still split (a team of D threads per subset; the operations of
// basic_direction_kernel in the same order -- the sample rows are staged as stored and centred
// where they are used, which yields the same float32 values), the projection of every row onto its
// subset's direction (the sum of basic_keys_kernel), then the selection and partition of the
// diagonalized subtree kernel.
// ---------------------------------------------------------------------------
// staged sample rows (later the scan and the digit counts): 16 subsets of 64 bf16 rows at d = 64, 4 at d = 128
template <int D> struct BasicStage { static constexpr int BYTES = D == 64 ? 135168 : 133120; };

template <int D>
struct BasicTailSmem {
  static constexpr int TEAMS = kSplitThreads / D;
  int32_t rows[2][kTailRowsMax];
  __align__(16) unsigned char stage[BasicStage<D>::BYTES];
  float dirs[2][kTailSegs][D];            // directions of this level's subsets and of the level above
  float mu[TEAMS][D], u[TEAMS][D], v[TEAMS][D], w[TEAMS][D], y[TEAMS][D], g[TEAMS][D];
  int seg_lo[2][2 * kTailSegs + 2];
  int seg_slot[2][2 * kTailSegs + 2];     // slot of a subset in the tree, at the level it stands on
  int seg_par[2][2 * kTailSegs + 2];      // subset of the level above it came from
  int seg_digit[kTailSegs], seg_rem[kTailSegs], seg_L[kTailSegs];
  int seg_cand[kTailSegs];                // candidates left after the first two digits; -1: threshold found
  int overflow;                           // some subset has more candidates than a warp takes
  uint32_t seg_prefix[kTailSegs];
  int split_list[kTailSegs];              // the subsets that still split
  int warp_tot[32];
  int nseg[2];
  int nsplit;
  int more;
};

template <typename T>
__device__ __forceinline__ float stored_value(const T* p);
template <>
__device__ __forceinline__ float stored_value<float>(const float* p) { return *p; }
template <>
__device__ __forceinline__ float stored_value<__nv_bfloat16>(const __nv_bfloat16* p) { return __bfloat162float(*p); }

template <typename T, int D>
__global__ void __launch_bounds__(kSplitThreads) basic_tail_kernel(const BasicParams prm, const SplitParams sp) {
  using Sm = BasicTailSmem<D>;
  extern __shared__ __align__(16) unsigned char smem_raw[];
  Sm& sm = *reinterpret_cast<Sm*>(smem_raw);
  constexpr int nt = kSplitThreads;
  constexpr int LD = D + (sizeof(T) == 2 ? 2 : 1);      // row stride of the staged rows (elements): odd in 4-byte words
  constexpr int NODE_BYTES = D * LD * (int)sizeof(T);
  constexpr int ROUND = (BasicStage<D>::BYTES / NODE_BYTES) < Sm::TEAMS ? (BasicStage<D>::BYTES / NODE_BYTES) : Sm::TEAMS;
  static_assert(ROUND >= 1, "a subset's sample must fit the staging area");
  constexpr int PT = kTailRowsMax / kSplitThreads;
  static_assert(PT == 4 && kTailRowsMax * 4 + kTailSegs * 256 * 4 <= BasicStage<D>::BYTES, "scan and digit counts live in the staging area");
  uint32_t* scan = reinterpret_cast<uint32_t*>(sm.stage);
  int* hist = reinterpret_cast<int*>(sm.stage + kTailRowsMax * 4);

  const int which = blockIdx.y / prm.problems, p = blockIdx.y % prm.problems;
  const BasicSide bs = prm.side[which];
  const SplitSide sd = sp.side[which];
  const int level0 = sd.tail_level;
  if (!sd.active || (int)blockIdx.x >= (1 << level0)) return;
  const SegmentRef root = locate_segment(sd.n, sd.c, level0, blockIdx.x);
  if (!root.active) return;
  const int tid = threadIdx.x;
  const int team = tid / D, member = tid % D;
  const int c = sd.c;
  const T* X = static_cast<const T*>(bs.X) + (size_t)p * sd.n * D;
  const float* Am = bs.A + (size_t)p * D * D;
  const float* noise = bs.noise + (size_t)p * bs.nodes * D;
  const int32_t* pin = sd.perm_in ? sd.perm_in + (size_t)p * sd.n : nullptr;
  int32_t* pout = sd.perm_out + (size_t)p * sd.n;
  const int lo = root.lo, s0 = root.size;

  for (int i = tid; i < s0; i += nt) sm.rows[0][i] = pin ? pin[lo + i] : lo + i;
  if (tid == 0) {
    sm.seg_lo[0][0] = 0; sm.seg_lo[0][1] = s0; sm.nseg[0] = 1; sm.more = s0 > c;
    sm.seg_slot[0][0] = (int)blockIdx.x; sm.seg_par[0][0] = -1;
    sm.split_list[0] = 0; sm.nsplit = s0 > c ? 1 : 0;
  }
  __syncthreads();

  int cur = 0, level = level0;
  while (sm.more) {
    const int nseg = sm.nseg[cur];
    const int* slo = sm.seg_lo[cur];
    const int32_t* rows = sm.rows[cur];
    int32_t* rows_next = sm.rows[cur ^ 1];
    const int nsplit = sm.nsplit;
    float (*dir_now)[D] = sm.dirs[cur];
    float (*dir_up)[D] = sm.dirs[cur ^ 1];

    // ---- 1. directions, ROUND subsets at a time (every stage boundary is a barrier of the CTA; teams
    // without a subset go through them idle)
    for (int r0 = 0; r0 < nsplit; r0 += ROUND) {
      const bool active = team < ROUND && r0 + team < nsplit;
      const int g = active ? sm.split_list[r0 + team] : 0;
      const int a = slo[g], sz = slo[g + 1] - a, m = min(D, sz);
      T* xs = reinterpret_cast<T*>(sm.stage + (size_t)(team < ROUND ? team : 0) * NODE_BYTES);
      if (active) {
        if (member < m) {
          const int pos = a + (int)(((long long)member * sz) / m);
          const T* xr = X + (size_t)rows[pos] * D;
          uint32_t* dst = reinterpret_cast<uint32_t*>(xs + (size_t)member * LD);     // LD * sizeof(T) is a multiple of 4
          constexpr int V = D * (int)sizeof(T) / 16;                                 // 16-byte loads of a row
#pragma unroll
          for (int k0 = 0; k0 < V; k0 += 8) {
            uint4 q[8];
#pragma unroll
            for (int k = 0; k < 8; ++k) if (k0 + k < V) q[k] = __ldg(reinterpret_cast<const uint4*>(xr) + k0 + k);
#pragma unroll
            for (int k = 0; k < 8; ++k)
              if (k0 + k < V) {
                dst[(k0 + k) * 4 + 0] = q[k].x; dst[(k0 + k) * 4 + 1] = q[k].y;
                dst[(k0 + k) * 4 + 2] = q[k].z; dst[(k0 + k) * 4 + 3] = q[k].w;
              }
          }
        }
        const int node = (1 << level) - 1 + sm.seg_slot[cur][g];
        sm.g[team][member] = noise[(size_t)node * D + member];
      }
      __syncthreads();
      if (active) {
        float mu = 0.f;                                      // column `member`, rows in order
        for (int i = 0; i < m; ++i) mu = __fadd_rn(mu, stored_value(xs + i * LD + member));
        mu = __fdiv_rn(mu, (float)m);
        sm.mu[team][member] = mu;
        const float gn = __fdiv_rn(sm.g[team][member], seq_norm(sm.g[team], D));
        float start = gn;
        if (level > 0) {
          const int par = sm.seg_par[cur][g];
          const float up = par >= 0 ? dir_up[par][member]
                                    : bs.dirs[((size_t)p * bs.nodes + (1 << (level - 1)) - 1 + (sm.seg_slot[cur][g] >> 1)) * D + member];
          start = __fmul_rn(__fadd_rn(up, gn), 0.5f);
        }
        sm.u[team][member] = start;
      }
      __syncthreads();
      for (int it = 0; it < prm.iterations; ++it) {
        if (active && member < m) {
          // (terms formed eight at a time, then added in order: the loads do not wait for the sum)
          float acc = 0.f;
#pragma unroll 1
          for (int k0 = 0; k0 < D; k0 += 8) {
            float term[8];
#pragma unroll
            for (int k = 0; k < 8; ++k)
              term[k] = __fmul_rn(__fsub_rn(stored_value(xs + member * LD + k0 + k), sm.mu[team][k0 + k]), sm.u[team][k0 + k]);
#pragma unroll
            for (int k = 0; k < 8; ++k) acc = __fadd_rn(acc, term[k]);
          }
          sm.v[team][member] = acc;
        }
        __syncthreads();
        if (active) {
          const float mk = sm.mu[team][member];
          float acc = 0.f;
          int i = 0;
#pragma unroll 1
          for (; i + 8 <= m; i += 8) {
            float term[8];
#pragma unroll
            for (int k = 0; k < 8; ++k)
              term[k] = __fmul_rn(__fsub_rn(stored_value(xs + (i + k) * LD + member), mk), sm.v[team][i + k]);
#pragma unroll
            for (int k = 0; k < 8; ++k) acc = __fadd_rn(acc, term[k]);
          }
          for (; i < m; ++i)
            acc = __fadd_rn(acc, __fmul_rn(__fsub_rn(stored_value(xs + i * LD + member), mk), sm.v[team][i]));
          sm.w[team][member] = acc;
        }
        __syncthreads();
        if (active) {
          const float4* Ar = reinterpret_cast<const float4*>(Am + (size_t)member * D);
          float acc = 0.f;
#pragma unroll 1
          for (int k0 = 0; k0 < D; k0 += 8) {
            const float4 a0 = __ldg(Ar + k0 / 4), a1 = __ldg(Ar + k0 / 4 + 1);
            const float av[8] = {a0.x, a0.y, a0.z, a0.w, a1.x, a1.y, a1.z, a1.w};
            float term[8];
#pragma unroll
            for (int k = 0; k < 8; ++k) term[k] = __fmul_rn(av[k], sm.w[team][k0 + k]);
#pragma unroll
            for (int k = 0; k < 8; ++k) acc = __fadd_rn(acc, term[k]);
          }
          sm.y[team][member] = acc;
        }
        __syncthreads();
        if (active) {
          const float nrm = seq_norm(sm.y[team], D);          // every thread takes the same sequential sum
          if (nrm > 0.f && isfinite(nrm)) sm.u[team][member] = __fdiv_rn(sm.y[team][member], nrm);
        }
        __syncthreads();
      }
      if (active) dir_now[g][member] = sm.u[team][member];
      __syncthreads();
    }
    if (tid < nseg) {
      const int a = slo[tid], sz = slo[tid + 1] - a;
      sm.seg_L[tid] = sz > c ? c * ((sz + c) / (2 * c)) : 0;
      sm.seg_prefix[tid] = 0u;
      sm.seg_rem[tid] = sm.seg_L[tid];
    }

    // ---- 2. keys: the projection of a row onto its subset's direction, terms in the order of the columns
    int my_seg[PT];
    uint32_t my_key[PT];
    {
      const int i0 = PT * tid;
      int g = 0;
      if (i0 < s0) {
        int hi = nseg;                                  // slo[g] <= i0 < slo[g+1]
        while (hi - g > 1) { const int mid = (g + hi) >> 1; if (slo[mid] <= i0) g = mid; else hi = mid; }
      }
#pragma unroll 1
      for (int u = 0; u < PT; ++u) {
        const int i = i0 + u;
        my_key[u] = 0u;
        if (i < s0) {
          while (slo[g + 1] <= i) ++g;
          const bool splits = slo[g + 1] - slo[g] > c;
          if (splits) {
            const T* xr = X + (size_t)rows[i] * D;
            const float* uu = dir_now[g];
            float t = 0.f;
            constexpr int E = 16 / (int)sizeof(T);       // elements of a 16-byte load
#pragma unroll
            for (int k0 = 0; k0 < D; k0 += 4 * E) {      // four loads in flight, then their terms in order
              uint4 q[4];
#pragma unroll
              for (int k = 0; k < 4; ++k) q[k] = __ldg(reinterpret_cast<const uint4*>(xr + k0) + k);
#pragma unroll
              for (int k = 0; k < 4; ++k) {
                const uint32_t wds[4] = {q[k].x, q[k].y, q[k].z, q[k].w};
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                  if (sizeof(T) == 2) {
                    const float x0 = __uint_as_float(wds[e] << 16), x1 = __uint_as_float(wds[e] & 0xffff0000u);
                    t = __fadd_rn(t, __fmul_rn(x0, uu[k0 + k * E + 2 * e]));
                    t = __fadd_rn(t, __fmul_rn(x1, uu[k0 + k * E + 2 * e + 1]));
                  } else {
                    t = __fadd_rn(t, __fmul_rn(__uint_as_float(wds[e]), uu[k0 + k * E + e]));
                  }
                }
              }
            }
            my_key[u] = order_key(t);
          }
          my_seg[u] = splits ? g : -1 - g;              // final subset: carried over unchanged
        } else {
          my_seg[u] = INT_MIN;
        }
      }
    }
    __syncthreads();                                    // the staging area becomes the scan and the digit counts

    tail_select_partition(sm, my_seg, my_key, nseg, slo, rows, rows_next, tid, hist, scan);

    // ---- next level's subsets
    if (tid == 0) {
      int* nlo = sm.seg_lo[cur ^ 1];
      int* nslot = sm.seg_slot[cur ^ 1];
      int* npar = sm.seg_par[cur ^ 1];
      int n2 = 0, more = 0, ns = 0;
      for (int g = 0; g < nseg; ++g) {
        const int a = slo[g], sz = slo[g + 1] - a;
        if (sz > c) {
          const int L = sm.seg_L[g];
          nlo[n2] = a;     nslot[n2] = 2 * sm.seg_slot[cur][g];     npar[n2] = g;
          if (L > c) sm.split_list[ns++] = n2;
          ++n2;
          nlo[n2] = a + L; nslot[n2] = 2 * sm.seg_slot[cur][g] + 1; npar[n2] = g;
          if (sz - L > c) sm.split_list[ns++] = n2;
          ++n2;
          more |= (L > c) | (sz - L > c);
        } else {
          nlo[n2] = a; nslot[n2] = 0; npar[n2] = g;      // a final subset: only carried along
          ++n2;
        }
      }
      nlo[n2] = s0;
      sm.nseg[cur ^ 1] = n2;
      sm.nsplit = ns;
      sm.more = more;
    }
    __syncthreads();
    cur ^= 1;
    ++level;
  }
  for (int i = tid; i < s0; i += nt) pout[lo + i] = sm.rows[cur][i];
}

template <typename T>
static int launch_split_basic_t(const T* Q, const T* K, const float* A_q, const float* A_k, const float* noise_q,
                                const float* noise_k, float* dirs_q, float* dirs_k, int iterations, int problems,
                                int D, int n_q, int n_k, int c_q, int c_k, int32_t* perm_q_out, int32_t* perm_q_tmp,
                                int32_t* perm_k_out, int32_t* perm_k_tmp, uint32_t* keybuf_q, uint32_t* keybuf_k,
                                cudaStream_t st) {
  auto level_kernel = D == 64 ? split_level_kernel<64> : split_level_kernel<128>;
  CA_RETURN_IF_CUDA(cudaFuncSetAttribute(level_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemRowsMax * 8));
  const int lev_q = split_levels_for(n_q, c_q), lev_k = split_levels_for(n_k, c_k);
  // Sets of more than kTailRowsMax rows take three launches per level (directions, projections,
  // select + partition); the subtree kernel finishes the rest.  Per-level launches write alternately
  // to tmp/out so that the subtree kernel, which runs last, reads the buffer that is not the output.
  const int tail_q = tail_level_for(n_q, c_q), tail_k = tail_level_for(n_k, c_k);
  const int top = tail_q > tail_k ? tail_q : tail_k;
  BasicParams bp;
  bp.problems = problems; bp.iterations = iterations;
  SplitParams prm;
  prm.D = D; prm.problems = problems; prm.keys_in = 1;
  auto fill = [&](int level) {
    for (int w = 0; w < 2; ++w) {
      const int tail = w == 0 ? tail_q : tail_k;
      int32_t* out = w == 0 ? perm_q_out : perm_k_out;
      int32_t* tmp = w == 0 ? perm_q_tmp : perm_k_tmp;
      SplitSide& sd = prm.side[w];
      sd.Y = nullptr;
      sd.Yt = nullptr;
      sd.keybuf = w == 0 ? keybuf_q : keybuf_k;
      sd.n = w == 0 ? n_q : n_k; sd.c = w == 0 ? c_q : c_k;
      sd.levels = w == 0 ? lev_q : lev_k;
      sd.tail_level = tail;
      sd.active = 1;
      const bool to_tmp = ((tail - 1 - level) % 2) == 0;
      if (level < tail) {
        sd.perm_out = to_tmp ? tmp : out;
        sd.perm_in = level == 0 ? nullptr : (to_tmp ? out : tmp);
      } else {
        sd.perm_out = out;
        sd.perm_in = tail == 0 ? nullptr : tmp;
      }
      BasicSide& bs = bp.side[w];
      bs.X = w == 0 ? static_cast<const void*>(Q) : static_cast<const void*>(K);
      bs.A = w == 0 ? A_q : A_k;
      bs.noise = w == 0 ? noise_q : noise_k;
      bs.dirs = w == 0 ? dirs_q : dirs_k;
      bs.perm_in = sd.perm_in; bs.keybuf = sd.keybuf;
      bs.n = sd.n; bs.c = sd.c;
      bs.levels = tail;                                    // the per-level kernels stop where the subtrees begin
      bs.nodes = (1 << (sd.levels > 0 ? sd.levels : 1)) - 1;
    }
  };
  for (int level = 0; level < top; ++level) {
    fill(level);
    bp.level = level; prm.level = level;
    const size_t dsmem = (size_t)D * (D + 1) * sizeof(float);
    if (D == 64) {
      auto dk = basic_direction_kernel<T, 64>;
      CA_RETURN_IF_CUDA(cudaFuncSetAttribute(dk, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)dsmem));
      dk<<<dim3(1u << level, 2 * problems), 64, dsmem, st>>>(bp);
    } else {
      auto dk = basic_direction_kernel<T, 128>;
      CA_RETURN_IF_CUDA(cudaFuncSetAttribute(dk, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)dsmem));
      dk<<<dim3(1u << level, 2 * problems), 128, dsmem, st>>>(bp);
    }
    CA_LAUNCH_CHECK();
    const int n_max = n_q > n_k ? n_q : n_k;
    if (D == 64) basic_keys_kernel<T, 64><<<dim3(ceil_div(n_max, 256), 2 * problems), 256, 0, st>>>(bp);
    else basic_keys_kernel<T, 128><<<dim3(ceil_div(n_max, 256), 2 * problems), 256, 0, st>>>(bp);
    CA_LAUNCH_CHECK();
    int max_seg = 1;
    if (level < tail_q) max_seg = max_segment_at_level(n_q, c_q, level);
    if (level < tail_k) { const int ms = max_segment_at_level(n_k, c_k, level); if (ms > max_seg) max_seg = ms; }
    int csize = 1;
    while (csize < kMaxCluster && max_seg > csize * 16384) csize *= 2;
    const int per_cta = (max_seg + csize - 1) / csize;
    prm.smem_rows = per_cta < kSmemRowsMax ? per_cta : kSmemRowsMax;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((1u << level) * csize, 2 * problems);
    int threads = 128;
    while (threads < kSplitThreads && threads * 4 < per_cta) threads *= 2;
    cfg.blockDim = dim3(threads);
    cfg.dynamicSmemBytes = (size_t)prm.smem_rows * 8 > 16 ? (size_t)prm.smem_rows * 8 : 16;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = csize; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    CA_RETURN_IF_CUDA(cudaLaunchKernelEx(&cfg, level_kernel, prm));
    CA_LAUNCH_CHECK();
  }
  fill(top);
  bp.level = top; prm.level = top;
  const int slots = 1 << top;
  if (D == 64) {
    auto tk = basic_tail_kernel<T, 64>;
    CA_RETURN_IF_CUDA(cudaFuncSetAttribute(tk, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sizeof(BasicTailSmem<64>)));
    tk<<<dim3(slots, 2 * problems), kSplitThreads, sizeof(BasicTailSmem<64>), st>>>(bp, prm);
  } else {
    auto tk = basic_tail_kernel<T, 128>;
    CA_RETURN_IF_CUDA(cudaFuncSetAttribute(tk, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sizeof(BasicTailSmem<128>)));
    tk<<<dim3(slots, 2 * problems), kSplitThreads, sizeof(BasicTailSmem<128>), st>>>(bp, prm);
  }
  CA_LAUNCH_CHECK();
  return CA_OK;
}

int launch_split_basic(const void* Q, const void* K, int dtype, const float* A_q, const float* A_k,
                       const float* noise_q, const float* noise_k, float* dirs_q, float* dirs_k, int iterations,
                       int problems, int D, int n_q, int n_k, int c_q, int c_k, int32_t* perm_q_out,
                       int32_t* perm_q_tmp, int32_t* perm_k_out, int32_t* perm_k_tmp, uint32_t* keybuf_q,
                       uint32_t* keybuf_k, cudaStream_t st) {
  if (dtype == CA_DTYPE_BF16)
    return launch_split_basic_t(static_cast<const __nv_bfloat16*>(Q), static_cast<const __nv_bfloat16*>(K), A_q, A_k,
                                noise_q, noise_k, dirs_q, dirs_k, iterations, problems, D, n_q, n_k, c_q, c_k,
                                perm_q_out, perm_q_tmp, perm_k_out, perm_k_tmp, keybuf_q, keybuf_k, st);
  return launch_split_basic_t(static_cast<const float*>(Q), static_cast<const float*>(K), A_q, A_k, noise_q, noise_k,
                              dirs_q, dirs_k, iterations, problems, D, n_q, n_k, c_q, c_k, perm_q_out, perm_q_tmp,
                              perm_k_out, perm_k_tmp, keybuf_q, keybuf_k, st);
}

}  // namespace ca
