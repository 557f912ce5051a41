// Principal components of the transformed rows (Section 3.2.1, diagonalized
// variant), one CTA per head and side: builds the d x d covariance, decomposes
// it, and writes the projection that the split coordinates are computed with.
//
// Prologue.  Keys: the transformed keys K F (F F^T = M the query metric, Section
// 3.2.2) have covariance F^T C_K F / n_k with C_K the centred scatter of the keys,
// formed here from the Gram matrix and the column sums of K (two d x d x d
// products in shared memory, no pass over the data).  Queries: the covariance of
// the representation r(q) from its Gram matrix and column sums.
//
// Decomposition (d = 64, 128; float32: the bases only feed fp32 coordinates):
// Householder reduction to tridiagonal form, then the implicit-shift QL
// iteration.  Phase 1 (all 8d threads, two barriers per reflector): for
// k = 0 .. d-3 the reflector H_k = I - beta v v^T annihilates A[k+2.., k]; the
// trailing block is updated as A - v w^T - w v^T with p = beta A v,
// w = p - (beta/2)(v.p) v, and the transposed accumulated transform
// Qt <- H_k Qt is updated in the same two stages.  Thread (r, q) =
// (tid / 8, tid % 8) keeps entries 4 (q + 8 t) + c of row r of A and of column r
// of Qt in registers for the whole phase (the loops are bound by instruction
// issue and latency, not by arithmetic); the eight owners of row k+1 build the
// next reflector right after their update, inside their warp, so no third
// barrier is needed.  Phase 2, divide and conquer: the QL iteration is one
// dependent chain of about 0.9 n^2 plane rotations for n rows, so the tridiagonal
// matrix is cut three times (a cut writes T = diag(T1, T2) + rho u u^T) and the four
// quarters are iterated side by side, a sixteenth of the chain each: per quarter
// one warp runs the iteration on (diag, sub-diag) -- the search for a negligible
// sub-diagonal entry uses all lanes, the rotation chase is one dependent chain on
// lane 0 -- and hands each chase's rotations through a list (two in rotation) to
// consumer threads, which apply them to the rows of Qt of that quarter (a thread
// per column), pipelined with the next chase by two named barriers.  Two extra
// columns that start as the u of the cuts go through the same rotations and end
// as z = Q^T u.  A merge solves diag(d) + rho z z^T: poles sorted, negligible
// weights and coinciding poles deflated, the roots of the secular equation by
// bisection on the offset from the nearer pole (eight threads per root; offsets
// keep the differences d_j - x accurate), the weights recomputed from the roots
// (Gu and Eisenstat) so that the eigenvectors stay orthogonal to rounding, and one
// product with the blocks' eigenvectors.  The quarters are merged into halves by
// the two halves of the CTA side by side, then the halves into the whole.
//
// Epilogue.  Components in order of descending eigenvalue.  With E the
// eigenvectors and F the factor that produced the transformed rows, the map from
// the original space to the coordinates is F E; component t is oriented so that
// the entry of largest magnitude (lowest row on ties) of column t of F E is
// positive -- a rule that gives the same signs whatever root of the metric F is.
// Written out: the projection matrix (F E for the keys, which are projected
// straight from K; E for the queries, whose representation is already stored),
// its bias -mean . W, and W^T as bf16 hi + lo parts for the tensor-core
// projection.
#include "kernels.h"

namespace ca {

namespace {

// named barriers with the id as an immediate (ids 1-8: the four QL groups, 9-10: the two half merges;
// barrier 0 stays the CTA's own: threads that finish early wait there while others still use theirs)
#define CA_BAR_CASE(OP, ID) case ID: asm volatile(OP " " #ID ", %0;" ::"r"(count) : "memory"); break;
__device__ __forceinline__ void named_sync(int id, int count) {
  switch (id) {
    CA_BAR_CASE("bar.sync", 0) CA_BAR_CASE("bar.sync", 1) CA_BAR_CASE("bar.sync", 2) CA_BAR_CASE("bar.sync", 3)
    CA_BAR_CASE("bar.sync", 4) CA_BAR_CASE("bar.sync", 5) CA_BAR_CASE("bar.sync", 6) CA_BAR_CASE("bar.sync", 7)
    CA_BAR_CASE("bar.sync", 8) CA_BAR_CASE("bar.sync", 9) CA_BAR_CASE("bar.sync", 10) CA_BAR_CASE("bar.sync", 11)
    CA_BAR_CASE("bar.sync", 12) CA_BAR_CASE("bar.sync", 13) CA_BAR_CASE("bar.sync", 14)
    default: asm volatile("bar.sync 15, %0;" ::"r"(count) : "memory"); break;
  }
}
__device__ __forceinline__ void named_arrive(int id, int count) {
  switch (id) {
    CA_BAR_CASE("bar.arrive", 0) CA_BAR_CASE("bar.arrive", 1) CA_BAR_CASE("bar.arrive", 2) CA_BAR_CASE("bar.arrive", 3)
    CA_BAR_CASE("bar.arrive", 4) CA_BAR_CASE("bar.arrive", 5) CA_BAR_CASE("bar.arrive", 6) CA_BAR_CASE("bar.arrive", 7)
    CA_BAR_CASE("bar.arrive", 8) CA_BAR_CASE("bar.arrive", 9) CA_BAR_CASE("bar.arrive", 10) CA_BAR_CASE("bar.arrive", 11)
    CA_BAR_CASE("bar.arrive", 12) CA_BAR_CASE("bar.arrive", 13) CA_BAR_CASE("bar.arrive", 14)
    default: asm volatile("bar.arrive 15, %0;" ::"r"(count) : "memory"); break;
  }
}
#undef CA_BAR_CASE

constexpr int kMaxQlIterations = 64;

// ---- implicit-shift QL on rows [l0, l1) of a tridiagonal matrix (de[i] = (diagonal i, coupling of
// i and i + 1); the coupling at l1 - 1 is not part of the block).  One warp: the search for a
// negligible sub-diagonal entry uses all lanes, the rotation chase is one dependent chain on lane 0.
// Each chase's rotations go through a list (rot, hdr; two in rotation, so that the next chase is
// written while the last one is applied) to the consumer threads, which apply them to the rows of
// Qt.  Two named barriers: bar_full hands a list over, bar_empty hands it back; a list is handed over
// only after the one before it has come back, so each barrier has one generation in flight.
__device__ __forceinline__ void ql_producer(float2* de, int l0, int l1, float* rot, int* hdr, int rot_stride,
                                            int bar_full, int bar_empty, int parties, int lane) {
  int bsel = 0, nlist = 0;
  const float eps = 6e-8f;
  for (int l = l0; l < l1; ++l) {
    for (int iter = 0; iter < kMaxQlIterations; ++iter) {
      // first m >= l whose sub-diagonal entry is negligible (m = l1 - 1 if none)
      int m = l1 - 1;
      for (int base = l; base < l1 - 1; base += 32) {
        const int idx = base + lane;
        bool small = false;
        if (idx < l1 - 1) {
          const float2 a = de[idx];
          small = fabsf(a.y) <= eps * (fabsf(a.x) + fabsf(de[idx + 1].x));
        }
        const unsigned bal = __ballot_sync(0xffffffffu, small);
        if (bal) { m = base + __ffs(bal) - 1; break; }
      }
      if (m == l) break;
      if (lane == 0) {
        float2* rt = reinterpret_cast<float2*>(rot + bsel * rot_stride);
        const float2 top = de[l];
        // the shift only steers the convergence (the rotations are formed from the matrix itself), so
        // approximate division and root are enough for it
        float g = __fdividef(de[l + 1].x - top.x, 2.f * top.y);
        float rr;
        asm("sqrt.approx.ftz.f32 %0, %1;" : "=f"(rr) : "f"(fmaf(g, g, 1.f)));
        g = de[m].x - top.x + __fdividef(top.y, g + (g >= 0.f ? rr : -rr));
        float s = 1.f, c = 1.f, p = 0.f;
        bool under = false;
        int i = m - 1;
        float2 cur = de[i];              // (d_i, e_i)
        float d_i1 = de[i + 1].x;
        for (; i >= l; --i) {
          // operands of the next rotation, fetched ahead of the dependent chain
          const float2 nxt = de[i > l ? i - 1 : l];
          const float f = s * cur.y, bb = c * cur.y;
          const float r2 = fmaf(f, f, g * g);
          float rinv;
          asm("rsqrt.approx.ftz.f32 %0, %1;" : "=f"(rinv) : "f"(r2));
          const float p_old = p, d_old = d_i1;
          s = f * rinv;
          c = g * rinv;
          g = d_i1 - p;
          rr = fmaf(c, bb + bb, (cur.x - g) * s);
          p = s * rr;
          de[i + 1] = make_float2(g + p, r2 * rinv);       // new d_{i+1}; e_{i+1} = hypot(f, g)
          g = fmaf(c, rr, -bb);
          rt[i] = make_float2(c, s);
          // The chase has died out (f = g = 0): deflate here.  Tested after the rotation has been
          // formed so that the test is off the dependent chain; its results are discarded.
          if (r2 < 1e-36f) {
            de[i + 1] = make_float2(d_old - p_old, 0.f);
            de[m].y = 0.f;
            under = true;
            break;
          }
          d_i1 = cur.x;          // d_i is the next step's d_{i+1}; it has not been modified yet
          cur = nxt;
        }
        int lo = l;
        if (!under) {
          de[l] = make_float2(top.x - p, g);
          de[m].y = 0.f;
        } else {
          lo = i + 1;
        }
        hdr[bsel * 4 + 0] = m - 1;
        hdr[bsel * 4 + 1] = lo;
        hdr[bsel * 4 + 2] = 0;
      }
      __syncwarp();
      __threadfence_block();
      if (nlist > 0) named_sync(bar_empty, parties);     // the list before this one has been applied
      named_arrive(bar_full, parties);
      ++nlist;
      bsel ^= 1;
    }
  }
  if (lane == 0) hdr[bsel * 4 + 2] = 1;                    // end marker
  __syncwarp();
  __threadfence_block();
  if (nlist > 0) named_sync(bar_empty, parties);
  named_arrive(bar_full, parties);
}

// consumer thread of column t (t >= ncols: only keeps the barriers going)
__device__ __forceinline__ void ql_consumer(float* Qt, int lda, int t, int ncols, const float* rot, const int* hdr,
                                            int rot_stride, int bar_full, int bar_empty, int parties) {
  int bsel = 0;
  while (true) {
    named_sync(bar_full, parties);
    if (hdr[bsel * 4 + 2]) break;
    if (t < ncols) {
      const int hi = hdr[bsel * 4 + 0], lo = hdr[bsel * 4 + 1];
      const float* rt = rot + bsel * rot_stride;
      float carry = Qt[(hi + 1) * lda + t];
      for (int i = hi; i >= lo; --i) {
        const float c = rt[2 * i], s = rt[2 * i + 1];
        const float zi = Qt[i * lda + t];
        Qt[(i + 1) * lda + t] = fmaf(s, zi, c * carry);
        carry = fmaf(c, zi, -s * carry);
      }
      Qt[lo * lda + t] = carry;
    }
    __threadfence_block();
    named_arrive(bar_empty, parties);
    bsel ^= 1;
  }
}

}  // namespace

// d x d x d products in shared memory, a 4 x 4 tile of the result per thread (the first d^2 / 16
// threads; every shared-memory load feeds four or sixteen multiply-adds, and the lanes of a
// quarter-warp read distinct banks).  Terms are added for k = 0, 1, ... in that order.
//   XT = false: acc[a][b] = sum_k X[(4 ti + a) lda + k] Y[k lda + 4 tj + b]
//   XT = true:  acc[a][b] = sum_k X[k lda + 4 ti + a]   Y[k lda + 4 tj + b]
template <int D, bool XT>
__device__ __forceinline__ void tile_product(const float* __restrict__ X, const float* __restrict__ Y, int lda,
                                             int ti, int tj, float (&acc)[4][4]) {
#pragma unroll
  for (int x = 0; x < 4; ++x)
#pragma unroll
    for (int y = 0; y < 4; ++y) acc[x][y] = 0.f;
#pragma unroll 2
  for (int k0 = 0; k0 < D; k0 += 4) {
    float xa[4][4];                                    // [row][k]
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      if (XT) {
        const float4 v = *reinterpret_cast<const float4*>(&X[(k0 + e) * lda + 4 * ti]);
        xa[0][e] = v.x; xa[1][e] = v.y; xa[2][e] = v.z; xa[3][e] = v.w;
      } else {
        const float4 v = *reinterpret_cast<const float4*>(&X[(4 * ti + e) * lda + k0]);
        xa[e][0] = v.x; xa[e][1] = v.y; xa[e][2] = v.z; xa[e][3] = v.w;
      }
    }
#pragma unroll
    for (int kk = 0; kk < 4; ++kk) {
      const float4 y = *reinterpret_cast<const float4*>(&Y[(k0 + kk) * lda + 4 * tj]);
#pragma unroll
      for (int x = 0; x < 4; ++x) {
        acc[x][0] = fmaf(xa[x][kk], y.x, acc[x][0]); acc[x][1] = fmaf(xa[x][kk], y.y, acc[x][1]);
        acc[x][2] = fmaf(xa[x][kk], y.z, acc[x][2]); acc[x][3] = fmaf(xa[x][kk], y.w, acc[x][3]);
      }
    }
  }
}

// acc[a][c] = sum_k X[(4 ti + a) lda + k] Yr[(tj + (D / 4) c) lda + k]   (both operands by rows)
template <int D>
__device__ __forceinline__ void tile_product_rows(const float* __restrict__ X, const float* __restrict__ Yr, int lda,
                                                  int ti, int tj, float (&acc)[4][4]) {
#pragma unroll
  for (int x = 0; x < 4; ++x)
#pragma unroll
    for (int y = 0; y < 4; ++y) acc[x][y] = 0.f;
#pragma unroll 2
  for (int k0 = 0; k0 < D; k0 += 4) {
    float4 xv[4], yv[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      xv[e] = *reinterpret_cast<const float4*>(&X[(4 * ti + e) * lda + k0]);
      yv[e] = *reinterpret_cast<const float4*>(&Yr[(tj + (D / 4) * e) * lda + k0]);
    }
#pragma unroll
    for (int x = 0; x < 4; ++x)
#pragma unroll
      for (int y = 0; y < 4; ++y) {
        acc[x][y] = fmaf(xv[x].x, yv[y].x, acc[x][y]); acc[x][y] = fmaf(xv[x].y, yv[y].y, acc[x][y]);
        acc[x][y] = fmaf(xv[x].z, yv[y].z, acc[x][y]); acc[x][y] = fmaf(xv[x].w, yv[y].w, acc[x][y]);
      }
  }
}

// ---- merge of two adjacent blocks of the tridiagonal matrix whose eigen-decompositions are known
// (rows [b0, b0 + NB) of Qt are their eigenvectors, de[].x their eigenvalues, column `zcol` of
// those rows z = Q^T u): eigen-decomposition of diag(d) + rho2 z z^T with z scaled to unit length
// (rho2 = 2 rho).  Sorted poles, deflation of negligible weights and of poles that coincide (a plane
// rotation of their two eigenvectors), the roots of the secular equation
// 1 + rho2 sum_j z_j^2 / (d_j - x) = 0 by bisection on the offset from the nearer pole (eight threads
// per root), the weights recomputed from the roots so that the eigenvectors come out orthogonal
// (Gu and Eisenstat), eigenvectors u_i[j] = zhat_j / (d_j - x_i), and the product with the blocks'
// eigenvectors.  Run by a group of GT threads (lt = index in the group, `sync` its barrier); the new
// rows go to rows [b0, b0 + NB) of L, with `carry` more columns after the D of the basis (the z of
// an enclosing merge); every array of `scratch` is used at [b0, b0 + NB), so groups on disjoint
// blocks run side by side.
template <int D, int NB, int GT, typename Sync>
__device__ __forceinline__ void merge_blocks(float* __restrict__ Qt, float* __restrict__ L, float* __restrict__ A,
                                             float2* de, float* scratch, int b0, int zcol, int carry, float rho,
                                             int lt, int grp, Sync sync) {
  constexpr int LDA = D + 4;
  static_assert(GT >= 8 * NB && GT >= D + 4 && (NB / 8) % 2 == 0, "eight threads per root, a thread per column");
  const int lane = lt & 31;
  float* ds = scratch + b0;                                // poles in ascending order
  float* zs = ds + D;
  int* ord = reinterpret_cast<int*>(zs + D);               // sorted position -> row of Qt
  int* keep_row = ord + D;                                 // kept pole -> row of Qt
  float* kd = reinterpret_cast<float*>(keep_row + D);      // kept poles, weights
  float* kz = kd + D;
  int* korg = reinterpret_cast<int*>(kz + D);              // root -> pole its offset is measured from
  float* kmu = reinterpret_cast<float*>(korg + D);
  float* kzh = kmu + D;
  float* gc = kzh + D;                                     // plane rotations of the deflation
  float* gs = gc + D;
  int* ga = reinterpret_cast<int*>(gs + D);
  int* gb = ga + D;
  int* defl_row = gb + D;                                  // deflated: row of Qt, eigenvalue
  float* defl_d = reinterpret_cast<float*>(defl_row + D);
  float* kz2 = defl_d + D;                                 // squared weights of the kept poles
  int* counts = reinterpret_cast<int*>(scratch + 16 * D) + 8 * grp;   // kept, rotations, deflated, skip
  float* z2sum = reinterpret_cast<float*>(counts + 4);
  const int W = D + carry;                                 // columns of a row that travel
  if (lt < NB) {
    const float mine = de[b0 + lt].x;
    int rank = 0;
#pragma unroll 16
    for (int k = 0; k < NB; ++k) {
      const float other = de[b0 + k].x;
      rank += (other < mine) || (other == mine && k < lt);
    }
    ord[rank] = b0 + lt;
  }
  sync();
  if (lt < NB) {
    ds[lt] = de[ord[lt]].x;
    zs[lt] = Qt[ord[lt] * LDA + zcol] * 0.70710678f;
  }
  sync();
  if (lt < 32) {
    const float rho2 = 2.f * rho;
    float dmax = 0.f, zmax = 0.f;
    for (int j = lane; j < NB; j += 32) { dmax = fmaxf(dmax, fabsf(ds[j])); zmax = fmaxf(zmax, fabsf(zs[j])); }
    for (int o = 16; o > 0; o >>= 1) {
      dmax = fmaxf(dmax, __shfl_xor_sync(0xffffffffu, dmax, o));
      zmax = fmaxf(zmax, __shfl_xor_sync(0xffffffffu, zmax, o));
    }
    const float tol = 8.f * 6e-8f * fmaxf(dmax, zmax);
    int K = 0, ng = 0, nd = 0;
    if (lt != 0) {
      // the scan below is one thread's
    } else if (rho2 * zmax <= tol) {
      counts[3] = 1;                                       // the blocks do not couple: nothing to merge
    } else {
      counts[3] = 0;
      // one pass over the sorted poles; the last kept pole and the next pole travel in registers
      // (every step would otherwise wait for the shared-memory round trip of the step before)
      float d_prev = 0.f, z_prev = 0.f;
      int o_prev = -1;
      float dj = ds[0], zj = zs[0];
      int oj = ord[0];
      for (int j = 0; j < NB; ++j) {
        const int jn = j + 1 < NB ? j + 1 : j;
        const float dn = ds[jn], zn = zs[jn];
        const int on = ord[jn];
        if (rho2 * fabsf(zj) <= tol) {
          defl_row[nd] = oj; defl_d[nd] = dj; ++nd;
        } else {
          // two poles coincide when |t c s| <= tol, c = z_j / tau, s = -z_prev / tau, tau^2 = z_j^2 + z_prev^2;
          // the test is made without the root and the divisions, which only a deflation needs
          if (o_prev >= 0 && fabsf((dj - d_prev) * zj * z_prev) <= tol * fmaf(zj, zj, z_prev * z_prev)) {
            float sn = z_prev, cs = zj;
            const float tau = sqrtf(fmaf(cs, cs, sn * sn));
            cs = cs / tau;
            sn = -sn / tau;
            // rotate the weight into pole j; the other of the two is deflated
            gc[ng] = cs; gs[ng] = sn; ga[ng] = o_prev; gb[ng] = oj; ++ng;
            const float tt = d_prev * cs * cs + dj * sn * sn;
            dj = d_prev * sn * sn + dj * cs * cs;
            zj = tau;
            --K;                                           // the last kept pole gives way
            defl_row[nd] = o_prev; defl_d[nd] = tt; ++nd;
          }
          keep_row[K] = oj; kd[K] = dj; kz[K] = zj; ++K;
          d_prev = dj; z_prev = zj; o_prev = oj;
        }
        dj = dn; zj = zn; oj = on;
      }
    }
    if (lt == 0) { counts[0] = K; counts[1] = ng; counts[2] = nd; }
  }
  sync();
  if (counts[3]) {
    // nothing to merge: the rows move as they are, so that every block ends in L
    for (int e = lt; e < NB * W; e += GT) L[(b0 + e / W) * LDA + e % W] = Qt[(b0 + e / W) * LDA + e % W];
    sync();
    return;
  }
  const int K = counts[0], ng = counts[1], nd = counts[2];
  const float rho2 = 2.f * rho;
  // squared weights of the kept poles and their sum (the last root's bracket)
  if (lt < NB) kz2[lt] = lt < K ? kz[lt] * kz[lt] : 0.f;
  if (lt < 32) {
    float z2 = 0.f;
    for (int j = lane; j < K; j += 32) z2 = fmaf(kz[j], kz[j], z2);
    for (int o = 16; o > 0; o >>= 1) z2 += __shfl_xor_sync(0xffffffffu, z2, o);
    if (lt == 0) *z2sum = z2;
  }
  sync();
  // rotations of the deflation on the rows of Qt (one column per thread, in the order recorded)
  if (lt < W) {
    for (int g = 0; g < ng; ++g) {
      const float x = Qt[ga[g] * LDA + lt], y = Qt[gb[g] * LDA + lt];
      Qt[ga[g] * LDA + lt] = gc[g] * x + gs[g] * y;
      Qt[gb[g] * LDA + lt] = gc[g] * y - gs[g] * x;
    }
  }
  // roots: group i = lt / 8 of eight threads, each with the poles j = sub (mod 8)
  const int gi = lt >> 3, sub = lt & 7;
  const bool live = gi < K;
  {
    const int i = live ? gi : 0;
    // this thread's poles j = sub + 8 t and their squared weights stay in registers for all the
    // halvings (past the last pole: weight 0 at a far distance); two terms share one reciprocal:
    // a / p + b / q = (a q + b p) / (p q)
    constexpr int TPR = NB / 8;
    float pole[TPR], wgt[TPR];
#pragma unroll
    for (int t = 0; t < TPR; ++t) {
      const int j = sub + 8 * t;
      pole[t] = j < K ? kd[j] : 0.f;
      wgt[t] = j < K ? kz2[j] : 0.f;
    }
    float dist[TPR];                                       // d_j - d_org
    auto set_origin = [&](int org) {
      const float d0 = kd[org];
#pragma unroll
      for (int t = 0; t < TPR; ++t) dist[t] = (sub + 8 * t < K) ? pole[t] - d0 : 1e18f;
    };
    auto fval = [&](float m) {
      float acc = 0.f;
#pragma unroll
      for (int t = 0; t < TPR; t += 2) {
        const float p0 = dist[t] - m, p1 = dist[t + 1] - m;
        float inv;                                          // one special-function operation, no rounding fix-up
        asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(inv) : "f"(p0 * p1));
        acc = fmaf(fmaf(wgt[t], p1, wgt[t + 1] * p0), inv, acc);
      }
      acc += __shfl_xor_sync(0xffffffffu, acc, 1);
      acc += __shfl_xor_sync(0xffffffffu, acc, 2);
      acc += __shfl_xor_sync(0xffffffffu, acc, 4);
      return fmaf(rho2, acc, 1.f);
    };
    // the last root lies in (d_{K-1}, d_{K-1} + rho2 |z|^2); every other one between two poles
    int org = i;
    const bool last = i >= K - 1;
    const float width = last ? rho2 * *z2sum : kd[i + 1] - kd[i];
    const float mid = 0.5f * width;
    set_origin(i);
    const float f_mid = fval(mid);                         // every thread of the warp takes part
    float lo_m = 0.f, hi_m = width;
    if (!last) {
      if (f_mid >= 0.f) hi_m = mid;                        // root in the left half: offset from pole i
      else { org = i + 1; lo_m = -mid; hi_m = 0.f; }       // offset from pole i + 1
    }
    set_origin(org);
    for (int it = 0; it < 44; ++it) {                      // a fixed count: the groups of a warp stay in step
      // (44 halvings take an interval of width w down to the float spacing of offsets >= 2^-20 w;
      // a root closer to its pole than that belongs to a weight that the deflation has removed)
      const float m = 0.5f * (lo_m + hi_m);
      const float fm = fval(m);
      if (m != lo_m && m != hi_m) {
        if (fm > 0.f) hi_m = m; else lo_m = m;
      }
    }
    if (live && sub == 0) { korg[gi] = org; kmu[gi] = 0.5f * (lo_m + hi_m); }
  }
  sync();
  // weights recomputed from the roots: zhat_j^2 = prod_i (x_i - d_j) / (rho2 prod_{i != j} (d_i - d_j))
  {
    const int j = live ? gi : 0;
    float prod = 1.f;
    for (int i = sub; i < K; i += 8) {
      const float num = (kd[korg[i]] - kd[j]) + kmu[i];
      prod *= __fdividef(num, (i == j) ? rho2 : kd[i] - kd[j]);
    }
    prod *= __shfl_xor_sync(0xffffffffu, prod, 1);
    prod *= __shfl_xor_sync(0xffffffffu, prod, 2);
    prod *= __shfl_xor_sync(0xffffffffu, prod, 4);
    if (live && sub == 0) kzh[gi] = copysignf(sqrtf(fabsf(prod)), kz[gi]);
  }
  sync();
  // eigenvector i over the kept poles, normalised, as row b0 + i of A
  {
    const int i = live ? gi : 0;
    const float d0 = kd[korg[i]], mu = kmu[i];
    float nrm = 0.f;
    for (int j = sub; j < K; j += 8) {
      const float v = __fdividef(kzh[j], (kd[j] - d0) - mu);
      nrm = fmaf(v, v, nrm);
    }
    nrm += __shfl_xor_sync(0xffffffffu, nrm, 1);
    nrm += __shfl_xor_sync(0xffffffffu, nrm, 2);
    nrm += __shfl_xor_sync(0xffffffffu, nrm, 4);
    const float inv = rsqrtf(nrm);
    if (live)
      for (int j = sub; j < K; j += 8) A[(b0 + gi) * LDA + j] = __fdividef(kzh[j], (kd[j] - d0) - mu) * inv;
  }
  sync();
  // rows of the merged basis into L: row b0 + i = sum_j A[b0 + i][j] Qt[keep_row[j]] (i < K), then
  // the deflated rows (a 4 x 4 tile per thread, terms in the order of j)
  {
    const int tile_i = lt / (D / 4), tile_j = lt % (D / 4);
    if (lt < NB * D / 16 && 4 * tile_i < K) {
      const int i0 = 4 * tile_i;
      float acc[4][4];
#pragma unroll
      for (int x = 0; x < 4; ++x)
#pragma unroll
        for (int y = 0; y < 4; ++y) acc[x][y] = 0.f;
      int j = 0;
      for (; j + 4 <= K; j += 4) {
        float xa[4][4];
#pragma unroll
        for (int x = 0; x < 4; ++x) {
          const float4 v = *reinterpret_cast<const float4*>(&A[(b0 + i0 + x) * LDA + j]);
          xa[x][0] = v.x; xa[x][1] = v.y; xa[x][2] = v.z; xa[x][3] = v.w;
        }
#pragma unroll
        for (int kk = 0; kk < 4; ++kk) {
          const float4 y = *reinterpret_cast<const float4*>(&Qt[keep_row[j + kk] * LDA + 4 * tile_j]);
#pragma unroll
          for (int x = 0; x < 4; ++x) {
            acc[x][0] = fmaf(xa[x][kk], y.x, acc[x][0]); acc[x][1] = fmaf(xa[x][kk], y.y, acc[x][1]);
            acc[x][2] = fmaf(xa[x][kk], y.z, acc[x][2]); acc[x][3] = fmaf(xa[x][kk], y.w, acc[x][3]);
          }
        }
      }
      for (; j < K; ++j) {
        const float4 y = *reinterpret_cast<const float4*>(&Qt[keep_row[j] * LDA + 4 * tile_j]);
#pragma unroll
        for (int x = 0; x < 4; ++x) {
          const float xv = A[(b0 + i0 + x) * LDA + j];
          acc[x][0] = fmaf(xv, y.x, acc[x][0]); acc[x][1] = fmaf(xv, y.y, acc[x][1]);
          acc[x][2] = fmaf(xv, y.z, acc[x][2]); acc[x][3] = fmaf(xv, y.w, acc[x][3]);
        }
      }
#pragma unroll
      for (int x = 0; x < 4; ++x)
        if (i0 + x < K)
          *reinterpret_cast<float4*>(&L[(b0 + i0 + x) * LDA + 4 * tile_j]) = make_float4(acc[x][0], acc[x][1], acc[x][2], acc[x][3]);
    }
  }
  // the columns that travel with the rows (the z of the enclosing merge)
  for (int e = lt; e < K * carry; e += GT) {
    const int i = e / carry, col = D + e % carry;
    float acc = 0.f;
    for (int j = 0; j < K; ++j) acc = fmaf(A[(b0 + i) * LDA + j], Qt[keep_row[j] * LDA + col], acc);
    L[(b0 + i) * LDA + col] = acc;
  }
  for (int e = lt; e < nd * W; e += GT) L[(b0 + K + e / W) * LDA + e % W] = Qt[defl_row[e / W] * LDA + e % W];
  sync();
  if (lt < NB) de[b0 + lt].x = lt < K ? kd[korg[lt]] + kmu[lt] : defl_d[lt - K];
  sync();
}

template <int D>
__global__ void __launch_bounds__(8 * D) eigh_tql_kernel(const PcaArgs a) {
  constexpr int NT = 8 * D, LDA = D + 4;
  constexpr int CH = D / 32;            // float4 chunks of a row per thread
  extern __shared__ __align__(16) unsigned char smem_raw[];
  float* A = reinterpret_cast<float*>(smem_raw);       // [D][LDA]
  float* Qt = A + D * LDA;                             // [D][LDA]   written after phase 1; rows become the eigenvectors
  float* L = Qt + D * LDA;                             // [D][LDA]   the factor F (prologue, sign rule); the merged basis in between
  float* vbuf = A + 3 * D * LDA;                       // [2][D]     reflector, zero above its first entry
  float* pbuf = vbuf + 2 * D;                          // [D]
  float* ubuf = pbuf + D;                              // [D]
  float2* de = reinterpret_cast<float2*>(ubuf + D);    // [D]        (diagonal i, sub-diagonal coupling i and i+1)
  float* beta = ubuf + 3 * D;                          // [2] (+2)
  float* rot = beta + 4;                               // [2][2D] (+4D) per buffer: (c, s) of the rotation of rows (i, i+1) at 2i
  int* hdr = reinterpret_cast<int*>(rot + 8 * D);      // [4][2][4]  per quarter and buffer: highest i, lowest i, end marker
  float* scratch = reinterpret_cast<float*>(hdr + 32); // [17 D]     arrays of the merge
  __shared__ double s_scale;

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int r = tid >> 3, q = tid & 7;
  const size_t mat = (size_t)blockIdx.x * D * D;
  // d x d x d products: a 4 x 4 tile per thread, the first d^2 / 16 threads
  constexpr int TILE_THREADS = D * D / 16;
  const int tile_i = tid / (D / 4), tile_j = tid % (D / 4);

  // ---- prologue: the matrix to decompose, in A
  if (a.lift) {
    const double* F = a.lift + mat;
    for (int e = tid; e < D * D; e += NT) L[(e / D) * LDA + e % D] = (float)F[e];
  }
  if (a.mode == kPcaKeys) {
    // C = (gram - s s^T / n) c_scale, the centred scatter of the keys; then alpha F^T C F
    // (double-precision operations are scarce on this part: no division per element)
    const double* G = a.gram + mat;
    const double* sm = a.sum + (size_t)blockIdx.x * D;
    const double cs = a.c_scale, cn = a.c_scale / a.n;
    for (int e = tid; e < D * D; e += NT) {
      const int i = e / D, j = e % D;
      A[i * LDA + j] = (float)fma(-cn * sm[i], sm[j], G[e] * cs);
    }
    __syncthreads();
    float acc[4][4];
    if (tid < TILE_THREADS) {
      tile_product<D, true>(L, A, LDA, tile_i, tile_j, acc);                              // F^T C
#pragma unroll
      for (int x = 0; x < 4; ++x)
        *reinterpret_cast<float4*>(&Qt[(4 * tile_i + x) * LDA + 4 * tile_j]) = make_float4(acc[x][0], acc[x][1], acc[x][2], acc[x][3]);
    }
    __syncthreads();
    if (tid < TILE_THREADS) {
      tile_product<D, false>(Qt, L, LDA, tile_i, tile_j, acc);                            // (F^T C) F
      const float al = (float)a.alpha;
#pragma unroll
      for (int x = 0; x < 4; ++x)
        *reinterpret_cast<float4*>(&A[(4 * tile_i + x) * LDA + 4 * tile_j]) =
            make_float4(al * acc[x][0], al * acc[x][1], al * acc[x][2], al * acc[x][3]);
    }
  } else if (a.mode == kPcaQueries) {
    // covariance of the stored representation: gram / n - mean mean^T
    const double* G = a.gram + mat;
    const double* sm = a.sum + (size_t)blockIdx.x * D;
    const double inv_n = 1.0 / a.n, inv_n2 = inv_n * inv_n;
    for (int e = tid; e < D * D; e += NT) {
      const int i = e / D, j = e % D;
      A[i * LDA + j] = (float)fma(-inv_n2 * sm[i], sm[j], G[e] * inv_n);
    }
  } else {
    const double* Ain = a.A_in + mat;
    for (int e = tid; e < D * D; e += NT) A[(e / D) * LDA + e % D] = (float)Ain[e];
  }
  __syncthreads();
  // symmetrise, and scale so that the largest diagonal entry is 1 (eigenvectors unchanged,
  // eigenvalues scaled back at the end)
  if (tid < 32) {
    float mx = 0.f;
    for (int i = tid; i < D; i += 32) mx = fmaxf(mx, fabsf(A[i * LDA + i]));
    for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
    if (tid == 0) s_scale = mx > 0.f ? (double)mx : 1.0;
  }
  float sym[CH][4];
#pragma unroll
  for (int t = 0; t < CH; ++t)
#pragma unroll
    for (int c = 0; c < 4; ++c) {
      const int j = 4 * (q + 8 * t) + c;
      sym[t][c] = 0.5f * (A[r * LDA + j] + A[j * LDA + r]);
    }
  __syncthreads();
  const double a_scale = s_scale;
  {
    const float inv = (float)(1.0 / a_scale);
#pragma unroll
    for (int t = 0; t < CH; ++t)
      *reinterpret_cast<float4*>(&A[r * LDA + 4 * (q + 8 * t)]) =
          make_float4(sym[t][0] * inv, sym[t][1] * inv, sym[t][2] * inv, sym[t][3] * inv);
  }
  __syncthreads();

  // This thread's parts of row r of A and of column r of Qt (the same index set: entries
  // 4 (q + 8 t) + c), kept in registers for the whole reduction.  Qt starts as the identity.
  float areg[CH][4], qreg[CH][4];
#pragma unroll
  for (int t = 0; t < CH; ++t) {
    const int j0 = 4 * (q + 8 * t);
    const float4 a = *reinterpret_cast<const float4*>(&A[r * LDA + j0]);
    areg[t][0] = a.x; areg[t][1] = a.y; areg[t][2] = a.z; areg[t][3] = a.w;
#pragma unroll
    for (int c = 0; c < 4; ++c) qreg[t][c] = (j0 + c == r) ? 1.f : 0.f;
  }

  // Iteration k applies reflector k (two stages) and then builds reflector k+1; k = -1 only builds.
  for (int k = -1; k < D - 2; ++k) {
    const int m0 = k + 1;
    const float* v = vbuf + (k & 1) * D;
    const float b = k >= 0 ? beta[k & 1] : 0.f;            // uniform over the CTA
    const int t_first = m0 >> 5;                           // chunks below it hold only zeros of v
    if (b != 0.f) {
      // p = beta A v (rows >= m0), u = beta v^T Qt
      float ps = 0.f, us = 0.f;
#pragma unroll
      for (int t = 0; t < CH; ++t) {
        if (t < t_first) continue;
        const float4 vv = *reinterpret_cast<const float4*>(&v[4 * (q + 8 * t)]);
        ps = fmaf(areg[t][0], vv.x, ps); ps = fmaf(areg[t][1], vv.y, ps);
        ps = fmaf(areg[t][2], vv.z, ps); ps = fmaf(areg[t][3], vv.w, ps);
        us = fmaf(qreg[t][0], vv.x, us); us = fmaf(qreg[t][1], vv.y, us);
        us = fmaf(qreg[t][2], vv.z, us); us = fmaf(qreg[t][3], vv.w, us);
      }
      ps += __shfl_xor_sync(0xffffffffu, ps, 1); us += __shfl_xor_sync(0xffffffffu, us, 1);
      ps += __shfl_xor_sync(0xffffffffu, ps, 2); us += __shfl_xor_sync(0xffffffffu, us, 2);
      ps += __shfl_xor_sync(0xffffffffu, ps, 4); us += __shfl_xor_sync(0xffffffffu, us, 4);
      if (q == 0) {
        pbuf[r] = (r >= m0) ? b * ps : 0.f;
        ubuf[r] = b * us;
      }
    }
    __syncthreads();
    if (b != 0.f) {
      float kp = 0.f;
      for (int j = lane; j < D; j += 32) kp = fmaf(v[j], pbuf[j], kp);
      for (int o = 16; o > 0; o >>= 1) kp += __shfl_xor_sync(0xffffffffu, kp, o);
      const float K = 0.5f * b * kp;
      const float v_r = v[r];
      const float w_r = pbuf[r] - K * v_r;
      const float u_r = ubuf[r];
      const bool live_row = r >= m0;
#pragma unroll
      for (int t = 0; t < CH; ++t) {
        if (t < t_first) continue;
        const int j0 = 4 * (q + 8 * t);
        const float4 vv = *reinterpret_cast<const float4*>(&v[j0]);
        if (live_row) {
          const float4 pp = *reinterpret_cast<const float4*>(&pbuf[j0]);
          areg[t][0] -= v_r * (pp.x - K * vv.x) + w_r * vv.x;
          areg[t][1] -= v_r * (pp.y - K * vv.y) + w_r * vv.y;
          areg[t][2] -= v_r * (pp.z - K * vv.z) + w_r * vv.z;
          areg[t][3] -= v_r * (pp.w - K * vv.w) + w_r * vv.w;
        }
        qreg[t][0] = fmaf(-vv.x, u_r, qreg[t][0]); qreg[t][1] = fmaf(-vv.y, u_r, qreg[t][1]);
        qreg[t][2] = fmaf(-vv.z, u_r, qreg[t][2]); qreg[t][3] = fmaf(-vv.w, u_r, qreg[t][3]);
      }
    }
  // Reflector for row kn = k+1, built by the whole warp that holds the row's eight owners
    // (the other groups of the warp go through the shuffles and write nothing).
    const int kn = k + 1;
    if (kn < D - 2 && warp == (kn >> 2)) {
      const int mn = kn + 1;
      float sig = 0.f, c_x0 = 0.f, c_kk = 0.f;              // candidates for A[kn][mn], A[kn][kn]
#pragma unroll
      for (int t = 0; t < CH; ++t) {
        const int j0 = 4 * (q + 8 * t);
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          const float a = areg[t][c];
          const float xv = (j0 + c >= mn) ? a : 0.f;
          sig = fmaf(xv, xv, sig);
          if (j0 + c == mn) c_x0 = a;
          if (j0 + c == kn) c_kk = a;
        }
      }
      sig += __shfl_xor_sync(0xffffffffu, sig, 1);
      sig += __shfl_xor_sync(0xffffffffu, sig, 2);
      sig += __shfl_xor_sync(0xffffffffu, sig, 4);
      const float x0 = __shfl_sync(0xffffffffu, c_x0, (lane & 24) | ((mn >> 2) & 7));
      const float akk = __shfl_sync(0xffffffffu, c_kk, (lane & 24) | ((kn >> 2) & 7));
      if (r == kn) {
        const float rest = sig - x0 * x0;
        float bn = 0.f, alpha = x0, v0 = 0.f;
        const bool reflect = rest > 1e-30f;       // already tridiagonal in this column otherwise
        if (reflect) {
          // approximate root and reciprocal (a unit in the last place or two): the reflector stays
          // orthogonal to the same order as the float32 updates that apply it, and the two IEEE
          // operations were on the critical path of every one of the d - 2 steps
          float rt;
          asm("sqrt.approx.ftz.f32 %0, %1;" : "=f"(rt) : "f"(sig));
          alpha = x0 >= 0.f ? -rt : rt;
          v0 = x0 - alpha;
          asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(bn) : "f"(sig + fabsf(x0) * rt));
        }
        float* vn = vbuf + (kn & 1) * D;
#pragma unroll
        for (int t = 0; t < CH; ++t) {
          const int j0 = 4 * (q + 8 * t);
          float4 o;
          o.x = (reflect && j0 + 0 >= mn) ? (j0 + 0 == mn ? v0 : areg[t][0]) : 0.f;
          o.y = (reflect && j0 + 1 >= mn) ? (j0 + 1 == mn ? v0 : areg[t][1]) : 0.f;
          o.z = (reflect && j0 + 2 >= mn) ? (j0 + 2 == mn ? v0 : areg[t][2]) : 0.f;
          o.w = (reflect && j0 + 3 >= mn) ? (j0 + 3 == mn ? v0 : areg[t][3]) : 0.f;
          *reinterpret_cast<float4*>(&vn[j0]) = o;
        }
        if (q == 0) {
          beta[kn & 1] = bn;
          de[kn] = make_float2(akk, alpha);
        }
      }
    }
    __syncthreads();
  }
  // the last 2 x 2 block; the accumulated transform goes to shared memory for the rotations
  if (q == 7 && r == D - 2) de[D - 2] = make_float2(areg[CH - 1][2], areg[CH - 1][3]);
  if (q == 7 && r == D - 1) de[D - 1] = make_float2(areg[CH - 1][3], 0.f);
#pragma unroll
  for (int t = 0; t < CH; ++t)
#pragma unroll
    for (int c = 0; c < 4; ++c) Qt[(4 * (q + 8 * t) + c) * LDA + r] = qreg[t][c];
  __syncthreads();

  // ---- phase 2: divide and conquer.  A cut between rows k-1 and k writes T = diag(T1, T2) + rho u u^T
  // with rho = |b|, b the coupling of the two rows, u = e_{k-1} + sign(b) e_k, and b subtracted from the
  // two diagonal entries it touches.  Three cuts make four quarters, independent tridiagonal
  // problems: each gets its own QL warp and its own consumer threads (the rows of Qt of its
  // quarter), side by side -- a sixteenth of the rotation chain of the whole matrix each.  Two extra
  // columns of Qt (in the row padding) start as the u of the middle cut (column D) and of the two
  // outer cuts (column D + 1, disjoint rows) and go through the same rotations: afterwards they hold
  // z = Q^T u.  The quarters are merged pairwise into halves by the two halves of the CTA side by
  // side (column D travels through that merge), then the halves into the whole.
  constexpr int KH = D / 2, KQ = D / 4;
  constexpr int kParties = D + 64;                         // a QL warp + D + 2 columns rounded up to warps
  constexpr int kGroup = D + 32;                           // consumer threads of a quarter
  __shared__ float s_rho[3], s_theta[3];                   // cuts at KQ, KH, 3 KQ
  if (tid < 3) {
    const int k = (tid + 1) * KQ;
    const float bk = de[k - 1].y;
    s_rho[tid] = fabsf(bk);
    s_theta[tid] = bk < 0.f ? -1.f : 1.f;
    de[k - 1] = make_float2(de[k - 1].x - fabsf(bk), 0.f);
    de[k].x -= fabsf(bk);
  }
  for (int i = tid; i < D; i += NT) { Qt[i * LDA + D] = 0.f; Qt[i * LDA + D + 1] = 0.f; }
  __syncthreads();
  if (tid == 0) {
    Qt[(KH - 1) * LDA + D] = 1.f;          Qt[KH * LDA + D] = s_theta[1];
    Qt[(KQ - 1) * LDA + D + 1] = 1.f;      Qt[KQ * LDA + D + 1] = s_theta[0];
    Qt[(3 * KQ - 1) * LDA + D + 1] = 1.f;  Qt[3 * KQ * LDA + D + 1] = s_theta[2];
  }
  __syncthreads();
  // rotation lists: one array per buffer parity, indexed by the row, shared by the quarters
  if (warp < 4) {
    ql_producer(de, warp * KQ, (warp + 1) * KQ, rot, hdr + 8 * warp, 2 * D, 1 + 2 * warp, 2 + 2 * warp, kParties, lane);
  } else if (tid < 128 + 4 * kGroup) {
    const int g = (tid - 128) / kGroup;
    ql_consumer(Qt, LDA, (tid - 128) % kGroup, D + 2, rot, hdr + 8 * g, 2 * D, 1 + 2 * g, 2 + 2 * g, kParties);
  }
  __syncthreads();
  {
    const int g2 = tid / (NT / 2);
    merge_blocks<D, KH, NT / 2>(Qt, L, A, de, scratch, g2 * KH, D + 1, 1, s_rho[g2 ? 2 : 0], tid % (NT / 2), g2,
                                [&]() { named_sync(9 + g2, NT / 2); });
  }
  __syncthreads();
  { float* swap = Qt; Qt = L; L = swap; }
  merge_blocks<D, D, NT>(Qt, L, A, de, scratch, 0, D, 0, s_rho[1], tid, 0, [&]() { __syncthreads(); });
  { float* swap = Qt; Qt = L; L = swap; }
  // the factor of the sign rule (its space served the prologue and the merge)
  if (a.lift) {
    const double* F = a.lift + mat;
    for (int e = tid; e < D * D; e += NT) L[(e / D) * LDA + e % D] = (float)F[e];
  }
  __syncthreads();

  // ---- the map from the original space, W = F E (W[i][j] = sum_k F[i][k] Qt[j][k]), into A
  if (a.lift && tid < TILE_THREADS) {
    float acc[4][4];
    tile_product_rows<D>(L, Qt, LDA, tile_i, tile_j, acc);
#pragma unroll
    for (int x = 0; x < 4; ++x)
#pragma unroll
      for (int y = 0; y < 4; ++y) A[(4 * tile_i + x) * LDA + tile_j + (D / 4) * y] = acc[x][y];
  }
  // ---- order, sign, bias
  double* lam = reinterpret_cast<double*>(vbuf);             // [D] doubles over vbuf's 2D floats
  int* rank_of = reinterpret_cast<int*>(pbuf);
  float* sign_of = ubuf;
  float* mean = rot;                                         // the rotation lists are free now
  if (tid < D) {
    lam[tid] = (double)de[tid].x * a_scale;
    mean[tid] = a.mean_sum ? (float)(a.mean_sum[(size_t)blockIdx.x * D + tid] / a.mean_n) : 0.f;
  }
  __syncthreads();
  const bool lifted_out = a.lift && a.out_lifted;
  if (tid < D) {
    const double mine = lam[tid];
    int rank = 0;
#pragma unroll 16
    for (int k = 0; k < D; ++k) {
      const double other = lam[k];
      rank += (other > mine) || (other == mine && k < tid);
    }
    // sign rule on column tid of F E (of E when no factor is given); bias = -mean . (output column)
    float best = -1.f, sgn = 1.f, dot = 0.f;
#pragma unroll 8
    for (int i = 0; i < D; ++i) {
      const float e_i = Qt[tid * LDA + i];
      const float w_i = a.lift ? A[i * LDA + tid] : e_i;
      if (fabsf(w_i) > best) { best = fabsf(w_i); sgn = (w_i < 0.f) ? -1.f : 1.f; }
      dot = fmaf(mean[i], lifted_out ? w_i : e_i, dot);
    }
    rank_of[tid] = rank;
    sign_of[tid] = sgn;
    if (a.bias) a.bias[(size_t)blockIdx.x * D + rank] = -sgn * dot;
    if (a.evals) a.evals[(size_t)blockIdx.x * D + rank] = mine;
  }
  __syncthreads();
  // projection matrix [in i][out rank(j)], fp32, and its transpose as bf16 hi + lo parts
  for (int e = tid; e < D * D; e += NT) {
    const int i = e / D, j = e % D;
    const float v = sign_of[j] * (lifted_out ? A[i * LDA + j] : Qt[j * LDA + i]);
    a.W32[mat + (size_t)i * D + rank_of[j]] = v;
  }
  if (a.wt_hi) {
    for (int e = tid; e < D * D; e += NT) {
      const int j = e / D, i = e % D;
      const float v = sign_of[j] * (lifted_out ? A[i * LDA + j] : Qt[j * LDA + i]);
      const __nv_bfloat16 h = __float2bfloat16_rn(v);
      a.wt_hi[mat + (size_t)rank_of[j] * D + i] = h;
      a.wt_lo[mat + (size_t)rank_of[j] * D + i] = __float2bfloat16_rn(v - __bfloat162float(h));
    }
  }
}

int launch_pca(const PcaArgs& args, int count, int D, cudaStream_t st) {
  const size_t smem = sizeof(float) * ((size_t)3 * D * (D + 4) + 6 * D + 4 + 8 * D + 17 * D) + 32 * sizeof(int);
  if (D == 64) {
    auto k = eigh_tql_kernel<64>;
    CA_RETURN_IF_CUDA(cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    k<<<count, 8 * 64, smem, st>>>(args);
  } else {
    auto k = eigh_tql_kernel<128>;
    CA_RETURN_IF_CUDA(cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    k<<<count, 8 * 128, smem, st>>>(args);
  }
  CA_LAUNCH_CHECK();
  return CA_OK;
}

}  // namespace ca
