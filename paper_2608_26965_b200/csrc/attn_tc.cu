// Block-sparse attention with striped mean-compensation on the sm_100a tensor
// cores (eq. 2 over the selected clusters; Appendix A: an excluded cluster
// enters through its centroid key/value with weight |c| exp(q . kbar / sqrt(d))).
//
// One CTA per tile of 128 query rows (one query cluster, or half of a 256-row
// one).  Key/value tiles of 128 rows stream through shared memory by TMA
// (128-byte swizzle, 64-column panels).  For every tile
//     S = Q K^T          tcgen05.mma, both operands in shared memory, S in TMEM
//     P = exp2(S*c - m)  four softmax warps, one query row per thread; P is
//                        written back over S in TMEM as packed bf16
//     O += P V           tcgen05.mma, P from TMEM, V from shared memory (MN-major)
// with a running maximum that is only raised when a tile exceeds it by 2^8
// (the rescale of O in TMEM is then done by the softmax warps).  After the
// selected clusters, the key centroids are streamed the same way as extra
// "keys" (split into bf16 hi + lo parts so the logits keep fp32-level accuracy),
// with logit bias ln|c| and selected clusters masked; their values are the
// value centroids.  Warp 0 issues TMA, warp 1 issues MMAs, warps 2-5 do the
// softmax and the epilogue (rows scattered back to the original order).
// Two CTAs share an SM so one's softmax overlaps the other's MMAs.
#include "kernels.h"
#include "tc_ptx.cuh"

namespace ca {

using namespace ptx;

constexpr int kTcThreads = 192;
constexpr int kTile = 128;                 // query rows per CTA, key rows per tile
constexpr uint32_t kTmemCols = 256;        // S: [0,128)  O: [128, 128+D)
constexpr float kRescaleThreshold = 8.0f;  // log2 units

template <int D>
struct TcCfg {
  static constexpr int PANELS = D / 64;
  static constexpr int PANEL_BYTES = kTile * 128;            // 128 rows x 128 bytes
  static constexpr int TILE_BYTES = PANELS * PANEL_BYTES;
  static constexpr int STAGES = (D == 64) ? 2 : 1;
  // shared memory layout (offsets from a 1024-byte aligned base)
  static constexpr int OFF_Q = 0;
  static constexpr int OFF_K = OFF_Q + TILE_BYTES;
  static constexpr int OFF_V = OFF_K + STAGES * TILE_BYTES;
  static constexpr int OFF_BIAS = OFF_V + STAGES * TILE_BYTES;     // 2 x 128 floats
  static constexpr int OFF_BAR = OFF_BIAS + 2 * kTile * 4;
  static constexpr int NUM_BARS = 4 + 4 * STAGES;
  static constexpr int OFF_MISC = OFF_BAR + NUM_BARS * 8;           // tmem base, abort flag
  static constexpr int OFF_BITMAP = OFF_MISC + 16;
};

struct TcParams {
  const int32_t* count_k;
  const int32_t* block_idx;
  const int32_t* perm_q;
  __nv_bfloat16* O;
  float* lse;
  int* status;
  int n_q, n_k, c_q, c_k, keep, n_qc, n_kc, n_kc_pad, compensate, bitmap_words;
  float scale_log2;
};

// key rows of the selected clusters are consumed in tiles of 128 rows
__host__ __device__ inline int selected_tiles(int keep, int c_k) {
  return c_k >= kTile ? keep * (c_k / kTile) : (keep * c_k + kTile - 1) / kTile;
}

template <int D>
__global__ void __launch_bounds__(kTcThreads, 2)
attn_tc_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
               const __grid_constant__ CUtensorMap tm_v, const __grid_constant__ CUtensorMap tm_ckhi,
               const __grid_constant__ CUtensorMap tm_cklo, const __grid_constant__ CUtensorMap tm_cv,
               const TcParams prm) {
  using C = TcCfg<D>;
  extern __shared__ unsigned char smem_unaligned[];
  unsigned char* smem = reinterpret_cast<unsigned char*>(
      (reinterpret_cast<uintptr_t>(smem_unaligned) + 1023) & ~uintptr_t(1023));
  const uint32_t s_base = smem_u32(smem);
  const uint32_t s_q = s_base + C::OFF_Q, s_k = s_base + C::OFF_K, s_v = s_base + C::OFF_V;
  float* bias = reinterpret_cast<float*>(smem + C::OFF_BIAS);
  const uint32_t bar0 = s_base + C::OFF_BAR;
  // barrier indices
  const uint32_t b_q_full = bar0, b_s_full = bar0 + 8, b_p_ready = bar0 + 16, b_o_done = bar0 + 24;
  auto b_k_full = [&](int s) { return bar0 + 32 + 8 * s; };
  auto b_k_empty = [&](int s) { return bar0 + 32 + 8 * (C::STAGES + s); };
  auto b_v_full = [&](int s) { return bar0 + 32 + 8 * (2 * C::STAGES + s); };
  auto b_v_empty = [&](int s) { return bar0 + 32 + 8 * (3 * C::STAGES + s); };
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + C::OFF_MISC);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + C::OFF_MISC + 4);
  unsigned* bitmap = reinterpret_cast<unsigned*>(smem + C::OFF_BITMAP);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int p = blockIdx.y;
  const int tiles_per_qc = prm.c_q / kTile;
  const int qc = blockIdx.x / tiles_per_qc, half = blockIdx.x % tiles_per_qc;
  const int32_t* sel = prm.block_idx + ((size_t)p * prm.n_qc + qc) * prm.keep;
  const int sel_tiles = selected_tiles(prm.keep, prm.c_k);
  const int cen_tiles = prm.compensate ? prm.n_kc_pad / kTile : 0;
  const int total_tiles = sel_tiles + cen_tiles;

  if (tid == 0) {
    mbar_init(b_q_full, 1);
    mbar_init(b_s_full, 1);
    mbar_init(b_p_ready, 128);
    mbar_init(b_o_done, 1);
    for (int s = 0; s < C::STAGES; ++s) {
      mbar_init(b_k_full(s), 1); mbar_init(b_k_empty(s), 1);
      mbar_init(b_v_full(s), 1); mbar_init(b_v_empty(s), 1);
    }
    *abort_flag = 0;
    fence_mbar_init();
  }
  if (warp == 1) {                       // this warp owns the TMEM allocation
    tmem_alloc(smem_u32(tmem_slot), kTmemCols);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  const uint32_t tmem_s = tmem_base, tmem_o = tmem_base + kTile;

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer
    if (lane == 0) {
      prefetch_tensormap(&tm_q); prefetch_tensormap(&tm_k); prefetch_tensormap(&tm_v);
      const int q_row = (p * prm.n_qc + qc) * prm.c_q + half * kTile;
      mbar_expect_tx(b_q_full, C::TILE_BYTES);
      for (int pn = 0; pn < C::PANELS; ++pn) tma_load_2d(s_q + pn * C::PANEL_BYTES, &tm_q, pn * 64, q_row, b_q_full);
      int kg = 0;                          // key load groups issued so far
      bool ok = true;
      auto load_rows = [&](uint32_t dst, const CUtensorMap* map, int row, uint32_t bar) {
        for (int pn = 0; pn < C::PANELS; ++pn) tma_load_2d(dst + pn * C::PANEL_BYTES, map, pn * 64, row, bar);
      };
      // rows of a selected-cluster tile: sub-boxes of min(c_k, 128) rows
      auto load_selected = [&](uint32_t dst, const CUtensorMap* map, int t, uint32_t bar) {
        if (prm.c_k >= kTile) {
          const int per = prm.c_k / kTile;
          const int j = sel[t / per];
          load_rows(dst, map, (p * prm.n_kc + j) * prm.c_k + (t % per) * kTile, bar);
        } else {
          const int per = kTile / prm.c_k;
          for (int u = 0; u < per; ++u) {
            int e = t * per + u;
            if (e >= prm.keep) e = prm.keep - 1;          // filler rows, masked by the softmax
            const int j = sel[e];
            for (int pn = 0; pn < C::PANELS; ++pn)
              tma_load_2d(dst + pn * C::PANEL_BYTES + u * prm.c_k * 128, map, pn * 64,
                          (p * prm.n_kc + j) * prm.c_k, bar);
          }
        }
      };
      for (int t = 0; t < total_tiles && ok; ++t) {
        const int groups = t < sel_tiles ? 1 : 2;
        for (int g = 0; g < groups && ok; ++g, ++kg) {
          const int s = kg % C::STAGES;
          if (kg >= C::STAGES) ok = mbar_wait(b_k_empty(s), ((kg / C::STAGES) - 1) & 1, abort_flag, prm.status);
          if (!ok) break;
          mbar_expect_tx(b_k_full(s), C::TILE_BYTES);
          if (t < sel_tiles) load_selected(s_k + s * C::TILE_BYTES, &tm_k, t, b_k_full(s));
          else load_rows(s_k + s * C::TILE_BYTES, g == 0 ? &tm_ckhi : &tm_cklo,
                         p * prm.n_kc_pad + (t - sel_tiles) * kTile, b_k_full(s));
        }
        if (!ok) break;
        const int s = t % C::STAGES;
        if (t >= C::STAGES) ok = mbar_wait(b_v_empty(s), ((t / C::STAGES) - 1) & 1, abort_flag, prm.status);
        if (!ok) break;
        mbar_expect_tx(b_v_full(s), C::TILE_BYTES);
        if (t < sel_tiles) load_selected(s_v + s * C::TILE_BYTES, &tm_v, t, b_v_full(s));
        else load_rows(s_v + s * C::TILE_BYTES, &tm_cv, p * prm.n_kc_pad + (t - sel_tiles) * kTile, b_v_full(s));
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      constexpr uint32_t idesc_qk = idesc_bf16_f32(kTile, kTile, 0, 0);
      constexpr uint32_t idesc_pv = idesc_bf16_f32(kTile, D, 0, 1);
      bool ok = mbar_wait(b_q_full, 0, abort_flag, prm.status);
      int kg = 0;
      for (int t = 0; t < total_tiles && ok; ++t) {
        const int groups = t < sel_tiles ? 1 : 2;
        for (int g = 0; g < groups && ok; ++g, ++kg) {
          const int s = kg % C::STAGES;
          ok = mbar_wait(b_k_full(s), (kg / C::STAGES) & 1, abort_flag, prm.status);
          if (!ok) break;
          tc_fence_after();
#pragma unroll
          for (int ks = 0; ks < D / 16; ++ks) {
            // K-major operands: 16 elements (32 bytes) per step inside a 64-column panel
            const uint32_t off = (ks / 4) * C::PANEL_BYTES + (ks % 4) * 32;
            const uint64_t a = smem_desc_sw128(s_q + off, 16, 1024);
            const uint64_t b = smem_desc_sw128(s_k + s * C::TILE_BYTES + off, 16, 1024);
            mma_ss(tmem_s, a, b, idesc_qk, (g > 0 || ks > 0) ? 1u : 0u);
          }
          mma_commit(b_k_empty(s));
        }
        if (!ok) break;
        mma_commit(b_s_full);
        const int s = t % C::STAGES;
        ok = mbar_wait(b_p_ready, t & 1, abort_flag, prm.status) &&
             mbar_wait(b_v_full(s), (t / C::STAGES) & 1, abort_flag, prm.status);
        if (!ok) break;
        tc_fence_after();
#pragma unroll
        for (int ks = 0; ks < kTile / 16; ++ks) {
          // V is MN-major: 16 key rows (2048 bytes) per step; panels along d
          const uint64_t b = smem_desc_sw128(s_v + s * C::TILE_BYTES + ks * 2048, C::PANEL_BYTES, 1024);
          mma_ts(tmem_o, tmem_s + ks * 8, b, idesc_pv, (t > 0 || ks > 0) ? 1u : 0u);
        }
        mma_commit(b_v_empty(s));
      }
      mma_commit(b_o_done);
    }
  } else {
    // ------------------------------------------------------------ softmax + epilogue (128 threads)
    const int st = tid - 64;                       // 0..127
    const int quarter = warp & 3;                  // TMEM lanes this warp may touch
    const int row = quarter * 32 + lane;           // query row within the tile
    const uint32_t lane_addr = (uint32_t)(quarter * 32) << 16;
    const int32_t* cnt = prm.count_k + (size_t)p * prm.n_kc;
    for (int w = st; w < prm.bitmap_words; w += 128) bitmap[w] = 0u;
    asm volatile("bar.sync 1, 128;" ::: "memory");
    if (prm.compensate)
      for (int e = st; e < prm.keep; e += 128) atomicOr(&bitmap[sel[e] >> 5], 1u << (sel[e] & 31));
    asm volatile("bar.sync 1, 128;" ::: "memory");

    float m_ref = -INFINITY, l_run = 0.f;
    bool ok = true;
    long long T0 = 0, T1 = 0, T2 = 0, T3 = 0, tA, tB;
    const bool dbg = (blockIdx.x == 5 && blockIdx.y == 0 && st == 0);
    for (int t = 0; t < total_tiles && ok; ++t) {
      // per-column additive term (log2 units): only tiles with masked or weighted columns need it.
      // `masked` depends on the tile only, so it is uniform over the 128 threads.
      bool masked = false;
      float* bz = bias + (t & 1) * kTile;
      if (t < sel_tiles) {
        bool use;
        if (prm.c_k >= kTile) {
          const int per = prm.c_k / kTile;
          const int members = cnt[sel[t / per]];
          masked = members < prm.c_k;
          use = st < members - (t % per) * kTile;
        } else {
          const int per = kTile / prm.c_k;
          for (int u = 0; u < per; ++u) {
            const int e = t * per + u;
            if (e >= prm.keep || cnt[sel[e]] < prm.c_k) masked = true;
          }
          const int e = t * per + st / prm.c_k;
          use = e < prm.keep && (st % prm.c_k) < cnt[sel[min(e, prm.keep - 1)]];
        }
        if (masked) bz[st] = use ? 0.f : -INFINITY;
      } else {
        masked = true;
        const int j = (t - sel_tiles) * kTile + st;
        const bool use = j < prm.n_kc && !((bitmap[j >> 5] >> (j & 31)) & 1u);
        bz[st] = use ? log2f((float)cnt[min(j, prm.n_kc - 1)]) : -INFINITY;
      }
      if (masked) asm volatile("bar.sync 1, 128;" ::: "memory");

      tA = clock64();
      ok = __all_sync(0xffffffffu, mbar_wait(b_s_full, t & 1, abort_flag, prm.status));
      if (!ok) break;
      tc_fence_after();
      tB = clock64(); T0 += tB - tA;
      // ---- pass 1: row maximum (TMEM chunks of 32 columns, the next load in flight while one is reduced)
      uint32_t ra[32], rb[32];
      float mx0 = -INFINITY, mx1 = -INFINITY, mx2 = -INFINITY, mx3 = -INFINITY;
      auto reduce_max = [&](const uint32_t (&r)[32], int c4) {
        if (masked) {
#pragma unroll
          for (int j = 0; j < 32; j += 4) {
            mx0 = fmaxf(mx0, fmaf(__uint_as_float(r[j]), prm.scale_log2, bz[c4 * 32 + j]));
            mx1 = fmaxf(mx1, fmaf(__uint_as_float(r[j + 1]), prm.scale_log2, bz[c4 * 32 + j + 1]));
            mx2 = fmaxf(mx2, fmaf(__uint_as_float(r[j + 2]), prm.scale_log2, bz[c4 * 32 + j + 2]));
            mx3 = fmaxf(mx3, fmaf(__uint_as_float(r[j + 3]), prm.scale_log2, bz[c4 * 32 + j + 3]));
          }
        } else {
#pragma unroll
          for (int j = 0; j < 32; j += 8) {
            mx0 = fmaxf(mx0, fmaxf(__uint_as_float(r[j]), __uint_as_float(r[j + 1])));
            mx1 = fmaxf(mx1, fmaxf(__uint_as_float(r[j + 2]), __uint_as_float(r[j + 3])));
            mx2 = fmaxf(mx2, fmaxf(__uint_as_float(r[j + 4]), __uint_as_float(r[j + 5])));
            mx3 = fmaxf(mx3, fmaxf(__uint_as_float(r[j + 6]), __uint_as_float(r[j + 7])));
          }
        }
      };
      tmem_ld32(tmem_s + lane_addr, ra);
      tmem_wait_ld();
      tmem_ld32(tmem_s + lane_addr + 32, rb);
      reduce_max(ra, 0);
      tmem_wait_ld();
      tmem_ld32(tmem_s + lane_addr + 64, ra);
      reduce_max(rb, 1);
      tmem_wait_ld();
      tmem_ld32(tmem_s + lane_addr + 96, rb);
      reduce_max(ra, 2);
      tmem_wait_ld();
      tmem_ld32(tmem_s + lane_addr, ra);             // first chunk again, for pass 2
      reduce_max(rb, 3);
      float tmax = fmaxf(fmaxf(mx0, mx1), fmaxf(mx2, mx3));
      if (!masked) tmax *= prm.scale_log2;
      tA = clock64(); T1 += tA - tB;
      // raise the reference maximum only when a tile exceeds it by the threshold
      const bool raise = tmax > m_ref + kRescaleThreshold || (m_ref == -INFINITY && tmax > -INFINITY);
      if (__any_sync(0xffffffffu, raise)) {
        float alpha = 1.f;
        if (raise) {
          alpha = (m_ref == -INFINITY) ? 0.f : ex2_approx(m_ref - tmax);
          m_ref = tmax;
        }
        l_run *= alpha;
        if (t > 0) {                               // O holds the earlier tiles (their MMAs completed before S)
          tmem_wait_ld();
#pragma unroll
          for (int c4 = 0; c4 < D / 32; ++c4) {
            uint32_t o[32];
            tmem_ld32(tmem_o + lane_addr + c4 * 32, o);
            tmem_wait_ld();
#pragma unroll
            for (int j = 0; j < 32; ++j) o[j] = __float_as_uint(__uint_as_float(o[j]) * alpha);
            tmem_st32(tmem_o + lane_addr + c4 * 32, o);
          }
        }
      }
      // ---- pass 2: P = exp2(x - m), packed to bf16 over the S columns already consumed
      const float neg_m = (m_ref == -INFINITY) ? 0.f : -m_ref;
      float ps0 = 0.f, ps1 = 0.f, ps2 = 0.f, ps3 = 0.f;
      auto exp_chunk = [&](const uint32_t (&r)[32], int c4) {
        uint32_t pk[16];
#pragma unroll
        for (int j = 0; j < 16; j += 2) {
          float x0 = __uint_as_float(r[2 * j]), x1 = __uint_as_float(r[2 * j + 1]);
          float x2 = __uint_as_float(r[2 * j + 2]), x3 = __uint_as_float(r[2 * j + 3]);
          if (masked) {
            x0 = fmaf(x0, prm.scale_log2, bz[c4 * 32 + 2 * j] + neg_m);
            x1 = fmaf(x1, prm.scale_log2, bz[c4 * 32 + 2 * j + 1] + neg_m);
            x2 = fmaf(x2, prm.scale_log2, bz[c4 * 32 + 2 * j + 2] + neg_m);
            x3 = fmaf(x3, prm.scale_log2, bz[c4 * 32 + 2 * j + 3] + neg_m);
          } else {
            x0 = fmaf(x0, prm.scale_log2, neg_m); x1 = fmaf(x1, prm.scale_log2, neg_m);
            x2 = fmaf(x2, prm.scale_log2, neg_m); x3 = fmaf(x3, prm.scale_log2, neg_m);
          }
          const float p0 = ex2_approx(x0), p1 = ex2_approx(x1), p2 = ex2_approx(x2), p3 = ex2_approx(x3);
          ps0 += p0; ps1 += p1; ps2 += p2; ps3 += p3;
          pk[j] = pack_bf16x2(p0, p1);
          pk[j + 1] = pack_bf16x2(p2, p3);
        }
        tmem_st16(tmem_s + lane_addr + c4 * 16, pk);
      };
      // P chunk c overwrites S columns [16c, 16c+16), which pass 2 has read before (chunk c covers
      // S columns [32c, 32c+32) >= 16c+16 only for c >= 1; chunk 0 is held in registers first)
      tmem_wait_ld();
      tmem_ld32(tmem_s + lane_addr + 32, rb);
      tmem_wait_ld();                                // chunks 0 and 1 in registers before any P store
      exp_chunk(ra, 0);
      tmem_ld32(tmem_s + lane_addr + 64, ra);
      exp_chunk(rb, 1);
      tmem_wait_ld();
      tmem_ld32(tmem_s + lane_addr + 96, rb);
      exp_chunk(ra, 2);
      tmem_wait_ld();
      exp_chunk(rb, 3);
      const float psum = (ps0 + ps1) + (ps2 + ps3);
      l_run += psum;
      tB = clock64(); T2 += tB - tA;
      tmem_wait_st();
      tc_fence_before();
      mbar_arrive(b_p_ready);
      tA = clock64(); T3 += tA - tB;
    }

    if (dbg) { prm.status[8] = (int)(T0 >> 4); prm.status[9] = (int)(T1 >> 4); prm.status[10] = (int)(T2 >> 4); prm.status[11] = (int)(T3 >> 4); prm.status[12] = total_tiles; }
    // epilogue: O / l, rows back to their original positions
    if (ok) ok = __all_sync(0xffffffffu, mbar_wait(b_o_done, 0, abort_flag, prm.status));
    tc_fence_after();
    if (ok) {                                          // warp-uniform: TMEM loads are warp-collective
      const int pos = qc * prm.c_q + half * kTile + row;
      const bool live = pos < prm.n_q;                 // rows of the padding are not written
      const int orig = live ? prm.perm_q[(size_t)p * prm.n_q + pos] : 0;
      const float inv = 1.f / l_run;
      __nv_bfloat16* out = prm.O + ((size_t)p * prm.n_q + orig) * D;
#pragma unroll
      for (int c4 = 0; c4 < D / 32; ++c4) {
        uint32_t o[32];
        tmem_ld32(tmem_o + lane_addr + c4 * 32, o);
        tmem_wait_ld();
        if (live) {
          uint4* dst = reinterpret_cast<uint4*>(out + c4 * 32);
#pragma unroll
          for (int v = 0; v < 4; ++v) {
            uint4 w;
            w.x = pack_bf16x2(__uint_as_float(o[8 * v + 0]) * inv, __uint_as_float(o[8 * v + 1]) * inv);
            w.y = pack_bf16x2(__uint_as_float(o[8 * v + 2]) * inv, __uint_as_float(o[8 * v + 3]) * inv);
            w.z = pack_bf16x2(__uint_as_float(o[8 * v + 4]) * inv, __uint_as_float(o[8 * v + 5]) * inv);
            w.w = pack_bf16x2(__uint_as_float(o[8 * v + 6]) * inv, __uint_as_float(o[8 * v + 7]) * inv);
            dst[v] = w;
          }
        }
      }
      if (live && prm.lse) prm.lse[(size_t)p * prm.n_q + orig] = (m_ref + log2f(l_run)) * 0.6931471805599453f;
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) tmem_dealloc(tmem_base, kTmemCols);
}

// ---------------------------------------------------------------------------
// Centroids for the tensor-core path: key centroids as bf16 hi + lo parts, value
// centroids as bf16, rows padded with zeros to a multiple of 128.
// ---------------------------------------------------------------------------
__global__ void centroid_prep_kernel(const float* __restrict__ ck, const float* __restrict__ cv, int n_kc,
                                     int n_kc_pad, int D, __nv_bfloat16* __restrict__ hi,
                                     __nv_bfloat16* __restrict__ lo, __nv_bfloat16* __restrict__ vb) {
  const int p = blockIdx.y;
  const int e = blockIdx.x * blockDim.x + threadIdx.x;
  if (e >= n_kc_pad * D) return;
  const int j = e / D;
  float k = 0.f, v = 0.f;
  if (j < n_kc) {
    k = ck[(size_t)p * n_kc * D + e];
    v = cv[(size_t)p * n_kc * D + e];
  }
  const __nv_bfloat16 h = __float2bfloat16_rn(k);
  const size_t o = (size_t)p * n_kc_pad * D + e;
  hi[o] = h;
  lo[o] = __float2bfloat16_rn(k - __bfloat162float(h));
  vb[o] = __float2bfloat16_rn(v);
}

// ---------------------------------------------------------------------------
// host side
// ---------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void* ptr = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) == cudaSuccess &&
        qres == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(ptr);
  }
  return fn;
}

// bf16 matrix [rows, D] row-major; box = 64 columns x box_rows rows, 128-byte swizzle
static bool make_map(CUtensorMap* map, const void* base, size_t rows, int D, int box_rows) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  cuuint64_t dims[2] = {(cuuint64_t)D, (cuuint64_t)rows};
  cuuint64_t strides[1] = {(cuuint64_t)D * 2};
  cuuint32_t box[2] = {64, (cuuint32_t)box_rows};
  cuuint32_t estr[2] = {1, 1};
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

bool attn_tc_supported(const ca_problem_t& pr) {
  if (pr.dtype != CA_DTYPE_BF16 || (pr.flags & CA_ATTN_FP32)) return false;
  if (pr.cluster_q != 128 && pr.cluster_q != 256) return false;
  if (pr.cluster_k < 16 || pr.cluster_k > 256) return false;
  const int n_kc = ceil_div(pr.n_k, pr.cluster_k);
  if ((n_kc + 31) / 32 * 4 > 16384) return false;          // selected-cluster bitmap in shared memory
  return true;
}

size_t attn_tc_workspace_bytes(const ca_problem_t& pr) {
  const size_t P = (size_t)pr.batch * pr.heads;
  const size_t n_kc_pad = (size_t)align_up(ceil_div(pr.n_k, pr.cluster_k), kTile);
  return kStatusBytes + 3 * align_up(P * n_kc_pad * pr.head_dim * sizeof(__nv_bfloat16), 256);
}

template <int D>
static int launch_tc_d(const ca_problem_t& pr, const CUtensorMap* maps, const TcParams& prm, dim3 grid,
                       cudaStream_t st) {
  using C = TcCfg<D>;
  const size_t smem = 1024 + C::OFF_BITMAP + (size_t)prm.bitmap_words * 4;
  auto k = attn_tc_kernel<D>;
  CA_RETURN_IF_CUDA(cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  k<<<grid, kTcThreads, smem, st>>>(maps[0], maps[1], maps[2], maps[3], maps[4], maps[5], prm);
  CA_LAUNCH_CHECK();
  return CA_OK;
}

int launch_attn_tc(const ca_problem_t& pr, const void* Qp, const void* Kp, const void* Vp, const float* ck,
                   const float* cv, const int32_t* count_k, const int32_t* block_idx, const int32_t* perm_q,
                   float scale, void* O, float* lse, void* ws, cudaStream_t st) {
  const int P = pr.batch * pr.heads, D = pr.head_dim;
  const int n_qc = ceil_div(pr.n_q, pr.cluster_q), n_kc = ceil_div(pr.n_k, pr.cluster_k);
  const int n_kc_pad = (int)align_up(n_kc, kTile);
  Carver c(ws);
  int* status = c.take<int>(kStatusBytes / sizeof(int));
  __nv_bfloat16* hi = c.take<__nv_bfloat16>((size_t)P * n_kc_pad * D);
  __nv_bfloat16* lo = c.take<__nv_bfloat16>((size_t)P * n_kc_pad * D);
  __nv_bfloat16* vb = c.take<__nv_bfloat16>((size_t)P * n_kc_pad * D);
  if (pr.compensate) {
    centroid_prep_kernel<<<dim3(ceil_div(n_kc_pad * D, 256), P), 256, 0, st>>>(ck, cv, n_kc, n_kc_pad, D, hi, lo, vb);
    CA_LAUNCH_CHECK();
  }
  CUtensorMap maps[6];
  const int kbox = pr.cluster_k < kTile ? pr.cluster_k : kTile;
  bool ok = make_map(&maps[0], Qp, (size_t)P * n_qc * pr.cluster_q, D, kTile) &&
            make_map(&maps[1], Kp, (size_t)P * n_kc * pr.cluster_k, D, kbox) &&
            make_map(&maps[2], Vp, (size_t)P * n_kc * pr.cluster_k, D, kbox) &&
            make_map(&maps[3], hi, (size_t)P * n_kc_pad, D, kTile) &&
            make_map(&maps[4], lo, (size_t)P * n_kc_pad, D, kTile) &&
            make_map(&maps[5], vb, (size_t)P * n_kc_pad, D, kTile);
  if (!ok) return CA_ERR_CUDA;
  TcParams prm;
  prm.count_k = count_k; prm.block_idx = block_idx; prm.perm_q = perm_q;
  prm.O = static_cast<__nv_bfloat16*>(O); prm.lse = lse; prm.status = status;
  prm.n_q = pr.n_q; prm.n_k = pr.n_k; prm.c_q = pr.cluster_q; prm.c_k = pr.cluster_k; prm.keep = pr.keep;
  prm.n_qc = n_qc; prm.n_kc = n_kc; prm.n_kc_pad = n_kc_pad; prm.compensate = pr.compensate;
  prm.bitmap_words = (n_kc_pad + 31) / 32;
  prm.scale_log2 = scale * 1.4426950408889634f;
  dim3 grid(n_qc * (pr.cluster_q / kTile), P);
  if (D == 64) return launch_tc_d<64>(pr, maps, prm, grid, st);
  return launch_tc_d<128>(pr, maps, prm, grid, st);
}

}  // namespace ca
