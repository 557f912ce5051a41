// Tensor-core (tcgen05 + TMEM + TMA) kernels for the tall-skinny linear algebra
// of the clustering stage (Section 3.2.2 metric matrices, Section 3.2.1
// covariance and projection on the principal components):
//   gram_tc       G = X^T X and column sums of X   (X [N, d] bf16, optionally hi + lo parts)
//   transform_tc  Y = g(X W + b), g = identity or row normalisation
//                 (W [d, d] fp32 used as bf16 hi + lo parts; Y fp32, or bf16 hi + lo parts)
// A value v stored as hi + lo (hi = bf16(v), lo = bf16(v - hi)) keeps 16 bits of
// mantissa; products use hi*hi + hi*lo + lo*hi with fp32 accumulation.
#include "kernels.h"
#include "tc_ptx.cuh"

namespace ca {

using namespace ptx;

constexpr int kLinThreads = 192;     // warp 0: TMA, warp 1: MMA, warps 2-5: epilogue
constexpr int kRows = 128;           // rows per tile

__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* map, int x, int y, int z,
                                            uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
      ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(z), "r"(bar)
      : "memory");
}
__device__ __forceinline__ void tma_store_3d(const CUtensorMap* map, int x, int y, int z, uint32_t src) {
  asm volatile("cp.async.bulk.tensor.3d.global.shared::cta.bulk_group [%0, {%1, %2, %3}], [%4];"
               ::"l"(map), "r"(x), "r"(y), "r"(z), "r"(src)
               : "memory");
}
__device__ __forceinline__ void tma_store_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
__device__ __forceinline__ void tma_store_wait_read() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }
__device__ __forceinline__ void tma_store_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }

// ===========================================================================
// Gram matrix + column sums
// ===========================================================================
template <int D>
struct GramCfg {
  static constexpr int PANELS = D / 64;
  static constexpr int PANEL_BYTES = kRows * 128;
  static constexpr int TILE_BYTES = PANELS * PANEL_BYTES;       // one part (hi or lo)
  static constexpr int M = D;                                   // 64 or 128 accumulator rows
};

struct GramParams {
  float* partial;        // [(p * n_chunks + chunk) * (D*D + D)]
  int* status;
  int n_rows, chunk_rows, n_chunks, has_lo, stages;
};

template <int D>
__global__ void __launch_bounds__(kLinThreads, 1)
gram_tc_kernel(const __grid_constant__ CUtensorMap tm_hi, const __grid_constant__ CUtensorMap tm_lo,
               const GramParams prm) {
  using C = GramCfg<D>;
  extern __shared__ unsigned char smem_unaligned[];
  unsigned char* smem = reinterpret_cast<unsigned char*>(
      (reinterpret_cast<uintptr_t>(smem_unaligned) + 1023) & ~uintptr_t(1023));
  const int parts = prm.has_lo ? 2 : 1;
  const int stage_bytes = parts * C::TILE_BYTES;
  const uint32_t s_base = smem_u32(smem);
  const uint32_t s_ones = s_base + prm.stages * stage_bytes;                // 2 KB of bf16 1.0
  const uint32_t bar0 = s_ones + 2048;
  auto b_full = [&](int s) { return bar0 + 8 * s; };
  auto b_empty = [&](int s) { return bar0 + 8 * (prm.stages + s); };
  const uint32_t b_done = bar0 + 8 * (2 * prm.stages);
  unsigned char* misc = smem + prm.stages * stage_bytes + 2048 + 8 * (2 * prm.stages + 1);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(misc);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(misc + 4);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int p = blockIdx.y, chunk = blockIdx.x;
  const int r_begin = chunk * prm.chunk_rows;
  const int r_end = min(prm.n_rows, r_begin + prm.chunk_rows);
  const int n_tiles = (r_end - r_begin + kRows - 1) / kRows;
  constexpr uint32_t kCols = (D + 16 <= 128) ? 128 : 256;

  if (tid == 0) {
    for (int s = 0; s < prm.stages; ++s) { mbar_init(b_full(s), 1); mbar_init(b_empty(s), 1); }
    mbar_init(b_done, 1);
    *abort_flag = 0;
    fence_mbar_init();
  }
  for (int e = tid; e < 1024; e += kLinThreads)
    reinterpret_cast<__nv_bfloat16*>(smem + prm.stages * stage_bytes)[e] = __float2bfloat16_rn(1.0f);
  fence_proxy_async();                 // the ones are read by the tensor core (async proxy)
  if (warp == 1) { tmem_alloc(smem_u32(tmem_slot), kCols); tmem_relinquish(); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_acc = *tmem_slot, tmem_sum = tmem_acc + D;

  if (warp == 0) {
    if (lane == 0) {
      bool ok = true;
      for (int t = 0; t < n_tiles && ok; ++t) {
        const int s = t % prm.stages;
        if (t >= prm.stages) ok = mbar_wait(b_empty(s), ((t / prm.stages) - 1) & 1, abort_flag, prm.status);
        if (!ok) break;
        mbar_expect_tx(b_full(s), stage_bytes);
        const uint32_t dst = s_base + s * stage_bytes;
        for (int pn = 0; pn < C::PANELS; ++pn) {
          tma_load_3d(dst + pn * C::PANEL_BYTES, &tm_hi, pn * 64, r_begin + t * kRows, p, b_full(s));
          if (prm.has_lo)
            tma_load_3d(dst + C::TILE_BYTES + pn * C::PANEL_BYTES, &tm_lo, pn * 64, r_begin + t * kRows, p, b_full(s));
        }
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      constexpr uint32_t idesc = idesc_bf16_f32(C::M, D, 1, 1);        // X^T X: both operands MN-major
      constexpr uint32_t idesc_sum = idesc_bf16_f32(C::M, 16, 1, 1);
      bool ok = true;
      for (int t = 0; t < n_tiles && ok; ++t) {
        const int s = t % prm.stages;
        ok = mbar_wait(b_full(s), (t / prm.stages) & 1, abort_flag, prm.status);
        if (!ok) break;
        tc_fence_after();
        const uint32_t hi = s_base + s * stage_bytes, lo = hi + C::TILE_BYTES;
#pragma unroll
        for (int ks = 0; ks < kRows / 16; ++ks) {
          // 16 rows (the contraction index) per step = 2048 bytes; 64-column panels along M and N
          const uint64_t dh = smem_desc_sw128(hi + ks * 2048, C::PANEL_BYTES, 1024);
          const uint64_t ones = smem_desc_sw128(s_ones, C::PANEL_BYTES, 1024);
          const uint32_t acc = (t > 0 || ks > 0) ? 1u : 0u;
          mma_ss(tmem_acc, dh, dh, idesc, acc);
          mma_ss(tmem_sum, dh, ones, idesc_sum, acc);
          if (prm.has_lo) {
            const uint64_t dl = smem_desc_sw128(lo + ks * 2048, C::PANEL_BYTES, 1024);
            mma_ss(tmem_acc, dh, dl, idesc, 1u);
            mma_ss(tmem_acc, dl, dh, idesc, 1u);
            mma_ss(tmem_sum, dl, ones, idesc_sum, 1u);
          }
        }
        mma_commit(b_empty(s));
      }
      mma_commit(b_done);
    }
  } else {
    const int quarter = warp & 3;
    const uint32_t lane_addr = (uint32_t)(quarter * 32) << 16;
    const bool ok = __all_sync(0xffffffffu, mbar_wait(b_done, 0, abort_flag, prm.status));
    tc_fence_after();
    if (ok) {
      // accumulator row m sits in lane m (M = 128) or in lane (m % 16) + 32 (m / 16) (M = 64)
      const int m = (C::M == 128) ? quarter * 32 + lane : quarter * 16 + lane;
      const bool live = (C::M == 128) || lane < 16;
      float* out = prm.partial + ((size_t)p * prm.n_chunks + chunk) * (D * D + D);
#pragma unroll
      for (int c4 = 0; c4 < D / 32; ++c4) {
        uint32_t v[32];
        tmem_ld32(tmem_acc + lane_addr + c4 * 32, v);
        tmem_wait_ld();
        if (live && n_tiles > 0) {
          float4* dst = reinterpret_cast<float4*>(out + m * D + c4 * 32);
#pragma unroll
          for (int j = 0; j < 8; ++j)
            dst[j] = make_float4(__uint_as_float(v[4 * j]), __uint_as_float(v[4 * j + 1]),
                                 __uint_as_float(v[4 * j + 2]), __uint_as_float(v[4 * j + 3]));
        }
      }
      uint32_t sv[32];
      tmem_ld32(tmem_sum + lane_addr, sv);          // 16 identical sums; columns beyond are unused
      tmem_wait_ld();
      if (live && n_tiles > 0) out[D * D + m] = __uint_as_float(sv[0]);
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) tmem_dealloc(tmem_acc, kCols);
}

// ===========================================================================
// Row transform
// ===========================================================================
template <int D>
struct LinCfg {
  static constexpr int PANELS = D / 64;
  static constexpr int PANEL_BYTES = kRows * 128;               // X panels: 128 rows x 128 bytes
  static constexpr int TILE_BYTES = PANELS * PANEL_BYTES;       // one part of an X tile
  static constexpr int W_PANEL_BYTES = D * 128;                 // W^T panels: D rows x 128 bytes
  static constexpr int W_BYTES = PANELS * W_PANEL_BYTES;        // one part of W^T
  static constexpr int OUT_BYTES = kRows * D * 4;               // fp32 tile, or hi + lo bf16 tiles
};

struct LinParams {
  const float* bias;      // [P][D] or null
  float* out_t;           // [P][D][n_rows] or null: the fp32 result once more, coordinate-major
  int* status;
  int n_rows, tiles_per_cta, has_lo, stages, normalize, out_split;
};

template <int D>
__global__ void __launch_bounds__(kLinThreads, 1)
transform_tc_kernel(const __grid_constant__ CUtensorMap tm_xhi, const __grid_constant__ CUtensorMap tm_xlo,
                    const __grid_constant__ CUtensorMap tm_whi, const __grid_constant__ CUtensorMap tm_wlo,
                    const __grid_constant__ CUtensorMap tm_out, const __grid_constant__ CUtensorMap tm_out_lo,
                    const LinParams prm) {
  using C = LinCfg<D>;
  extern __shared__ unsigned char smem_unaligned[];
  unsigned char* smem = reinterpret_cast<unsigned char*>(
      (reinterpret_cast<uintptr_t>(smem_unaligned) + 1023) & ~uintptr_t(1023));
  const int parts = prm.has_lo ? 2 : 1;
  const int stage_bytes = parts * C::TILE_BYTES;
  const uint32_t s_base = smem_u32(smem);
  const uint32_t s_w = s_base;                                   // W^T hi, W^T lo
  const uint32_t s_x = s_w + 2 * C::W_BYTES;
  const uint32_t s_out = s_x + prm.stages * stage_bytes;
  unsigned char* out_ptr = smem + 2 * C::W_BYTES + prm.stages * stage_bytes;
  const uint32_t bar0 = s_out + C::OUT_BYTES;
  const uint32_t b_w = bar0;
  auto b_full = [&](int s) { return bar0 + 8 + 8 * s; };
  auto b_empty = [&](int s) { return bar0 + 8 + 8 * (prm.stages + s); };
  auto b_acc_full = [&](int a) { return bar0 + 8 + 8 * (2 * prm.stages + a); };
  auto b_acc_empty = [&](int a) { return bar0 + 8 + 8 * (2 * prm.stages + 2 + a); };
  unsigned char* misc = out_ptr + C::OUT_BYTES + 8 * (2 * prm.stages + 5);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(misc);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(misc + 4);
  float* s_bias = reinterpret_cast<float*>(misc + 16);            // [D]

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int p = blockIdx.y;
  const int total_tiles = (prm.n_rows + kRows - 1) / kRows;
  const int t_begin = blockIdx.x * prm.tiles_per_cta;
  const int n_tiles = max(0, min(total_tiles, t_begin + prm.tiles_per_cta) - t_begin);
  constexpr uint32_t kCols = 2 * D;                              // two accumulators

  if (tid == 0) {
    mbar_init(b_w, 1);
    for (int s = 0; s < prm.stages; ++s) { mbar_init(b_full(s), 1); mbar_init(b_empty(s), 1); }
    for (int a = 0; a < 2; ++a) { mbar_init(b_acc_full(a), 1); mbar_init(b_acc_empty(a), 128); }
    *abort_flag = 0;
    fence_mbar_init();
  }
  for (int j = tid; j < D; j += kLinThreads) s_bias[j] = prm.bias ? prm.bias[(size_t)p * D + j] : 0.f;
  if (warp == 1) { tmem_alloc(smem_u32(tmem_slot), kCols); tmem_relinquish(); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    if (lane == 0) {
      mbar_expect_tx(b_w, 2 * C::W_BYTES);
      for (int pn = 0; pn < C::PANELS; ++pn) {
        tma_load_2d(s_w + pn * C::W_PANEL_BYTES, &tm_whi, pn * 64, p * D, b_w);
        tma_load_2d(s_w + C::W_BYTES + pn * C::W_PANEL_BYTES, &tm_wlo, pn * 64, p * D, b_w);
      }
      bool ok = true;
      for (int t = 0; t < n_tiles && ok; ++t) {
        const int s = t % prm.stages;
        if (t >= prm.stages) ok = mbar_wait(b_empty(s), ((t / prm.stages) - 1) & 1, abort_flag, prm.status);
        if (!ok) break;
        mbar_expect_tx(b_full(s), stage_bytes);
        const uint32_t dst = s_x + s * stage_bytes;
        const int row = (t_begin + t) * kRows;
        for (int pn = 0; pn < C::PANELS; ++pn) {
          tma_load_3d(dst + pn * C::PANEL_BYTES, &tm_xhi, pn * 64, row, p, b_full(s));
          if (prm.has_lo) tma_load_3d(dst + C::TILE_BYTES + pn * C::PANEL_BYTES, &tm_xlo, pn * 64, row, p, b_full(s));
        }
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      constexpr uint32_t idesc = idesc_bf16_f32(kRows, D, 0, 0);    // X (K-major) times W^T (K-major)
      bool ok = mbar_wait(b_w, 0, abort_flag, prm.status);
      for (int t = 0; t < n_tiles && ok; ++t) {
        const int s = t % prm.stages, a = t & 1;
        if (t >= 2) ok = mbar_wait(b_acc_empty(a), ((t >> 1) - 1) & 1, abort_flag, prm.status);
        if (ok) ok = mbar_wait(b_full(s), (t / prm.stages) & 1, abort_flag, prm.status);
        if (!ok) break;
        tc_fence_after();
        const uint32_t xh = s_x + s * stage_bytes, xl = xh + C::TILE_BYTES;
        const uint32_t acc = tmem_base + a * D;
#pragma unroll
        for (int ks = 0; ks < D / 16; ++ks) {
          const uint32_t xo = (ks / 4) * C::PANEL_BYTES + (ks % 4) * 32;
          const uint32_t wo = (ks / 4) * C::W_PANEL_BYTES + (ks % 4) * 32;
          const uint64_t dxh = smem_desc_sw128(xh + xo, 16, 1024);
          const uint64_t dwh = smem_desc_sw128(s_w + wo, 16, 1024);
          const uint64_t dwl = smem_desc_sw128(s_w + C::W_BYTES + wo, 16, 1024);
          mma_ss(acc, dxh, dwh, idesc, ks > 0 ? 1u : 0u);
          mma_ss(acc, dxh, dwl, idesc, 1u);
          if (prm.has_lo) mma_ss(acc, smem_desc_sw128(xl + xo, 16, 1024), dwh, idesc, 1u);
        }
        mma_commit(b_empty(s));
        mma_commit(b_acc_full(a));
      }
    }
  } else {
    const int st = tid - 64;
    const int quarter = warp & 3;
    const int row = quarter * 32 + lane;
    const uint32_t lane_addr = (uint32_t)(quarter * 32) << 16;
    bool ok = true;
    for (int t = 0; t < n_tiles && ok; ++t) {
      const int a = t & 1;
      ok = __all_sync(0xffffffffu, mbar_wait(b_acc_full(a), (t >> 1) & 1, abort_flag, prm.status));
      if (!ok) break;
      tc_fence_after();
      float v[D];
#pragma unroll
      for (int c4 = 0; c4 < D / 32; ++c4) {
        uint32_t r[32];
        tmem_ld32(tmem_base + a * D + lane_addr + c4 * 32, r);
        tmem_wait_ld();
#pragma unroll
        for (int j = 0; j < 32; ++j) v[c4 * 32 + j] = __uint_as_float(r[j]) + s_bias[c4 * 32 + j];
      }
      tc_fence_before();
      mbar_arrive(b_acc_empty(a));                    // the accumulator may be overwritten
      if (prm.normalize) {
        float ss = 0.f;
#pragma unroll
        for (int j = 0; j < D; ++j) ss = fmaf(v[j], v[j], ss);
        const float nrm = sqrtf(ss);
        const float inv = nrm >= 1e-30f ? 1.f / nrm : 0.f;
#pragma unroll
        for (int j = 0; j < D; ++j) v[j] *= inv;
      }
      if (prm.out_t) {
        // coordinate-major copy: for one coordinate the 128 threads of the tile write 512
        // consecutive bytes.  The splitter gathers one coordinate of scattered rows per level; from
        // this layout that is a 4-byte read inside an L2-resident column instead of one DRAM line
        // per row of the row-major result.
        const int grow = (t_begin + t) * kRows + row;
        if (grow < prm.n_rows) {
          float* dst = prm.out_t + (size_t)p * D * prm.n_rows + grow;
#pragma unroll
          for (int j = 0; j < D; ++j) dst[(size_t)j * prm.n_rows] = v[j];
        }
      }
      // the previous tile's stores must have finished reading the staging buffer
      if (st == 0) tma_store_wait_read();
      asm volatile("bar.sync 1, 128;" ::: "memory");
      if (!prm.out_split) {
        // fp32 tile as 32-column panels with the 128-byte swizzle the store expects
#pragma unroll
        for (int pn = 0; pn < D / 32; ++pn)
#pragma unroll
          for (int c = 0; c < 8; ++c) {
            float4 w = make_float4(v[pn * 32 + 4 * c], v[pn * 32 + 4 * c + 1], v[pn * 32 + 4 * c + 2], v[pn * 32 + 4 * c + 3]);
            *reinterpret_cast<float4*>(out_ptr + pn * 16384 + row * 128 + ((c ^ (row & 7)) * 16)) = w;
          }
      } else {
        // bf16 hi and lo tiles as 64-column panels
#pragma unroll
        for (int pn = 0; pn < D / 64; ++pn)
#pragma unroll
          for (int c = 0; c < 8; ++c) {
            uint32_t h[4], l[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
              const float x0 = v[pn * 64 + 8 * c + 2 * j], x1 = v[pn * 64 + 8 * c + 2 * j + 1];
              const __nv_bfloat16 h0 = __float2bfloat16_rn(x0), h1 = __float2bfloat16_rn(x1);
              h[j] = pack_bf16x2(__bfloat162float(h0), __bfloat162float(h1));
              l[j] = pack_bf16x2(x0 - __bfloat162float(h0), x1 - __bfloat162float(h1));
            }
            const int off = pn * 16384 + row * 128 + ((c ^ (row & 7)) * 16);
            *reinterpret_cast<uint4*>(out_ptr + off) = make_uint4(h[0], h[1], h[2], h[3]);
            *reinterpret_cast<uint4*>(out_ptr + C::OUT_BYTES / 2 + off) = make_uint4(l[0], l[1], l[2], l[3]);
          }
      }
      fence_proxy_async();
      asm volatile("bar.sync 1, 128;" ::: "memory");
      if (st == 0) {
        const int grow = (t_begin + t) * kRows;
        if (!prm.out_split) {
          for (int pn = 0; pn < D / 32; ++pn) tma_store_3d(&tm_out, pn * 32, grow, p, s_out + pn * 16384);
        } else {
          for (int pn = 0; pn < D / 64; ++pn) {
            tma_store_3d(&tm_out, pn * 64, grow, p, s_out + pn * 16384);
            tma_store_3d(&tm_out_lo, pn * 64, grow, p, s_out + C::OUT_BYTES / 2 + pn * 16384);
          }
        }
        tma_store_commit();
      }
    }
    if (st == 0) tma_store_wait_all();
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) tmem_dealloc(tmem_base, kCols);
}

// W [P][D in][D out] fp32  ->  W^T hi / lo [P][D out][D in] bf16
__global__ void weight_prep_kernel(const float* __restrict__ W, int D, __nv_bfloat16* __restrict__ hi,
                                   __nv_bfloat16* __restrict__ lo) {
  const int p = blockIdx.y;
  const int e = blockIdx.x * blockDim.x + threadIdx.x;
  if (e >= D * D) return;
  const int n = e / D, k = e % D;
  const float w = W[(size_t)p * D * D + k * D + n];
  const __nv_bfloat16 h = __float2bfloat16_rn(w);
  hi[(size_t)p * D * D + e] = h;
  lo[(size_t)p * D * D + e] = __float2bfloat16_rn(w - __bfloat162float(h));
}

// ---------------------------------------------------------------------------
// host side
// ---------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

static EncodeTiledFn lin_encode_fn() {
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

// [P][n][D] tensor; box = box_cols x box_rows x 1, 128-byte swizzle
static bool map_3d(CUtensorMap* map, const void* base, int P, int n, int D, int elem_bytes, int box_cols,
                   int box_rows) {
  EncodeTiledFn fn = lin_encode_fn();
  if (!fn) return false;
  cuuint64_t dims[3] = {(cuuint64_t)D, (cuuint64_t)n, (cuuint64_t)P};
  cuuint64_t strides[2] = {(cuuint64_t)D * elem_bytes, (cuuint64_t)n * D * elem_bytes};
  cuuint32_t box[3] = {(cuuint32_t)box_cols, (cuuint32_t)box_rows, 1};
  cuuint32_t estr[3] = {1, 1, 1};
  return fn(map, elem_bytes == 2 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3,
            const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
            CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}
static bool map_2d(CUtensorMap* map, const void* base, size_t rows, int D, int box_rows) {
  EncodeTiledFn fn = lin_encode_fn();
  if (!fn) return false;
  cuuint64_t dims[2] = {(cuuint64_t)D, (cuuint64_t)rows};
  cuuint64_t strides[1] = {(cuuint64_t)D * 2};
  cuuint32_t box[2] = {64, (cuuint32_t)box_rows};
  cuuint32_t estr[2] = {1, 1};
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Chunks of rows per problem, one CTA each, `ctas_per_sm` of them resident per SM: the count that
// minimises rounds x (tiles per chunk + 3), the time of the launch in tiles when every CTA pays
// about three tiles' worth of start-up and epilogue and a last round that is nearly empty costs a
// full round (320 CTAs on 148 slots run as long as 444); chunks of at least four tiles.
int gram_tc_chunking(int n_rows, int problems, int ctas_per_sm, int* chunk_rows, int* n_chunks) {
  int sms = 148, dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess ||
      cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms < 1) {
    (void)cudaGetLastError();
    sms = 148;
  }
  const long long slots = (long long)sms * (ctas_per_sm > 0 ? ctas_per_sm : 1);
  const int tiles = ceil_div(n_rows, kRows);
  int best_c = 1, best_cr = tiles * kRows;
  long long best_cost = -1;
  for (int c = 1; c <= tiles; ++c) {
    const int ct = ceil_div(tiles, c);                     // tiles per chunk
    if (c > 1 && ct < 4) break;
    const int cr = ct * kRows;
    const int chunks = ceil_div(n_rows, cr);
    const long long total = (long long)chunks * problems;
    const long long rounds = (total + slots - 1) / slots;
    const long long cost = rounds * (ct + 3);
    if (best_cost < 0 || cost < best_cost) { best_cost = cost; best_c = chunks; best_cr = cr; }
    if (rounds > 8) break;
  }
  // the buffer of partial sums is sized for the chunk count of the CUDA-core moments kernel
  int m_cr, m_chunks;
  moments_chunking(n_rows, problems, &m_cr, &m_chunks);
  if (best_c > m_chunks) {
    best_cr = ceil_div(ceil_div(n_rows, m_chunks), kRows) * kRows;
    best_c = ceil_div(n_rows, best_cr);
  }
  *chunk_rows = best_cr;
  *n_chunks = best_c;
  return 0;
}

int launch_gram_tc(const void* X_hi, const void* X_lo, int problems, int n_rows, int D, float* partial,
                   double* gram, double* colsum, int* status, cudaStream_t st) {
  GramParams prm;
  prm.partial = partial; prm.status = status; prm.n_rows = n_rows; prm.has_lo = X_lo ? 1 : 0;
  const int tile = kRows * D * 2 * (X_lo ? 2 : 1);
  prm.stages = (200 * 1024 - 4096) / tile;
  if (prm.stages > 6) prm.stages = 6;
  // one part per tile (32 KB at d = 128): three stages, so that two CTAs share an SM and one's
  // start-up and epilogue overlap the other's streaming (video480: 0.36 -> 0.34 ms for the step's
  // three launches)
  if (!X_lo && prm.stages > 3) prm.stages = 3;
  {
    const size_t smem_cta = 1024 + (size_t)prm.stages * tile + 2048 + 8 * (2 * prm.stages + 1) + 64 + 1024;
    int per_sm = (int)((227 * 1024) / smem_cta);
    const int by_tmem = 512 / ((D + 16 <= 128) ? 128 : 256);
    if (per_sm > by_tmem) per_sm = by_tmem;
    gram_tc_chunking(n_rows, problems, per_sm, &prm.chunk_rows, &prm.n_chunks);
  }
  CUtensorMap mh, ml;
  if (!map_3d(&mh, X_hi, problems, n_rows, D, 2, 64, kRows)) return CA_ERR_CUDA;
  if (!map_3d(&ml, X_lo ? X_lo : X_hi, problems, n_rows, D, 2, 64, kRows)) return CA_ERR_CUDA;
  const size_t smem = 1024 + (size_t)prm.stages * tile + 2048 + 8 * (2 * prm.stages + 1) + 64;
  dim3 grid(prm.n_chunks, problems);
  if (D == 64) {
    auto k = gram_tc_kernel<64>;
    CA_RETURN_IF_CUDA(cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    k<<<grid, kLinThreads, smem, st>>>(mh, ml, prm);
  } else {
    auto k = gram_tc_kernel<128>;
    CA_RETURN_IF_CUDA(cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    k<<<grid, kLinThreads, smem, st>>>(mh, ml, prm);
  }
  CA_LAUNCH_CHECK();
  return launch_gram_finalize(partial, problems, prm.n_chunks, D, gram, colsum, st);
}

int launch_transform_tc(const void* X_hi, const void* X_lo, int problems, int n_rows, int D, const float* W,
                        const float* bias, int normalize, float* out, void* out_hi, void* out_lo,
                        void* wt_hi, void* wt_lo, int* status, cudaStream_t st, float* out_t, bool weights_ready) {
  if (!weights_ready) {               // otherwise the kernel that produced W has laid it out
    weight_prep_kernel<<<dim3(ceil_div(D * D, 256), problems), 256, 0, st>>>(
        W, D, static_cast<__nv_bfloat16*>(wt_hi), static_cast<__nv_bfloat16*>(wt_lo));
    CA_LAUNCH_CHECK();
  }
  LinParams prm;
  prm.bias = bias; prm.out_t = out ? out_t : nullptr; prm.status = status; prm.n_rows = n_rows; prm.has_lo = X_lo ? 1 : 0;
  prm.normalize = normalize; prm.out_split = out ? 0 : 1;
  const int tile = kRows * D * 2 * (X_lo ? 2 : 1);
  const int fixed = 2 * D * D * 2 + kRows * D * 4 + 4096;
  prm.stages = (200 * 1024 - fixed) / tile;
  if (prm.stages > 4) prm.stages = 4;
  if (prm.stages < 1) return CA_ERR_UNSUPPORTED;
  const int total_tiles = ceil_div(n_rows, kRows);
  int ctas = 296 / problems;
  if (ctas < 1) ctas = 1;
  prm.tiles_per_cta = ceil_div(total_tiles, ctas);
  if (prm.tiles_per_cta < 2) prm.tiles_per_cta = 2;
  CUtensorMap mxh, mxl, mwh, mwl, mo, mol;
  bool ok = map_3d(&mxh, X_hi, problems, n_rows, D, 2, 64, kRows) &&
            map_3d(&mxl, X_lo ? X_lo : X_hi, problems, n_rows, D, 2, 64, kRows) &&
            map_2d(&mwh, wt_hi, (size_t)problems * D, D, D) && map_2d(&mwl, wt_lo, (size_t)problems * D, D, D);
  if (out) ok = ok && map_3d(&mo, out, problems, n_rows, D, 4, 32, kRows) && map_3d(&mol, out, problems, n_rows, D, 4, 32, kRows);
  else ok = ok && map_3d(&mo, out_hi, problems, n_rows, D, 2, 64, kRows) && map_3d(&mol, out_lo, problems, n_rows, D, 2, 64, kRows);
  if (!ok) return CA_ERR_CUDA;
  const size_t smem = 1024 + (size_t)fixed + (size_t)prm.stages * tile + D * 4;
  dim3 grid(ceil_div(total_tiles, prm.tiles_per_cta), problems);
  if (D == 64) {
    auto k = transform_tc_kernel<64>;
    CA_RETURN_IF_CUDA(cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    k<<<grid, kLinThreads, smem, st>>>(mxh, mxl, mwh, mwl, mo, mol, prm);
  } else {
    auto k = transform_tc_kernel<128>;
    CA_RETURN_IF_CUDA(cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    k<<<grid, kLinThreads, smem, st>>>(mxh, mxl, mwh, mwl, mo, mol, prm);
  }
  CA_LAUNCH_CHECK();
  return CA_OK;
}

}  // namespace ca
