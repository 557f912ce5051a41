// Block-sparse attention with striped mean-compensation on the sm_100a tensor
// cores (eq. 2 over the selected clusters; Appendix A: an excluded cluster
// enters through its centroid key/value with weight |c| exp(q . kbar / sqrt(d))).
//
// One CTA per tile of 128 query rows (one query cluster, half of a 256-row one,
// or a 64-row one in a half-filled tile).  Per CTA the half-steps of 64 keys form
// one dependent chain, so what counts is the number of chains per SM: at d = 64 a
// CTA holds one 64-column score buffer and 64 output columns in tensor memory and
// four CTAs share an SM; at d = 128 two score buffers and 128 output columns, two
// CTAs per SM (TcCfg).  Key and value rows stream through shared memory by TMA in
// slots of 64 rows (128-byte swizzle, 64-column panels), loaded in the order the
// tensor core consumes them:
//     S_b = Q K_h^T        tcgen05.mma, Q and K from shared memory (K-major)
//     P_b = exp2(S_b c - m) four softmax warps, one query row per thread; P is
//                          written back over S_b as packed bf16; row sums in fp32
//                          registers
//     O  += P_b V_h        tcgen05.mma, P from tensor memory, V from shared memory (MN-major)
// issued as S(0) [S(1)] | PV(0) S(NBUF) | PV(1) S(NBUF + 1) | ...  The softmax keeps
// a reference m per row instead of the exact running maximum: it is measured on a
// row's first half-step, afterwards gathered with the exponentials and raised one
// half-step late (by an integer, when a half-step exceeded it by 2^8), the softmax
// warps then rescale O in tensor memory themselves after waiting for the one
// product that can still be in flight; a climb beyond 2^96 inside one half-step
// marks the tile for the second pass of the fp32 kernel.  After the selected
// clusters the key centroids are streamed as extra keys, 64 per half-step: their
// tile holds bf16 hi parts in rows 0-63 and lo parts in rows 64-127, accumulated
// by two products so the centroid logits keep fp32-level accuracy; logit bias
// ln|c|, selected clusters masked; values are the value centroids.  Block lists
// may be ragged (a length per query cluster).  Warp 0 issues TMA, warp 1 issues
// MMAs (all lanes run the loop, one elected lane issues), warps 2-5 do the softmax
// and the epilogue (rows scattered back to the original order).
// Indices that come from the caller (block lists, list lengths, perm_q) are range-
// checked before use: a bad one sets CA_ERR_BAD_INDEX in the status word and the
// access is skipped (the cluster is masked, the row is not written).
#include "kernels.h"
#include "tc_ptx.cuh"

namespace ca {

using namespace ptx;

constexpr int kTcThreads = 192;
constexpr int kTile = 128;                 // query rows per CTA, key rows per tile
constexpr int kHalf = 64;                  // keys per half-step
constexpr float kRescaleThreshold = 8.0f;  // log2 units
constexpr float kDanger = 96.0f;            // log2 units: exp2 arguments stay below this

// F8: queries, keys and key centroids arrive as E4M3 codes (one byte per element: a 128-byte row
// of a panel holds 128 of them) and Q K^T runs as kind::f8f6f4 products; values stay bf16.
template <int D, bool F8 = false>
struct TcCfg {
  static constexpr int PANELS = D / 64;                      // value panels (bf16: 64 elements per 128-byte row)
  static constexpr int QK_PANELS = F8 ? D / 128 : D / 64;    // query / key panels
  static constexpr int QK_PANEL_COLS = F8 ? 128 : 64;        // elements per panel row
  static constexpr int QK_KSTEP = F8 ? 32 : 16;              // elements per tensor-core instruction (32 bytes)
  static constexpr int PANEL_BYTES = kTile * 128;            // query tile: 128 rows x 128 bytes per panel
  static constexpr int TILE_BYTES = QK_PANELS * PANEL_BYTES;
  static constexpr int HALF_PANEL_BYTES = kHalf * 128;       // key/value slot: 64 rows x 128 bytes per panel
  static constexpr int HALF_BYTES = PANELS * HALF_PANEL_BYTES;        // a value slot
  static constexpr int KHALF_BYTES = QK_PANELS * HALF_PANEL_BYTES;    // a key slot
  static constexpr int CEN_PARTS = F8 ? 1 : 2;               // key slots of a centroid half-step (bf16: hi and lo parts)
  // Per CTA the half-steps form one dependent chain (scores -> softmax -> P V -> next scores) whose
  // length is set by latencies, not by any pipe, and an SM has throughput to spare: what counts is
  // the number of such chains per SM.  d = 64: one 64-column score buffer + 64 output columns =
  // 128 columns of tensor memory and 48 KB of shared memory per CTA, four CTAs per SM.  d = 128: the
  // output alone takes 128 columns; two score buffers, 256 columns, two CTAs per SM.
  static constexpr int NBUF = (D == 64) ? 1 : 2;
  static constexpr int NBAR = 2;                              // barrier rings (>= every lead below)
  static constexpr uint32_t TMEM_COLS = (D == 64) ? 128 : 256;
  static constexpr int CTAS_PER_SM = (D == 64) ? 4 : 2;
  // key and value slots of 64 rows (one half-step each; a centroid half-step takes two key slots).
  // The keys of half-step i are loaded once S(i - K_LEAD) has completed, so the slots of at most
  // K_LEAD half-steps are live (K_LEAD_CEN for centroid half-steps); likewise for the values.
  static constexpr int NK = 2;
  static constexpr int NV = 2;
  static constexpr int K_LEAD = 2;
  static constexpr int K_LEAD_CEN = 1;
  static constexpr int PV_N = D;
  // How the softmax notices a probability above 2^threshold.  d = 128: it keeps the largest
  // exponent of the half-step.  d = 64: no exponent is tracked; such a probability shows in its
  // chunk's row sum, and the sum bounds it from above, so the reference moves up by the sum's
  // exponent (too far by at most log2(32), which costs nothing in fp32 / bf16).  Measured: d = 64
  // 0.916 -> 0.895 ms without the tracking, d = 128 2.90 -> 2.95 ms.
  static constexpr bool TRACK_MAX = D != 64;
  static constexpr bool Q_IN_TMEM = false;
  static constexpr int TMEM_Q = 0;
  // shared memory layout (offsets from a 1024-byte aligned base)
  static constexpr int OFF_Q = 0;
  static constexpr int OFF_K = OFF_Q + TILE_BYTES;
  static constexpr int OFF_V = OFF_K + NK * KHALF_BYTES;
  static constexpr int OFF_BIAS = OFF_V + NV * HALF_BYTES;                     // 8 x 64 floats
  static constexpr int OFF_BAR = OFF_BIAS + 8 * kHalf * 4;
  static constexpr int NUM_BARS = 3 + 3 * NBAR + NK + NV;           // q_full, o_done, q_tmem, three rings, per slot
  static constexpr int OFF_MISC = OFF_BAR + NUM_BARS * 8;           // tmem base, abort flag
  static constexpr int OFF_BITMAP = OFF_MISC + 16;
};

struct TcParams {
  const int32_t* count_k;
  const int32_t* block_idx;
  const int32_t* keep_count;      // per query cluster list length, or null: every list holds `keep` entries
  const int32_t* perm_q;
  __nv_bfloat16* O;
  float* lse;
  int* status;
  int32_t* redo;                  // [B*H, n_qc, 2] per CTA: scores left the range of the fast softmax
  int n_q, n_k, c_q, c_k, keep, list_stride, n_qc, n_kc, cen_tiles, compensate, bitmap_words;
  float scale_log2;
  // quantised Q K^T: de-quantisation scales of the query rows [B*H*n_qc*c_q], of the key clusters
  // [B*H*n_kc] and of the runs of 64 key centroids [B*H*cen_tiles]; null otherwise
  const float* q_scale;
  const float* k_scale;
  const float* c_scale;
  long long wait_limit;           // SM cycles after which a barrier wait gives up (CA_ERR_TIMEOUT)
  int skip_key_load;              // diagnostic hook: the loader leaves out the keys of this half-step (-1: none)
};

constexpr int kErrBadIndex = 6;   // CA_ERR_BAD_INDEX

// key rows of the selected clusters are consumed in tiles of 128 rows
__host__ __device__ inline int selected_tiles(int keep, int c_k) {
  return c_k >= kTile ? keep * (c_k / kTile) : (keep * c_k + kTile - 1) / kTile;
}

template <int D, bool F8>
__global__ void __launch_bounds__(kTcThreads, TcCfg<D, F8>::CTAS_PER_SM)
attn_tc_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
               const __grid_constant__ CUtensorMap tm_v, const __grid_constant__ CUtensorMap tm_ck,
               const __grid_constant__ CUtensorMap tm_cv, const TcParams prm) {
  using C = TcCfg<D, F8>;
  extern __shared__ unsigned char smem_unaligned[];
  unsigned char* smem = reinterpret_cast<unsigned char*>(
      (reinterpret_cast<uintptr_t>(smem_unaligned) + 1023) & ~uintptr_t(1023));
  const uint32_t s_base = smem_u32(smem);
  const uint32_t s_q = s_base + C::OFF_Q, s_k = s_base + C::OFF_K, s_v = s_base + C::OFF_V;
  float* bias = reinterpret_cast<float*>(smem + C::OFF_BIAS);
  const uint32_t bar0 = s_base + C::OFF_BAR;
  const uint32_t b_q_full = bar0, b_o_done = bar0 + 8, b_q_tmem = bar0 + 16;
  auto b_s_full = [&](int b) { return bar0 + 24 + 8 * b; };
  auto b_p_ready = [&](int b) { return bar0 + 24 + 8 * (C::NBAR + b); };
  auto b_pv_done = [&](int b) { return bar0 + 24 + 8 * (2 * C::NBAR + b); };
  auto b_k_full = [&](int s) { return bar0 + 24 + 8 * (3 * C::NBAR + s); };
  auto b_v_full = [&](int s) { return bar0 + 24 + 8 * (3 * C::NBAR + C::NK + s); };
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + C::OFF_MISC);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + C::OFF_MISC + 4);
  volatile int* redo_flag = reinterpret_cast<volatile int*>(smem + C::OFF_MISC + 8);
  unsigned* bitmap = reinterpret_cast<unsigned*>(smem + C::OFF_BITMAP);
  // member counts of the selected clusters, in list order: looked up every half-step, so they are
  // fetched from global memory once instead of sitting on each half-step's critical path
  uint16_t* members_of = reinterpret_cast<uint16_t*>(bitmap + prm.bitmap_words);
  // quantised Q K^T: de-quantisation scale of every selected key cluster, in list order
  float* kscale_of = reinterpret_cast<float*>(reinterpret_cast<unsigned char*>(members_of) +
                                              (((size_t)prm.list_stride * 2 + 15) & ~(size_t)15));

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int p = blockIdx.y;
  // a query cluster of 256 rows takes two CTAs; one of 64 rows fills the upper half of a tile
  // (the lower half is zeros and the warps that own those rows only keep the barriers going)
  const int tiles_per_qc = prm.c_q >= kTile ? prm.c_q / kTile : 1;
  const int q_rows = prm.c_q >= kTile ? kTile : prm.c_q;
  const int qc = blockIdx.x / tiles_per_qc, half = blockIdx.x % tiles_per_qc;
  const int32_t* sel = prm.block_idx + ((size_t)p * prm.n_qc + qc) * prm.list_stride;
  int keep = prm.keep_count ? prm.keep_count[(size_t)p * prm.n_qc + qc] : prm.keep;
  if (keep < 0 || keep > prm.list_stride) {            // a list length that does not fit its row
    if (tid == 0) atomicCAS(prm.status, 0, kErrBadIndex);
    keep = keep < 0 ? 0 : prm.list_stride;
  }
  const int sel_tiles = selected_tiles(keep, prm.c_k);
  const int cen_tiles = prm.compensate ? prm.cen_tiles : 0;
  const int steps = 2 * sel_tiles + cen_tiles;         // half-steps of 64 keys

  if (tid == 0) {
    mbar_init(b_q_full, 1);
    mbar_init(b_q_tmem, 4);
    mbar_init(b_o_done, 1);
    for (int b = 0; b < C::NBAR; ++b) { mbar_init(b_s_full(b), 1); mbar_init(b_p_ready(b), 4); mbar_init(b_pv_done(b), 1); }
    for (int s = 0; s < C::NK; ++s) mbar_init(b_k_full(s), 1);
    for (int s = 0; s < C::NV; ++s) mbar_init(b_v_full(s), 1);
    *abort_flag = 0;
    *redo_flag = 0;
    fence_mbar_init();
  }
  if (q_rows < kTile) {
    // rows [q_rows, 128) of every Q panel: zeros (read by the tensor core through the async proxy)
    for (int e = tid; e < C::QK_PANELS * (kTile - q_rows) * 8; e += kTcThreads) {
      const int pn = e / ((kTile - q_rows) * 8), rem = e % ((kTile - q_rows) * 8);
      *reinterpret_cast<uint4*>(smem + C::OFF_Q + pn * C::PANEL_BYTES + q_rows * 128 + rem * 16) = make_uint4(0u, 0u, 0u, 0u);
    }
    fence_proxy_async();
  }
  if (warp == 1) {                       // this warp owns the TMEM allocation
    tmem_alloc(smem_u32(tmem_slot), C::TMEM_COLS);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  const uint32_t tmem_s = tmem_base, tmem_o = tmem_base + C::NBUF * kHalf;
  // key slots used before half-step u (a centroid half-step takes two: hi and lo parts)
  auto kslot_of = [&](int u) { return u < 2 * sel_tiles ? u : 2 * sel_tiles + C::CEN_PARTS * (u - 2 * sel_tiles); };

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer
    // Loads run in the order the tensor core consumes them: the keys of half-step i (needed by
    // S(i), issued NBUF half-steps early) and the values of half-step i - NBUF.  A slot is free
    // again when the product that read it has completed, which is what the barriers s_full and
    // pv_done of that half-step announce; no separate "empty" barriers or commits.
    if (lane == 0) {
      prefetch_tensormap(&tm_q); prefetch_tensormap(&tm_k); prefetch_tensormap(&tm_v);
      const int q_row = (p * prm.n_qc + qc) * prm.c_q + half * kTile;
      mbar_expect_tx(b_q_full, C::QK_PANELS * q_rows * 128);
      for (int pn = 0; pn < C::QK_PANELS; ++pn)
        tma_load_2d(s_q + pn * C::PANEL_BYTES, &tm_q, pn * C::QK_PANEL_COLS, q_row, b_q_full);
      bool ok = true;
      // `key`: rows of keys or key centroids (their panels), otherwise rows of values
      auto load_rows = [&](uint32_t dst, const CUtensorMap* map, int row, uint32_t bar, bool key) {
        const int panels = key ? C::QK_PANELS : C::PANELS, cols = key ? C::QK_PANEL_COLS : 64;
        for (int pn = 0; pn < panels; ++pn) tma_load_2d(dst + pn * C::HALF_PANEL_BYTES, map, pn * cols, row, bar);
      };
      // the 64 rows of half-step u of the selected clusters: one box, or several boxes of c_k rows
      auto load_selected = [&](uint32_t dst, const CUtensorMap* map, int u, uint32_t bar, bool key) {
        if (prm.c_k >= kHalf) {
          const int pos = u * kHalf;                       // position in the concatenated selected rows
          int j = sel[min(pos / prm.c_k, keep - 1)];     // a filler half-step repeats the last cluster (masked)
          j = min(max(j, 0), prm.n_kc - 1);                // out-of-range entries are flagged and masked by the softmax warps
          load_rows(dst, map, (p * prm.n_kc + j) * prm.c_k + pos % prm.c_k, bar, key);
        } else {
          const int per = kHalf / prm.c_k;
          for (int x = 0; x < per; ++x) {
            int e = u * per + x;
            if (e >= keep) e = keep - 1;                   // filler rows, masked by the softmax
            const int j = min(max(sel[e], 0), prm.n_kc - 1);
            const int panels = key ? C::QK_PANELS : C::PANELS, cols = key ? C::QK_PANEL_COLS : 64;
            for (int pn = 0; pn < panels; ++pn)
              tma_load_2d(dst + pn * C::HALF_PANEL_BYTES + x * prm.c_k * 128, map, pn * cols,
                          (p * prm.n_kc + j) * prm.c_k, bar);
          }
        }
      };
      // A slot is reused when the product that read it has completed.  Products complete in the
      // order of their issue, so it is enough to wait for a later one; the one waited for is chosen
      // so that its barrier cannot complete another phase before this thread has looked (the next
      // product on the same score buffer needs the very load that follows the wait).
      for (int i = 0; i < steps + C::NBUF && ok; ++i) {
        if (i < steps) {
          const bool centroid = i >= 2 * sel_tiles;
          const int parts = centroid ? C::CEN_PARTS : 1;
          const int w = i - (centroid ? C::K_LEAD_CEN : C::K_LEAD);
          if (w >= 0) ok = mbar_wait_relaxed(b_s_full(w % C::NBAR), (w / C::NBAR) & 1, abort_flag, prm.status, prm.wait_limit);
          for (int g = 0; g < parts && ok; ++g) {
            const int kc = kslot_of(i) + g, slot = kc % C::NK;
            if (i == prm.skip_key_load) continue;          // diagnostic: this slot never fills, its waiters time out
            mbar_expect_tx(b_k_full(slot), C::KHALF_BYTES);
            const uint32_t dst = s_k + slot * C::KHALF_BYTES;
            if (!centroid) load_selected(dst, &tm_k, i, b_k_full(slot), true);
            else load_rows(dst, &tm_ck, (p * prm.cen_tiles + (i - 2 * sel_tiles)) * (C::CEN_PARTS * kHalf) + g * kHalf,
                           b_k_full(slot), true);
          }
        }
        const int j = i - C::NBUF;
        if (j >= 0 && ok) {
          const int slot = j % C::NV;
          const int w = j - C::NV;
          if (w >= 0) ok = mbar_wait_relaxed(b_pv_done(w % C::NBAR), (w / C::NBAR) & 1, abort_flag, prm.status, prm.wait_limit);
          if (!ok) break;
          mbar_expect_tx(b_v_full(slot), C::HALF_BYTES);
          const uint32_t dst = s_v + slot * C::HALF_BYTES;
          if (j < 2 * sel_tiles) load_selected(dst, &tm_v, j, b_v_full(slot), false);
          else load_rows(dst, &tm_cv, (p * prm.cen_tiles + (j - 2 * sel_tiles)) * kHalf, b_v_full(slot), false);
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer
    // every lane runs the loop (waits and descriptor arithmetic stay warp-uniform); one elected
    // lane issues the tensor-core instructions
    {
      constexpr uint32_t idesc_qk = F8 ? idesc_e4m3_f32(kTile, kHalf) : idesc_bf16_f32(kTile, kHalf, 0, 0);
      constexpr uint32_t idesc_pv = idesc_bf16_f32(kTile, C::PV_N, 0, 1);
      bool ok = __all_sync(0xffffffffu, mbar_wait(b_q_full, 0, abort_flag, prm.status, prm.wait_limit));
      // descriptors differ from a base one only in the start-address field (units of 16 bytes):
      // the base descriptors are built once, the per-instruction part is an addition
      const uint64_t q_desc0 = smem_desc_sw128(s_q, 16, 1024);
      const uint64_t k_desc0 = smem_desc_sw128(s_k, 16, 1024);
      const uint64_t v_desc0 = smem_desc_sw128(s_v, C::HALF_PANEL_BYTES, 1024);
      // The tensor core sits idle between the softmax's arrival and the next product, so that
      // stretch is kept short: everything a product needs besides the probabilities -- its key and
      // value slots (loaded long before) and their descriptors -- is waited for and computed BEFORE
      // the wait for the softmax, and P V (u) and S(u + NBUF) are then issued back to back.
      auto wait_keys = [&](int un) {
        const int parts = un >= 2 * sel_tiles ? C::CEN_PARTS : 1;      // centroid keys as bf16: hi parts, then lo parts
        bool got = true;
        for (int g = 0; g < parts && got; ++g) {
          const int kc = kslot_of(un) + g;
          got = __all_sync(0xffffffffu, mbar_wait(b_k_full(kc % C::NK), (kc / C::NK) & 1, abort_flag, prm.status, prm.wait_limit));
        }
        return got;
      };
      // first key slot and number of parts of S(un); fire_s (elected lane) issues it
      auto fire_s = [&](uint32_t d_cols, int kc0, int parts, uint32_t bar) {
        for (int g = 0; g < parts; ++g) {
          const uint64_t kd = k_desc0 + ((((kc0 + g) % C::NK) * C::KHALF_BYTES) >> 4);
#pragma unroll
          for (int ks = 0; ks < D / C::QK_KSTEP; ++ks) {
            // K-major operands: 32 bytes (16 bf16 or 32 E4M3 elements) per step, four steps per panel
            const uint32_t qoff = ((ks / 4) * C::PANEL_BYTES + (ks % 4) * 32) >> 4;
            const uint32_t koff = ((ks / 4) * C::HALF_PANEL_BYTES + (ks % 4) * 32) >> 4;
            if (F8) mma_ss_f8(d_cols, q_desc0 + qoff, kd + koff, idesc_qk, (g > 0 || ks > 0) ? 1u : 0u);
            else mma_ss(d_cols, q_desc0 + qoff, kd + koff, idesc_qk, (g > 0 || ks > 0) ? 1u : 0u);
          }
        }
        mma_commit(bar);
      };
      for (int u = 0; u < C::NBUF && u < steps && ok; ++u) {
        ok = wait_keys(u);
        if (!ok) break;
        tc_fence_after();
        if (elect_one())
          fire_s(tmem_s + (u % C::NBUF) * kHalf, kslot_of(u), u >= 2 * sel_tiles ? C::CEN_PARTS : 1, b_s_full(u % C::NBAR));
        __syncwarp();
      }
      for (int u = 0; u < steps && ok; ++u) {
        const int slot = u % C::NV, un = u + C::NBUF;
        ok = __all_sync(0xffffffffu, mbar_wait(b_v_full(slot), (u / C::NV) & 1, abort_flag, prm.status, prm.wait_limit));
        if (ok && un < steps) ok = wait_keys(un);
        // V is MN-major: 16 key rows (2048 bytes) per instruction; panels along d
        const uint64_t vd = v_desc0 + ((slot * C::HALF_BYTES) >> 4);
        const uint32_t p_cols = tmem_s + (u % C::NBUF) * kHalf;
        const uint32_t s_cols = tmem_s + (un % C::NBUF) * kHalf, s_bar = b_s_full(un % C::NBAR), pv_bar = b_pv_done(u % C::NBAR);
        const int s_kc0 = kslot_of(un), s_parts = un >= steps ? 0 : (un >= 2 * sel_tiles ? C::CEN_PARTS : 1);
        if (ok) ok = __all_sync(0xffffffffu, mbar_wait(b_p_ready(u % C::NBAR), (u / C::NBAR) & 1, abort_flag, prm.status, prm.wait_limit));
        if (!ok) break;
        tc_fence_after();
        if (elect_one()) {
#pragma unroll
          for (int ks = 0; ks < kHalf / 16; ++ks)
            mma_ts(tmem_o, p_cols + ks * 8, vd + (uint64_t)(ks * (2048 >> 4)), idesc_pv, (u > 0 || ks > 0) ? 1u : 0u);
          mma_commit(pv_bar);
          if (s_parts) fire_s(s_cols, s_kc0, s_parts, s_bar);
        }
        __syncwarp();
      }
      if (elect_one()) mma_commit(b_o_done);
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
    for (int e = st; e < keep; e += 128) {
      const int j = sel[e];
      if (j < 0 || j >= prm.n_kc) {                        // not a key cluster: flagged, all of its columns masked
        atomicCAS(prm.status, 0, kErrBadIndex);
        members_of[e] = 0;
        if (F8) kscale_of[e] = 0.f;
        continue;
      }
      members_of[e] = (uint16_t)min(max(cnt[j], 0), prm.c_k);
      if (F8) kscale_of[e] = prm.k_scale[(size_t)p * prm.n_kc + j];
      if (prm.compensate) atomicOr(&bitmap[j >> 5], 1u << (j & 31));
    }
    asm volatile("bar.sync 1, 128;" ::: "memory");

    if (C::Q_IN_TMEM) {
      // this thread's query row: eight 16-byte chunks, stored at chunk position c ^ (row & 7)
      bool q_ok = __all_sync(0xffffffffu, mbar_wait(b_q_full, 0, abort_flag, prm.status, prm.wait_limit));
      uint32_t qw[32];
#pragma unroll
      for (int c = 0; c < 8; ++c) {
        const uint4 v = *reinterpret_cast<const uint4*>(smem + C::OFF_Q + row * 128 + ((c ^ (row & 7)) << 4));
        qw[4 * c] = v.x; qw[4 * c + 1] = v.y; qw[4 * c + 2] = v.z; qw[4 * c + 3] = v.w;
      }
      (void)q_ok;
      tmem_st32(tmem_base + C::TMEM_Q + lane_addr, qw);
      tmem_wait_st();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(b_q_tmem);
    }
    float m_ref = -INFINITY, l_run = 0.f, pend = 0.f;
    const int ck_shift = __ffs(prm.c_k) - 1;
    // factor from a raw score to log2 units: the softmax scale, and with quantised Q K^T the scale
    // of this thread's query row (times, per half-step, the scale of the key cluster or centroid run)
    float row_sc = prm.scale_log2;
    if (F8) {
      const int qrow = (p * prm.n_qc + qc) * prm.c_q + half * kTile + (row < q_rows ? row : 0);
      row_sc *= prm.q_scale[qrow];
    }
    // A warp whose wait gave up goes through the remaining half-steps without touching anything
    // (`dead`), so that it still meets the other softmax warps at the barriers they share.
    bool dead = false;
    for (int u = 0; u < steps; ++u) {
      const int b = u & 1;                               // half of a 128-row tile (geometry of the keys)
      const int buf = u % C::NBUF;                       // score buffer
      const uint32_t t_s = tmem_s + lane_addr + buf * kHalf;
      // per-column additive term (log2 units): only half-steps with masked or weighted columns need
      // it.  `masked` depends on the half-step only, so it is uniform over the 128 threads.
      bool masked = false;
      // eight buffers: a thread can run at most NBUF half-steps ahead of the slowest one
      float* bz = bias + (u & 7) * kHalf;
      if (u < 2 * sel_tiles) {
        // cluster sizes are powers of two: positions are split with shifts and masks
        const int t = u >> 1;
        bool use = true;
        if (prm.c_k >= kTile) {
          const int e = t >> (ck_shift - 7);                      // c_k / 128 tiles per cluster
          const int members = members_of[e];
          const int first = ((t << 7) & (prm.c_k - 1)) + b * kHalf;   // row of this half-step's first column
          masked = members < first + kHalf;
          use = first + (st & 63) < members;
        } else {
          const int col0 = t * kTile + b * kHalf;                // position in the list of selected rows
          const int e_first = col0 >> ck_shift, e_last = (col0 + kHalf - 1) >> ck_shift;
          for (int e = e_first; e <= e_last; ++e)
            if (e >= keep || members_of[e] < prm.c_k) masked = true;
          const int e = (col0 + (st & 63)) >> ck_shift;
          use = e < keep && ((col0 + (st & 63)) & (prm.c_k - 1)) < members_of[min(e, keep - 1)];
        }
        if (masked && st < kHalf) bz[st] = use ? 0.f : -INFINITY;
      } else {
        masked = true;
        const int j = (u - 2 * sel_tiles) * kHalf + (st & 63);
        const bool use = j < prm.n_kc && !((bitmap[j >> 5] >> (j & 31)) & 1u);
        if (st < kHalf) bz[st] = use ? log2f((float)cnt[min(j, prm.n_kc - 1)]) : -INFINITY;
      }
      if (masked) asm volatile("bar.sync 1, 128;" ::: "memory");
      if (dead) continue;
      // scale of this half-step's scores.  A zero scale (an all-zero query row or key group) makes
      // every logit 0: the raw scores are then dropped and the additive terms enter with scale 1.
      float sc_used = prm.scale_log2;
      bool keep_raw = true;
      if (F8) {
        const float ks = u < 2 * sel_tiles ? kscale_of[min((u * kHalf) >> ck_shift, max(keep - 1, 0))]
                                           : prm.c_scale[(size_t)p * prm.cen_tiles + (u - 2 * sel_tiles)];
        const float sc_eff = row_sc * ks;
        keep_raw = sc_eff > 0.f;
        sc_used = keep_raw ? sc_eff : (masked ? 1.f : 0.f);
      }

      if (!__all_sync(0xffffffffu, mbar_wait(b_s_full(u % C::NBAR), (u / C::NBAR) & 1, abort_flag, prm.status, prm.wait_limit))) {
        dead = true;
        continue;
      }
      tc_fence_after();
      if (quarter * 32 >= q_rows) {          // this warp's rows are padding of a 64-row query cluster
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(b_p_ready(u % C::NBAR));
        continue;
      }
      // The loops over the two 32-column chunks are kept rolled: the body of a half-step is
      // executed by every softmax warp of both resident CTAs at different places, and an unrolled
      // body does not stay in the instruction cache.
      // ---- masked / weighted half-steps (short clusters, centroid columns): the additive term is
      // folded into the scores in tensor memory first, so that the common path below has no bias
      if (masked) {
        const float inv_scale_log2 = __fdividef(1.f, sc_used);
        const float raw_factor = keep_raw ? 1.f : 0.f;
#pragma unroll 1
        for (int c4 = 0; c4 < 2; ++c4) {
          uint32_t r[32];
          tmem_ld32(t_s + c4 * 32, r);
          tmem_wait_ld();
#pragma unroll
          for (int j = 0; j < 32; ++j) {
            const float raw = F8 ? __uint_as_float(r[j]) * raw_factor : __uint_as_float(r[j]);
            r[j] = __float_as_uint(fmaf(bz[c4 * 32 + j], inv_scale_log2, raw));
          }
          tmem_st32(t_s + c4 * 32, r);
        }
        tmem_wait_st();
      }
      // ---- reference maximum.  The softmax needs no exact row maximum, only a reference m_ref
      // that keeps exp2(x - m_ref) in range.  The first half-step of a row (and any later one while
      // the row has seen only masked columns) measures the maximum of its scores first; afterwards
      // the maximum of a half-step is gathered while its exponentials are computed, and a row
      // whose values exceeded 2^threshold moves its reference up at the start of the NEXT
      // half-step (`pend`).  Values between 2^threshold and 2^kDanger are exact all the same: P is
      // bf16, which has the exponent range of fp32, and O and l are fp32.  A jump beyond 2^kDanger
      // within one half-step may overflow: the CTA then marks its query tile in `redo`, and the
      // launcher's second pass recomputes marked tiles with the fp32 kernel (exact row maxima).
      float alpha = 1.f;
      bool rescale = false;
      if (__any_sync(0xffffffffu, m_ref == -INFINITY || pend > 0.f)) {
        bool raise = false;
        float tmax = 0.f;
        if (__any_sync(0xffffffffu, m_ref == -INFINITY)) {
          float mx0 = -INFINITY, mx1 = -INFINITY, mx2 = -INFINITY, mx3 = -INFINITY;
#pragma unroll 1
          for (int c4 = 0; c4 < 2; ++c4) {
            uint32_t r[32];
            tmem_ld32(t_s + c4 * 32, r);
            tmem_wait_ld();
#pragma unroll
            for (int j = 0; j < 32; j += 8) {
              mx0 = max3(mx0, __uint_as_float(r[j]), __uint_as_float(r[j + 1]));
              mx1 = max3(mx1, __uint_as_float(r[j + 2]), __uint_as_float(r[j + 3]));
              mx2 = max3(mx2, __uint_as_float(r[j + 4]), __uint_as_float(r[j + 5]));
              mx3 = max3(mx3, __uint_as_float(r[j + 6]), __uint_as_float(r[j + 7]));
            }
          }
          tmax = fmaxf(fmaxf(mx0, mx1), fmaxf(mx2, mx3)) * sc_used;
          raise = tmax > m_ref + kRescaleThreshold || (m_ref == -INFINITY && tmax > -INFINITY);
        }
        if (raise) {
          alpha = (m_ref == -INFINITY) ? 0.f : ex2_approx(m_ref - tmax);
          m_ref = tmax;
        } else if (pend > 0.f) {
          alpha = ex2_approx(-pend);
          m_ref += pend;
        }
        rescale = __any_sync(0xffffffffu, raise || pend > 0.f);
      }
      pend = 0.f;
      if (rescale) {
        l_run *= alpha;
        if (u > 0) {
          // products complete in the order of their issue: once P V (u-1) is complete, all earlier are
          if (!__all_sync(0xffffffffu, mbar_wait(b_pv_done((u - 1) % C::NBAR), ((u - 1) / C::NBAR) & 1, abort_flag, prm.status, prm.wait_limit))) {
            dead = true;
            continue;
          }
          tc_fence_after();
#pragma unroll 1
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
      // ---- P = exp2(x - m_ref), packed to bf16 over the first 32 columns of the buffer (chunk 0
      // goes to columns [0,16) while chunk 1 is still unread in [32,64); chunk 1 to [16,32))
      float neg_m = (m_ref == -INFINITY) ? 0.f : -m_ref;
      const f32x2 sc2 = pack2(sc_used, sc_used);
      float cm0 = -INFINITY, cm1 = -INFINITY;            // maximum of x - m_ref over the half-step
      float big = 0.f;                                   // larger of the two chunk sums of the half-step
#pragma unroll 1
      for (int c4 = 0; c4 < 2; ++c4) {
        uint32_t r[32];
        tmem_ld32(t_s + c4 * 32, r);
        tmem_wait_ld();
        // The special-function unit takes one exponential per 8 cycles and sub-core and is the
        // busiest unit of the kernel at d = 64: scaling and sums use two-value fp32 instructions,
        // and the other work of the chunk is interleaved with the exponentials in groups of four,
        // two groups behind, so that it issues in the shadow of that unit.
        float x[32];
        uint32_t pk[16];
        const f32x2 nm2 = pack2(neg_m, neg_m);
        f32x2 s01 = pack2(0.f, 0.f), s23 = s01;
        auto scale4 = [&](int j) {
          unpack2(fma2(pack2(__uint_as_float(r[j]), __uint_as_float(r[j + 1])), sc2, nm2), x[j], x[j + 1]);
          unpack2(fma2(pack2(__uint_as_float(r[j + 2]), __uint_as_float(r[j + 3])), sc2, nm2), x[j + 2], x[j + 3]);
        };
        scale4(0);
        scale4(4);
#pragma unroll
        for (int g = 0; g < 10; ++g) {
          if (g < 8) {
            const int j = 4 * g;
            if (C::TRACK_MAX) {
              cm0 = max3(cm0, x[j], x[j + 1]);
              cm1 = max3(cm1, x[j + 2], x[j + 3]);
            }
#pragma unroll
            for (int e = j; e < j + 4; ++e) x[e] = ex2_approx(x[e]);
          }
          if (g + 2 < 8) scale4(4 * (g + 2));
          if (g >= 2) {
            const int j = 4 * (g - 2);
            s01 = add2(s01, pack2(x[j], x[j + 1]));
            s23 = add2(s23, pack2(x[j + 2], x[j + 3]));
            pk[j / 2] = pack_bf16x2(x[j], x[j + 1]);
            pk[j / 2 + 1] = pack_bf16x2(x[j + 2], x[j + 3]);
          }
        }
        float sa, sb, sc, sd;
        unpack2(s01, sa, sb);
        unpack2(s23, sc, sd);
        const float chunk_sum = (sa + sb) + (sc + sd);
        l_run += chunk_sum;
        if (!C::TRACK_MAX) big = fmaxf(big, chunk_sum);
        tmem_st16(t_s + c4 * 16, pk);
      }
      if (C::TRACK_MAX) {
        const float hm = fmaxf(cm0, cm1);
        if (hm > kRescaleThreshold) pend = ceilf(hm);
        if (__any_sync(0xffffffffu, hm > kDanger)) *redo_flag = 1;
      } else {
        // a sum that is not below 2^kDanger (infinite or NaN included) marks the tile
        if (big > 256.0f) pend = ceilf(log2f(big));
        if (__any_sync(0xffffffffu, !(big < 7.9228163e28f))) *redo_flag = 1;
      }
      // one arrival per warp: 128 arrivals on one barrier word would be serialised in shared memory
      tmem_wait_st();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(b_p_ready(u % C::NBAR));
    }

    // epilogue: O / l, rows back to their original positions
    bool ok = !dead;
    if (ok) ok = __all_sync(0xffffffffu, mbar_wait(b_o_done, 0, abort_flag, prm.status, prm.wait_limit));
    tc_fence_after();
    if (ok) {                                          // warp-uniform: TMEM loads are warp-collective
      const int pos = qc * prm.c_q + half * kTile + row;
      bool live = row < q_rows && pos < prm.n_q;        // rows of the padding are not written
      int orig = live ? prm.perm_q[(size_t)p * prm.n_q + pos] : 0;
      if (orig < 0 || orig >= prm.n_q) {                // not a row of O: flagged, nothing written
        atomicCAS(prm.status, 0, kErrBadIndex);
        live = false;
        orig = 0;
      }
      // a row without a single live entry (an empty list without compensation): zeros, lse = -inf
      const bool empty = !(l_run > 0.f);
      const float inv = empty ? 0.f : 1.f / l_run;
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
            if (empty) w = make_uint4(0u, 0u, 0u, 0u);   // no product was issued: the accumulator holds no data
            dst[v] = w;
          }
        }
      }
      if (live && prm.lse)
        prm.lse[(size_t)p * prm.n_q + orig] = empty ? -INFINITY : (m_ref + log2f(l_run)) * 0.6931471805599453f;
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) tmem_dealloc(tmem_base, C::TMEM_COLS);
  // one word per CTA, written on every launch: 1 = this tile is to be recomputed
  if (tid == 0) prm.redo[((size_t)p * prm.n_qc + qc) * 2 + half] = *redo_flag;
}

// ---------------------------------------------------------------------------
// Centroids for the tensor-core path, 64 per tile: key tile = 64 rows of bf16 hi
// parts followed by 64 rows of lo parts; value centroids as bf16.  Rows beyond
// the last centroid are zero.
// ---------------------------------------------------------------------------
__global__ void centroid_prep_kernel(const float* __restrict__ ck, const float* __restrict__ cv, int n_kc,
                                     int cen_tiles, int D, __nv_bfloat16* __restrict__ kmix,
                                     __nv_bfloat16* __restrict__ vb) {
  const int p = blockIdx.y;
  const int e = blockIdx.x * blockDim.x + threadIdx.x;
  if (e >= cen_tiles * kHalf * D) return;
  const int j = e / D, col = e % D;
  float k = 0.f, v = 0.f;
  if (j < n_kc) {
    k = ck[(size_t)p * n_kc * D + e];
    v = cv[(size_t)p * n_kc * D + e];
  }
  const __nv_bfloat16 h = __float2bfloat16_rn(k);
  const size_t tile = (size_t)p * cen_tiles + j / kHalf;
  kmix[(tile * kTile + (j % kHalf)) * D + col] = h;
  kmix[(tile * kTile + kHalf + (j % kHalf)) * D + col] = __float2bfloat16_rn(k - __bfloat162float(h));
  vb[((size_t)p * cen_tiles * kHalf + j) * D + col] = __float2bfloat16_rn(v);
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

// matrix [rows, D] row-major of bf16 (or of one-byte codes); box = one 128-byte panel row (64 bf16
// or 128 codes) x box_rows rows, 128-byte swizzle
static bool make_map(CUtensorMap* map, const void* base, size_t rows, int D, int box_rows, bool bytes = false) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  cuuint64_t dims[2] = {(cuuint64_t)D, (cuuint64_t)rows};
  cuuint64_t strides[1] = {(cuuint64_t)D * (bytes ? 1 : 2)};
  cuuint32_t box[2] = {bytes ? 128u : 64u, (cuuint32_t)box_rows};
  cuuint32_t estr[2] = {1, 1};
  return fn(map, bytes ? CU_TENSOR_MAP_DATA_TYPE_UINT8 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

bool attn_tc_supported(const ca_problem_t& pr) {
  if (pr.dtype != CA_DTYPE_BF16 || (pr.flags & CA_ATTN_FP32)) return false;
  if (pr.cluster_q != 64 && pr.cluster_q != 128 && pr.cluster_q != 256) return false;
  if (pr.cluster_k < 16 || pr.cluster_k > 256) return false;
  const int n_kc = ceil_div(pr.n_k, pr.cluster_k);
  if ((n_kc + 31) / 32 * 4 > 16384) return false;          // selected-cluster bitmap in shared memory
  return true;
}

// quantised Q K^T: head dimension 128 (one 128-byte panel row of codes), key clusters of at least
// 64 rows (one scale per half-step)
bool attn_tc_fp8_supported(const ca_problem_t& pr) {
  return attn_tc_supported(pr) && pr.head_dim == 128 && pr.cluster_k >= kHalf;
}

size_t attn_tc_workspace_bytes(const ca_problem_t& pr) {
  const size_t P = (size_t)pr.batch * pr.heads;
  const size_t cen_tiles = (size_t)ceil_div(ceil_div(pr.n_k, pr.cluster_k), kHalf);
  const size_t n_qc = (size_t)ceil_div(pr.n_q, pr.cluster_q);
  size_t bytes = kStatusBytes + align_up(P * cen_tiles * kTile * pr.head_dim * sizeof(__nv_bfloat16), 256) +
                 align_up(P * cen_tiles * kHalf * pr.head_dim * sizeof(__nv_bfloat16), 256) +
                 align_up(P * n_qc * 2 * sizeof(int32_t), 256);
  if (pr.flags & CA_ATTN_FP8_QK) {
    const size_t n_kc = (size_t)ceil_div(pr.n_k, pr.cluster_k), D = pr.head_dim;
    const size_t q_rows = P * n_qc * pr.cluster_q, k_rows = P * n_kc * pr.cluster_k;
    bytes += align_up(q_rows * D, 256) + align_up(q_rows * 4, 256) + align_up(k_rows * D, 256) +
             align_up(P * n_kc * 4, 256) + align_up(P * cen_tiles * kHalf * D, 256) + align_up(P * cen_tiles * 4, 256);
  }
  return bytes;
}

template <int D, bool F8>
static int launch_tc_d(const CUtensorMap* maps, const TcParams& prm, dim3 grid, cudaStream_t st) {
  using C = TcCfg<D, F8>;
  const size_t smem = 1024 + C::OFF_BITMAP + (size_t)prm.bitmap_words * 4 + (((size_t)prm.list_stride * 2 + 15) & ~(size_t)15) +
                      (F8 ? (size_t)prm.list_stride * 4 : 0);
  auto k = attn_tc_kernel<D, F8>;
  CA_RETURN_IF_CUDA(cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  k<<<grid, kTcThreads, smem, st>>>(maps[0], maps[1], maps[2], maps[3], maps[4], prm);
  CA_LAUNCH_CHECK();
  return CA_OK;
}

namespace {
long long g_wait_limit = kWaitLimitCycles;   // host-side settings of the diagnostic hook
int g_skip_key_load = -1;
}  // namespace
void attn_tc_set_debug(long long wait_limit_cycles, int skip_key_load) {
  g_wait_limit = wait_limit_cycles > 0 ? wait_limit_cycles : kWaitLimitCycles;
  g_skip_key_load = skip_key_load;
}

int launch_attn_tc(const ca_problem_t& pr, const void* Qp, const void* Kp, const void* Vp, const float* ck,
                   const float* cv, const int32_t* count_k, const int32_t* block_idx, const int32_t* keep_count,
                   int list_stride, const int32_t* perm_q, float scale, void* O, float* lse, void* ws,
                   cudaStream_t st) {
  const int P = pr.batch * pr.heads, D = pr.head_dim;
  const int n_qc = ceil_div(pr.n_q, pr.cluster_q), n_kc = ceil_div(pr.n_k, pr.cluster_k);
  const int cen_tiles = ceil_div(n_kc, kHalf);
  Carver c(ws);
  int* status = c.take<int>(kStatusBytes / sizeof(int));
  __nv_bfloat16* kmix = c.take<__nv_bfloat16>((size_t)P * cen_tiles * kTile * D);
  __nv_bfloat16* vb = c.take<__nv_bfloat16>((size_t)P * cen_tiles * kHalf * D);
  int32_t* redo = c.take<int32_t>((size_t)P * n_qc * 2);
  const bool f8 = (pr.flags & CA_ATTN_FP8_QK) != 0;
  unsigned char *q8 = nullptr, *k8 = nullptr, *c8 = nullptr;
  float *sq = nullptr, *sk = nullptr, *sc = nullptr;
  if (f8) {
    // queries, keys and key centroids as E4M3 codes with their scales (quantize.cu)
    const size_t q_rows = (size_t)P * n_qc * pr.cluster_q, k_rows = (size_t)P * n_kc * pr.cluster_k;
    q8 = c.take<unsigned char>(q_rows * D);  sq = c.take<float>(q_rows);
    k8 = c.take<unsigned char>(k_rows * D);  sk = c.take<float>((size_t)P * n_kc);
    c8 = c.take<unsigned char>((size_t)P * cen_tiles * kHalf * D);  sc = c.take<float>((size_t)P * cen_tiles);
    ProfScope ps(kProfAttnPrep, st);
    const int rq = launch_quantize_qk(Qp, Kp, pr.compensate ? ck : nullptr, P, n_qc, pr.cluster_q, n_kc, pr.cluster_k,
                                      cen_tiles, D, q8, sq, k8, sk, c8, sc, st);
    if (rq != CA_OK) return rq;
  }
  if (pr.compensate) {
    ProfScope ps(kProfAttnPrep, st);
    centroid_prep_kernel<<<dim3(ceil_div(cen_tiles * kHalf * D, 256), P), 256, 0, st>>>(ck, cv, n_kc, cen_tiles, D,
                                                                                        kmix, vb);
    CA_LAUNCH_CHECK();
  }
  CUtensorMap maps[5];
  const int kbox = pr.cluster_k < kHalf ? pr.cluster_k : kHalf;      // key/value slots hold 64 rows
  const int qbox = pr.cluster_q < kTile ? pr.cluster_q : kTile;
  bool ok = make_map(&maps[2], Vp, (size_t)P * n_kc * pr.cluster_k, D, kbox) &&
            make_map(&maps[4], vb, (size_t)P * cen_tiles * kHalf, D, kHalf);
  if (f8)
    ok = ok && make_map(&maps[0], q8, (size_t)P * n_qc * pr.cluster_q, D, qbox, true) &&
         make_map(&maps[1], k8, (size_t)P * n_kc * pr.cluster_k, D, kbox, true) &&
         make_map(&maps[3], c8, (size_t)P * cen_tiles * kHalf, D, kHalf, true);
  else
    ok = ok && make_map(&maps[0], Qp, (size_t)P * n_qc * pr.cluster_q, D, qbox) &&
         make_map(&maps[1], Kp, (size_t)P * n_kc * pr.cluster_k, D, kbox) &&
         make_map(&maps[3], kmix, (size_t)P * cen_tiles * kTile, D, kHalf);
  if (!ok) return CA_ERR_CUDA;
  TcParams prm;
  prm.count_k = count_k; prm.block_idx = block_idx; prm.keep_count = keep_count; prm.perm_q = perm_q;
  prm.list_stride = list_stride;
  prm.O = static_cast<__nv_bfloat16*>(O); prm.lse = lse; prm.status = status; prm.redo = redo;
  prm.n_q = pr.n_q; prm.n_k = pr.n_k; prm.c_q = pr.cluster_q; prm.c_k = pr.cluster_k; prm.keep = pr.keep;
  prm.n_qc = n_qc; prm.n_kc = n_kc; prm.cen_tiles = cen_tiles; prm.compensate = pr.compensate;
  prm.bitmap_words = (cen_tiles * kHalf + 31) / 32;
  prm.scale_log2 = scale * 1.4426950408889634f;
  prm.wait_limit = g_wait_limit;
  prm.skip_key_load = g_skip_key_load;
  prm.q_scale = sq; prm.k_scale = sk; prm.c_scale = sc;
  dim3 grid(n_qc * (pr.cluster_q >= kTile ? pr.cluster_q / kTile : 1), P);
  int rc;
  {
    ProfScope ps(kProfAttn, st);
    if (f8) rc = launch_tc_d<128, true>(maps, prm, grid, st);
    else rc = D == 64 ? launch_tc_d<64, false>(maps, prm, grid, st) : launch_tc_d<128, false>(maps, prm, grid, st);
  }
  if (rc != CA_OK) return rc;
  ProfScope ps(kProfAttnSecond, st);
  // second pass: query tiles whose scores left the range of the fast softmax (a climb of more than
  // 2^96 within 64 keys) are recomputed by the fp32 kernel; its CTAs return at once for the others
  return launch_attn_ref(pr, Qp, Kp, Vp, ck, cv, count_k, block_idx, keep_count, list_stride, perm_q, scale, O, lse,
                         status, st, redo, (int)grid.x / n_qc, status + kRecomputedWord);
}

}  // namespace ca
