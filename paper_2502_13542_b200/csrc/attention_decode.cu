// Step 5 for short steps (decode, Eq. 3): attention of n_tokens <= 128 / G new tokens over
//   [initial tokens | selected blocks | local past | the new tokens (causal)]
// for bf16, D = 128, 16-token pages.  The work per key is 4 * D * G flops against 4 * D bytes of
// K and V, so the stage is bound by the K/V stream, not by arithmetic.
//
// One CTA = one KV head of one (sequence, layer) and one contiguous share ("split") of its key
// tiles.  The 128-row M tile packs the G query heads of the KV group: row r = token r / G, query
// head g * G + r % G, so K and V are streamed once for the whole group; rows past n_tokens * G
// are padding whose results are dropped.  Machinery as in the prefill kernel: TMA page gather
// into K and V rings, tcgen05.mma with TMEM accumulators (M = 128 is the narrowest tile the
// pipeline takes here; the tensor pipe has the headroom), two softmax threads per row, P as
// hi + lo bf16 terms.
//
// With one split the CTA writes the normalised output.  With several (few sequences, long
// contexts: not enough (sequence, KV head) pairs to fill the SMs) every split writes its
// normalised partial output and its base-2 log-sum-exp to a workspace, and a second kernel
// merges them per (token, head) in a fixed order.
// Every wait on an mbarrier is bounded; on expiry the CTA flags ACTQKV_DEV_TIMEOUT, stops
// issuing work, drains and frees its TMEM.
#include <algorithm>

#include "tc_common.cuh"

using namespace actqkv;
using namespace actqkv::tc;

namespace {

constexpr int kBM = 128, kBN = 128, kD = 128;
constexpr int kRing = 3;                                 // K tiles in flight, and V tiles in flight
constexpr int kSBuf = 3;                                 // S/P buffers in TMEM
constexpr int kPvRing = 4;                               // barriers that count completed P V products
constexpr int kThreads = 384;                            // 3 warpgroups
constexpr uint32_t kSubTileBytes = 128 * 128;            // [128 rows x 64 bf16], 16 KiB
constexpr uint32_t kTileBytes = 2 * kSubTileBytes;       // 32 KiB: one K or V or Q tile
constexpr uint32_t kSmemTiles = (1 + 2 * kRing) * kTileBytes;
constexpr int kNumBars = 1 + 4 * kRing + 2 * kSBuf + kPvRing + 1;
constexpr uint32_t kBarBytes = 256;                      // barriers, TMEM slot, abort flag
constexpr uint32_t kXchgBytes = 2 * 2 * 128 * 4;         // [tile parity][column half][row] floats
constexpr uint32_t kSmemNeeded = kSmemTiles + kBarBytes + kXchgBytes;
constexpr uint32_t kSmemBytes = 227 * 1024;              // everything an SM offers one CTA
static_assert(8 * kNumBars + 16 <= kBarBytes, "barrier area too small");
static_assert(kSmemNeeded <= kSmemBytes, "shared memory budget");


struct DecodeParams {
  uint32_t spin_limit; // iterations a device-side wait may take (kSpinLimit; shorter only under test)
  int drop_k_tile;     // test hook: the K copy of this tile of every CTA is not issued (-1: none)
  int n_splits;        // CTAs per (unit, KV head)
  float* part_o;       // [U][n_tokens][Hq][n_splits][D] normalised partial outputs (n_splits > 1)
  float* part_lse;     // [U][n_tokens][Hq][n_splits] base-2 log-sum-exp of each split (-inf: empty)
};

// ---------------------------------------------------------------- kernel
__global__ void __launch_bounds__(kThreads, 1)
attention_decode_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_kw,
                    const __grid_constant__ CUtensorMap tm_vw, const __grid_constant__ CUtensorMap tm_kp,
                       const __grid_constant__ CUtensorMap tm_vp, TcParams p, DecodeParams dp) {
  extern __shared__ unsigned char smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  const bool smem_short = base - raw + kSmemNeeded > kSmemBytes;   // never with a 1 KiB-aligned window
  const uint32_t q_smem = base;
  const uint32_t k_ring = base + kTileBytes;
  const uint32_t v_ring = k_ring + kRing * kTileBytes;
  const uint32_t bars = base + kSmemTiles;
  // barrier slots (8 bytes each)
  const uint32_t bar_q = bars;
  auto bar_kfull = [&](int s) { return bars + 8u * (1 + s); };
  auto bar_kempty = [&](int s) { return bars + 8u * (1 + kRing + s); };
  auto bar_vfull = [&](int s) { return bars + 8u * (1 + 2 * kRing + s); };
  auto bar_vempty = [&](int s) { return bars + 8u * (1 + 3 * kRing + s); };
  auto bar_sfull = [&](int b) { return bars + 8u * (1 + 4 * kRing + b); };
  auto bar_pfull = [&](int b) { return bars + 8u * (1 + 4 * kRing + kSBuf + b); };
  auto bar_pvdone = [&](int i) { return bars + 8u * (1 + 4 * kRing + 2 * kSBuf + i); };
  const uint32_t bar_done = bars + 8u * (kNumBars - 1);
  unsigned char* base_generic = smem_raw + (base - raw);
  unsigned char* bars_generic = base_generic + kSmemTiles;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars_generic + 8 * kNumBars);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(bars_generic + 8 * kNumBars + 8);
  float* xchg = reinterpret_cast<float*>(bars_generic + kBarBytes);   // [2][2][128]

  const int sp = blockIdx.x, g = blockIdx.y, unit = blockIdx.z;
  const int G = p.group;
  const int seq = unit / p.n_layers, layer_local = unit - seq * p.n_layers;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int nt = p.a.n_tokens;

  // ---- geometry (uniform over the CTA)
  const Geometry geo = make_geometry(p.a.pos0[seq], p.n_init, p.block, p.n_local_prev);
  int c = p.a.sel_count ? p.a.sel_count[unit] : 0;
  bool bad = false;
  if (c < 0 || c > p.cap_blocks || c > geo.n_cand) {
    bad = true;
    c = max(0, min(c, min(p.cap_blocks, geo.n_cand)));
  }
  KeyStream ks;
  ks.sel = p.a.sel_idx + (size_t(unit) * p.n_kv_heads + g) * p.cap_blocks;
  ks.pt = p.a.page_table + size_t(seq) * p.max_pages;
  ks.gpb = p.block / 16;                                 // page granules per block
  ks.g_init = geo.init_len / 16;
  ks.g_sel = c * ks.gpb;
  const int64_t local_len = geo.p0 - geo.local_start;
  ks.g_past = ks.g_init + ks.g_sel + int((local_len + 15) / 16);   // the last local page may be partly filled
  ks.n_cand = geo.n_cand; ks.n_init = p.n_init; ks.block = p.block; ks.max_pages = p.max_pages;
  ks.n_phys_pages = p.n_phys_pages; ks.page_base = layer_local * p.n_phys_pages;
  ks.page_oob = p.n_layers * p.n_phys_pages;             // beyond the tensor: zero fill
  ks.local_start = geo.local_start;
  const bool misaligned = smem_short;
  const int n_past = geo.init_len + c * p.block + int(local_len);     // exact: the tail of the last page is masked
  const int past_tiles = (n_past + kBN - 1) / kBN;
  // this split's share of the tiles: the past tiles, then one tile holding the new tokens
  const int all_tiles = past_tiles + 1;
  const int per_split = (all_tiles + dp.n_splits - 1) / dp.n_splits;
  const int j_lo = sp * per_split;
  const int n_tiles = max(0, min(all_tiles, j_lo + per_split) - j_lo);
  // A split that contributes nothing says so with a log-sum-exp of minus infinity: the merge then
  // skips its partial output, whatever an earlier call left at that place of the workspace.
  auto mark_split_empty = [&]() {
    if (dp.n_splits <= 1) return;
    for (int i = tid; i < nt * G; i += kThreads) {
      const int t = i / G, hh = g * G + i % G;
      dp.part_lse[((size_t(unit) * nt + t) * p.n_q_heads + hh) * dp.n_splits + sp] = -INFINITY;
    }
  };
  if (n_tiles == 0) {          // uniform over the CTA: more splits than tiles
    mark_split_empty();
    return;
  }

  if (tid == 0) {
    if (bad || misaligned) set_status(p.a.status, ACTQKV_DEV_BAD_SELECTION);
    mbar_init(bar_q, 1);
    for (int s = 0; s < kRing; ++s) {
      mbar_init(bar_kfull(s), 1); mbar_init(bar_kempty(s), 1);
      mbar_init(bar_vfull(s), 1); mbar_init(bar_vempty(s), 1);
    }
    for (int b = 0; b < kSBuf; ++b) { mbar_init(bar_sfull(b), 1); mbar_init(bar_pfull(b), 256); }
    for (int i = 0; i < kPvRing; ++i) mbar_init(bar_pvdone(i), 1);
    mbar_init(bar_done, 1);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(512));
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  if (misaligned) {           // uniform: nothing was issued yet
    mark_split_empty();
    __syncthreads();
    if (warp == 1) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(512));
    return;
  }

  if (warp == 0 || warp == 2) {
    // =========================== TMA producers: warp 0 -> K (and Q), warp 2 -> V ===========================
    const bool is_v = warp == 2;
    const uint32_t ring = is_v ? v_ring : k_ring;
    const CUtensorMap* tm_pages = is_v ? &tm_vp : &tm_kp;
    const CUtensorMap* tm_win = is_v ? &tm_vw : &tm_kw;
    if (!is_v && lane == 0) {
      mbar_expect_tx(bar_q, kTileBytes);
      tma_load_3d(q_smem, &tm_q, bar_q, 0, g * G, unit * nt);              // box: 64 channels x G heads x 128/G tokens
      tma_load_3d(q_smem + kSubTileBytes, &tm_q, bar_q, 64, g * G, unit * nt);
    }
    const int half = (lane >> 3) & 1, slot = lane & 7;     // lanes 0-15: one box each
    // Page lookups (sel_idx -> page_table, two dependent loads) are taken 32 granules = 4 tiles at
    // a time, one granule per lane, one chunk ahead of the tiles being issued, so their latency
    // is off the per-tile path; the issuing lane fetches its page with a shuffle.
    auto resolve = [&](int chunk) {
      const int gi = (j_lo + chunk * 4) * 8 + lane;
      return gi < past_tiles * 8 ? granule_page(ks, gi, p.a.status, !is_v) : ks.page_oob;
    };
    int page_cur = 0, page_next = resolve(0);
    bool ok = true;
    int issued = 0;
    for (int j = 0; j < n_tiles && ok; ++j) {
      const int s = j % kRing, it = j / kRing;
      if ((j & 3) == 0) page_cur = page_next;
      const int page = __shfl_sync(0xffffffffu, page_cur, (j & 3) * 8 + slot);
      if (it > 0) ok = mbar_wait(is_v ? bar_vempty(s) : bar_kempty(s), (it - 1) & 1, abort_flag, dp.spin_limit);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      const uint32_t full = is_v ? bar_vfull(s) : bar_kfull(s);
      const uint32_t sbase = ring + s * kTileBytes;
      const bool dropped = !is_v && j == dp.drop_k_tile;   // test hook: this copy is never made, so the wait for it runs out
      if (lane == 0 && !dropped) mbar_expect_tx(full, kTileBytes);
      __syncwarp();
      if (dropped) {
      } else if (j_lo + j < past_tiles) {
        if (lane < 16) tma_load_4d(sbase + half * kSubTileBytes + slot * 2048u, tm_pages, full, half * 64, 0, g, page);
      } else if (lane < 2) {
        tma_load_3d(sbase + lane * kSubTileBytes, tm_win, full, lane * 64, g, unit * nt);
      }
      issued = j + 1;
      if ((j & 3) == 0) page_next = resolve((j >> 2) + 1);   // after the issue: its stall is behind the ring
    }
    // drain: every issued copy must have landed before the CTA may exit on the abort path
    if (!ok) {
      for (int j = max(0, issued - kRing); j < issued; ++j) {
        if (!is_v && j == dp.drop_k_tile) continue;
        const uint32_t full = is_v ? bar_vfull(j % kRing) : bar_kfull(j % kRing);
        for (uint32_t i = 0; i < dp.spin_limit && !mbar_try_wait(full, (j / kRing) & 1); ++i) {}
      }
      if (!is_v) for (uint32_t i = 0; i < dp.spin_limit && !mbar_try_wait(bar_q, 0); ++i) {}
    }
  } else if (warp == 1) {
    // =========================== MMA issuer ===========================
    if (lane == 0) {
      constexpr uint32_t idesc_qk = make_idesc(false, kBM, kBN);
      constexpr uint32_t idesc_pv = make_idesc(true, kBM, kBN);
      const uint32_t tmem_o = tmem + kSBuf * 128;
      bool ok = mbar_wait(bar_q, 0, abort_flag, dp.spin_limit);
      auto issue_qk = [&](int j) {
        const int s = j % kRing;
        ok = ok && mbar_wait(bar_kfull(s), (j / kRing) & 1, abort_flag, dp.spin_limit);
        if (!ok) return;
        tc_fence_after();
        const uint32_t kbase = k_ring + s * kTileBytes;
        const uint32_t s_tmem = tmem + (j % kSBuf) * 128;
#pragma unroll
        for (int k = 0; k < kD / 16; ++k) {
          const uint32_t off = (k >> 2) * kSubTileBytes + (k & 3) * 32u;
          mma_ss(s_tmem, make_desc(q_smem + off, 16u, 1024u), make_desc(kbase + off, 16u, 1024u), idesc_qk,
                 k > 0 ? 1u : 0u);
        }
        tc_commit(bar_kempty(s));
        tc_commit(bar_sfull(j % kSBuf));
      };
      auto issue_pv = [&](int i) {
        const int s = i % kRing, b = i % kSBuf;
        ok = ok && mbar_wait(bar_vfull(s), (i / kRing) & 1, abort_flag, dp.spin_limit);
        ok = ok && mbar_wait(bar_pfull(b), (i / kSBuf) & 1, abort_flag, dp.spin_limit);
        if (!ok) return;
        tc_fence_after();
        const uint32_t vbase = v_ring + s * kTileBytes;
        const uint32_t p_tmem = tmem + b * 128;
#pragma unroll
        for (int k = 0; k < kBN / 16; ++k) {
          // 16 keys per step: B advances 16 rows of 128 bytes; A = 8 packed columns of the hi
          // term, then the 8 columns of the lo term of the same keys against the same V rows.
          const uint64_t bdesc = make_desc(vbase + k * 2048u, kSubTileBytes, 1024u);
          const uint32_t pa = p_tmem + (k >> 1) * 32 + (k & 1) * 8;
          mma_ts(tmem_o, pa, bdesc, idesc_pv, (i > 0 || k > 0) ? 1u : 0u);
          mma_ts(tmem_o, pa + 16, bdesc, idesc_pv, 1u);
        }
        tc_commit(bar_vempty(s));
        tc_commit(bar_pvdone(i % kPvRing));
      };
      issue_qk(0);
      if (n_tiles > 1) issue_qk(1);
      for (int i = 0; i < n_tiles && ok; ++i) {
        if (i + 2 < n_tiles) issue_qk(i + 2);
        issue_pv(i);
      }
      tc_commit(bar_done);
      // when a wait gave up nobody else waits for this barrier: the issuer itself sees the products
      // it has issued through, so that TMEM is not freed under them
      if (!ok) for (uint32_t i = 0; i < dp.spin_limit && !mbar_try_wait(bar_done, 0); ++i) {}
    }
    __syncwarp();
  } else if (warp >= 4) {
    // =========================== softmax / epilogue ===========================
    const int b = (warp >> 2) - 1;                        // column half of every tile
    const int q4 = warp & 3;                              // TMEM lane quadrant of this warp
    const int row = q4 * 32 + lane;                       // query row inside the tile
    const uint32_t lane_addr = uint32_t(q4 * 32) << 16;
    const uint32_t o_addr = tmem + lane_addr + kSBuf * 128 + b * 64;
    float m_used = -INFINITY, l = 0.f;
    bool ok = true;
    // A warp whose 32 rows hold no query (single-token decode fills G rows of the tile) only keeps
    // the barrier phases in step: nothing is read from its rows of P or O, and the exponentials,
    // issue slots and TMEM traffic it would spend go to the warps that have rows.
    const bool warp_used = q4 * 32 < nt * G;
    if (!warp_used) {
      for (int j = 0; j < n_tiles && ok; ++j) {
        const int sb = j % kSBuf;
        ok = mbar_wait(bar_sfull(sb), (j / kSBuf) & 1, abort_flag, dp.spin_limit);
        mbar_arrive(bar_pfull(sb));
      }
    }
    for (int j = 0; warp_used && j < n_tiles; ++j) {
      const int sb = j % kSBuf;
      ok = ok && mbar_wait(bar_sfull(sb), (j / kSBuf) & 1, abort_flag, dp.spin_limit);
      tc_fence_after();
      const uint32_t s_addr = tmem + lane_addr + sb * 128 + b * 64;
      uint64_t sv[32];
      TMEM_LD64P_WAIT(s_addr, sv);
      // key-validity limit: ragged last past tile, or the causal diagonal of the last tile
      const int jj = j_lo + j;                            // tile index in the whole key stream
      int limit = kBN;
      if (jj < past_tiles) limit = min(kBN, n_past - jj * kBN);
      else limit = min(nt, row / G + 1);                  // the new tokens, causal; row = token * G + head
      limit -= b * 64;                                    // in this thread's column numbering
      const bool masked = jj == past_tiles || (jj == past_tiles - 1 && (n_past % kBN) != 0);   // CTA-uniform
      float mx = -INFINITY, mx2 = -INFINITY;
      if (masked) {
#pragma unroll
        for (int i = 0; i < 32; ++i) {
          const float x0 = 2 * i < limit ? lo2(sv[i]) : -INFINITY;
          const float x1 = 2 * i + 1 < limit ? hi2(sv[i]) : -INFINITY;
          sv[i] = pack2(x0, x1);
          mx = max3(mx, x0, x1);
        }
      } else {
        float mx3 = -INFINITY, mx4 = -INFINITY;           // four independent chains
#pragma unroll
        for (int i = 0; i < 32; i += 4) {
          mx = max3(mx, lo2(sv[i]), hi2(sv[i]));
          mx2 = max3(mx2, lo2(sv[i + 1]), hi2(sv[i + 1]));
          mx3 = max3(mx3, lo2(sv[i + 2]), hi2(sv[i + 2]));
          mx4 = max3(mx4, lo2(sv[i + 3]), hi2(sv[i + 3]));
        }
        mx = fmaxf(max3(mx, mx2, mx3), mx4);
      }
      // the row's maximum over both column halves
      float* xrow = xchg + (j & 1) * 256 + row;
      xrow[b * 128] = mx;
      ok = pair_sync_and(q4, ok);
      if (!ok) break;                                     // both threads of a row leave together
      mx = fmaxf(mx, xrow[(1 - b) * 128]);
      const float m_new = fmaxf(m_used, mx * p.scale_log2);
      const bool grow = m_new - m_used > kRescaleThreshold;     // also true for the first tile
      if (j == 0) {
        m_used = m_new;
      } else if (__any_sync(0xffffffffu, grow)) {
        // O must be quiescent: P V of every earlier tile complete (tile j's is not issued before
        // this thread publishes P(j)).  One barrier per tile in a ring of 4, so the parity of the
        // awaited phase cannot be confused with a later one.
        ok = mbar_wait(bar_pvdone((j - 1) % kPvRing), ((j - 1) / kPvRing) & 1, abort_flag, dp.spin_limit);
        tc_fence_after();
        const float f = grow ? ex2(m_used - m_new) : 1.f;
        if (grow) { m_used = m_new; l *= f; }
#pragma unroll
        for (int cc = 0; cc < 2; ++cc) {
          uint32_t orr[32];
          TMEM_LD32_WAIT(o_addr + cc * 32, orr);
#pragma unroll
          for (int i = 0; i < 32; ++i) orr[i] = __float_as_uint(__uint_as_float(orr[i]) * f);
          TMEM_ST32(o_addr + cc * 32, orr);
        }
      }
      // P = exp2(x - m) split into two bf16 terms (hi + lo): with outlier value channels a
      // single bf16 P (8 significant bits) would cost up to |v| * 2^-9 of absolute error.
      const uint64_t scale2 = pack2(p.scale_log2, p.scale_log2), negm2 = pack2(-m_used, -m_used);
      uint64_t sum_a = 0, sum_b = 0;                      // two (+0, +0) pairs
#pragma unroll
      for (int cc = 0; cc < 2; ++cc) {
        uint32_t pk[32];
#pragma unroll
        for (int i = 0; i < 16; ++i) {
          const uint64_t x = fma2(sv[16 * cc + i], scale2, negm2);
          const float e0 = ex2(lo2(x)), e1 = ex2(hi2(x));
          const uint64_t e = pack2(e0, e1);
          if (i & 1) sum_b = add2(sum_b, e); else sum_a = add2(sum_a, e);
          const uint32_t hi = pack_bf16(e0, e1);
          pk[i] = hi;
          const uint64_t lo = sub2(e, (uint64_t(hi & 0xFFFF0000u) << 32) | (hi << 16));
          pk[16 + i] = pack_bf16(lo2(lo), hi2(lo));
        }
        TMEM_ST32(s_addr + cc * 32, pk);
      }
      sum_a = add2(sum_a, sum_b);
      l += lo2(sum_a) + hi2(sum_a);
      tmem_wait_st();
      tc_fence_before();
      mbar_arrive(bar_pfull(sb));
    }
    // ---- epilogue: the row sum over both column halves, then this thread's 64 channels of O / l
    ok = ok && warp_used && mbar_wait(bar_done, 0, abort_flag, dp.spin_limit);
    float* xrow = xchg + (n_tiles & 1) * 256 + row;
    if (warp_used) {
      xrow[b * 128] = l;
      ok = pair_sync_and(q4, ok);
    }
    if (ok) {
      tc_fence_after();
      const float lsum = l + xrow[(1 - b) * 128];
      const float inv = lsum > 0.f ? 1.f / lsum : 0.f;
      const int t = row / G, hh = g * G + row % G;       // this row's token and query head
      const bool valid = t < nt;
      const size_t th = (size_t(unit) * nt + t) * p.n_q_heads + hh;
#pragma unroll
      for (int cc = 0; cc < 2; ++cc) {
        const int col = b * 64 + cc * 32;
        uint32_t orr[32];
        TMEM_LD32_WAIT(o_addr + cc * 32, orr);
        if (!valid) continue;
        if (dp.n_splits > 1) {
          float* of = dp.part_o + (th * dp.n_splits + sp) * kD + col;
#pragma unroll
          for (int i = 0; i < 8; ++i) {
            float4 v;
            v.x = __uint_as_float(orr[4 * i + 0]) * inv; v.y = __uint_as_float(orr[4 * i + 1]) * inv;
            v.z = __uint_as_float(orr[4 * i + 2]) * inv; v.w = __uint_as_float(orr[4 * i + 3]) * inv;
            *reinterpret_cast<float4*>(of + 4 * i) = v;
          }
        } else if (p.out_bf16) {
          __nv_bfloat16* ob = static_cast<__nv_bfloat16*>(p.a.out) + th * kD + col;
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            uint4 v;
            v.x = pack_bf16(__uint_as_float(orr[8 * i + 0]) * inv, __uint_as_float(orr[8 * i + 1]) * inv);
            v.y = pack_bf16(__uint_as_float(orr[8 * i + 2]) * inv, __uint_as_float(orr[8 * i + 3]) * inv);
            v.z = pack_bf16(__uint_as_float(orr[8 * i + 4]) * inv, __uint_as_float(orr[8 * i + 5]) * inv);
            v.w = pack_bf16(__uint_as_float(orr[8 * i + 6]) * inv, __uint_as_float(orr[8 * i + 7]) * inv);
            *reinterpret_cast<uint4*>(ob + 8 * i) = v;
          }
        } else {
          float* of = static_cast<float*>(p.a.out) + th * kD + col;
#pragma unroll
          for (int i = 0; i < 8; ++i) {
            float4 v;
            v.x = __uint_as_float(orr[4 * i + 0]) * inv; v.y = __uint_as_float(orr[4 * i + 1]) * inv;
            v.z = __uint_as_float(orr[4 * i + 2]) * inv; v.w = __uint_as_float(orr[4 * i + 3]) * inv;
            *reinterpret_cast<float4*>(of + 4 * i) = v;
          }
        }
      }
      if (valid && b == 0) {
        const float lse2 = lsum > 0.f ? m_used + log2f(lsum) : -INFINITY;
        if (dp.n_splits > 1) dp.part_lse[th * dp.n_splits + sp] = lse2;
        else if (p.a.lse) p.a.lse[(size_t(unit) * p.n_q_heads + hh) * nt + t] = lse2 * 0.6931471805599453f;
      }
    }
  }

  // ---- teardown
  tc_fence_before();
  __syncthreads();
  if (*abort_flag) {            // a wait gave up: this split's partial result is not to be used
    mark_split_empty();
    if (tid == 0) set_status(p.a.status, ACTQKV_DEV_TIMEOUT);
  }
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(512));
  }
}

// Merge of the splits' partial results, one warp per (unit, token, query head): weights
// 2^(lse_s - max lse) in split order.
__global__ void __launch_bounds__(128)
decode_merge_kernel(const float* __restrict__ part_o, const float* __restrict__ part_lse, void* out, float* lse,
                    int n_rows, int n_splits, int n_tokens, int n_q_heads, int out_bf16) {
  const int rowi = blockIdx.x * 4 + (threadIdx.x >> 5), lane = threadIdx.x & 31;
  if (rowi >= n_rows) return;                         // rowi = (unit * n_tokens + t) * Hq + h
  const float* ls = part_lse + size_t(rowi) * n_splits;
  float mx = -INFINITY;
  for (int s = 0; s < n_splits; ++s) mx = fmaxf(mx, ls[s]);
  float acc[4] = {0.f, 0.f, 0.f, 0.f}, wsum = 0.f;
  for (int s = 0; s < n_splits; ++s) {
    const float l2 = ls[s];
    if (l2 == -INFINITY) continue;                    // empty split: its partial output was never written
    const float w = exp2f(l2 - mx);
    wsum += w;
    const float4 v = *reinterpret_cast<const float4*>(part_o + (size_t(rowi) * n_splits + s) * kD + lane * 4);
    acc[0] = fmaf(w, v.x, acc[0]); acc[1] = fmaf(w, v.y, acc[1]);
    acc[2] = fmaf(w, v.z, acc[2]); acc[3] = fmaf(w, v.w, acc[3]);
  }
  const float inv = wsum > 0.f ? 1.f / wsum : 0.f;
  if (out_bf16) {
    uint2 v;
    v.x = pack_bf16(acc[0] * inv, acc[1] * inv);
    v.y = pack_bf16(acc[2] * inv, acc[3] * inv);
    *reinterpret_cast<uint2*>(static_cast<__nv_bfloat16*>(out) + size_t(rowi) * kD + lane * 4) = v;
  } else {
    *reinterpret_cast<float4*>(static_cast<float*>(out) + size_t(rowi) * kD + lane * 4) =
        make_float4(acc[0] * inv, acc[1] * inv, acc[2] * inv, acc[3] * inv);
  }
  if (lse && lane == 0) {
    const int h = rowi % n_q_heads, ut = rowi / n_q_heads, t = ut % n_tokens, unit = ut / n_tokens;
    lse[(size_t(unit) * n_q_heads + h) * n_tokens + t] = wsum > 0.f ? (mx + log2f(wsum)) * 0.6931471805599453f : -INFINITY;
  }
}

}  // namespace

namespace actqkv {

bool attention_decode_supported(const actqkv_config* cfg, int n_tokens) {
  const int group = cfg->n_q_heads / cfg->n_kv_heads;
  return cfg->dtype == ACTQKV_BF16 && cfg->head_dim == 128 && cfg->page_tokens == 16 && cfg->block % 16 == 0 &&
         cfg->n_init % 16 == 0 && cfg->n_local_prev % 16 == 0 && kBM % group == 0 && n_tokens * group <= kBM;
}

int64_t attention_decode_workspace_bytes(const actqkv_config* cfg, const Batch& b, int n_tokens, int n_splits) {
  if (n_splits <= 1) return 0;
  const int64_t rows = int64_t(b.units()) * n_tokens * cfg->n_q_heads;
  return rows * n_splits * (kD + 1) * int64_t(sizeof(float));
}

// Splits per (unit, KV head) that fill the SMs once; 1 when the batch already does.
int attention_decode_auto_splits(const actqkv_config* cfg, const Batch& b) {
  int n_sm = 148;
  int dev = 0;
  if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev);
  const int pairs = b.units() * cfg->n_kv_heads;
  int s = n_sm / std::max(1, pairs);
  return std::max(1, std::min(s, 16));
}

// The caller passes pos0 of the positions BEFORE the new tokens, as for the prefill kernels.  p0
// need not sit on a page boundary: the last, partly filled page of the local segment is loaded
// whole and the rows past p0 are masked out of the softmax (they must hold finite values).
int launch_attention_decode(const actqkv_config* cfg, const Batch& b, const AttnArgs& a, int n_splits,
                            void* workspace, cudaStream_t st) {
  const int U = b.units(), nt = a.n_tokens, Hq = cfg->n_q_heads, Hkv = cfg->n_kv_heads, G = Hq / Hkv;
  CUtensorMap tm_q, tm_kw, tm_vw, tm_kp, tm_vp;
  {
    const cuuint64_t dims[3] = {cuuint64_t(kD), cuuint64_t(Hq), cuuint64_t(U) * nt};
    const cuuint64_t str[2] = {cuuint64_t(kD) * 2, cuuint64_t(Hq) * kD * 2};
    const cuuint32_t box[3] = {64, cuuint32_t(G), cuuint32_t(kBM / G)};
    if (!encode(&tm_q, a.q, 3, dims, str, box)) return ACTQKV_ERR_LAUNCH;
  }
  {
    const cuuint64_t dims[3] = {cuuint64_t(kD), cuuint64_t(Hkv), cuuint64_t(U) * nt};
    const cuuint64_t str[2] = {cuuint64_t(kD) * 2, cuuint64_t(Hkv) * kD * 2};
    const cuuint32_t box[3] = {64, 1, cuuint32_t(kBN)};
    if (!encode(&tm_kw, a.k_win, 3, dims, str, box)) return ACTQKV_ERR_LAUNCH;
    if (!encode(&tm_vw, a.v_win, 3, dims, str, box)) return ACTQKV_ERR_LAUNCH;
  }
  {
    const cuuint64_t dims[4] = {cuuint64_t(kD), 16, cuuint64_t(Hkv), cuuint64_t(b.n_layers) * cfg->n_phys_pages};
    const cuuint64_t str[3] = {cuuint64_t(kD) * 2, cuuint64_t(kD) * 2 * 16, cuuint64_t(kD) * 2 * 16 * Hkv};
    const cuuint32_t box[4] = {64, 16, 1, 1};
    if (!encode(&tm_kp, a.k_pages, 4, dims, str, box)) return ACTQKV_ERR_LAUNCH;
    if (!encode(&tm_vp, a.v_pages, 4, dims, str, box)) return ACTQKV_ERR_LAUNCH;
  }
  TcParams p;
  p.a = a;
  p.n_q_heads = Hq; p.n_kv_heads = Hkv; p.group = G; p.block = cfg->block; p.n_init = cfg->n_init;
  p.n_local_prev = cfg->n_local_prev; p.cap_blocks = cfg->cap_blocks; p.max_pages = cfg->max_pages;
  p.n_phys_pages = cfg->n_phys_pages; p.n_layers = b.n_layers; p.out_bf16 = cfg->out_dtype == ACTQKV_BF16;
  const float scale = cfg->sm_scale > 0.f ? cfg->sm_scale : 1.f / sqrtf(float(kD));
  p.scale_log2 = scale * 1.4426950408889634f;
  DecodeParams dp;
  dp.spin_limit = cfg->test_wait_limit > 0 ? uint32_t(cfg->test_wait_limit) : kSpinLimit;
  dp.drop_k_tile = cfg->test_wait_limit > 0 ? cfg->test_drop_k_tile : -1;
  dp.n_splits = std::max(1, n_splits);
  const size_t rows = size_t(U) * nt * Hq;
  dp.part_o = static_cast<float*>(workspace);
  dp.part_lse = dp.part_o ? dp.part_o + rows * dp.n_splits * kD : nullptr;
  if (dp.n_splits > 1 && !workspace) return ACTQKV_ERR_NULL;
  static std::atomic<bool> opted_in[kMaxDevices];
  if (!opt_in_shared_memory(attention_decode_kernel, int(kSmemBytes), opted_in)) return ACTQKV_ERR_LAUNCH;
  dim3 grid(dp.n_splits, Hkv, U);
  attention_decode_kernel<<<grid, kThreads, kSmemBytes, st>>>(tm_q, tm_kw, tm_vw, tm_kp, tm_vp, p, dp);
  if (cudaGetLastError() != cudaSuccess) return ACTQKV_ERR_LAUNCH;
  if (dp.n_splits > 1) {
    decode_merge_kernel<<<unsigned((rows + 3) / 4), 128, 0, st>>>(dp.part_o, dp.part_lse, a.out, a.lse, int(rows),
                                                                dp.n_splits, nt, Hq, p.out_bf16);
  }
  return launch_status();
}

}  // namespace actqkv

// ---------------------------------------------------------------- entry point that allocates nothing
namespace {

// Scratch for the split form of the decode attention, owned by the library image itself: the
// array is part of the module, so every device that loads the library reserves these bytes from
// load until the process exits, and no allocation call is ever needed to use them.
static __device__ __align__(256) unsigned char g_decode_scratch[ACTQKV_STATIC_SCRATCH_BYTES];

// In host code `g_decode_scratch` is only a handle for the runtime, not a device address; the
// address of each device's copy is asked for once, with that device current, and remembered.
std::atomic<void*> g_scratch_addr[actqkv::kMaxDevices];

int static_scratch(void** ptr) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= actqkv::kMaxDevices) return ACTQKV_ERR_LAUNCH;
  void* addr = g_scratch_addr[dev].load(std::memory_order_acquire);
  if (!addr) {      // two threads may both ask; they get the same answer
    if (cudaGetSymbolAddress(&addr, g_decode_scratch) != cudaSuccess || !addr) {
      (void)cudaGetLastError();
      return ACTQKV_ERR_LAUNCH;
    }
    g_scratch_addr[dev].store(addr, std::memory_order_release);
  }
  *ptr = addr;
  return ACTQKV_OK;
}

}  // namespace

extern "C" int actqkv_decode_attention_static(const actqkv_config* cfg, const actqkv_batch* batch, const void* q,
                                              const void* k_win, const void* v_win, int32_t n_tokens,
                                              const void* k_pages, const void* v_pages, const int32_t* page_table,
                                              const int64_t* pos0, const int32_t* sel_idx, const int32_t* sel_count,
                                              void* out, float* lse, int32_t n_splits, int32_t* status, void* stream) {
  const Batch b = get_batch(batch);
  int rc = check_config(cfg, b);
  if (rc) return rc;
  ACTQKV_REQUIRE_PTR(q);
  ACTQKV_REQUIRE_PTR(k_win);
  ACTQKV_REQUIRE_PTR(v_win);
  ACTQKV_REQUIRE_PTR(k_pages);
  ACTQKV_REQUIRE_PTR(v_pages);
  ACTQKV_REQUIRE_PTR(out);
  ACTQKV_OPTIONAL_PTR(lse);
  if (!page_table || !pos0) return ACTQKV_ERR_NULL;
  if (cfg->cap_blocks > 0 && (!sel_idx || !sel_count)) return ACTQKV_ERR_NULL;
  if (n_tokens <= 0 || n_tokens > cfg->window) return ACTQKV_ERR_SHAPE;
  if (!attention_decode_supported(cfg, n_tokens)) return ACTQKV_ERR_UNSUPPORTED;
  if (n_splits <= 0) n_splits = attention_decode_auto_splits(cfg, b);
  if (n_splits > 64) return ACTQKV_ERR_SHAPE;
  if (attention_decode_workspace_bytes(cfg, b, n_tokens, n_splits) > int64_t(ACTQKV_STATIC_SCRATCH_BYTES))
    return ACTQKV_ERR_SCRATCH_LIMIT;
  void* scratch = nullptr;
  rc = static_scratch(&scratch);
  if (rc) return rc;
  AttnArgs a;
  a.q = q; a.k_win = k_win; a.v_win = v_win; a.k_pages = k_pages; a.v_pages = v_pages;
  a.page_table = page_table; a.pos0 = pos0; a.sel_idx = sel_idx; a.sel_count = sel_count;
  a.out = out; a.lse = lse; a.status = status; a.n_tokens = n_tokens;
  // Nothing in the scratch has to start at zero: every split writes its log-sum-exp -- minus
  // infinity when it holds no tile, or when it gave up on a bounded wait -- and the merge reads a
  // partial output only where that value is finite, so what an earlier call left behind is never
  // read.
  return launch_attention_decode(cfg, b, a, n_splits, scratch, reinterpret_cast<cudaStream_t>(stream));
}

