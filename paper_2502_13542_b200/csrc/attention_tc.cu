// Step 5, tensor-core kernel: attention of one window over
//   [initial tokens | selected blocks | local past | window tokens (causal)]     (Eq. 2)
// for bf16, D = 128, 16-token pages, on the 5th-generation tensor cores.
//
// One CTA = one 128-row query tile (128 consecutive window tokens of one query head).
// Key tiles of 128 keys are gathered page by page: each 16-token page is one TMA box of
// 16 rows x 128 bytes per 64-channel half, written with the 128-byte swizzle the MMA
// descriptors expect, so a [128 x 64] operand sub-tile is 8 boxes stacked in shared memory.
// The block -> page indirection (sel_idx, page_table) is resolved by the producer warps, one
// lane per box.  The window's own keys / values come from k_win / v_win with one box per half.
//
// Three warpgroups (384 threads):
//   warp 0        TMA producer of the K tiles (ring of 3) and of the Q tile
//   warp 1        tcgen05.mma issuer (one lane), owns the TMEM allocation
//   warp 2        TMA producer of the V tiles (ring of 3, released separately from K)
//   warps 4-7     softmax, key columns [0, 64) of every tile (packed f32x2 arithmetic)
//   warps 8-11    softmax, key columns [64, 128) of every tile
// A query row (= TMEM lane) is shared by two softmax threads, one per column half; they
// exchange their half-row maxima through shared memory once per tile.  Running max / sum are
// kept in base 2; P is written back over the S columns as two bf16 terms (hi + lo); O is
// rescaled in TMEM only when a row's max grew by more than 2^32 (lazy rescale).
//
// TMEM columns: S/P buffers 0..2 at [0,128) [128,256) [256,384), O at [384,512).
// S = Q K^T uses both operands from shared memory (K-major, SW128); O += P V takes P from
// TMEM and V from shared memory as an MN-major operand (the V tile is [keys x channels]).
// P of keys [32c, 32c+32) of a tile lives in columns [32c, 32c+16) (hi) and [32c+16, 32c+32) (lo).
// The tensor pipe executes in issue order QK(0) QK(1) | QK(j+2) PV(j) ..., so S(j+2) is computed
// while the softmax of tile j+1 runs and QK(j+3) cannot overwrite buffer j%3 before PV(j) read it.
// Every wait on an mbarrier is bounded; on expiry the CTA flags ACTQKV_DEV_TIMEOUT, stops
// issuing work, drains and frees its TMEM.
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


// ---------------------------------------------------------------- kernel
__global__ void __launch_bounds__(kThreads, 1)
attention_tc_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_kw,
                    const __grid_constant__ CUtensorMap tm_vw, const __grid_constant__ CUtensorMap tm_kp,
                    const __grid_constant__ CUtensorMap tm_vp, TcParams p) {
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

  const int mt = blockIdx.x, h = blockIdx.y, unit = blockIdx.z;
  const int g = h / p.group, seq = unit / p.n_layers, layer_local = unit - seq * p.n_layers;
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
  const int n_tiles = past_tiles + mt + 1;

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
      tma_load_3d(q_smem, &tm_q, bar_q, 0, h, unit * nt + mt * kBM);
      tma_load_3d(q_smem + kSubTileBytes, &tm_q, bar_q, 64, h, unit * nt + mt * kBM);
    }
    const int half = (lane >> 3) & 1, slot = lane & 7;     // lanes 0-15: one box each
    // Page lookups (sel_idx -> page_table, two dependent loads) are taken 32 granules = 4 tiles at
    // a time, one granule per lane, one chunk ahead of the tiles being issued, so their latency
    // is off the per-tile path; the issuing lane fetches its page with a shuffle.
    auto resolve = [&](int chunk) {
      const int gi = chunk * 32 + lane;
      return gi < past_tiles * 8 ? granule_page(ks, gi, p.a.status, !is_v) : ks.page_oob;
    };
    int page_cur = 0, page_next = resolve(0);
    bool ok = true;
    int issued = 0;
    for (int j = 0; j < n_tiles && ok; ++j) {
      const int s = j % kRing, it = j / kRing;
      if ((j & 3) == 0) page_cur = page_next;
      const int page = __shfl_sync(0xffffffffu, page_cur, (j & 3) * 8 + slot);
      if (it > 0) ok = mbar_wait(is_v ? bar_vempty(s) : bar_kempty(s), (it - 1) & 1, abort_flag);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      const uint32_t full = is_v ? bar_vfull(s) : bar_kfull(s);
      const uint32_t sbase = ring + s * kTileBytes;
      if (lane == 0) mbar_expect_tx(full, kTileBytes);
      __syncwarp();
      if (j < past_tiles) {
        if (lane < 16) tma_load_4d(sbase + half * kSubTileBytes + slot * 2048u, tm_pages, full, half * 64, 0, g, page);
      } else if (lane < 2) {
        tma_load_3d(sbase + lane * kSubTileBytes, tm_win, full, lane * 64, g, unit * nt + (j - past_tiles) * kBN);
      }
      issued = j + 1;
      if ((j & 3) == 0) page_next = resolve((j >> 2) + 1);   // after the issue: its stall is behind the ring
    }
    // drain: every issued copy must have landed before the CTA may exit on the abort path
    if (!ok) {
      for (int j = max(0, issued - kRing); j < issued; ++j) {
        const uint32_t full = is_v ? bar_vfull(j % kRing) : bar_kfull(j % kRing);
        for (uint32_t i = 0; i < kSpinLimit && !mbar_try_wait(full, (j / kRing) & 1); ++i) {}
      }
      if (!is_v) for (uint32_t i = 0; i < kSpinLimit && !mbar_try_wait(bar_q, 0); ++i) {}
    }
  } else if (warp == 1) {
    // =========================== MMA issuer ===========================
    if (lane == 0) {
      constexpr uint32_t idesc_qk = make_idesc(false, kBM, kBN);
      constexpr uint32_t idesc_pv = make_idesc(true, kBM, kBN);
      const uint32_t tmem_o = tmem + kSBuf * 128;
      bool ok = mbar_wait(bar_q, 0, abort_flag);
      auto issue_qk = [&](int j) {
        const int s = j % kRing;
        ok = ok && mbar_wait(bar_kfull(s), (j / kRing) & 1, abort_flag);
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
        ok = ok && mbar_wait(bar_vfull(s), (i / kRing) & 1, abort_flag);
        ok = ok && mbar_wait(bar_pfull(b), (i / kSBuf) & 1, abort_flag);
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
      if (ok) tc_commit(bar_done);
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
    for (int j = 0; j < n_tiles; ++j) {
      const int sb = j % kSBuf;
      ok = ok && mbar_wait(bar_sfull(sb), (j / kSBuf) & 1, abort_flag);
      tc_fence_after();
      const uint32_t s_addr = tmem + lane_addr + sb * 128 + b * 64;
      uint64_t sv[32];
      TMEM_LD64P_WAIT(s_addr, sv);
      // key-validity limit: ragged last past tile, or the causal diagonal of the last tile
      int limit = kBN;
      if (j < past_tiles) limit = min(kBN, n_past - j * kBN);
      else if (j == n_tiles - 1) limit = row + 1;
      limit -= b * 64;                                    // in this thread's column numbering
      const bool masked = (j == n_tiles - 1) || (j == past_tiles - 1 && (n_past % kBN) != 0);   // CTA-uniform
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
        ok = mbar_wait(bar_pvdone((j - 1) % kPvRing), ((j - 1) / kPvRing) & 1, abort_flag);
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
    ok = ok && mbar_wait(bar_done, 0, abort_flag);
    float* xrow = xchg + (n_tiles & 1) * 256 + row;
    xrow[b * 128] = l;
    ok = pair_sync_and(q4, ok);
    if (ok) {
      tc_fence_after();
      const float lsum = l + xrow[(1 - b) * 128];
      const float inv = lsum > 0.f ? 1.f / lsum : 0.f;
      const size_t tok = size_t(unit) * nt + size_t(mt) * kBM + row;
#pragma unroll
      for (int cc = 0; cc < 2; ++cc) {
        const int col = b * 64 + cc * 32;
        uint32_t orr[32];
        TMEM_LD32_WAIT(o_addr + cc * 32, orr);
        if (p.out_bf16) {
          __nv_bfloat16* ob = static_cast<__nv_bfloat16*>(p.a.out) + (tok * p.n_q_heads + h) * kD + col;
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
          float* of = static_cast<float*>(p.a.out) + (tok * p.n_q_heads + h) * kD + col;
#pragma unroll
          for (int i = 0; i < 8; ++i) {
            float4 v;
            v.x = __uint_as_float(orr[4 * i + 0]) * inv; v.y = __uint_as_float(orr[4 * i + 1]) * inv;
            v.z = __uint_as_float(orr[4 * i + 2]) * inv; v.w = __uint_as_float(orr[4 * i + 3]) * inv;
            *reinterpret_cast<float4*>(of + 4 * i) = v;
          }
        }
      }
      if (p.a.lse && b == 0)
        p.a.lse[(size_t(unit) * p.n_q_heads + h) * nt + size_t(mt) * kBM + row] =
            (m_used + log2f(lsum)) * 0.6931471805599453f;
    }
  }

  // ---- teardown
  tc_fence_before();
  __syncthreads();
  if (tid == 0 && *abort_flag) set_status(p.a.status, ACTQKV_DEV_TIMEOUT);
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(512));
  }
}

}  // namespace

namespace actqkv {

bool attention_tc_supported(const actqkv_config* cfg, int n_tokens) {
  return cfg->dtype == ACTQKV_BF16 && cfg->head_dim == 128 && cfg->page_tokens == 16 && n_tokens % kBM == 0 &&
         cfg->block % 16 == 0 && cfg->n_init % 16 == 0 && cfg->n_local_prev % 16 == 0;
}

int launch_attention_tc(const actqkv_config* cfg, const Batch& b, const AttnArgs& a, cudaStream_t st) {
  const int U = b.units(), nt = a.n_tokens, Hq = cfg->n_q_heads, Hkv = cfg->n_kv_heads;
  CUtensorMap tm_q, tm_kw, tm_vw, tm_kp, tm_vp;
  {
    const cuuint64_t dims[3] = {cuuint64_t(kD), cuuint64_t(Hq), cuuint64_t(U) * nt};
    const cuuint64_t str[2] = {cuuint64_t(kD) * 2, cuuint64_t(Hq) * kD * 2};
    const cuuint32_t box[3] = {64, 1, cuuint32_t(kBM)};
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
  p.n_q_heads = Hq; p.n_kv_heads = Hkv; p.group = Hq / Hkv; p.block = cfg->block; p.n_init = cfg->n_init;
  p.n_local_prev = cfg->n_local_prev; p.cap_blocks = cfg->cap_blocks; p.max_pages = cfg->max_pages;
  p.n_phys_pages = cfg->n_phys_pages; p.n_layers = b.n_layers; p.out_bf16 = cfg->out_dtype == ACTQKV_BF16;
  const float scale = cfg->sm_scale > 0.f ? cfg->sm_scale : 1.f / sqrtf(float(kD));
  p.scale_log2 = scale * 1.4426950408889634f;
  static std::atomic<bool> opted_in[kMaxDevices];
  if (!opt_in_shared_memory(attention_tc_kernel, int(kSmemBytes), opted_in)) return ACTQKV_ERR_LAUNCH;
  dim3 grid(nt / kBM, Hq, U);
  attention_tc_kernel<<<grid, kThreads, kSmemBytes, st>>>(tm_q, tm_kw, tm_vw, tm_kp, tm_vp, p);
  return launch_status();
}

}  // namespace actqkv
