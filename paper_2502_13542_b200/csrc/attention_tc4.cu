// Step 5, tensor-core kernel for a whole KV group: the attention of Eq. 2,
//   [initial tokens | selected blocks | local past | window tokens (causal)],
// for bf16, D = 128, 16-token pages and G = Hq / Hkv a multiple of 4.
//
// Work unit = 128 window tokens x 4 query heads of one KV head.  A cluster of 4 CTAs takes it:
//   * CTAs (0, 1) and (2, 3) are two PAIRS.  A pair runs tcgen05.mma.cta_group::2 products of
//     M = 256: CTA r of a pair holds the Q tiles of heads 2r ("set X") and 2r + 1 ("set Y"), so one
//     K / V tile serves four heads, and it supplies HALF of every B operand -- 64 of the tile's
//     128 keys for S = Q K^T, 64 of the 128 channels of V for O += P V.  Per key tile a CTA
//     therefore gathers 32 KiB for 2 x 2 x 128 x 128 x 128 x 2 flop of its own: half the copy
//     requests per product of the two-head pair kernel (attention_tc2.cu).
//   * The two pairs split the key stream: pair 0 takes the first half of the key tiles, pair 1
//     the rest (with the causal diagonal).  At the end each CTA hands the partial result
//     (O, running maximum, row sum) of ONE set to its counterpart in the other pair through
//     distributed shared memory and finishes the other set: pair 0 writes set X, pair 1 set Y.
//     No workspace in global memory, no second kernel, and 8 x 4 units fill 128 SMs.
//
// Roles per CTA (512 threads):
//   warp 0      K producer (TMA page gather) and the Q tiles
//   warps 1, 3  MMA issuers (leader CTA of the pair only), one thread each: warp 1 issues the
//               products of set X, warp 3 those of set Y, each in order.  A key tile is handled as
//               two BLOCKS of 64 keys; block b of a set uses S buffer b % 2:
//                   ... PV(b)  QK(b+2)  PV(b+1)  QK(b+3) ...
//               The tensor pipe executes one thread's products in issue order, so QK(b+2) overwrites
//               its S buffer only after PV(b) has read P(b) from it, and while a softmax thread works
//               on block b the scores of block b + 1 are already waiting for it.  A ring slot is
//               released when both issuers have committed their last product on it.
//   warp 2      V producer
//   warps 4-7   softmax of set X, one thread per query row (a block's 64 fp32 scores in registers:
//               no shuffles for the row maximum or sum)
//   warps 8-11  softmax of set Y.  Every scheduler of the SM holds one warp of each set.
//   warps 12-15 V conversion (bf16 -> fp16 in place, two tiles ahead) and O correction
// P is fp16 (11 significant bits) and overwrites the first 32 columns of its S buffer; the running
// maximum used for P may lag the true one by up to 2^8 (fp16 range), and when it moves O is
// rescaled by the correction warps, off the softmax threads' path.
// TMEM columns (every CTA): S_X [0,64) [64,128)  S_Y [128,192) [192,256)  O_X [256,384)  O_Y [384,512).
// Measured on the LLaMA3-8B layer at 32k context: 60.8 us per call against 55.8 us for the two-head
// pair kernel, so the dispatcher takes this kernel only when asked to (ACTQKV_ATTN_CLUSTER4).  A
// tcgen05.mma of M = 256 occupies the tensor pipe ~62 cycles for every N <= 128, so the 64-key
// blocks that double-buffered S needs (TMEM has 512 columns: two sets x (2 x 64 S + 128 O)) spend
// twice the pipe time on Q K^T; with 128-key blocks and one S buffer per set the pipe waits for the
// softmax -> P -> P V -> Q K^T chain instead (4,350 cycles per key tile measured).
// No TMA multicast anywhere.  Every wait on an mbarrier is bounded; on expiry the CTA flags
// ACTQKV_DEV_TIMEOUT, stops issuing work and drains; every CTA of the cluster always reaches the
// cluster barriers of the hand-over, so nobody waits for a CTA that gave up.
#include "tc_common.cuh"

using namespace actqkv;
using namespace actqkv::tc;

namespace {

constexpr int kBM = 128, kBN = 128, kD = 128;
constexpr int kRingK = 5;                                // K halves in flight
constexpr int kRingV = 5;                                // V halves in flight
constexpr int kLag = 2;                                  // V is converted this many tiles ahead of its use
constexpr float kRescaleF16 = 8.0f;                      // the maximum used for P may lag by 2^8 (fp16 tops out at 65504)
constexpr int kThreads = 512;
constexpr uint32_t kSubTileBytes = 128 * 128;            // [128 rows x 64 bf16], 16 KiB
constexpr uint32_t kTileBytes = 2 * kSubTileBytes;       // 32 KiB: one Q tile
constexpr uint32_t kHalfBytes = 16 * 1024;               // what one CTA holds of a K or V tile
constexpr uint32_t kKSubBytes = 64 * 128;                // [64 keys x 64 channels] sub-tile of a K half
constexpr uint32_t kQBytes = 2 * kTileBytes;             // the Q tiles of sets X and Y
constexpr uint32_t kSmemTiles = kQBytes + (kRingK + kRingV) * kHalfBytes;
constexpr int kBlk = 64;                                 // keys per block = columns of an S buffer
constexpr int kNumBars = 1 + 2 * kRingK + 3 * kRingV + 4 * 4 + 2 + 1;
constexpr uint32_t kBarBytes = 384;                      // barriers, TMEM slot, abort flag
constexpr uint32_t kXchgBytes = 4 * 128 * 4;             // O factors [set][buffer][row]; reused for the hand-over of (maximum, sum) [row][2]
constexpr uint32_t kSmemNeeded = kSmemTiles + kBarBytes + kXchgBytes;
constexpr uint32_t kSmemBytes = 227 * 1024;              // everything an SM offers one CTA
constexpr uint32_t kStageBytes = 128 * 128 * 4;          // one set's partial O in fp32, staged over the rings
static_assert(8 * kNumBars + 16 <= kBarBytes, "barrier area too small");
static_assert(kSmemNeeded <= kSmemBytes, "shared memory budget");
static_assert(kStageBytes <= (kRingK + kRingV) * kHalfBytes, "the hand-over stage must fit in the rings");

// ---------------------------------------------------------------- cluster-wide PTX wrappers
__device__ __forceinline__ uint32_t cluster_rank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
// Address of CTA `rank`'s copy of a shared-memory object, in the cluster window.
__device__ __forceinline__ uint32_t cta_addr(uint32_t local, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(local), "r"(rank));
  return r;
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_bar) {
  asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(cluster_bar) : "memory");
}
__device__ __forceinline__ void st_cluster_f32x4(uint32_t addr, float a, float b, float c, float d) {
  asm volatile("st.shared::cluster.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "f"(a), "f"(b), "f"(c), "f"(d) : "memory");
}
__device__ __forceinline__ void st_cluster_f32x2(uint32_t addr, float a, float b) {
  asm volatile("st.shared::cluster.v2.f32 [%0], {%1, %2};" ::"r"(addr), "f"(a), "f"(b) : "memory");
}
// TMA loads whose completion is signalled on the pair leader's barrier (`bar` in the cluster window).
__device__ __forceinline__ void tma2_load_3d(uint32_t dst, const CUtensorMap* tm, uint32_t bar, int c0, int c1, int c2) {
  asm volatile(
      "cp.async.bulk.tensor.3d.cta_group::2.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
      ::"r"(dst), "l"(tm), "r"(bar), "r"(c0), "r"(c1), "r"(c2) : "memory");
}
__device__ __forceinline__ void tma2_load_4d(uint32_t dst, const CUtensorMap* tm, uint32_t bar, int c0, int c1, int c2,
                                             int c3) {
  asm volatile(
      "cp.async.bulk.tensor.4d.cta_group::2.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
      ::"r"(dst), "l"(tm), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3) : "memory");
}
__device__ __forceinline__ void prefetch_tensormap(const CUtensorMap* tm) {
  asm volatile("prefetch.tensormap [%0];" ::"l"(tm) : "memory");
}
// Arrives on the barrier at this offset in BOTH CTAs of the pair once every MMA issued so far has
// completed; `mask` holds the two CTAs' ranks in the cluster.
__device__ __forceinline__ void pair_commit(uint32_t bar, uint16_t mask) {
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
               ::"r"(bar), "h"(mask) : "memory");
}
// Descriptors are passed as (low, high) words; kAcc = accumulate into D (else overwrite).
template <bool kAcc>
__device__ __forceinline__ void mma2_ss(uint32_t d_tmem, uint32_t a_lo, uint32_t b_lo, uint32_t hi, uint32_t idesc) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\tsetp.ne.b32 p, %5, 0;\n\t"
      "mov.b64 da, {%1, %3};\n\tmov.b64 db, {%2, %3};\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], da, db, %4, p;\n\t}"
      ::"r"(d_tmem), "r"(a_lo), "r"(b_lo), "r"(hi), "r"(idesc), "n"(kAcc ? 1 : 0) : "memory");
}
__device__ __forceinline__ void mma2_ts(uint32_t d_tmem, uint32_t a_tmem, uint32_t b_lo, uint32_t hi, uint32_t idesc, uint32_t acc) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t.reg .b64 db;\n\tsetp.ne.b32 p, %5, 0;\n\t"
      "mov.b64 db, {%2, %3};\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], [%1], db, %4, p;\n\t}"
      ::"r"(d_tmem), "r"(a_tmem), "r"(b_lo), "r"(hi), "r"(idesc), "r"(acc) : "memory");
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}

// ---------------------------------------------------------------- kernel
__global__ void __launch_bounds__(kThreads, 1)
attention_tc4_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_kw,
                     const __grid_constant__ CUtensorMap tm_vw, const __grid_constant__ CUtensorMap tm_kp,
                     const __grid_constant__ CUtensorMap tm_vp, TcParams p) {
  extern __shared__ __align__(1024) unsigned char smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  const bool smem_short = base - raw + kSmemNeeded > kSmemBytes;   // never with a 1 KiB-aligned window
  const uint32_t q_smem = base;                                    // [set][128 rows x 128 channels]
  const uint32_t k_ring = base + kQBytes;
  const uint32_t v_ring = k_ring + kRingK * kHalfBytes;
  const uint32_t bars = base + kSmemTiles;
  // barrier slots (8 bytes each)
  const uint32_t bar_q = bars;
  auto bar_kfull = [&](int s) { return bars + 8u * (1 + s); };
  auto bar_kempty = [&](int s) { return bars + 8u * (1 + kRingK + s); };
  auto bar_vfull = [&](int s) { return bars + 8u * (1 + 2 * kRingK + s); };
  auto bar_vempty = [&](int s) { return bars + 8u * (1 + 2 * kRingK + kRingV + s); };
  auto bar_vready = [&](int s) { return bars + 8u * (1 + 2 * kRingK + 2 * kRingV + s); };
  constexpr int kB0 = 1 + 2 * kRingK + 3 * kRingV;
  // per (set t, S buffer u): index 2 t + u
  auto bar_sfull = [&](int t, int u) { return bars + 8u * (kB0 + 2 * t + u); };        // S is complete
  auto bar_pfull = [&](int t, int u) { return bars + 8u * (kB0 + 4 + 2 * t + u); };    // P is published (leader)
  auto bar_f = [&](int t, int u) { return bars + 8u * (kB0 + 8 + 2 * t + u); };        // O factors are in shared memory
  auto bar_corr = [&](int t, int u) { return bars + 8u * (kB0 + 12 + 2 * t + u); };    // O is on P's maximum (leader)
  auto bar_pvdone = [&](int t) { return bars + 8u * (kB0 + 16 + t); };                 // a P V of set t has completed
  const uint32_t bar_done = bars + 8u * (kNumBars - 1);
  unsigned char* base_generic = smem_raw + (base - raw);
  unsigned char* bars_generic = base_generic + kSmemTiles;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars_generic + 8 * kNumBars);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(bars_generic + 8 * kNumBars + 8);
  float* f_share = reinterpret_cast<float*>(bars_generic + kBarBytes);   // [set][buffer][128] O correction factors
  float* ml_share = f_share;     // the factors are dead when the hand-over begins (after cluster barrier 1)                                   // [2][128] counterpart's (maximum, sum) of the set this CTA finishes
  float* stage = reinterpret_cast<float*>(base_generic + kQBytes);       // [32 column quads][128 rows][4]: counterpart's partial O

  const int quad = blockIdx.x >> 2, mt = blockIdx.y, unit = blockIdx.z;
  const uint32_t rank = cluster_rank();                               // 0..3
  const uint32_t split = rank >> 1, r = rank & 1;                     // pair (= share of the key stream), CTA inside the pair
  const bool leader = r == 0;
  const uint32_t lead_rank = rank & ~1u;
  const uint16_t pair_mask = uint16_t(3u << lead_rank);
  auto leader_addr = [&](uint32_t local) { return cta_addr(local, lead_rank); };
  const int h0 = quad * 4 + int(r) * 2;                               // heads h0 (set X) and h0 + 1 (set Y)
  const int g = (quad * 4) / p.group, seq = unit / p.n_layers, layer_local = unit - seq * p.n_layers;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int nt = p.a.n_tokens;

  // ---- set-up that depends on no earlier kernel: barriers, TMEM, descriptor prefetch
  if (tid == 0) {
    mbar_init(bar_q, 1);
    for (int s = 0; s < kRingK; ++s) { mbar_init(bar_kfull(s), 1); mbar_init(bar_kempty(s), 2); }
    for (int s = 0; s < kRingV; ++s) { mbar_init(bar_vfull(s), 1); mbar_init(bar_vempty(s), 2); mbar_init(bar_vready(s), 8); }
    for (int t = 0; t < 2; ++t) {
      for (int u = 0; u < 2; ++u) {
        mbar_init(bar_sfull(t, u), 1); mbar_init(bar_pfull(t, u), 8);
        mbar_init(bar_f(t, u), 4); mbar_init(bar_corr(t, u), 8);
      }
      mbar_init(bar_pvdone(t), 1);
    }
    mbar_init(bar_done, 2);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 0 && lane < 3) prefetch_tensormap(lane == 0 ? &tm_q : lane == 1 ? &tm_kp : &tm_kw);
  if (warp == 2 && lane < 2) prefetch_tensormap(lane == 0 ? &tm_vp : &tm_vw);
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(512));
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;");
  }
  tc_fence_before();
  cluster_sync_all();         // every CTA's barriers are initialised and every pair holds its TMEM
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  grid_dependency_wait();            // the selection (and whatever produced Q / K / V) is complete from here on
  // ---- geometry (uniform over the cluster)
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
  const int n_past = geo.init_len + c * p.block + int(local_len);     // exact: the tail of the last page is masked
  const int past_tiles = (n_past + kBN - 1) / kBN;
  const int all_tiles = past_tiles + mt + 1;
  // this pair's share of the key tiles: [j_lo, j_lo + n_tiles)
  const int first_half = (all_tiles + 1) / 2;
  const int j_lo = split == 0 ? 0 : first_half;
  const int n_tiles = smem_short ? 0 : (split == 0 ? first_half : all_tiles - first_half);

  if (tid == 0 && (bad || smem_short)) set_status(p.a.status, ACTQKV_DEV_BAD_SELECTION);

  // The hand-over at the end has three cluster barriers; every thread of the cluster takes part in
  // all of them, whatever its role and whether or not it gave up on a wait.  Roles other than the
  // softmax pass the first two here; the third is in the common teardown.
  auto pass_handover_barriers = [&]() {
    tc_fence_before();
    cluster_sync_all();
    cluster_sync_all();
  };

  // state of a softmax thread (one query row of one set), needed again in the hand-over
  float m_run = -INFINITY, l_run = 0.f;                  // running maximum (log2 units) and row sum
  bool row_ok = true;

  if (warp < 4) {
    if (warp == 0 || warp == 2) {
      // =========================== TMA producers: warp 0 -> K half (and Q), warp 2 -> V half ===========================
      // This CTA's half of a tile: keys [64 r, +64) of K (all channels), channels [64 r, +64) of V
      // (all keys).  K halves of both CTAs complete on the leader's barrier (the leader posts the
      // bytes of both); a V half completes on its own CTA's barrier, where the converter warps wait.
      const bool is_v = warp == 2;
      const uint32_t ring = is_v ? v_ring : k_ring;
      const CUtensorMap* tm_pages = is_v ? &tm_vp : &tm_kp;
      const CUtensorMap* tm_win = is_v ? &tm_vw : &tm_kw;
      if (!is_v && lane == 0 && n_tiles > 0) {
        if (leader) mbar_expect_tx(bar_q, 2 * kQBytes);
        const uint32_t qb = leader_addr(bar_q);
        const int row0 = unit * nt + mt * kBM;
#pragma unroll
        for (int t = 0; t < 2; ++t) {
          tma2_load_3d(q_smem + t * kTileBytes, &tm_q, qb, 0, h0 + t, row0);
          tma2_load_3d(q_smem + t * kTileBytes + kSubTileBytes, &tm_q, qb, 64, h0 + t, row0);
        }
      }
      // lanes 0-7 issue one box each.  V: granule = lane.  K: (channel half, slot); the CTA's 64
      // key rows are [32 keys of block 0 | 32 keys of block 1], i.e. 16-key granules
      // 2 r, 2 r + 1, 4 + 2 r, 5 + 2 r of the tile, so that block b is keys [64 b, 64 b + 64) in order.
      const int half = (lane >> 2) & 1, slot = lane & 3;
      const int my_granule = is_v ? (lane & 7) : (slot >> 1) * 4 + int(r) * 2 + (slot & 1);
      // Page lookups (sel_idx -> page_table, two dependent loads) are taken 32 granules = 4 tiles at
      // a time, one granule per lane, one chunk ahead of the tiles being issued.
      auto resolve = [&](int chunk) {
        const int gi = (j_lo + chunk * 4) * 8 + lane;
        return gi < past_tiles * 8 ? granule_page(ks, gi, p.a.status, !is_v && rank == 0) : ks.page_oob;
      };
      int page_cur = 0, page_next = n_tiles > 0 ? resolve(0) : 0;
      bool ok = true;
      int issued = 0;
      const int ring_n = is_v ? kRingV : kRingK;
      for (int j = 0; j < n_tiles && ok; ++j) {
        const int s = j % ring_n, it = j / ring_n;
        if ((j & 3) == 0) page_cur = page_next;
        const int page = __shfl_sync(0xffffffffu, page_cur, (j & 3) * 8 + my_granule);
        if (it > 0) ok = mbar_wait(is_v ? bar_vempty(s) : bar_kempty(s), (it - 1) & 1, abort_flag);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        const uint32_t full_local = is_v ? bar_vfull(s) : bar_kfull(s);
        const uint32_t full = is_v ? full_local : leader_addr(full_local);
        const uint32_t sbase = ring + s * kHalfBytes;
        if (lane == 0) {
          if (is_v) mbar_expect_tx(full_local, kHalfBytes);
          else if (leader) mbar_expect_tx(full_local, 2 * kHalfBytes);
        }
        __syncwarp();
        const int jj = j_lo + j;                          // tile index in the whole key stream
        if (jj < past_tiles) {
          if (lane < 8) {
            if (is_v) tma_load_4d(sbase + lane * 2048u, tm_pages, full, int(r) * 64, 0, g, page);
            else tma2_load_4d(sbase + half * kKSubBytes + slot * 2048u, tm_pages, full, half * 64, 0, g, page);
          }
        } else {
          const int row0 = unit * nt + (jj - past_tiles) * kBN;
          if (is_v) {
            if (lane == 0) tma_load_3d(sbase, tm_win, full, int(r) * 64, g, row0);
          } else if (lane < 4) {        // (channel half, block): 32 keys each
            const int hf = lane & 1, blk = lane >> 1;
            tma2_load_3d(sbase + hf * kKSubBytes + blk * 4096u, tm_win, full, hf * 64, g, row0 + blk * kBlk + int(r) * 32);
          }
        }
        issued = j + 1;
        if ((j & 3) == 0) page_next = resolve((j >> 2) + 1);   // after the issue: its stall is behind the ring
      }
      // drain: what this CTA issued must have landed before it may go on to the hand-over on the
      // abort path; K copies complete on the leader's barriers, which only the leader can poll, so
      // the other CTA waits out the worst-case copy time instead
      if (!ok) {
        if (leader || is_v) {
          for (int j = max(0, issued - ring_n); j < issued; ++j) {
            const uint32_t fl = is_v ? bar_vfull(j % ring_n) : bar_kfull(j % ring_n);
            for (uint32_t i = 0; i < kSpinLimit && !mbar_try_wait(fl, (j / ring_n) & 1); ++i) {}
          }
          if (!is_v && leader) for (uint32_t i = 0; i < kSpinLimit && !mbar_try_wait(bar_q, 0); ++i) {}
        } else {
          __nanosleep(200000);
        }
      }
    } else if (warp == 1 || warp == 3) {
      // =========================== MMA issuers: warp 1 set X, warp 3 set Y (leader CTA of the pair) ===========================
      // One thread, one order.  Per 64-key block b:  PV_X(b)  QK_X(b+2)  PV_Y(b)  QK_Y(b+2).  The
      // pipe runs products in issue order, so nothing else orders the reuse of an S / P buffer.
      if (lane == 0 && leader && n_tiles > 0) {
        constexpr uint32_t kHi = desc_hi(1024u);       // descriptor high words are constants
        constexpr uint32_t idesc_qk = make_idesc(false, 2 * kBM, kBlk);
        constexpr uint32_t idesc_pv = make_idesc_f16(true, 2 * kBM, kBN);
        const int n_blocks = 2 * n_tiles;
        bool ok = mbar_wait(bar_q, 0, abort_flag);
        // S(t, b) = Q_t K(b)^T: A = this CTA's 128 query rows, B = this CTA's 32 keys of the block
        auto qk = [&](int t, int b) {
          const uint32_t q_lo = desc_lo(q_smem + t * kTileBytes, 16u);
          const uint32_t k_lo = desc_lo(k_ring + ((b >> 1) % kRingK) * kHalfBytes + (b & 1) * 4096u, 16u);
          const uint32_t s_tmem = tmem + t * 128 + (b & 1) * kBlk;
          mma2_ss<false>(s_tmem, q_lo, k_lo, kHi, idesc_qk);
#pragma unroll
          for (int k = 1; k < kD / 16; ++k) {          // both operands advance 16 channels per step
            constexpr uint32_t kUnit = 16;             // descriptor addresses count 16-byte units
            const uint32_t a_off = ((k >> 2) * kSubTileBytes + (k & 3) * 32u) / kUnit;
            const uint32_t b_off = ((k >> 2) * kKSubBytes + (k & 3) * 32u) / kUnit;
            mma2_ss<true>(s_tmem, q_lo + a_off, k_lo + b_off, kHi, idesc_qk);
          }
        };
        // O_t += P(t, b) V(b): A = 64 keys of P as 32 packed fp16 columns, B = this CTA's 64 channels
        auto pv = [&](int t, int b) {
          const uint32_t v_lo = desc_lo(v_ring + ((b >> 1) % kRingV) * kHalfBytes, kSubTileBytes) + (b & 1) * (4 * 2048u / 16u);
          const uint32_t p_tmem = tmem + t * 128 + (b & 1) * kBlk, o_tmem = tmem + 256 + t * 128;
#pragma unroll
          for (int k = 0; k < kBlk / 16; ++k)     // 16 keys per step: B advances 16 rows of 128 bytes, A 8 packed fp16 columns
            mma2_ts(o_tmem, p_tmem + k * 8, v_lo + k * (2048u / 16u), kHi, idesc_pv, (b > 0 || k > 0) ? 1u : 0u);
        };
        const int t = warp == 1 ? 0 : 1;                 // this thread's set
        ok = ok && mbar_wait(bar_kfull(0), 0, abort_flag);
        if (ok) {
          tc_fence_after();
          qk(t, 0); pair_commit(bar_sfull(t, 0), pair_mask);
          qk(t, 1); pair_commit(bar_kempty(0), pair_mask); pair_commit(bar_sfull(t, 1), pair_mask);
        }
        for (int b = 0; b < n_blocks && ok; ++b) {
          const int j = b >> 1, u = b & 1;
          const uint32_t ph = (b >> 1) & 1;             // phase of the per-(set, buffer) barriers
          const bool more = b + 2 < n_blocks;
          if (u == 0) ok = mbar_wait(bar_vready(j % kRingV), (j / kRingV) & 1, abort_flag);   // V(j) is fp16 in both CTAs
          ok = ok && mbar_wait(bar_corr(t, u), ph, abort_flag);                  // O is on P(b)'s maximum
          ok = ok && mbar_wait(bar_pfull(t, u), ph, abort_flag);                 // P(b) published by both CTAs
          if (!ok) break;
          tc_fence_after();
          pv(t, b);
          if (u == 1) pair_commit(bar_vempty(j % kRingV), pair_mask);
          pair_commit(bar_pvdone(t), pair_mask);
          if (more) {
            if (u == 0) {
              ok = mbar_wait(bar_kfull((j + 1) % kRingK), ((j + 1) / kRingK) & 1, abort_flag);
              if (!ok) break;
              tc_fence_after();
            }
            qk(t, b + 2);
            if (u == 1) pair_commit(bar_kempty((j + 1) % kRingK), pair_mask);
            pair_commit(bar_sfull(t, u), pair_mask);
          }
        }
        if (ok) pair_commit(bar_done, pair_mask);
      }
      __syncwarp();
    }
    __syncwarp();
    pass_handover_barriers();
  }
  else if (warp >= 12) {
    // =========================== V converters / O correction ===========================
    // This CTA's half of every V tile, as it landed (bf16), becomes fp16 in place, 128 bytes per
    // thread, kLag tiles ahead of its use; one arrival per warp on the leader's "V ready" barrier.
    const int ct = tid - 12 * 32;                         // 0..127 = this thread's query row in both sets
    const int q4 = warp & 3;                              // TMEM lane quadrant of this warp
    const uint32_t o_lane = tmem + (uint32_t(q4 * 32) << 16) + 256;
    bool ok = true;
    for (int it = 0; it < n_tiles + kLag && ok; ++it) {
      if (it < n_tiles) {
        const int vs = it % kRingV;
        ok = mbar_wait(bar_vfull(vs), (it / kRingV) & 1, abort_flag);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        uint4* vp = reinterpret_cast<uint4*>(base_generic + (v_ring - base) + vs * kHalfBytes);
        uint4 a[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) a[i] = vp[i * 128 + ct];      // consecutive threads, consecutive 16 bytes
#pragma unroll
        for (int i = 0; i < 8; ++i) vp[i * 128 + ct] = bf16x8_to_f16x8(a[i]);
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // visible to the tensor core's reads
        __syncwarp();
        if (lane == 0) mbar_arrive_cluster(leader_addr(bar_vready(vs)));
      }
      const int j = it - kLag;
      if (j >= 0) {
        // The maxima of the two blocks of tile j are known: where a row's maximum grew, its O (on
        // the old maximum) is scaled down before P V of that block is added.  The softmax threads
        // do not wait for this.  Order as the issuer's: (block, set) = (2j, X) (2j, Y) (2j+1, X) (2j+1, Y).
        for (int bt = 0; bt < 4 && ok; ++bt) {
          const int u = bt >> 1, t = bt & 1, b = 2 * j + u;
          ok = mbar_wait(bar_f(t, u), j & 1, abort_flag);
          ok = __all_sync(0xffffffffu, ok);
          if (!ok) break;
          const float f = f_share[(t * 2 + u) * 128 + ct];
          if (__any_sync(0xffffffffu, f != 1.f)) {          // never for the first block
            // O must be quiescent: P V of every earlier block of this set complete
            ok = mbar_wait(bar_pvdone(t), (b - 1) & 1, abort_flag);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            tc_fence_after();
#pragma unroll
            for (int cc = 0; cc < 4; ++cc) {
              uint32_t orr[32];
              TMEM_LD32_WAIT(o_lane + t * 128 + cc * 32, orr);
#pragma unroll
              for (int i = 0; i < 32; ++i) orr[i] = __float_as_uint(__uint_as_float(orr[i]) * f);
              TMEM_ST32(o_lane + t * 128 + cc * 32, orr);
            }
            tmem_wait_st();
            tc_fence_before();
          }
          __syncwarp();
          if (lane == 0) mbar_arrive_cluster(leader_addr(bar_corr(t, u)));
        }
      }
    }
    __syncwarp();
    pass_handover_barriers();
  }
  else {
    // =========================== softmax: warps 4-7 set X, warps 8-11 set Y ===========================
    // One thread per query row: the row's 64 scores of a block sit in its registers, so the maximum
    // and the sum need no exchange with other threads.
    const int t = warp >= 8 ? 1 : 0;
    const int q4 = warp & 3, row = q4 * 32 + lane;
    const uint32_t s_row = tmem + (uint32_t(q4 * 32) << 16) + t * 128;
    for (int b = 0; b < 2 * n_tiles; ++b) {
      const int u = b & 1;
      row_ok = mbar_wait(bar_sfull(t, u), (b >> 1) & 1, abort_flag);
      row_ok = __all_sync(0xffffffffu, row_ok);
      if (!row_ok) break;
      tc_fence_after();
      const uint32_t s_addr = s_row + u * kBlk;
      uint64_t sv[32];                                    // sv[i] = columns 2i, 2i + 1 of this block
      TMEM_LD64P_WAIT(s_addr, sv);
      // key-validity limit: ragged last past tile, or the causal diagonal of the last tile
      const int jj = j_lo + (b >> 1);
      int lim = kBN;
      if (jj < past_tiles) lim = min(kBN, n_past - jj * kBN);
      else if (jj == all_tiles - 1) lim = row + 1;
      lim -= u * kBlk;                                    // in this block's column numbering
      const bool masked = (jj == all_tiles - 1) || (jj == past_tiles - 1 && (n_past % kBN) != 0);   // CTA-uniform
      float mx0 = -INFINITY, mx1 = -INFINITY, mx2 = -INFINITY, mx3 = -INFINITY;
      if (masked) {
#pragma unroll
        for (int i = 0; i < 32; ++i) {
          const float a0 = 2 * i < lim ? lo2(sv[i]) : -INFINITY, a1 = 2 * i + 1 < lim ? hi2(sv[i]) : -INFINITY;
          sv[i] = pack2(a0, a1);
          mx0 = max3(mx0, a0, a1);
        }
      } else {
#pragma unroll
        for (int i = 0; i < 32; i += 4) {                 // four chains
          mx0 = max3(mx0, lo2(sv[i]), hi2(sv[i]));
          mx1 = max3(mx1, lo2(sv[i + 1]), hi2(sv[i + 1]));
          mx2 = max3(mx2, lo2(sv[i + 2]), hi2(sv[i + 2]));
          mx3 = max3(mx3, lo2(sv[i + 3]), hi2(sv[i + 3]));
        }
      }
      const float mx = fmaxf(fmaxf(mx0, mx1), fmaxf(mx2, mx3));
      // (a block of the diagonal tile can be masked entirely for a row: mx = -inf, nothing changes)
      const float m_new = fmaxf(m_run, mx * p.scale_log2);
      const bool grow = m_new - m_run > kRescaleF16;      // also true for the first block
      // Where the maximum grew, O has to be scaled by f before P(b) V(b) is added: the correction
      // warps do that, off this thread's path; the first block starts O, so its factor is 1.
      const float f = grow ? ex2(m_run - m_new) : 1.f;
      f_share[(t * 2 + u) * 128 + row] = b > 0 ? f : 1.f;
      __syncwarp();
      if (lane == 0) mbar_arrive(bar_f(t, u));
      if (grow) { m_run = m_new; l_run *= f; }
      // P = exp2(x - m) in fp16, written over the first 32 columns of this row of the S buffer (all
      // of which this thread already holds).  The row sum adds the values as rounded to fp16, the
      // ones P V multiplies, so numerator and denominator carry the same rounding.
      const uint64_t scale2 = pack2(p.scale_log2, p.scale_log2), negm = pack2(-m_run, -m_run);
      float sa = 0.f, sb = 0.f;
#pragma unroll
      for (int cq = 0; cq < 2; ++cq) {
        uint32_t pk[16];
#pragma unroll
        for (int i = 0; i < 16; ++i) {
          const uint64_t x = fma2(sv[16 * cq + i], scale2, negm);
          pk[i] = pack_f16(ex2(lo2(x)), ex2(hi2(x)));
          add_f16x2(sa, sb, pk[i]);
        }
        TMEM_ST16(s_addr + cq * 16, pk);
      }
      l_run += sa + sb;
      tmem_wait_st();
      tc_fence_before();
      __syncwarp();                                       // one arrival per warp: 8 of both CTAs' warps of this set
      if (lane == 0) mbar_arrive_cluster(leader_addr(bar_pfull(t, u)));
    }
    // the last P V depends, through the softmax, on every Q K^T: O is final once this completes
    if (n_tiles > 0) {
      row_ok = row_ok && mbar_wait(bar_done, 0, abort_flag);
      row_ok = __all_sync(0xffffffffu, row_ok);
    }

    // ---- hand-over between the two pairs (the other roles only pass the three cluster barriers)
    const int set = t;
    const uint32_t o_addr = tmem + (uint32_t(q4 * 32) << 16) + 256 + set * 128;
    const bool have = n_tiles > 0 && row_ok;                // this CTA holds a partial result for its rows
    __syncwarp();
    tc_fence_before();
    cluster_sync_all();       // 1: every product of the cluster has completed: O is final, the rings are free
    tc_fence_after();
    if (uint32_t(set) != split) {
      // this set is finished by the counterpart CTA of the other pair: send (O, maximum, sum)
      const uint32_t peer = rank ^ 2u;
      const uint32_t stage_peer = cta_addr(smem_u32(stage), peer), ml_peer = cta_addr(smem_u32(ml_share), peer);
#pragma unroll
      for (int cc = 0; cc < 4; ++cc) {
        uint32_t orr[32];
        if (have) {
          TMEM_LD32_WAIT(o_addr + cc * 32, orr);
        } else {
#pragma unroll
          for (int i = 0; i < 32; ++i) orr[i] = 0u;
        }
#pragma unroll
        for (int i = 0; i < 8; ++i)       // [column quad][row][4]: consecutive rows, consecutive 16 bytes
          st_cluster_f32x4(stage_peer + uint32_t(((cc * 8 + i) * 128 + row) * 16), __uint_as_float(orr[4 * i]),
                           __uint_as_float(orr[4 * i + 1]), __uint_as_float(orr[4 * i + 2]), __uint_as_float(orr[4 * i + 3]));
      }
      st_cluster_f32x2(ml_peer + uint32_t(row * 8), have ? m_run : -INFINITY, have ? l_run : 0.f);
    }
    cluster_sync_all();       // 2: the partial results have landed in their counterparts' shared memory
    if (uint32_t(set) == split) {
      // finish this set: merge the counterpart's partial result with this CTA's own
      const float m_b = ml_share[row * 2], l_b = ml_share[row * 2 + 1];
      const float m_a = have ? m_run : -INFINITY, l_a = have ? l_run : 0.f;
      const float m_all = fmaxf(m_a, m_b);
      float w_a = m_a == -INFINITY ? 0.f : ex2(m_a - m_all), w_b = m_b == -INFINITY ? 0.f : ex2(m_b - m_all);
      const float lsum = l_a * w_a + l_b * w_b;
      const float inv = lsum > 0.f ? 1.f / lsum : 0.f;
      w_a *= inv; w_b *= inv;
      const int h = h0 + set;
      const size_t tok = size_t(unit) * nt + size_t(mt) * kBM + row;
      const float4* st4 = reinterpret_cast<const float4*>(stage);
#pragma unroll
      for (int cc = 0; cc < 4; ++cc) {
        uint32_t orr[32];
        if (have) {
          TMEM_LD32_WAIT(o_addr + cc * 32, orr);
        } else {
#pragma unroll
          for (int i = 0; i < 32; ++i) orr[i] = 0u;
        }
        float o[32];
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          const float4 b = st4[(cc * 8 + i) * 128 + row];
          o[4 * i + 0] = __uint_as_float(orr[4 * i + 0]) * w_a + b.x * w_b;
          o[4 * i + 1] = __uint_as_float(orr[4 * i + 1]) * w_a + b.y * w_b;
          o[4 * i + 2] = __uint_as_float(orr[4 * i + 2]) * w_a + b.z * w_b;
          o[4 * i + 3] = __uint_as_float(orr[4 * i + 3]) * w_a + b.w * w_b;
        }
        const int col = cc * 32;
        if (p.out_bf16) {
          __nv_bfloat16* ob = static_cast<__nv_bfloat16*>(p.a.out) + (tok * p.n_q_heads + h) * kD + col;
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            uint4 v;
            v.x = pack_bf16(o[8 * i + 0], o[8 * i + 1]);
            v.y = pack_bf16(o[8 * i + 2], o[8 * i + 3]);
            v.z = pack_bf16(o[8 * i + 4], o[8 * i + 5]);
            v.w = pack_bf16(o[8 * i + 6], o[8 * i + 7]);
            *reinterpret_cast<uint4*>(ob + 8 * i) = v;
          }
        } else {
          float* of = static_cast<float*>(p.a.out) + (tok * p.n_q_heads + h) * kD + col;
#pragma unroll
          for (int i = 0; i < 8; ++i)
            *reinterpret_cast<float4*>(of + 4 * i) = make_float4(o[4 * i], o[4 * i + 1], o[4 * i + 2], o[4 * i + 3]);
        }
      }
      if (p.a.lse)
        p.a.lse[(size_t(unit) * p.n_q_heads + h) * nt + size_t(mt) * kBM + row] =
            lsum > 0.f ? (m_all + log2f(lsum)) * 0.6931471805599453f : -INFINITY;
    }

  }

  // ---- teardown
  tc_fence_before();
  cluster_sync_all();       // 3: no CTA frees TMEM or leaves while its pair or its counterpart may still touch it
  if (tid == 0 && *abort_flag) set_status(p.a.status, ACTQKV_DEV_TIMEOUT);
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(512));
  }
}

}  // namespace

namespace actqkv {

bool attention_tc4_supported(const actqkv_config* cfg, int n_tokens) {
  const int group = cfg->n_q_heads / cfg->n_kv_heads;
  return attention_tc_supported(cfg, n_tokens) && group % 4 == 0;
}

int launch_attention_tc4(const actqkv_config* cfg, const Batch& b, const AttnArgs& a, cudaStream_t st) {
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
    const cuuint32_t box_k[3] = {64, 1, 32};                       // one channel half of 32 keys
    const cuuint32_t box_v[3] = {64, 1, cuuint32_t(kBN)};          // one channel half of 128 keys
    if (!encode(&tm_kw, a.k_win, 3, dims, str, box_k)) return ACTQKV_ERR_LAUNCH;
    if (!encode(&tm_vw, a.v_win, 3, dims, str, box_v)) return ACTQKV_ERR_LAUNCH;
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
  if (!opt_in_shared_memory(attention_tc4_kernel, int(kSmemBytes), opted_in)) return ACTQKV_ERR_LAUNCH;
  cudaLaunchConfig_t lc = {};
  lc.gridDim = dim3(Hq, nt / kBM, U);          // 4 consecutive CTAs in x = one cluster = one unit of 4 heads
  lc.blockDim = dim3(kThreads, 1, 1);
  lc.dynamicSmemBytes = kSmemBytes;
  lc.stream = st;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 4;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  allow_early_launch(attr[1]);
  lc.attrs = attr;
  lc.numAttrs = 2;
  if (cudaLaunchKernelEx(&lc, attention_tc4_kernel, tm_q, tm_kw, tm_vw, tm_kp, tm_vp, p) != cudaSuccess)
    return ACTQKV_ERR_LAUNCH;
  return launch_status();
}

}  // namespace actqkv
