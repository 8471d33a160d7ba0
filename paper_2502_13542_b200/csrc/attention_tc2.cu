// Step 5, tensor-core kernel for CTA pairs: the same attention as attention_tc.cu,
//   [initial tokens | selected blocks | local past | window tokens (causal)]     (Eq. 2)
// for bf16, D = 128, 16-token pages, with two CTAs (a cluster of 2, on two SMs) sharing every
// K / V tile.  The keys are visited in the order [initial | local past | window | selected]: all
// but the selected blocks are known before this step's selection exists, so the kernel is launched
// while the selection is still being computed (programmatic dependent launch), works through those
// tiles, and takes the dependency wait only where the selected blocks begin.
//
// The single-CTA kernel streams a whole 64 KiB K+V tile into every CTA for 128 query rows and is
// bound by that L2 -> shared-memory traffic.  Here the two CTAs of a pair hold the same 128 window
// tokens of two query heads of one KV group, and every product is one tcgen05.mma.cta_group::2
// of M = 256: each CTA supplies its own 128 rows of A (Q from shared memory, P from TMEM) and
// HALF of B -- 64 of the tile's 128 keys for S = Q K^T, 64 of the 128 channels of V for
// O += P V -- and receives its own 128 rows of the result in its TMEM.  A CTA therefore loads
// 32 KiB per tile instead of 64, and the rings hold 6 K halves and 5 V halves.  No TMA multicast
// is used: each CTA fetches its own halves.
//
// Roles per CTA (512 threads): warp 0 K producer, warp 2 V producer, warps 1 and 3 the MMA issuers
// (leader CTA = cluster rank 0 only; warp 1: S = Q K^T, warp 3: O += P V), warps 4-11 softmax: each
// owns 16 query rows (TMEM lanes) and reads all 128 key columns of their S rows with one 16x256b
// load, so a row's maximum and sum are finished by shuffles inside a quad of threads and no softmax
// warp waits for another one inside a tile; warps 12-15 V conversion and O correction.
//
// P is kept in fp16 (11 significant bits; one tcgen05.mma per 16 keys, half the tensor-pipe time of
// a bf16 high + low pair), so V must be fp16 too (kind::f16 wants both operands alike): warps 12-15
// convert each CTA's half of a V tile in place after it landed, two tiles ahead of its use.  The row
// sum adds the fp16-rounded P, so numerator and denominator carry the same rounding.  fp16 tops out
// at 65504, so the running maximum used for P may lag the true one by at most 2^8; when it has to
// move, O is rescaled by warps 12-15 between two P V products, off the softmax threads' path.
// Cross-CTA signalling:
//   K loads of both CTAs complete on the LEADER's "full" barriers (cta_group::2 form of the load);
//   V loads complete on the loading CTA's barrier; its converter warps then arrive on the leader's
//   "V ready" barrier;
//   the leader's commits are multicast to the barriers of both CTAs (slot released, S ready, P V done);
//   the softmax warps of both CTAs arrive on the leader's "P ready" barrier (one arrival per warp),
//   the correction warps on its "O corrected" barrier.
// TMEM columns (both CTAs alike): S/P buffers 0..2 at [0,128) [128,256) [256,384), O at [384,512).
// Every wait on an mbarrier is bounded; on expiry the CTA flags ACTQKV_DEV_TIMEOUT, stops issuing
// work and drains; both CTAs meet at a cluster barrier before they free their TMEM.
#include "tc_common.cuh"

using namespace actqkv;
using namespace actqkv::tc;

namespace {

constexpr int kBM = 128, kBN = 128, kD = 128;
constexpr int kRing = 6;                                 // K halves in flight
constexpr int kRingV = 5;                                // V halves in flight
// fp16 P: exp2(x - m) must stay below 65504, so the running maximum may lag by at most 2^8
constexpr float kRescaleF16 = 8.0f;
constexpr int kSoftmaxWarps = 8;                         // each owns 16 query rows (TMEM lanes) and all 128 key columns of a tile
constexpr int kSBuf = 3;                                 // S/P buffers in TMEM
constexpr int kPvRing = 4;                               // barriers that count completed P V products
constexpr int kThreads = 128 + kSoftmaxWarps * 32 + 128; // producers + MMA issuers, softmax warps, V converters / O correction
constexpr int kConvWarp0 = 4 + kSoftmaxWarps;            // first warp of the converter warpgroup
constexpr uint32_t kSubTileBytes = 128 * 128;            // [128 rows x 64 bf16], 16 KiB
constexpr uint32_t kTileBytes = 2 * kSubTileBytes;       // 32 KiB: the Q tile, or a whole K or V tile
constexpr uint32_t kHalfBytes = kTileBytes / 2;          // 16 KiB: what one CTA holds of a K or V tile
constexpr uint32_t kKSubBytes = 64 * 128;                // [64 keys x 64 channels] sub-tile of a K half
constexpr uint32_t kSmemTiles = kTileBytes + (kRing + kRingV) * kHalfBytes;
constexpr int kFRing = 4;                                // O correction factors in flight
constexpr int kNumBars = 1 + 2 * kRing + 3 * kRingV + 2 * kSBuf + kPvRing + 2 * kFRing + 2;
constexpr uint32_t kBarBytes = 448;                      // barriers, TMEM slot, abort flag
constexpr uint32_t kXchgBytes = (2 + kFRing) * 128 * 4;  // final row sums and maxima [row], O factors [ring][row]
constexpr uint32_t kSmemNeeded = kSmemTiles + kBarBytes + kXchgBytes;
constexpr uint32_t kSmemBytes = 227 * 1024;              // everything an SM offers one CTA
static_assert(8 * kNumBars + 16 <= kBarBytes, "barrier area too small");
static_assert(kSmemNeeded <= kSmemBytes, "shared memory budget");


// ---------------------------------------------------------------- pair-wide PTX wrappers
__device__ __forceinline__ uint32_t cluster_rank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
// Address of the leader CTA's copy of a shared-memory object, in the cluster window.
__device__ __forceinline__ uint32_t leader_addr(uint32_t local) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, 0;" : "=r"(r) : "r"(local));
  return r;
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_bar) {
  asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(cluster_bar) : "memory");
}
// TMA loads whose completion may be signalled on the peer CTA's barrier (`bar` in the cluster window).
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
// Arrives on the barrier at this offset in BOTH CTAs once every MMA issued so far has completed.
__device__ __forceinline__ void tc2_commit(uint32_t bar) {
  const uint16_t both = 3;
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
               ::"r"(bar), "h"(both) : "memory");
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

// ---------------------------------------------------------------- the paged key stream, in two parts
struct PairKeys {
  const int32_t* sel;
  const int32_t* pt;
  int g_init, g_a, g_b, gpb, n_cand, n_init, block, max_pages, n_phys_pages, page_base, page_oob;
  int gpp;                   // 16-token granules per cache page (1, 2, 4 or 8)
  int64_t local_page0;       // first granule of the local past, counted from token 0
};
// The key stream is addressed in granules of 16 tokens whatever the page size; a page of
// 16 * gpp tokens holds gpp consecutive granules, and every part of the stream starts on a page.
// Row of the 4-D tensor map of the page that holds granule lg (counted from token 0); page_oob
// (outside the tensor: TMA fills zeros) for rejected table entries.
__device__ __forceinline__ int physical_page(const PairKeys& ks, int64_t lg, int32_t* status, bool report) {
  const int64_t lp = lg / ks.gpp;
  const int phys = lp < ks.max_pages ? ks.pt[lp] : -1;
  if (phys < 0 || phys >= ks.n_phys_pages) {
    if (report) set_status(status, ACTQKV_DEV_BAD_PAGE);
    return ks.page_oob;
  }
  return ks.page_base + phys;
}
// Part A, 16-token granule gi: the initial tokens, then the local past up to p0.
__device__ __forceinline__ int page_a(const PairKeys& ks, int gi, int32_t* status, bool report) {
  if (gi >= ks.g_a) return ks.page_oob;
  return physical_page(ks, gi < ks.g_init ? int64_t(gi) : ks.local_page0 + (gi - ks.g_init), status, report);
}
// Part B, granule gi: the selected blocks in the order of sel_idx.
// (blk = the entry of sel_idx that granule gi falls into, read by the caller)
__device__ __forceinline__ int page_b_of_block(const PairKeys& ks, int gi, int blk, int32_t* status, bool report) {
  if (gi >= ks.g_b) return ks.page_oob;
  if (blk < 0 || blk >= ks.n_cand) {
    if (report) set_status(status, ACTQKV_DEV_BAD_SELECTION);
    return ks.page_oob;
  }
  return physical_page(ks, (int64_t(ks.n_init) + int64_t(blk) * ks.block) / 16 + gi % ks.gpb, status, report);
}
__device__ __forceinline__ int page_b(const PairKeys& ks, int gi, int32_t* status, bool report) {
  if (gi >= ks.g_b) return ks.page_oob;
  return page_b_of_block(ks, gi, ks.sel[gi / ks.gpb], status, report);
}

// ---------------------------------------------------------------- kernel
__global__ void __launch_bounds__(kThreads, 1)
attention_tc2_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_kw,
                    const __grid_constant__ CUtensorMap tm_vw, const __grid_constant__ CUtensorMap tm_kp,
                    const __grid_constant__ CUtensorMap tm_vp, TcParams p) {
  extern __shared__ unsigned char smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  const bool smem_short = base - raw + kSmemNeeded > kSmemBytes;   // never with a 1 KiB-aligned window
  const uint32_t q_smem = base;
  const uint32_t k_ring = base + kTileBytes;
  const uint32_t v_ring = k_ring + kRing * kHalfBytes;
  const uint32_t bars = base + kSmemTiles;
  // barrier slots (8 bytes each)
  const uint32_t bar_q = bars;
  auto bar_kfull = [&](int s) { return bars + 8u * (1 + s); };
  auto bar_kempty = [&](int s) { return bars + 8u * (1 + kRing + s); };
  auto bar_vfull = [&](int s) { return bars + 8u * (1 + 2 * kRing + s); };
  auto bar_vempty = [&](int s) { return bars + 8u * (1 + 2 * kRing + kRingV + s); };
  auto bar_sfull = [&](int b) { return bars + 8u * (1 + 2 * kRing + 2 * kRingV + b); };
  auto bar_pfull = [&](int b) { return bars + 8u * (1 + 2 * kRing + 2 * kRingV + kSBuf + b); };
  auto bar_pvdone = [&](int i) { return bars + 8u * (1 + 2 * kRing + 2 * kRingV + 2 * kSBuf + i); };
  auto bar_vready = [&](int s) { return bars + 8u * (1 + 2 * kRing + 2 * kRingV + 2 * kSBuf + kPvRing + s); };
  auto bar_f = [&](int i) { return bars + 8u * (1 + 2 * kRing + 3 * kRingV + 2 * kSBuf + kPvRing + i); };
  auto bar_corr = [&](int i) { return bars + 8u * (1 + 2 * kRing + 3 * kRingV + 2 * kSBuf + kPvRing + kFRing + i); };
  const uint32_t bar_done = bars + 8u * (kNumBars - 2);
  const uint32_t bar_sel = bars + 8u * (kNumBars - 1);      // the selection has arrived (this CTA's K producer)
  unsigned char* base_generic = smem_raw + (base - raw);
  unsigned char* bars_generic = base_generic + kSmemTiles;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars_generic + 8 * kNumBars);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(bars_generic + 8 * kNumBars + 8);
  float* l_share = reinterpret_cast<float*>(bars_generic + kBarBytes);   // [128] row sums, for the epilogue
  float* m_share = l_share + 128;                                        // [128] running maxima, for the log-sum-exp
  float* f_share = m_share + 128;                                        // [kFRing][128] O correction factors

  // the query tiles with the most keys (the last of the window) are launched first
  const int h = blockIdx.x, mt = int(gridDim.y) - 1 - int(blockIdx.y), unit = blockIdx.z;      // the pair = heads (h & ~1, h | 1)
  const uint32_t rank = cluster_rank();                               // 0 = leader
  const bool leader = rank == 0;
  const int g = h / p.group, seq = unit / p.n_layers, layer_local = unit - seq * p.n_layers;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int nt = p.a.n_tokens;

  // ---- set-up that depends on no earlier kernel: barriers, TMEM
  if (tid == 0) {
    mbar_init(bar_q, 1);
    for (int s = 0; s < kRing; ++s) { mbar_init(bar_kfull(s), 1); mbar_init(bar_kempty(s), 1); }
    for (int s = 0; s < kRingV; ++s) { mbar_init(bar_vfull(s), 1); mbar_init(bar_vempty(s), 1); mbar_init(bar_vready(s), 8); }
    for (int b = 0; b < kSBuf; ++b) { mbar_init(bar_sfull(b), 1); mbar_init(bar_pfull(b), 2 * kSoftmaxWarps); }
    for (int i = 0; i < kPvRing; ++i) mbar_init(bar_pvdone(i), 1);
    for (int i = 0; i < kFRing; ++i) { mbar_init(bar_f(i), kSoftmaxWarps); mbar_init(bar_corr(i), 8); }
    mbar_init(bar_done, 1);
    mbar_init(bar_sel, 1);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(512));
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;");
  }
  tc_fence_before();
  cluster_sync_all();         // both CTAs' barriers are initialised and both hold their TMEM
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  // ---- the key stream in two parts.  Part A needs nothing of this step's selection: the initial
  // tokens and the local past (one run of 16-token pages, a ragged last tile masked), then the
  // window's own tiles (causal on the last).  Part B, the selected blocks, follows the dependency
  // wait.  The softmax is running, so the order of the tiles changes the rounding only.  The kernel
  // launched just before this one may still be running while part A is worked on (programmatic
  // dependent launch): every kernel of the library waits for its own predecessor before it writes,
  // and none of those that let their successor start early writes the position, the page table,
  // the cache pages of past tokens or the step's own Q / K / V.  Only sel_idx / sel_count must wait.
  const Geometry geo = make_geometry(p.a.pos0[seq], p.n_init, p.block, p.n_local_prev);
  const int64_t local_len = geo.p0 - geo.local_start;
  PairKeys ks;
  ks.sel = p.a.sel_idx + (size_t(unit) * p.n_kv_heads + g) * p.cap_blocks;
  ks.pt = p.a.page_table + size_t(seq) * p.max_pages;
  ks.gpb = p.block / 16;                                 // granules per block
  ks.gpp = p.page_tokens / 16;
  ks.g_init = geo.init_len / 16;
  ks.g_a = ks.g_init + int((local_len + 15) / 16);       // the last local page may be partly filled
  ks.g_b = 0;
  ks.local_page0 = geo.local_start / 16;
  ks.n_cand = geo.n_cand; ks.n_init = p.n_init; ks.block = p.block; ks.max_pages = p.max_pages;
  ks.n_phys_pages = p.n_phys_pages; ks.page_base = layer_local * p.n_phys_pages;
  ks.page_oob = p.n_layers * p.n_phys_pages;             // beyond the tensor: zero fill
  const int n_a = geo.init_len + int(local_len);         // exact: the tail of the last page is masked
  const int tiles_a = (n_a + kBN - 1) / kBN;
  const int n1 = tiles_a + mt + 1;                       // tiles before the dependency wait
  int n_b = 0;                                           // keys of the selected blocks, known after the wait
  // Every thread that needs the total takes the wait itself (it is the launch dependency, so it
  // always ends) and reads the count: no role then waits on another one for it.
  auto total_after_wait = [&](bool report) -> int {
    grid_dependency_wait();            // the selection is complete from here on
    int c = p.a.sel_count ? p.a.sel_count[unit] : 0;
    if (c < 0 || c > p.cap_blocks || c > geo.n_cand) {
      if (report) set_status(p.a.status, ACTQKV_DEV_BAD_SELECTION);
      c = max(0, min(c, min(p.cap_blocks, geo.n_cand)));
    }
    n_b = c * p.block;
    ks.g_b = c * ks.gpb;
    return n1 + (n_b + kBN - 1) / kBN;
  };

  if (smem_short) {           // uniform over the pair: nothing was issued yet
    if (tid == 0) set_status(p.a.status, ACTQKV_DEV_BAD_SELECTION);
    cluster_sync_all();
    if (warp == 1) asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(512));
    return;
  }

  if (warp == 0 || warp == 2) {
    // =========================== TMA producers: warp 0 -> K half (and Q), warp 2 -> V half ===========================
    // This CTA's half of a tile: keys [64 * rank, +64) of K (all channels), channels [64 * rank, +64)
    // of V (all keys).  K copies complete on the leader's barriers (the leader posts the byte count
    // of both halves), a V half on its own CTA's barrier, where that CTA's converter warps pick it up.
    const bool is_v = warp == 2;
    const uint32_t ring = is_v ? v_ring : k_ring;
    const CUtensorMap* tm_pages = is_v ? &tm_vp : &tm_kp;
    const CUtensorMap* tm_win = is_v ? &tm_vw : &tm_kw;
    const int ring_n = is_v ? kRingV : kRing;
    if (!is_v && lane == 0) {
      if (leader) mbar_expect_tx(bar_q, 2 * kTileBytes);
      tma2_load_3d(q_smem, &tm_q, leader_addr(bar_q), 0, h, unit * nt + mt * kBM);
      tma2_load_3d(q_smem + kSubTileBytes, &tm_q, leader_addr(bar_q), 64, h, unit * nt + mt * kBM);
    }
    // One box per page (or per part of a page that belongs to this CTA's share of the tile) and,
    // for K, per 64-channel half: with 16-token pages lanes 0-7 issue one box of 16 rows each
    // (K: channel half, granule 4 * rank + slot; V: granule = lane), with larger pages fewer lanes
    // issue taller boxes.  A box costs the copy engine about the same whatever its height.
    const int box_g = min(ks.gpp, is_v ? 8 : 4);           // granules per box
    const int n_box = is_v ? 8 / box_g : 2 * (4 / box_g);  // boxes of this CTA per tile
    const int per_half = is_v ? n_box : n_box / 2;
    const int half = lane / per_half, slot = lane % per_half;
    const int my_granule = (is_v ? 0 : int(rank) * 4) + slot * box_g;          // first granule of the box, in the tile
    const int tok_in_page = (my_granule % ks.gpp) * 16;
    const uint32_t box_off = (is_v ? 0u : uint32_t(half) * kKSubBytes) + uint32_t(slot * box_g) * 2048u;
    const bool report = !is_v && leader;
    bool ok = true;
    int issued = 0;
    // waits for the ring slot of tile j and posts the bytes to come; returns the slot's base address
    auto claim = [&](int j, uint32_t& full) -> uint32_t {
      const int s = j % ring_n, it = j / ring_n;
      if (it > 0) ok = mbar_wait(is_v ? bar_vempty(s) : bar_kempty(s), (it - 1) & 1, abort_flag);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) return 0;
      const uint32_t full_local = is_v ? bar_vfull(s) : bar_kfull(s);
      full = is_v ? full_local : leader_addr(full_local);
      if (lane == 0) {
        if (is_v) mbar_expect_tx(full_local, kHalfBytes);
        else if (leader) mbar_expect_tx(full_local, kTileBytes);
      }
      __syncwarp();
      return ring + s * kHalfBytes;
    };
    // `cnt` tiles of cache pages from tile j_base on.  Page look-ups (for part B sel_idx ->
    // page_table, two dependent loads) are taken 32 granules = 4 tiles at a time, one granule per
    // lane, one chunk ahead of the tiles being issued, so that their latency is off the per-tile
    // path; the issuing lane fetches its page with a shuffle.
    auto paged_tiles = [&](int j_base, int cnt, auto&& page_of, int first_chunk) {
      int page_cur = 0, page_next = first_chunk;
      for (int t = 0; t < cnt && ok; ++t) {
        if ((t & 3) == 0) page_cur = page_next;
        const int page = __shfl_sync(0xffffffffu, page_cur, (t & 3) * 8 + my_granule);
        uint32_t full = 0;
        const uint32_t sbase = claim(j_base + t, full);
        if (!ok) break;
        if (lane < n_box) {
          if (is_v) tma_load_4d(sbase + box_off, tm_pages, full, int(rank) * 64, tok_in_page, g, page);
          else tma2_load_4d(sbase + box_off, tm_pages, full, half * 64, tok_in_page, g, page);
        }
        issued = j_base + t + 1;
        // the next chunk of look-ups after the issue: its stall is behind the ring
        if ((t & 3) == 0) page_next = page_of(((t >> 2) + 1) * 32 + lane);
      }
    };
    paged_tiles(0, tiles_a, [&](int gi) { return page_a(ks, gi, p.a.status, report); }, page_a(ks, lane, p.a.status, report));
    for (int w = 0; w <= mt && ok; ++w) {
      uint32_t full = 0;
      const uint32_t sbase = claim(tiles_a + w, full);
      if (!ok) break;
      const int row0 = unit * nt + w * kBN;
      if (is_v) {
        if (lane == 0) tma_load_3d(sbase, tm_win, full, int(rank) * 64, g, row0);
      } else if (lane < 2) {
        tma2_load_3d(sbase + lane * kKSubBytes, tm_win, full, lane * 64, g, row0 + int(rank) * 64);
      }
      issued = tiles_a + w + 1;
    }
    if (ok) {
      // the page-table entries of every candidate block start their way into L2 while this warp
      // sits in the wait: the look-ups of the selected blocks that follow it then find them there
      if (!is_v) {
        const char* pt0 = reinterpret_cast<const char*>(ks.pt + p.n_init / p.page_tokens);
        const int lines = min(ks.max_pages - p.n_init / p.page_tokens, ks.n_cand * ks.gpb / ks.gpp) / 32;     // 32 entries per 128 bytes
        for (int l = lane; l < lines; l += 32)
          asm volatile("prefetch.global.L2 [%0];" ::"l"(pt0 + size_t(l) * 128));
      }
      // the first look-up into the selection goes out together with the load of the count
      grid_dependency_wait();
      const int e0 = lane / ks.gpb;
      const int blk0 = e0 < p.cap_blocks ? ks.sel[e0] : -1;
      const int n_tiles = total_after_wait(report && lane == 0);
      if (!is_v && lane == 0) mbar_arrive(bar_sel);      // the converter warps poll this instead of blocking
      paged_tiles(n1, n_tiles - n1, [&](int gi) { return page_b(ks, gi, p.a.status, report); },
                  page_b_of_block(ks, lane, blk0, p.a.status, report));
    }
    // drain: what this CTA issued must have landed before it may leave on the abort path; its
    // copies complete on the leader's barriers, which only the leader can poll, so the peer waits
    // out the worst-case copy time instead
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
    // =========================== MMA issuers (leader CTA): warp 1 -> S = Q K^T, warp 3 -> O += P V ===========================
    // Two issuing threads, so that a wait of one product (a late K tile; P not yet published) does
    // not stop the issue of the other: a thread that issues tcgen05.mma is held back to the pipe's
    // pace, and whatever it waits for in between leaves the pipe idle.  Products of different
    // threads are not ordered by the pipe, so the reuse of an S/P buffer is ordered explicitly:
    // QK(j) waits until PV(j - kSBuf), which read that buffer, has completed.
    if (lane == 0 && leader) {
      constexpr uint32_t kHi = desc_hi(1024u);       // descriptor high words are constants
      bool ok = true;
      if (warp == 1) {
        constexpr uint32_t idesc_qk = make_idesc(false, 2 * kBM, kBN);
        const uint32_t q_lo = desc_lo(q_smem, 16u);
        ok = mbar_wait(bar_q, 0, abort_flag);
        int n_tiles = n1;
        for (int j = 0; ok; ++j) {
          if (j == n1) n_tiles = total_after_wait(false);
          if (j >= n_tiles) break;
          const int s = j % kRing;
          if (j >= kSBuf) ok = mbar_wait(bar_pvdone((j - kSBuf) % kPvRing), ((j - kSBuf) / kPvRing) & 1, abort_flag);
          ok = ok && mbar_wait(bar_kfull(s), (j / kRing) & 1, abort_flag);
          if (!ok) break;
          tc_fence_after();
          const uint32_t k_lo = desc_lo(k_ring + s * kHalfBytes, 16u);
          const uint32_t s_tmem = tmem + (j % kSBuf) * 128;
          // A: this CTA's 128 query rows; B: this CTA's 64 keys; both advance 16 channels per step
          mma2_ss<false>(s_tmem, q_lo, k_lo, kHi, idesc_qk);
#pragma unroll
          for (int k = 1; k < kD / 16; ++k) {
            constexpr uint32_t kUnit = 16;     // descriptor addresses count 16-byte units
            const uint32_t a_off = ((k >> 2) * kSubTileBytes + (k & 3) * 32u) / kUnit;
            const uint32_t b_off = ((k >> 2) * kKSubBytes + (k & 3) * 32u) / kUnit;
            mma2_ss<true>(s_tmem, q_lo + a_off, k_lo + b_off, kHi, idesc_qk);
          }
          tc2_commit(bar_kempty(s));
          tc2_commit(bar_sfull(j % kSBuf));
        }
      } else {
        constexpr uint32_t idesc_pv = make_idesc_f16(true, 2 * kBM, kBN);
        const uint32_t tmem_o = tmem + kSBuf * 128;
        int n_tiles = n1;
        for (int i = 0; ok; ++i) {
          if (i == n1) n_tiles = total_after_wait(false);
          if (i >= n_tiles) break;
          const int s = i % kRingV, b = i % kSBuf;
          // P(i) published by every softmax warp of both CTAs, which also turned V(i) into fp16
          ok = mbar_wait(bar_vready(s), (i / kRingV) & 1, abort_flag);          // V(i) is fp16 in both CTAs
          ok = ok && mbar_wait(bar_corr(i % kFRing), (i / kFRing) & 1, abort_flag);   // O is on P(i)'s maximum in both CTAs
          ok = ok && mbar_wait(bar_pfull(b), (i / kSBuf) & 1, abort_flag);      // P(i) published by both CTAs
          if (!ok) break;
          tc_fence_after();
          const uint32_t v_lo = desc_lo(v_ring + s * kHalfBytes, kSubTileBytes);
          const uint32_t p_tmem = tmem + b * 128;
#pragma unroll
          for (int k = 0; k < kBN / 16; ++k) {
            // 16 keys per step: B advances 16 rows of 128 bytes, A 8 packed fp16 columns
            const uint32_t b_lo = v_lo + k * (2048u / 16u);
            const uint32_t pa = p_tmem + k * 8;
            mma2_ts(tmem_o, pa, b_lo, kHi, idesc_pv, (i > 0 || k > 0) ? 1u : 0u);
          }
          tc2_commit(bar_vempty(s));
          tc2_commit(bar_pvdone(i % kPvRing));
        }
        if (ok) tc2_commit(bar_done);      // the last P V depends, through the softmax, on every Q K^T
      }
    }
    __syncwarp();
  } else if (warp >= kConvWarp0) {
    // =========================== V converters ===========================
    // This CTA's half of every V tile, as it landed (bf16), becomes fp16 in place, 128 bytes per
    // thread; one arrival per warp on the leader's "V ready" barrier.
    const int ct = tid - kConvWarp0 * 32;
    const int q4 = warp & 3;                              // TMEM lane quadrant of this warp
    const uint32_t o_row = tmem + (uint32_t(q4 * 32) << 16) + kSBuf * 128;
    constexpr int kLag = 2;                               // V is converted this many tiles ahead of the correction
    bool ok = true;
    // ci: next tile to convert, ri: next tile whose O correction is due.  Conversions lead by kLag.
    // Where part A ends the total is not known yet: the K producer signals the arrival of the
    // selection, and these warps only poll that signal while corrections of part A are still due
    // (a blocking wait here would hold back the last products of part A).
    int ci = 0, ri = 0, known = n1;
    bool final = false;
    while (ok) {
      if (!final && ci >= known) {
        bool ready = ri >= known || mbar_test_wait(bar_sel, 0);
        ready = __shfl_sync(0xffffffffu, ready, 0);
        if (ready) {
          known = total_after_wait(false);
          final = true;
        }
      }
      if (ri >= known) break;                             // only once the total is final
      if (ci < known && ci <= ri + kLag) {
        const int vs = ci % kRingV;
        ok = mbar_wait(bar_vfull(vs), (ci / kRingV) & 1, abort_flag);
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
        ++ci;
      } else {
        const int j = ri;
        // The running maximum of tile j is known: where it grew, O (on the old maximum) is scaled
        // down before P(j) V(j) is added.  The softmax threads do not wait for this.
        ok = mbar_wait(bar_f(j % kFRing), (j / kFRing) & 1, abort_flag);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        const float f = f_share[(j % kFRing) * 128 + ct];
        if (__any_sync(0xffffffffu, f != 1.f)) {          // never for tile 0
          // O must be quiescent: P V of every earlier tile complete
          ok = mbar_wait(bar_pvdone((j - 1) % kPvRing), ((j - 1) / kPvRing) & 1, abort_flag);
          ok = __all_sync(0xffffffffu, ok);
          if (!ok) break;
          tc_fence_after();
#pragma unroll
          for (int cc = 0; cc < 4; ++cc) {
            uint32_t orr[32];
            TMEM_LD32_WAIT(o_row + cc * 32, orr);
#pragma unroll
            for (int i = 0; i < 32; ++i) orr[i] = __float_as_uint(__uint_as_float(orr[i]) * f);
            TMEM_ST32(o_row + cc * 32, orr);
          }
          tmem_wait_st();
          tc_fence_before();
        }
        __syncwarp();
        if (lane == 0) mbar_arrive_cluster(leader_addr(bar_corr(j % kFRing)));
        ++ri;
      }
    }
  } else if (warp >= 4) {
    // =========================== softmax / epilogue ===========================
    // A warp owns 16 query rows (TMEM lanes) and reads all 128 key columns of their S rows with ONE
    // 16x256b load: the four threads of a quad share two rows (lane g and g + 8; thread q of the
    // quad holds columns 8k + 2q, 8k + 2q + 1 of both, k = 0..15).  A row's maximum and sum are
    // finished by two shuffles inside the quad, so no warp ever waits for another one inside a
    // tile, and the eight softmax warps drift apart: while one is bound by the special-function
    // unit (exponentials) another reads TMEM and takes maxima.  The packed fp16 pair of columns
    // (8k + 2q, +1) is P column 4k + q: exactly the register layout of the 16x128b store.
    const int sw = warp - 4;
    const int q4 = sw & 3, hw = sw >> 2;                  // TMEM lane quadrant (= warp % 4); lower / upper 16 lanes
    const int qd = lane & 3, g8 = lane >> 2;
    const int row0 = q4 * 32 + hw * 16 + g8, row1 = row0 + 8;      // this thread's two query rows inside the tile
    const uint32_t lane16 = uint32_t(q4 * 32 + hw * 16) << 16;
    float m0 = -INFINITY, m1 = -INFINITY, l0 = 0.f, l1 = 0.f;     // running maxima (log2 units) and partial row sums
    bool ok = true;
    int n_tiles = n1;
    for (int j = 0;; ++j) {
      if (j == n1) n_tiles = total_after_wait(false);
      if (j >= n_tiles) break;
      const int sb = j % kSBuf;
      ok = mbar_wait(bar_sfull(sb), (j / kSBuf) & 1, abort_flag);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tc_fence_after();
      const uint32_t s_addr = tmem + lane16 + sb * 128;
      uint64_t sv[32];                                    // sv[2k] row0, sv[2k + 1] row1
      TMEM_LD16X256P_WAIT(s_addr, sv);
      // key-validity limits: ragged last past tile, or the causal diagonal of the last tile
      int lim0 = kBN, lim1 = kBN;
      if (j < tiles_a) lim0 = lim1 = min(kBN, n_a - j * kBN);
      else if (j == n1 - 1) { lim0 = row0 + 1; lim1 = row1 + 1; }
      else if (j >= n1) lim0 = lim1 = min(kBN, n_b - (j - n1) * kBN);
      const bool masked = j == n1 - 1 || lim0 < kBN;      // CTA-uniform
      float mx0 = -INFINITY, mx1 = -INFINITY;
      if (masked) {
#pragma unroll
        for (int k = 0; k < 16; ++k) {
          const int col = 8 * k + 2 * qd;
          const float a0 = col < lim0 ? lo2(sv[2 * k]) : -INFINITY, a1 = col + 1 < lim0 ? hi2(sv[2 * k]) : -INFINITY;
          const float b0 = col < lim1 ? lo2(sv[2 * k + 1]) : -INFINITY, b1 = col + 1 < lim1 ? hi2(sv[2 * k + 1]) : -INFINITY;
          sv[2 * k] = pack2(a0, a1);
          sv[2 * k + 1] = pack2(b0, b1);
          mx0 = max3(mx0, a0, a1);
          mx1 = max3(mx1, b0, b1);
        }
      } else {
        float mx0b = -INFINITY, mx1b = -INFINITY;         // two chains per row
#pragma unroll
        for (int k = 0; k < 16; k += 2) {
          mx0 = max3(mx0, lo2(sv[2 * k]), hi2(sv[2 * k]));
          mx1 = max3(mx1, lo2(sv[2 * k + 1]), hi2(sv[2 * k + 1]));
          mx0b = max3(mx0b, lo2(sv[2 * k + 2]), hi2(sv[2 * k + 2]));
          mx1b = max3(mx1b, lo2(sv[2 * k + 3]), hi2(sv[2 * k + 3]));
        }
        mx0 = fmaxf(mx0, mx0b);
        mx1 = fmaxf(mx1, mx1b);
      }
      // the rows' maxima over the quad
      mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 1));
      mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 1));
      mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 2));
      mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 2));
      const float n0 = fmaxf(m0, mx0 * p.scale_log2), n1 = fmaxf(m1, mx1 * p.scale_log2);
      const bool grow0 = n0 - m0 > kRescaleF16, grow1 = n1 - m1 > kRescaleF16;   // also true for the first tile
      // Where the maximum grew, O has to be scaled by f before P(j) V(j) is added: the correction
      // warps do that, off this thread's path; tile 0 starts O, so its factor is 1.
      const float f0 = grow0 ? ex2(m0 - n0) : 1.f, f1 = grow1 ? ex2(m1 - n1) : 1.f;   // 0 for the first tile (l = 0)
      if (qd == 0) {
        f_share[(j % kFRing) * 128 + row0] = j > 0 ? f0 : 1.f;
        f_share[(j % kFRing) * 128 + row1] = j > 0 ? f1 : 1.f;
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(bar_f(j % kFRing));
      if (grow0) { m0 = n0; l0 *= f0; }
      if (grow1) { m1 = n1; l1 *= f1; }
      // P = exp2(x - m) in fp16 (11 significant bits): with outlier value channels |v| ~ 40 a bf16
      // P (8 bits) would cost up to |v| * 2^-9 = 0.08 of absolute error, fp16 at most |v| * 2^-12.
      // The row sum adds the values as rounded to fp16, the ones P V multiplies.  P overwrites the
      // first 64 columns of these rows of S, all of which this warp already holds.
      const uint64_t scale2 = pack2(p.scale_log2, p.scale_log2);
      const uint64_t negm0 = pack2(-m0, -m0), negm1 = pack2(-m1, -m1);
      float s0a = 0.f, s0b = 0.f, s1a = 0.f, s1b = 0.f;
#pragma unroll
      for (int hh = 0; hh < 2; ++hh) {
        uint32_t pk[16];
#pragma unroll
        for (int kk = 0; kk < 8; ++kk) {
          const int k = 8 * hh + kk;
          const uint64_t x0 = fma2(sv[2 * k], scale2, negm0), x1 = fma2(sv[2 * k + 1], scale2, negm1);
          pk[2 * kk] = pack_f16(ex2(lo2(x0)), ex2(hi2(x0)));
          pk[2 * kk + 1] = pack_f16(ex2(lo2(x1)), ex2(hi2(x1)));
          add_f16x2(s0a, s0b, pk[2 * kk]);
          add_f16x2(s1a, s1b, pk[2 * kk + 1]);
        }
        TMEM_ST16X128_X8(s_addr + hh * 32, pk);
      }
      l0 += s0a + s0b;
      l1 += s1a + s1b;
      tmem_wait_st();
      tc_fence_before();
      __syncwarp();                                       // one arrival per warp: 16 of both CTAs' warps in all
      if (lane == 0) mbar_arrive_cluster(leader_addr(bar_pfull(sb)));
    }
    // ---- epilogue: the rows' sums over the quad, handed over in shared memory; then thread = row,
    // warp hw takes channels [64 hw, 64 hw + 64) of O / l
    l0 += __shfl_xor_sync(0xffffffffu, l0, 1);
    l1 += __shfl_xor_sync(0xffffffffu, l1, 1);
    l0 += __shfl_xor_sync(0xffffffffu, l0, 2);
    l1 += __shfl_xor_sync(0xffffffffu, l1, 2);
    if (qd == 0) {
      l_share[row0] = l0; l_share[row1] = l1;
      m_share[row0] = m0; m_share[row1] = m1;
    }
    ok = ok && mbar_wait(bar_done, 0, abort_flag);
    ok = pair_sync_and(q4, ok);                           // the two warps of a lane quadrant
    if (ok) {
      tc_fence_after();
      const int row = q4 * 32 + lane;
      const float lsum = l_share[row];
      const float inv = lsum > 0.f ? 1.f / lsum : 0.f;
      const size_t tok = size_t(unit) * nt + size_t(mt) * kBM + row;
      const uint32_t o_row = tmem + (uint32_t(q4 * 32) << 16) + kSBuf * 128;
#pragma unroll
      for (int cc = 0; cc < 2; ++cc) {
        const int col = hw * 64 + cc * 32;
        uint32_t orr[32];
        TMEM_LD32_WAIT(o_row + col, orr);
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
      if (p.a.lse && hw == 0)
        p.a.lse[(size_t(unit) * p.n_q_heads + h) * nt + size_t(mt) * kBM + row] =
            (m_share[row] + log2f(lsum)) * 0.6931471805599453f;
    }
  }

  // ---- teardown
  tc_fence_before();
  cluster_sync_all();       // neither CTA frees TMEM or leaves while the pair's MMAs or signals may touch it
  if (tid == 0 && *abort_flag) set_status(p.a.status, ACTQKV_DEV_TIMEOUT);
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(512));
  }
}

}  // namespace

namespace actqkv {

bool attention_tc2_supported(const actqkv_config* cfg, int n_tokens) {
  const int group = cfg->n_q_heads / cfg->n_kv_heads, P = cfg->page_tokens;
  const bool page_ok = P == 16 || P == 32 || P == 64 || P == 128;
  return cfg->dtype == ACTQKV_BF16 && cfg->head_dim == 128 && page_ok && n_tokens % kBM == 0 && cfg->block % P == 0 &&
         cfg->n_init % P == 0 && cfg->n_local_prev % 16 == 0 && group % 2 == 0;
}

int launch_attention_tc2(const actqkv_config* cfg, const Batch& b, const AttnArgs& a, cudaStream_t st) {
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
    const cuuint32_t box_k[3] = {64, 1, 64};                       // one channel half of 64 keys
    const cuuint32_t box_v[3] = {64, 1, cuuint32_t(kBN)};          // one channel half of 128 keys
    if (!encode(&tm_kw, a.k_win, 3, dims, str, box_k)) return ACTQKV_ERR_LAUNCH;
    if (!encode(&tm_vw, a.v_win, 3, dims, str, box_v)) return ACTQKV_ERR_LAUNCH;
  }
  {
    const cuuint64_t P = cuuint64_t(cfg->page_tokens);
    const cuuint64_t dims[4] = {cuuint64_t(kD), P, cuuint64_t(Hkv), cuuint64_t(b.n_layers) * cfg->n_phys_pages};
    const cuuint64_t str[3] = {cuuint64_t(kD) * 2, cuuint64_t(kD) * 2 * P, cuuint64_t(kD) * 2 * P * Hkv};
    // a CTA holds 64 keys of a K tile and all 128 keys of its channel half of a V tile: a box is a
    // whole page, or the part of a larger page that falls into that share
    const cuuint32_t box_k[4] = {64, cuuint32_t(std::min(cfg->page_tokens, 64)), 1, 1};
    const cuuint32_t box_v[4] = {64, cuuint32_t(std::min(cfg->page_tokens, 128)), 1, 1};
    if (!encode(&tm_kp, a.k_pages, 4, dims, str, box_k)) return ACTQKV_ERR_LAUNCH;
    if (!encode(&tm_vp, a.v_pages, 4, dims, str, box_v)) return ACTQKV_ERR_LAUNCH;
  }
  TcParams p;
  p.a = a;
  p.n_q_heads = Hq; p.n_kv_heads = Hkv; p.group = Hq / Hkv; p.block = cfg->block; p.n_init = cfg->n_init;
  p.n_local_prev = cfg->n_local_prev; p.cap_blocks = cfg->cap_blocks; p.max_pages = cfg->max_pages;
  p.n_phys_pages = cfg->n_phys_pages; p.n_layers = b.n_layers; p.out_bf16 = cfg->out_dtype == ACTQKV_BF16;
  p.page_tokens = cfg->page_tokens;
  const float scale = cfg->sm_scale > 0.f ? cfg->sm_scale : 1.f / sqrtf(float(kD));
  p.scale_log2 = scale * 1.4426950408889634f;
  static std::atomic<bool> opted_in[kMaxDevices];
  if (!opt_in_shared_memory(attention_tc2_kernel, int(kSmemBytes), opted_in)) return ACTQKV_ERR_LAUNCH;
  cudaLaunchConfig_t lc = {};
  lc.gridDim = dim3(Hq, nt / kBM, U);
  lc.blockDim = dim3(kThreads, 1, 1);
  lc.dynamicSmemBytes = kSmemBytes;
  lc.stream = st;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  allow_early_launch(attr[1]);
  lc.attrs = attr;
  lc.numAttrs = 2;
  if (cudaLaunchKernelEx(&lc, attention_tc2_kernel, tm_q, tm_kw, tm_vw, tm_kp, tm_vp, p) != cudaSuccess)
    return ACTQKV_ERR_LAUNCH;
  return launch_status();
}

}  // namespace actqkv
