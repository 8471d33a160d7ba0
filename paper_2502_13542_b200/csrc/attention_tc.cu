// Step 5, tensor-core kernel: attention of one window over
//   [initial tokens | selected blocks | local past | window tokens (causal)]     (Eq. 2)
// for bf16, D = 128, 16-token pages, on the 5th-generation tensor cores.
//
// One CTA = one 128-row query tile (128 consecutive window tokens of one query head).
// Key tiles of 128 keys are gathered page by page: each 16-token page is one TMA box of
// 16 rows x 128 bytes per 64-channel half, written with the 128-byte swizzle the MMA
// descriptors expect, so a [128 x 64] operand sub-tile is 8 boxes stacked in shared memory.
// The block -> page indirection (sel_idx, page_table) is resolved by the producer warp, one
// lane per box.  The window's own keys / values come from k_win / v_win with one box per half.
//
// Three warpgroups:
//   warp 0        TMA producer (3-stage ring of K+V tiles)
//   warp 1        tcgen05.mma issuer (one lane), owns the TMEM allocation
//   warps 4-7     softmax of the even key tiles, accumulator O0
//   warps 8-11    softmax of the odd key tiles, accumulator O1
// Each softmax thread owns one query row (= TMEM lane): running max / sum in base 2, P written
// back over the S columns as two bf16 terms (hi + lo), its O rescaled in TMEM only when the
// row's max grew by more than 2^8 (lazy rescale).  The two warpgroups keep independent
// (max, sum, O) triples, so the tensor pipe works on one tile's P V while the other tile's
// softmax runs; the epilogue merges the two partial results per row.
//
// TMEM columns: S0/P0 [0,128)  S1/P1 [128,256)  O0 [256,384)  O1 [384,512).
// S = Q K^T uses both operands from shared memory (K-major, SW128); O += P V takes P from
// TMEM and V from shared memory as an MN-major operand (the V tile is [keys x channels]).
// P of keys [32c, 32c+32) of a tile lives in columns [32c, 32c+16) (hi) and [32c+16, 32c+32) (lo).
// Every wait on an mbarrier is bounded; on expiry the CTA flags ACTQKV_DEV_TIMEOUT, stops
// issuing work, drains and frees its TMEM.
#include <cuda.h>

#include "common.cuh"
#include "stages.cuh"

using namespace actqkv;

namespace {

constexpr int kBM = 128, kBN = 128, kD = 128;
constexpr int kStages = 3;
constexpr int kThreads = 384;                           // 3 warpgroups
constexpr uint32_t kSubTileBytes = 128 * 128;            // [128 rows x 64 bf16], 16 KiB
constexpr uint32_t kTileBytes = 2 * kSubTileBytes;       // 32 KiB: one K or V or Q tile
constexpr uint32_t kStageBytes = 2 * kTileBytes;         // K + V
constexpr uint32_t kSmemData = kTileBytes + kStages * kStageBytes;
constexpr uint32_t kSmemBytes = kSmemData + 1024 /*align*/ + 256 /*barriers*/;
constexpr uint32_t kSpinLimit = 1u << 24;
constexpr float kRescaleThreshold = 8.0f;                // log2 units

struct TcParams {
  AttnArgs a;
  int n_q_heads, n_kv_heads, group, block, n_init, n_local_prev, cap_blocks;
  int max_pages, n_phys_pages, n_layers, out_bf16;
  float scale_log2;
};

// ---------------------------------------------------------------- PTX wrappers
__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.b32 %0, 1, 0, p;\n\t}"
      : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok != 0;
}
// Bounded wait.  Returns false when the limit expired or another role already gave up.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
  for (uint32_t i = 0; i < kSpinLimit; ++i) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((i & 1023u) == 1023u && *abort_flag) return false;
  }
  *abort_flag = 1;
  return false;
}
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* tm, uint32_t bar, int c0, int c1, int c2) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
      ::"r"(dst), "l"(tm), "r"(bar), "r"(c0), "r"(c1), "r"(c2) : "memory");
}
__device__ __forceinline__ void tma_load_4d(uint32_t dst, const CUtensorMap* tm, uint32_t bar, int c0, int c1, int c2,
                                            int c3) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
      ::"r"(dst), "l"(tm), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// D[tmem] (+)= A[smem] * B[smem]
__device__ __forceinline__ void mma_ss(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t acc) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(acc) : "memory");
}
// D[tmem] (+)= A[tmem] * B[smem]
__device__ __forceinline__ void mma_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc, uint32_t acc) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
      ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(acc) : "memory");
}
#define TMEM_LD32(taddr, r)                                                                      \
  asm volatile(                                                                                  \
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,"  \
      "%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"         \
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]),      \
        "=r"(r[7]), "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]),  \
        "=r"(r[14]), "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]),            \
        "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]),            \
        "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])             \
      : "r"(taddr))
// Four 32-column loads and the wait in ONE asm statement: no consumer of the registers can be
// scheduled ahead of tcgen05.wait::ld.
#define TMEM_LD128_WAIT(taddr, r)                                                              \
  asm volatile(                                                                                \
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%128];\n\t"                            \
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%32,%33,%34,%35,%36,%37,%38,%39,%40,%41,%42,%43,%44,%45,%46,%47,%48,%49,%50,%51,%52,%53,%54,%55,%56,%57,%58,%59,%60,%61,%62,%63}, [%129];\n\t"                            \
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%64,%65,%66,%67,%68,%69,%70,%71,%72,%73,%74,%75,%76,%77,%78,%79,%80,%81,%82,%83,%84,%85,%86,%87,%88,%89,%90,%91,%92,%93,%94,%95}, [%130];\n\t"                            \
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%96,%97,%98,%99,%100,%101,%102,%103,%104,%105,%106,%107,%108,%109,%110,%111,%112,%113,%114,%115,%116,%117,%118,%119,%120,%121,%122,%123,%124,%125,%126,%127}, [%131];\n\t"                            \
      "tcgen05.wait::ld.sync.aligned;"                                                         \
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31]), "=r"(r[32]), "=r"(r[33]), "=r"(r[34]), "=r"(r[35]), "=r"(r[36]), "=r"(r[37]), "=r"(r[38]), "=r"(r[39]), "=r"(r[40]), "=r"(r[41]), "=r"(r[42]), "=r"(r[43]), "=r"(r[44]), "=r"(r[45]), "=r"(r[46]), "=r"(r[47]), "=r"(r[48]), "=r"(r[49]), "=r"(r[50]), "=r"(r[51]), "=r"(r[52]), "=r"(r[53]), "=r"(r[54]), "=r"(r[55]), "=r"(r[56]), "=r"(r[57]), "=r"(r[58]), "=r"(r[59]), "=r"(r[60]), "=r"(r[61]), "=r"(r[62]), "=r"(r[63]), "=r"(r[64]), "=r"(r[65]), "=r"(r[66]), "=r"(r[67]), "=r"(r[68]), "=r"(r[69]), "=r"(r[70]), "=r"(r[71]), "=r"(r[72]), "=r"(r[73]), "=r"(r[74]), "=r"(r[75]), "=r"(r[76]), "=r"(r[77]), "=r"(r[78]), "=r"(r[79]), "=r"(r[80]), "=r"(r[81]), "=r"(r[82]), "=r"(r[83]), "=r"(r[84]), "=r"(r[85]), "=r"(r[86]), "=r"(r[87]), "=r"(r[88]), "=r"(r[89]), "=r"(r[90]), "=r"(r[91]), "=r"(r[92]), "=r"(r[93]), "=r"(r[94]), "=r"(r[95]), "=r"(r[96]), "=r"(r[97]), "=r"(r[98]), "=r"(r[99]), "=r"(r[100]), "=r"(r[101]), "=r"(r[102]), "=r"(r[103]), "=r"(r[104]), "=r"(r[105]), "=r"(r[106]), "=r"(r[107]), "=r"(r[108]), "=r"(r[109]), "=r"(r[110]), "=r"(r[111]), "=r"(r[112]), "=r"(r[113]), "=r"(r[114]), "=r"(r[115]), "=r"(r[116]), "=r"(r[117]), "=r"(r[118]), "=r"(r[119]), "=r"(r[120]), "=r"(r[121]), "=r"(r[122]), "=r"(r[123]), "=r"(r[124]), "=r"(r[125]), "=r"(r[126]), "=r"(r[127])                                                                                     \
      : "r"(taddr), "r"((taddr) + 32), "r"((taddr) + 64), "r"((taddr) + 96)                    \
      : "memory")
#define TMEM_LD32_WAIT(taddr, r)                                                               \
  asm volatile(                                                                                \
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];\n\t"                             \
      "tcgen05.wait::ld.sync.aligned;"                                                         \
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])                                                                                     \
      : "r"(taddr)                                                                             \
      : "memory")
#define TMEM_ST32(taddr, r)                                                                      \
  asm volatile(                                                                                  \
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,"   \
      "%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31,%32};"        \
      ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), \
        "r"(r[7]), "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]),         \
        "r"(r[14]), "r"(r[15]), "r"(r[16]), "r"(r[17]), "r"(r[18]), "r"(r[19]), "r"(r[20]),      \
        "r"(r[21]), "r"(r[22]), "r"(r[23]), "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]),      \
        "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31])                                           \
      : "memory")
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

// Shared-memory matrix descriptor, 128-byte swizzle, version 1 (sm_100).
__device__ __forceinline__ uint64_t make_desc(uint32_t saddr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
  uint64_t d = 0;
  d |= uint64_t((saddr & 0x3FFFFu) >> 4);
  d |= uint64_t((lbo_bytes >> 4) & 0x3FFFu) << 16;
  d |= uint64_t((sbo_bytes >> 4) & 0x3FFFu) << 32;
  d |= uint64_t(1) << 46;        // descriptor version
  d |= uint64_t(2) << 61;        // SWIZZLE_128B
  return d;
}
// Instruction descriptor: bf16 x bf16 -> fp32, M = 128, N = 128.
__host__ __device__ constexpr uint32_t make_idesc(bool b_mn_major) {
  return (1u << 4) | (1u << 7) | (1u << 10) | (uint32_t(b_mn_major) << 16) | (uint32_t(kBN >> 3) << 17) |
         (uint32_t(kBM >> 4) << 24);
}

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}

// ---------------------------------------------------------------- kernel
__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
// Barrier among the 256 softmax threads only (hardware barrier 1; barrier 0 is __syncthreads).
__device__ __forceinline__ void softmax_sync() { asm volatile("bar.sync 1, 256;" ::: "memory"); }

__global__ void __launch_bounds__(kThreads, 1)
attention_tc_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_kw,
                    const __grid_constant__ CUtensorMap tm_vw, const __grid_constant__ CUtensorMap tm_kp,
                    const __grid_constant__ CUtensorMap tm_vp, TcParams p) {
  extern __shared__ unsigned char smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t q_smem = base;
  const uint32_t stage0 = base + kTileBytes;
  const uint32_t bars = base + kSmemData;
  // barrier slots (8 bytes each)
  const uint32_t bar_q = bars;
  auto bar_kfull = [&](int s) { return bars + 8u * (1 + s); };
  auto bar_vfull = [&](int s) { return bars + 8u * (1 + kStages + s); };
  auto bar_empty = [&](int s) { return bars + 8u * (1 + 2 * kStages + s); };
  auto bar_sfull = [&](int b) { return bars + 8u * (1 + 3 * kStages + b); };
  auto bar_pfull = [&](int b) { return bars + 8u * (3 + 3 * kStages + b); };
  const uint32_t bar_done = bars + 8u * (5 + 3 * kStages);
  unsigned char* base_generic = smem_raw + (base - smem_u32(smem_raw));
  unsigned char* bars_generic = base_generic + kSmemData;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars_generic + 8 * (6 + 3 * kStages));
  volatile int* abort_flag = reinterpret_cast<volatile int*>(bars_generic + 8 * (6 + 3 * kStages) + 8);
  // after the last MMA has completed the Q tile is dead: its first 2 KiB carry the two
  // warpgroups' (max, sum) pairs to the merge
  float2* merge_ml = reinterpret_cast<float2*>(base_generic);

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
  const int gpb = p.block / 16;                          // page granules per block
  const int g_init = geo.init_len / 16;
  const int g_sel = c * gpb;
  const int64_t local_len = geo.p0 - geo.local_start;
  const int g_past = g_init + g_sel + int(local_len / 16);
  const bool misaligned = (local_len % 16) != 0;
  const int n_past = g_past * 16;
  const int past_tiles = (n_past + kBN - 1) / kBN;
  const int n_tiles = past_tiles + mt + 1;

  if (tid == 0) {
    if (bad) set_status(p.a.status, ACTQKV_DEV_BAD_SELECTION);
    if (misaligned) set_status(p.a.status, ACTQKV_DEV_BAD_SELECTION);
    mbar_init(bar_q, 1);
    for (int s = 0; s < kStages; ++s) { mbar_init(bar_kfull(s), 1); mbar_init(bar_vfull(s), 1); mbar_init(bar_empty(s), 1); }
    for (int b = 0; b < 2; ++b) { mbar_init(bar_sfull(b), 1); mbar_init(bar_pfull(b), 128); }
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

  if (warp < 4) {
    asm volatile("setmaxnreg.dec.sync.aligned.u32 56;");
    if (warp == 0) {
      // =========================== TMA producer ===========================
      const int32_t* sel = p.a.sel_idx + (size_t(unit) * p.n_kv_heads + g) * p.cap_blocks;
      const int32_t* pt = p.a.page_table + size_t(seq) * p.max_pages;
      const int page_oob = p.n_layers * p.n_phys_pages;              // beyond the tensor: zero fill
      if (lane == 0) {
        mbar_expect_tx(bar_q, kTileBytes);
        tma_load_3d(q_smem, &tm_q, bar_q, 0, h, unit * nt + mt * kBM);
        tma_load_3d(q_smem + kSubTileBytes, &tm_q, bar_q, 64, h, unit * nt + mt * kBM);
      }
      bool ok = true;
      int issued = 0;
      for (int j = 0; j < n_tiles && ok; ++j) {
        const int s = j % kStages, it = j / kStages;
        if (it > 0) ok = mbar_wait(bar_empty(s), (it - 1) & 1, abort_flag);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        const uint32_t sbase = stage0 + s * kStageBytes;
        if (lane == 0) {
          mbar_expect_tx(bar_kfull(s), kTileBytes);
          mbar_expect_tx(bar_vfull(s), kTileBytes);
        }
        __syncwarp();
        if (j < past_tiles) {
          const int is_v = lane >> 4, half = (lane >> 3) & 1, slot = lane & 7;
          const int gi = j * 8 + slot;
          int page = page_oob;
          if (gi < g_past) {
            int64_t lp;
            if (gi < g_init) {
              lp = gi;
            } else if (gi < g_init + g_sel) {
              const int r = gi - g_init;
              const int blk = sel[r / gpb];
              lp = (blk >= 0 && blk < geo.n_cand) ? (int64_t(p.n_init) + int64_t(blk) * p.block) / 16 + r % gpb : -1;
              if (lp < 0 && half == 0 && is_v == 0) set_status(p.a.status, ACTQKV_DEV_BAD_SELECTION);
            } else {
              lp = geo.local_start / 16 + (gi - g_init - g_sel);
            }
            if (lp >= 0) {
              const int phys = lp < p.max_pages ? pt[lp] : -1;
              if (phys < 0 || phys >= p.n_phys_pages) {
                if (half == 0 && is_v == 0) set_status(p.a.status, ACTQKV_DEV_BAD_PAGE);
              } else {
                page = layer_local * p.n_phys_pages + phys;
              }
            }
          }
          const uint32_t dst = sbase + is_v * kTileBytes + half * kSubTileBytes + slot * 2048u;
          tma_load_4d(dst, is_v ? &tm_vp : &tm_kp, is_v ? bar_vfull(s) : bar_kfull(s), half * 64, 0, g, page);
        } else if (lane < 4) {
          const int is_v = lane >> 1, half = lane & 1;
          const int kt = j - past_tiles;
          const uint32_t dst = sbase + is_v * kTileBytes + half * kSubTileBytes;
          tma_load_3d(dst, is_v ? &tm_vw : &tm_kw, is_v ? bar_vfull(s) : bar_kfull(s), half * 64, g,
                      unit * nt + kt * kBN);
        }
        issued = j + 1;
      }
      // drain: every issued copy must have landed before the CTA may exit on the abort path
      if (!ok) {
        for (int j = max(0, issued - kStages); j < issued; ++j) {
          const int s = j % kStages, par = (j / kStages) & 1;
          for (uint32_t i = 0; i < kSpinLimit && !mbar_try_wait(bar_kfull(s), par); ++i) {}
          for (uint32_t i = 0; i < kSpinLimit && !mbar_try_wait(bar_vfull(s), par); ++i) {}
        }
        for (uint32_t i = 0; i < kSpinLimit && !mbar_try_wait(bar_q, 0); ++i) {}
      }
    } else if (warp == 1) {
      // =========================== MMA issuer ===========================
      // Issue order QK(0), QK(1), PV(0), QK(2), PV(1), ...: the tensor pipe executes in issue
      // order, so QK(j+2) cannot overwrite S/P buffer j&1 before PV(j) has read P(j), and a
      // completed QK(j) implies a completed PV(j-2).
      if (lane == 0) {
        constexpr uint32_t idesc_qk = make_idesc(false);
        constexpr uint32_t idesc_pv = make_idesc(true);
        bool ok = mbar_wait(bar_q, 0, abort_flag);
        auto issue_pv = [&](int i) {
          const int s = i % kStages, b = i & 1;
          ok = ok && mbar_wait(bar_vfull(s), (i / kStages) & 1, abort_flag);
          ok = ok && mbar_wait(bar_pfull(b), (i >> 1) & 1, abort_flag);
          if (!ok) return;
          tc_fence_after();
          const uint32_t vbase = stage0 + s * kStageBytes + kTileBytes;
          const uint32_t p_tmem = tmem + b * 128;
          const uint32_t o_tmem = tmem + 256 + b * 128;
#pragma unroll
          for (int k = 0; k < kBN / 16; ++k) {
            // 16 keys per step: B advances 16 rows of 128 bytes; A = 8 packed columns of the hi
            // term, then the 8 columns of the lo term of the same keys against the same V rows.
            const uint64_t bdesc = make_desc(vbase + k * 2048u, kSubTileBytes, 1024u);
            const uint32_t pa = p_tmem + (k >> 1) * 32 + (k & 1) * 8;
            mma_ts(o_tmem, pa, bdesc, idesc_pv, (i >= 2 || k > 0) ? 1u : 0u);
            mma_ts(o_tmem, pa + 16, bdesc, idesc_pv, 1u);
          }
          tc_commit(bar_empty(s));
        };
        for (int j = 0; j < n_tiles && ok; ++j) {
          const int s = j % kStages;
          ok = mbar_wait(bar_kfull(s), (j / kStages) & 1, abort_flag);
          if (!ok) break;
          tc_fence_after();
          const uint32_t kbase = stage0 + s * kStageBytes;
#pragma unroll
          for (int k = 0; k < kD / 16; ++k) {
            const uint32_t off = (k >> 2) * kSubTileBytes + (k & 3) * 32u;
            const uint64_t adesc = make_desc(q_smem + off, 16u, 1024u);
            const uint64_t bdesc = make_desc(kbase + off, 16u, 1024u);
            mma_ss(tmem + (j & 1) * 128, adesc, bdesc, idesc_qk, k > 0 ? 1u : 0u);
          }
          tc_commit(bar_sfull(j & 1));
          if (j >= 1) issue_pv(j - 1);
        }
        if (ok) issue_pv(n_tiles - 1);
        if (ok) tc_commit(bar_done);
      }
      __syncwarp();
    }
  } else {
    asm volatile("setmaxnreg.inc.sync.aligned.u32 224;");
    // =========================== softmax / epilogue ===========================
    const int b = (warp >> 2) - 1;                        // 0: even tiles, 1: odd tiles
    const int q4 = warp & 3;                              // TMEM lane quadrant of this warp
    const int row = q4 * 32 + lane;                       // query row inside the tile
    const uint32_t lane_addr = uint32_t(q4 * 32) << 16;
    const uint32_t s_addr = tmem + lane_addr + b * 128;
    const uint32_t o_addr = tmem + lane_addr + 256 + b * 128;
    float m_used = -INFINITY, l = 0.f;
    bool ok = true;
    for (int j = b, kk = 0; j < n_tiles; j += 2, ++kk) {
      ok = ok && mbar_wait(bar_sfull(b), kk & 1, abort_flag);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tc_fence_after();
      uint32_t sr[128];
      TMEM_LD128_WAIT(s_addr, sr);
      // key-validity limit: ragged last past tile, or the causal diagonal of the last tile
      int limit = kBN;
      if (j < past_tiles) limit = min(kBN, n_past - j * kBN);
      else if (j == n_tiles - 1) limit = row + 1;
      const bool masked = (j == n_tiles - 1) || (j == past_tiles - 1 && (n_past % kBN) != 0);   // CTA-uniform
      float mx = -INFINITY;
      if (masked) {
#pragma unroll
        for (int i = 0; i < 128; ++i) {
          const float x = i < limit ? __uint_as_float(sr[i]) : -INFINITY;
          sr[i] = __float_as_uint(x);
          mx = fmaxf(mx, x);
        }
      } else {
        float mx2 = -INFINITY;
#pragma unroll
        for (int i = 0; i < 128; i += 2) {
          mx = fmaxf(mx, __uint_as_float(sr[i]));
          mx2 = fmaxf(mx2, __uint_as_float(sr[i + 1]));
        }
        mx = fmaxf(mx, mx2);
      }
      const float m_new = fmaxf(m_used, mx * p.scale_log2);
      const bool grow = m_new - m_used > kRescaleThreshold;     // also true for the first tile
      if (kk == 0) {
        m_used = m_new;
      } else if (__any_sync(0xffffffffu, grow)) {
        // S(j) complete implies PV(j-2) complete: this warpgroup's O is quiescent until it
        // publishes P(j)
        const float f = grow ? ex2(m_used - m_new) : 1.f;
        if (grow) { m_used = m_new; l *= f; }
#pragma unroll
        for (int cc = 0; cc < 4; ++cc) {
          uint32_t orr[32];
          TMEM_LD32_WAIT(o_addr + cc * 32, orr);
#pragma unroll
          for (int i = 0; i < 32; ++i) orr[i] = __float_as_uint(__uint_as_float(orr[i]) * f);
          TMEM_ST32(o_addr + cc * 32, orr);
        }
      }
      // P = exp2(x - m) split into two bf16 terms (hi + lo): with outlier value channels a
      // single bf16 P (8 significant bits) would cost up to |v| * 2^-9 of absolute error.
      const float neg_m = -m_used;
      float sum0 = 0.f, sum1 = 0.f;
#pragma unroll
      for (int cc = 0; cc < 4; ++cc) {
        uint32_t pk[32];
#pragma unroll
        for (int i = 0; i < 16; ++i) {
          const float e0 = ex2(fmaf(__uint_as_float(sr[32 * cc + 2 * i]), p.scale_log2, neg_m));
          const float e1 = ex2(fmaf(__uint_as_float(sr[32 * cc + 2 * i + 1]), p.scale_log2, neg_m));
          sum0 += e0;
          sum1 += e1;
          const uint32_t hi = pack_bf16(e0, e1);
          pk[i] = hi;
          pk[16 + i] = pack_bf16(e0 - __uint_as_float(hi << 16), e1 - __uint_as_float(hi & 0xFFFF0000u));
        }
        TMEM_ST32(s_addr + cc * 32, pk);
      }
      l += sum0 + sum1;
      tmem_wait_st();
      tc_fence_before();
      mbar_arrive(bar_pfull(b));
    }
    // ---- merge of the two warpgroups' partial results and epilogue
    ok = ok && mbar_wait(bar_done, 0, abort_flag);
    if (ok) merge_ml[b * 128 + row] = make_float2(m_used, l);
    softmax_sync();
    if (*abort_flag == 0) {
      tc_fence_after();
      const float2 a0 = merge_ml[row], a1 = merge_ml[128 + row];
      const float m = fmaxf(a0.x, a1.x);
      float f0 = a0.y > 0.f ? ex2(a0.x - m) : 0.f;
      float f1 = a1.y > 0.f ? ex2(a1.x - m) : 0.f;
      const float lsum = a0.y * f0 + a1.y * f1;
      const float inv = lsum > 0.f ? 1.f / lsum : 0.f;
      f0 *= inv;
      f1 *= inv;
      const bool use1 = f1 != 0.f;                          // O1 was never written when the CTA has one tile
      const size_t tok = size_t(unit) * nt + size_t(mt) * kBM + row;
      const uint32_t o0 = tmem + lane_addr + 256, o1 = tmem + lane_addr + 384;
#pragma unroll
      for (int cc = 0; cc < 2; ++cc) {
        const int col = b * 64 + cc * 32;                   // this warpgroup's half of the channels
        uint32_t r0[32], r1[32];
        TMEM_LD32_WAIT(o0 + col, r0);
        TMEM_LD32_WAIT(o1 + col, r1);
        float o[32];
#pragma unroll
        for (int i = 0; i < 32; ++i) {
          const float x1 = use1 ? __uint_as_float(r1[i]) * f1 : 0.f;
          o[i] = fmaf(__uint_as_float(r0[i]), f0, x1);
        }
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
      if (p.a.lse && b == 0)
        p.a.lse[(size_t(unit) * p.n_q_heads + h) * nt + size_t(mt) * kBM + row] =
            (m + log2f(lsum)) * 0.6931471805599453f;
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

// ---------------------------------------------------------------- host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode() {
  static EncodeTiledFn fn = nullptr;
  static bool tried = false;
  if (!tried) {
    tried = true;
    void* sym = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &qres) == cudaSuccess &&
        qres == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(sym);
  }
  return fn;
}

// bf16 tensor map with 128-byte swizzle; dims / strides innermost first, strides in bytes (rank - 1 of them).
bool encode(CUtensorMap* tm, const void* base, int rank, const cuuint64_t* dims, const cuuint64_t* strides,
            const cuuint32_t* box) {
  EncodeTiledFn fn = get_encode();
  if (!fn) return false;
  cuuint32_t estr[5] = {1, 1, 1, 1, 1};
  return fn(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, rank, const_cast<void*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
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
  static bool attr_set = false;
  if (!attr_set) {
    if (cudaFuncSetAttribute(attention_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, int(kSmemBytes)) !=
        cudaSuccess)
      return ACTQKV_ERR_LAUNCH;
    attr_set = true;
  }
  dim3 grid(nt / kBM, Hq, U);
  attention_tc_kernel<<<grid, kThreads, kSmemBytes, st>>>(tm_q, tm_kw, tm_vw, tm_kp, tm_vp, p);
  return launch_status();
}

}  // namespace actqkv
