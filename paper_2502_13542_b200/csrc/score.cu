// Step 3: cosine scores of the probe-query against every candidate block's representative
// keys (Eq. 10) and the information density of each head's score distribution (Eq. 11).
//
// The representative-key table is streamed once with 16-byte loads.  One warp scores four
// blocks: a row of D elements is covered by D*sizeof(T)/16 lanes, all of the warp's loads for
// the block are issued before the first is used, the dot products are finished with warp
// shuffles inside each row's lane group.  With one block per warp the grid is wide enough to
// keep every SM's memory pipeline busy on tables of a few MB.
#include "common.cuh"
#include "stages.cuh"

using namespace actqkv;

namespace {

constexpr int kScoreThreads = 256;
constexpr int kBlocksPerWarp = 4;                   // candidate blocks scored by one warp, loads of all in flight
constexpr int kBlocksPerCta = (kScoreThreads / 32) * kBlocksPerWarp;
constexpr int kMaxPasses = 2;                       // row groups of one block held in registers

// kMean: block score = mean of the r cosines.  Then every lane scales its partial dot product by
// its row's inverse norm and ONE shuffle tree over the warp finishes the block; the max
// aggregation needs the r cosines separately and reduces row by row.
template <typename T, int D, bool kMean>
__global__ void __launch_bounds__(kScoreThreads, 2)
score_kernel(const float* __restrict__ probe_kv, const T* __restrict__ repr_k,
             const float* __restrict__ repr_inv_norm, const int32_t* __restrict__ n_cand,
             float* __restrict__ scores, int n_kv_heads, int r, int n_cap, int n_layers, int groups,
             int32_t* status) {
  const int g = blockIdx.y, unit = blockIdx.z;
  const int seq = unit / n_layers;
  int n = n_cand[seq];
  if (n > n_cap) {
    n = n_cap;
    if (threadIdx.x == 0 && blockIdx.x == 0 && g == 0) set_status(status, ACTQKV_DEV_NCAND_CLAMPED);
  }
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  // a warp scores `groups` groups of kBlocksPerWarp consecutive blocks
  const int b0 = (blockIdx.x * (kScoreThreads / 32) + warp) * kBlocksPerWarp * groups;
  if (b0 >= n) return;                    // warp-uniform; no block-wide barrier below

  constexpr int VN = Vec16<T>::N;
  constexpr int LPR = D / VN;           // lanes per row: 8, 16 or 32
  constexpr int RPP = 32 / LPR;         // rows per pass
  const int sub = lane / LPR, lir = lane - sub * LPR;
  const size_t head_rows = (size_t(unit) * n_kv_heads + g) * size_t(n_cap) * r;
  const int n_pass = (r + RPP - 1) / RPP;
  const T* tab = repr_k + head_rows * D + lir * VN;
  const float* inv = repr_inv_norm + head_rows;

  // One group's rows: raw 16-byte vectors (unpacked at use) and the rows' inverse norms.
  struct Group {
    uint4 kv[kBlocksPerWarp][kMaxPasses];
    float nrm[kBlocksPerWarp][kMaxPasses];
  };
  auto load_group = [&](int bg, Group& gr) {
#pragma unroll
    for (int bi = 0; bi < kBlocksPerWarp; ++bi) {
#pragma unroll
      for (int ps = 0; ps < kMaxPasses; ++ps) {
        const int i = ps * RPP + sub;
        const bool on = bg + bi < n && i < r;
        const size_t row = size_t(bg + bi) * r + i;
        gr.nrm[bi][ps] = on ? __ldg(inv + row) : 0.f;
        gr.kv[bi][ps] = on ? __ldg(reinterpret_cast<const uint4*>(tab + row * D)) : make_uint4(0, 0, 0, 0);
      }
    }
  };
  // Fast path (mean aggregation): a group of four blocks is 4 KiB of contiguous rows when
  // r * D * sizeof(T) = 1 KiB per block: eight 512-byte warp loads at fixed offsets from one base,
  // the sixteen inverse norms by one load and shuffles.  Whole groups only; a ragged last group
  // takes the general loads.
  constexpr int kVec = 8;                                // 512-byte vectors per group
  struct Raw { uint4 v[kVec]; float nrm; };
  const bool fast_shape = kMean && size_t(r) * D * sizeof(T) == 1024;
  auto load_fast = [&](int bg, Raw& x) {
    const uint4* pch = reinterpret_cast<const uint4*>(repr_k + (head_rows + size_t(bg) * r) * D) + lane;
#pragma unroll
    for (int u = 0; u < kVec; ++u) x.v[u] = __ldg(pch + u * 32);
    x.nrm = lane < kBlocksPerWarp * r ? __ldg(inv + size_t(bg) * r + lane) : 0.f;
  };
  auto full = [&](int gi) { return gi < groups && b0 + (gi + 1) * kBlocksPerWarp <= n; };
  auto exists = [&](int gi) { return gi < groups && b0 + gi * kBlocksPerWarp < n; };
  // the first group's loads go out before anything else, then the probe
  Group ga, gb;
  Raw ra, rb;
  const bool first_fast = fast_shape && full(0);
  if (first_fast) load_fast(b0, ra); else load_group(b0, ga);
  grid_launch_dependents();
  grid_dependency_wait();            // the table is older than the stream's previous kernel; the probe is not
  const float* pg = probe_kv + (size_t(unit) * n_kv_heads + g) * D;
  float pv[VN];
  Vec16<float>::load_nc(pg + lir * VN, reinterpret_cast<float(&)[4]>(pv[0]));
  if constexpr (VN == 8) Vec16<float>::load_nc(pg + lir * VN + 4, reinterpret_cast<float(&)[4]>(pv[4]));
  // probe norm: every group of LPR lanes holds the whole probe
  float sq = 0.f;
#pragma unroll
  for (int e = 0; e < VN; ++e) sq = fmaf(pv[e], pv[e], sq);
#pragma unroll
  for (int o = LPR >> 1; o > 0; o >>= 1) sq += __shfl_xor_sync(0xffffffffu, sq, o);
  const bool bad = !(sq > 0.f) || !isfinite(sq);
  if (bad && lane == 0 && b0 == 0) set_status(status, ACTQKV_DEV_BAD_PROBE);
  const float inv_pn = bad ? 0.f : rsqrtf(sq);
  float* out = scores + (size_t(unit) * n_kv_heads + g) * n_cap;

  auto score_group = [&](int bg, const Group& gr) {
#pragma unroll
    for (int bi = 0; bi < kBlocksPerWarp; ++bi) {
      const int b = bg + bi;
      if (b >= n) break;                  // warp-uniform
      if constexpr (kMean) {
        float acc = 0.f;                  // sum over this lane's rows of (partial dot) / ||R_i||
        for (int p0 = 0; p0 < n_pass; p0 += kMaxPasses) {
#pragma unroll
          for (int ps = 0; ps < kMaxPasses; ++ps) {
            float row[VN];
            float w = gr.nrm[bi][ps];
            if (p0 == 0) {
              Vec16<T>::unpack(gr.kv[bi][ps], row);
            } else {                      // more row groups than the registers hold
              const int i = (p0 + ps) * RPP + sub;
              w = 0.f;
#pragma unroll
              for (int e = 0; e < VN; ++e) row[e] = 0.f;
              if (i < r) {
                w = __ldg(inv + size_t(b) * r + i);
                Vec16<T>::load_nc(tab + (size_t(b) * r + i) * D, row);
              }
            }
            float dot = 0.f;
#pragma unroll
            for (int e = 0; e < VN; ++e) dot = fmaf(pv[e], row[e], dot);
            acc = fmaf(dot, w, acc);
          }
        }
        acc = warp_sum(acc);
        if (lane == 0) out[b] = acc * inv_pn / float(r);
      } else {
        float agg = -INFINITY;
        for (int ps = 0; ps < n_pass; ++ps) {
          const int i = ps * RPP + sub;
          float row[VN];
          float w = 0.f;
#pragma unroll
          for (int e = 0; e < VN; ++e) row[e] = 0.f;
          if (i < r) {
            w = __ldg(inv + size_t(b) * r + i);
            Vec16<T>::load_nc(tab + (size_t(b) * r + i) * D, row);
          }
          float dot = 0.f;
#pragma unroll
          for (int e = 0; e < VN; ++e) dot = fmaf(pv[e], row[e], dot);
#pragma unroll
          for (int o = LPR >> 1; o > 0; o >>= 1) dot += __shfl_xor_sync(0xffffffffu, dot, o);
          float cosv = i < r ? dot * inv_pn * w : -INFINITY;
          // maximum over the row groups of this pass (group leaders hold the cosines)
#pragma unroll
          for (int o = LPR; o < 32; o <<= 1) cosv = fmaxf(cosv, __shfl_xor_sync(0xffffffffu, cosv, o));
          agg = fmaxf(agg, cosv);
        }
        if (lane == 0) out[b] = agg;
      }
    }
  };
  if constexpr (kMean) if (fast_shape) {
    // the four block sums of a group are reduced together (6 shuffles instead of 20): halves swap
    // block pairs, quarters swap blocks, then three steps inside each quarter
    auto score_fast = [&](int bg, const Raw& x) {
      float accb[kBlocksPerWarp];
#pragma unroll
      for (int bi = 0; bi < kBlocksPerWarp; ++bi) {
        accb[bi] = 0.f;
#pragma unroll
        for (int k = 0; k < 2; ++k) {                    // the block's two vectors
          const int u = 2 * bi + k;
          float row[VN];
          Vec16<T>::unpack(x.v[u], row);
          float dot = 0.f;
#pragma unroll
          for (int e = 0; e < VN; ++e) dot = fmaf(pv[e], row[e], dot);
          const float w = __shfl_sync(0xffffffffu, x.nrm, u * RPP + sub);   // row u * RPP + sub of the group
          accb[bi] = fmaf(dot, w, accb[bi]);
        }
      }
      const bool up16 = lane & 16, up8 = lane & 8;
      const float t0 = __shfl_xor_sync(0xffffffffu, up16 ? accb[0] : accb[2], 16);
      const float t1 = __shfl_xor_sync(0xffffffffu, up16 ? accb[1] : accb[3], 16);
      const float k0 = (up16 ? accb[2] : accb[0]) + t0, k1 = (up16 ? accb[3] : accb[1]) + t1;
      float k = (up8 ? k1 : k0) + __shfl_xor_sync(0xffffffffu, up8 ? k0 : k1, 8);
      k += __shfl_xor_sync(0xffffffffu, k, 4);
      k += __shfl_xor_sync(0xffffffffu, k, 2);
      k += __shfl_xor_sync(0xffffffffu, k, 1);
      if ((lane & 7) == 0) out[bg + 2 * (lane >> 4) + ((lane >> 3) & 1)] = k * inv_pn / float(r);
    };
    auto ragged = [&](int gi) {                            // a last, partly filled group: general loads
      const int bg = b0 + gi * kBlocksPerWarp;
      load_group(bg, ga);
      score_group(bg, ga);
    };
    if (!first_fast) { score_group(b0, ga); return; }      // b0 + 4 > n: the only group of this warp
    // invariant at the loop head: if group gi is whole, ra holds it
    for (int gi = 0; exists(gi);) {
      if (!full(gi)) { ragged(gi); break; }
      if (full(gi + 1)) load_fast(b0 + (gi + 1) * kBlocksPerWarp, rb);
      score_fast(b0 + gi * kBlocksPerWarp, ra);
      ++gi;
      if (!exists(gi)) break;
      if (!full(gi)) { ragged(gi); break; }
      if (full(gi + 1)) load_fast(b0 + (gi + 1) * kBlocksPerWarp, ra);
      score_fast(b0 + gi * kBlocksPerWarp, rb);
      ++gi;
    }
    return;
  }
  // double-buffered: the next group's loads are in flight while the current group is scored
  for (int gi = 0; gi < groups; gi += 2) {
    const int bg = b0 + gi * kBlocksPerWarp;
    if (bg >= n) break;
    if (gi + 1 < groups) load_group(bg + kBlocksPerWarp, gb);
    score_group(bg, ga);
    if (gi + 2 < groups) load_group(bg + 2 * kBlocksPerWarp, ga);
    if (gi + 1 < groups) score_group(bg + kBlocksPerWarp, gb);
  }
}

constexpr int kEntropyThreads = 256;

__global__ void __launch_bounds__(kEntropyThreads)
entropy_kernel(const float* __restrict__ scores, const int32_t* __restrict__ n_cand,
               float* __restrict__ theta, int n_kv_heads, int n_cap, int n_layers, float beta) {
  __shared__ float red[3 * (kEntropyThreads / 32)];
  const int g = blockIdx.x, unit = blockIdx.y;
  grid_launch_dependents();
  grid_dependency_wait();            // the scores come from the stream's previous kernel
  const int n = min(n_cand[unit / n_layers], n_cap);
  const float th = block_entropy<kEntropyThreads>(scores + (size_t(unit) * n_kv_heads + g) * n_cap, n, beta, red);
  if (threadIdx.x == 0) theta[size_t(unit) * n_kv_heads + g] = th;
}

}  // namespace

namespace actqkv {

template <typename T, int D>
void launch_scores_t(const actqkv_config* cfg, const Batch& b, const float* probe_kv, const void* repr_k,
                     const float* repr_inv_norm, const int32_t* n_cand, float* scores, int32_t* status,
                     cudaStream_t st) {
  // blocks per warp: one group of kBlocksPerWarp when the call is small (latency matters, spread
  // it over as many CTAs as possible), more groups (software-pipelined) once the grid would
  // exceed a few CTAs per SM anyway
  const int ctas_1 = (cfg->n_cap + kBlocksPerCta - 1) / kBlocksPerCta;
  const long long total_1 = (long long)ctas_1 * cfg->n_kv_heads * b.units();
  int groups = 1;
  while (groups < 8 && total_1 / (2 * groups) >= 4 * 148 && ctas_1 / (2 * groups) >= 1) groups *= 2;
  dim3 grid((cfg->n_cap + kBlocksPerCta * groups - 1) / (kBlocksPerCta * groups), cfg->n_kv_heads, b.units());
  prefer_max_shared(score_kernel<T, D, false>);
  prefer_max_shared(score_kernel<T, D, true>);
  cudaLaunchConfig_t lc = {};
  lc.gridDim = grid;
  lc.blockDim = dim3(kScoreThreads, 1, 1);
  lc.stream = st;
  cudaLaunchAttribute attr[1];
  allow_early_launch(attr[0]);
  lc.attrs = attr;
  lc.numAttrs = 1;
  const T* tab = static_cast<const T*>(repr_k);
  if (cfg->agg_mode == ACTQKV_AGG_MAX)
    (void)cudaLaunchKernelEx(&lc, score_kernel<T, D, false>, probe_kv, tab, repr_inv_norm, n_cand, scores,
                             cfg->n_kv_heads, cfg->n_repr, cfg->n_cap, b.n_layers, groups, status);
  else
    (void)cudaLaunchKernelEx(&lc, score_kernel<T, D, true>, probe_kv, tab, repr_inv_norm, n_cand, scores,
                             cfg->n_kv_heads, cfg->n_repr, cfg->n_cap, b.n_layers, groups, status);
}

int launch_scores(const actqkv_config* cfg, const Batch& b, const float* probe_kv, const void* repr_k,
                  const float* repr_inv_norm, const int32_t* n_cand, float* scores, int32_t* status,
                  cudaStream_t st) {
  if (cfg->n_cap == 0) return ACTQKV_OK;
  const bool bf16 = cfg->dtype == ACTQKV_BF16;
  if (cfg->head_dim == 64) {
    if (bf16) launch_scores_t<__nv_bfloat16, 64>(cfg, b, probe_kv, repr_k, repr_inv_norm, n_cand, scores, status, st);
    else launch_scores_t<float, 64>(cfg, b, probe_kv, repr_k, repr_inv_norm, n_cand, scores, status, st);
  } else {
    if (bf16) launch_scores_t<__nv_bfloat16, 128>(cfg, b, probe_kv, repr_k, repr_inv_norm, n_cand, scores, status, st);
    else launch_scores_t<float, 128>(cfg, b, probe_kv, repr_k, repr_inv_norm, n_cand, scores, status, st);
  }
  return launch_status();
}

int launch_entropy(const actqkv_config* cfg, const Batch& b, const float* scores, const int32_t* n_cand,
                   float* theta, cudaStream_t st) {
  prefer_max_shared(entropy_kernel);
  cudaLaunchConfig_t lc = {};
  lc.gridDim = dim3(cfg->n_kv_heads, b.units(), 1);
  lc.blockDim = dim3(kEntropyThreads, 1, 1);
  lc.stream = st;
  cudaLaunchAttribute attr[1];
  allow_early_launch(attr[0]);       // resident while the score kernel drains; waits for it before reading
  lc.attrs = attr;
  lc.numAttrs = 1;
  if (cudaLaunchKernelEx(&lc, entropy_kernel, scores, n_cand, theta, cfg->n_kv_heads, cfg->n_cap, b.n_layers,
                         cfg->beta) != cudaSuccess)
    return ACTQKV_ERR_LAUNCH;
  return launch_status();
}

}  // namespace actqkv

extern "C" int actqkv_score_blocks(const actqkv_config* cfg, const actqkv_batch* batch,
                                   const float* probe_kv, const void* repr_k, const float* repr_inv_norm,
                                   const int32_t* n_cand, float* scores, float* theta, int32_t* status,
                                   void* stream) {
  const Batch b = get_batch(batch);
  int rc = check_config(cfg, b);
  if (rc) return rc;
  ACTQKV_REQUIRE_PTR(probe_kv);
  ACTQKV_REQUIRE_PTR(repr_k);
  ACTQKV_REQUIRE_PTR(repr_inv_norm);
  if (!n_cand) return ACTQKV_ERR_NULL;
  ACTQKV_REQUIRE_PTR(scores);
  if (!theta) return ACTQKV_ERR_NULL;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  rc = launch_scores(cfg, b, probe_kv, repr_k, repr_inv_norm, n_cand, scores, status, st);
  if (rc) return rc;
  return launch_entropy(cfg, b, scores, n_cand, theta, st);
}
