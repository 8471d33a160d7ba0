// Step 3: cosine scores of the probe-query against every candidate block's representative
// keys (Eq. 10) and the information density of each head's score distribution (Eq. 11).
//
// The representative-key table is streamed once with 16-byte loads.  One warp scores one
// block: a row of D elements is covered by D*sizeof(T)/16 lanes, all of the warp's loads for
// the block are issued before the first is used, the dot products are finished with warp
// shuffles inside each row's lane group.  With one block per warp the grid is wide enough to
// keep every SM's memory pipeline busy on tables of a few MB.
#include "common.cuh"
#include "stages.cuh"

using namespace actqkv;

namespace {

constexpr int kScoreThreads = 256;
constexpr int kBlocksPerCta = kScoreThreads / 32;   // one candidate block per warp
constexpr int kMaxPasses = 4;                       // row groups of a block loaded together

template <typename T>
__global__ void __launch_bounds__(kScoreThreads)
score_kernel(const float* __restrict__ probe_kv, const T* __restrict__ repr_k,
             const float* __restrict__ repr_inv_norm, const int32_t* __restrict__ n_cand,
             float* __restrict__ scores, int n_kv_heads, int D, int r, int n_cap, int n_layers,
             int agg_mode, int32_t* status) {
  const int g = blockIdx.y, unit = blockIdx.z;
  const int seq = unit / n_layers;
  int n = n_cand[seq];
  if (n > n_cap) {
    n = n_cap;
    if (threadIdx.x == 0 && blockIdx.x == 0 && g == 0) set_status(status, ACTQKV_DEV_NCAND_CLAMPED);
  }
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int b = blockIdx.x * kBlocksPerCta + warp;
  if (b >= n) return;                     // warp-uniform; no block-wide barrier below

  constexpr int VN = Vec16<T>::N;
  const int lpr = D / VN;               // lanes per row: 8, 16 or 32
  const int rows_per_pass = 32 / lpr;
  const int sub = lane / lpr, lir = lane - sub * lpr;
  const size_t head_rows = (size_t(unit) * n_kv_heads + g) * size_t(n_cap) * r;
  const T* tab = repr_k + (head_rows + size_t(b) * r) * D;
  const float* inv = repr_inv_norm + head_rows + size_t(b) * r;

  // the block's rows first (independent loads), then the probe
  float kv[kMaxPasses][VN];
  const int n_pass = (r + rows_per_pass - 1) / rows_per_pass;
#pragma unroll
  for (int ps = 0; ps < kMaxPasses; ++ps) {
    const int i = ps * rows_per_pass + sub;
    if (ps < n_pass && i < r) Vec16<T>::load_nc(tab + size_t(i) * D + lir * VN, kv[ps]);
    else {
#pragma unroll
      for (int e = 0; e < VN; ++e) kv[ps][e] = 0.f;
    }
  }
  const float inv_row = lane < r ? __ldg(inv + lane) : 0.f;          // lane i holds 1 / ||R_i||
  const float* pg = probe_kv + (size_t(unit) * n_kv_heads + g) * D;
  float pv[VN];
  Vec16<float>::load_nc(pg + lir * VN, reinterpret_cast<float(&)[4]>(pv[0]));
  if constexpr (VN == 8) Vec16<float>::load_nc(pg + lir * VN + 4, reinterpret_cast<float(&)[4]>(pv[4]));
  // probe norm: every lane group of lpr lanes holds the whole probe
  float sq = 0.f;
#pragma unroll
  for (int e = 0; e < VN; ++e) sq = fmaf(pv[e], pv[e], sq);
  for (int o = lpr >> 1; o > 0; o >>= 1) sq += __shfl_xor_sync(0xffffffffu, sq, o);
  const bool bad = !(sq > 0.f) || !isfinite(sq);
  if (bad && lane == 0 && b == 0) set_status(status, ACTQKV_DEV_BAD_PROBE);
  const float inv_pn = bad ? 0.f : rsqrtf(sq);

  float agg = agg_mode == ACTQKV_AGG_MAX ? -INFINITY : 0.f;
  for (int p0 = 0; p0 < n_pass; p0 += kMaxPasses) {
    if (p0 > 0) {                        // more than kMaxPasses row groups: fetch the next batch
#pragma unroll
      for (int ps = 0; ps < kMaxPasses; ++ps) {
        const int i = (p0 + ps) * rows_per_pass + sub;
        if (p0 + ps < n_pass && i < r) Vec16<T>::load_nc(tab + size_t(i) * D + lir * VN, kv[ps]);
      }
    }
#pragma unroll
    for (int ps = 0; ps < kMaxPasses; ++ps) {
      if (p0 + ps >= n_pass) break;
      const int i0 = (p0 + ps) * rows_per_pass;
      float dot = 0.f;
#pragma unroll
      for (int e = 0; e < VN; ++e) dot = fmaf(pv[e], kv[ps][e], dot);
      for (int o = lpr >> 1; o > 0; o >>= 1) dot += __shfl_xor_sync(0xffffffffu, dot, o);
      // combine the row groups of this pass (group leaders hold the dot products)
      for (int s = 0; s < rows_per_pass; ++s) {
        const int i = i0 + s;
        const float d = __shfl_sync(0xffffffffu, dot, s * lpr);
        const float nrm = i < 32 ? __shfl_sync(0xffffffffu, inv_row, i & 31) : __ldg(inv + min(i, r - 1));
        if (i < r) {
          const float cv = d * inv_pn * nrm;
          agg = agg_mode == ACTQKV_AGG_MAX ? fmaxf(agg, cv) : agg + cv;
        }
      }
    }
  }
  if (lane == 0)
    scores[(size_t(unit) * n_kv_heads + g) * n_cap + b] = agg_mode == ACTQKV_AGG_MAX ? agg : agg / float(r);
}

__global__ void __launch_bounds__(32)
entropy_kernel(const float* __restrict__ scores, const int32_t* __restrict__ n_cand,
               float* __restrict__ theta, int n_kv_heads, int n_cap, int n_layers, float beta) {
  const int g = blockIdx.x, unit = blockIdx.y;
  const int n = min(n_cand[unit / n_layers], n_cap);
  const float th = warp_entropy(scores + (size_t(unit) * n_kv_heads + g) * n_cap, n, beta);
  if (threadIdx.x == 0) theta[size_t(unit) * n_kv_heads + g] = th;
}

}  // namespace

namespace actqkv {

int launch_scores(const actqkv_config* cfg, const Batch& b, const float* probe_kv, const void* repr_k,
                  const float* repr_inv_norm, const int32_t* n_cand, float* scores, int32_t* status,
                  cudaStream_t st) {
  if (cfg->n_cap == 0) return ACTQKV_OK;
  dim3 grid((cfg->n_cap + kBlocksPerCta - 1) / kBlocksPerCta, cfg->n_kv_heads, b.units());
  if (cfg->dtype == ACTQKV_BF16)
    score_kernel<__nv_bfloat16><<<grid, kScoreThreads, 0, st>>>(
        probe_kv, static_cast<const __nv_bfloat16*>(repr_k), repr_inv_norm, n_cand, scores,
        cfg->n_kv_heads, cfg->head_dim, cfg->n_repr, cfg->n_cap, b.n_layers, cfg->agg_mode, status);
  else
    score_kernel<float><<<grid, kScoreThreads, 0, st>>>(
        probe_kv, static_cast<const float*>(repr_k), repr_inv_norm, n_cand, scores, cfg->n_kv_heads,
        cfg->head_dim, cfg->n_repr, cfg->n_cap, b.n_layers, cfg->agg_mode, status);
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
  entropy_kernel<<<dim3(cfg->n_kv_heads, b.units()), 32, 0, st>>>(
      scores, n_cand, theta, cfg->n_kv_heads, cfg->n_cap, b.n_layers, cfg->beta);
  return launch_status();
}
