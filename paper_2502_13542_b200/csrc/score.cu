// Step 3: cosine scores of the probe-query against every candidate block's representative
// keys (Eq. 10) and the information density of each head's score distribution (Eq. 11).
//
// The representative-key table is streamed once with 16-byte loads; a row of D elements is
// covered by D*sizeof(T)/16 lanes, the dot product is finished with warp shuffles inside
// that lane group, and one warp produces the scores of kBlocksPerIter blocks per iteration
// so that several loads are in flight per lane.
#include "common.cuh"
#include "stages.cuh"

using namespace actqkv;

namespace {

constexpr int kScoreThreads = 256;
constexpr int kBlocksPerCta = 64;   // candidate blocks per CTA (grid.x covers n_cap)

template <typename T>
__global__ void __launch_bounds__(kScoreThreads)
score_kernel(const float* __restrict__ probe_kv, const T* __restrict__ repr_k,
             const float* __restrict__ repr_inv_norm, const int32_t* __restrict__ n_cand,
             float* __restrict__ scores, int n_kv_heads, int D, int r, int n_cap, int n_layers,
             int agg_mode, int32_t* status) {
  __shared__ float probe_s[128];
  __shared__ float red_s[kScoreThreads / 32];
  const int g = blockIdx.y, unit = blockIdx.z;
  const int seq = unit / n_layers;
  int n = n_cand[seq];
  if (n > n_cap) {
    n = n_cap;
    if (threadIdx.x == 0 && blockIdx.x == 0 && g == 0) set_status(status, ACTQKV_DEV_NCAND_CLAMPED);
  }
  const int b_lo = blockIdx.x * kBlocksPerCta;
  if (b_lo >= n) return;
  const int b_hi = min(n, b_lo + kBlocksPerCta);
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

  // probe and its norm
  const float* pg = probe_kv + (size_t(unit) * n_kv_heads + g) * D;
  float sq = 0.f;
  if (tid < D) {
    const float v = pg[tid];
    probe_s[tid] = v;
    sq = v * v;
  }
  sq = warp_sum(sq);
  if (lane == 0) red_s[warp] = sq;
  __syncthreads();
  float pn2 = 0.f;
  for (int i = 0; i < kScoreThreads / 32; ++i) pn2 += red_s[i];
  const bool bad = !(pn2 > 0.f) || !isfinite(pn2);
  if (bad && tid == 0 && blockIdx.x == 0) set_status(status, ACTQKV_DEV_BAD_PROBE);
  const float inv_pn = bad ? 0.f : rsqrtf(pn2);

  constexpr int VN = Vec16<T>::N;
  const int lpr = D / VN;               // lanes per row: 8, 16 or 32
  const int rows_per_pass = 32 / lpr;
  const int sub = lane / lpr, lir = lane - sub * lpr;
  float pv[VN];
#pragma unroll
  for (int i = 0; i < VN; ++i) pv[i] = probe_s[lir * VN + i];

  const size_t head_rows = (size_t(unit) * n_kv_heads + g) * size_t(n_cap) * r;
  const T* tab = repr_k + head_rows * D;
  const float* inv = repr_inv_norm + head_rows;
  float* out = scores + (size_t(unit) * n_kv_heads + g) * n_cap;

  for (int b = b_lo + warp; b < b_hi; b += kScoreThreads / 32) {
    float agg = agg_mode == ACTQKV_AGG_MAX ? -INFINITY : 0.f;
    for (int i0 = 0; i0 < r; i0 += rows_per_pass) {
      const int i = i0 + sub;
      float dot = 0.f;
      if (i < r) {
        float kv[VN];
        Vec16<T>::load_nc(tab + (size_t(b) * r + i) * D + lir * VN, kv);
#pragma unroll
        for (int e = 0; e < VN; ++e) dot = fmaf(pv[e], kv[e], dot);
      }
      for (int o = lpr >> 1; o > 0; o >>= 1) dot += __shfl_xor_sync(0xffffffffu, dot, o);
      const float cosv = i < r ? dot * inv_pn * __ldg(inv + size_t(b) * r + i) : 0.f;
      // combine the row groups of this pass (group leaders hold the cosines)
      for (int s = 0; s < rows_per_pass; ++s) {
        const float cv = __shfl_sync(0xffffffffu, cosv, s * lpr);
        if (i0 + s < r) agg = agg_mode == ACTQKV_AGG_MAX ? fmaxf(agg, cv) : agg + cv;
      }
    }
    if (lane == 0) out[b] = agg_mode == ACTQKV_AGG_MAX ? agg : agg / float(r);
  }
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
