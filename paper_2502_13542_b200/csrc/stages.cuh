// Internal launchers shared between translation units of the library.
#pragma once
#include "common.cuh"

namespace actqkv {

// Eq. 11 for one head, by one warp: theta = ln Z - sum_i e_i x_i / Z with
// x_i = beta * s_i - max, e_i = exp(x_i), Z = sum_i e_i.  All lanes return theta.
__device__ __forceinline__ float warp_entropy(const float* __restrict__ s, int n, float beta) {
  if (n <= 0) return 0.f;
  const int lane = threadIdx.x & 31;
  float m = -INFINITY;
  for (int i = lane; i < n; i += 32) m = fmaxf(m, beta * s[i]);
  m = warp_max(m);
  float z = 0.f, ex = 0.f;
  for (int i = lane; i < n; i += 32) {
    const float x = beta * s[i] - m;
    const float e = expf(x);
    z += e;
    ex = fmaf(e, x, ex);
  }
  z = warp_sum(z);
  ex = warp_sum(ex);
  return fmaxf(logf(z) - ex / z, 0.f);
}

// Eq. 11 for one head by a whole CTA of kCtaThreads threads: the same quantities as warp_entropy,
// partial sums per thread, then per warp, then over the warps in a fixed order.  Every thread
// returns theta.  red: 3 * (kCtaThreads / 32) floats of shared memory; contains a CTA barrier.
template <int kCtaThreads>
__device__ __forceinline__ float block_entropy(const float* sc, int n, float beta, float* red) {
  constexpr int NW = kCtaThreads / 32;
  if (n <= 0) return 0.f;                       // uniform over the CTA
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  float m = -INFINITY;
  for (int i = tid; i < n; i += kCtaThreads) m = fmaxf(m, beta * sc[i]);
  m = warp_max(m);
  if (lane == 0) red[warp] = m;
  __syncthreads();
#pragma unroll
  for (int w = 0; w < NW; ++w) m = fmaxf(m, red[w]);
  float z = 0.f, ex = 0.f;
  for (int i = tid; i < n; i += kCtaThreads) {
    const float x = beta * sc[i] - m;
    const float e = expf(x);
    z += e;
    ex = fmaf(e, x, ex);
  }
  z = warp_sum(z);
  ex = warp_sum(ex);
  if (lane == 0) { red[NW + warp] = z; red[2 * NW + warp] = ex; }
  __syncthreads();
  z = 0.f; ex = 0.f;
#pragma unroll
  for (int w = 0; w < NW; ++w) { z += red[NW + w]; ex += red[2 * NW + w]; }
  return fmaxf(logf(z) - ex / z, 0.f);
}

int launch_scores(const actqkv_config* cfg, const Batch& b, const float* probe_kv, const void* repr_k,
                  const float* repr_inv_norm, const int32_t* n_cand, float* scores, int32_t* status,
                  cudaStream_t st);

// Eq. 11 for every (unit, KV head), one CTA each.
int launch_entropy(const actqkv_config* cfg, const Batch& b, const float* scores, const int32_t* n_cand,
                   float* theta, cudaStream_t st);

// Retrieval attention kernels: the general fp32-accumulate kernel and the tcgen05 kernel.
struct AttnArgs {
  const void *q, *k_win, *v_win, *k_pages, *v_pages;
  const int32_t* page_table;
  const int64_t* pos0;
  const int32_t *sel_idx, *sel_count;
  void* out;
  float* lse;
  int32_t* status;
  int n_tokens;
};
int launch_attention_simt(const actqkv_config* cfg, const Batch& b, const AttnArgs& a, cudaStream_t st);
bool attention_tc_supported(const actqkv_config* cfg, int n_tokens);
int launch_attention_tc(const actqkv_config* cfg, const Batch& b, const AttnArgs& a, cudaStream_t st);
// The same kernel for pairs of CTAs sharing each K / V tile (needs an even number of query heads per KV head).
bool attention_tc2_supported(const actqkv_config* cfg, int n_tokens);
int launch_attention_tc2(const actqkv_config* cfg, const Batch& b, const AttnArgs& a, cudaStream_t st);
// Four query heads of a KV group per CTA pair, the key stream split over the two pairs of a 4-CTA
// cluster (needs a multiple of 4 query heads per KV head).  Not the default: see attention_tc4.cu.
bool attention_tc4_supported(const actqkv_config* cfg, int n_tokens);
int launch_attention_tc4(const actqkv_config* cfg, const Batch& b, const AttnArgs& a, cudaStream_t st);

// Short steps (decode): one CTA per (unit, KV head, split of the key stream), G query heads packed
// in the M tile; n_splits > 1 needs a workspace of attention_decode_workspace_bytes().
bool attention_decode_supported(const actqkv_config* cfg, int n_tokens);
int attention_decode_auto_splits(const actqkv_config* cfg, const Batch& b);
int64_t attention_decode_workspace_bytes(const actqkv_config* cfg, const Batch& b, int n_tokens, int n_splits);
int launch_attention_decode(const actqkv_config* cfg, const Batch& b, const AttnArgs& a, int n_splits,
                            void* workspace, cudaStream_t st);

}  // namespace actqkv
