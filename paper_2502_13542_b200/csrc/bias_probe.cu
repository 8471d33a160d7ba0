// Steps 1 and 2: Activation Bias (Eq. 7, statistics Eq. 8) and the activation-aware
// probe-query (Eq. 9).
//
// One CTA per (unit, query head).  The head's [n_tokens x D] query tile is read from HBM
// once into shared memory (rows of D elements, 16-byte loads); the window's per-channel
// mean and sum of squared deviations are taken two-pass from shared memory and merged
// into the running statistics, so Eq. 8 over all windows costs one HBM pass per window.
// The G CTAs of one KV head form a thread-block cluster; rank 0 averages the G probes
// through distributed shared memory in a fixed order (bitwise reproducible).
#include <cooperative_groups.h>

#include "common.cuh"

namespace cg = cooperative_groups;
using namespace actqkv;

namespace {

constexpr int kThreads = 512;

struct BiasProbeParams {
  const void* q;
  int n_tokens, n_q_heads, n_kv_heads, head_dim, group;
  int64_t* stats_count;
  float* stats_mean;
  float* stats_m2;
  float* phi_l1;
  float* phi_full;
  float* probe_qh;
  float* probe_kv;
  float var_eps;
  int stats_mode;
  int do_bias;    // compute statistics + phi (else phi_l1 is an input)
  int do_probe;   // compute probes
  int32_t* status;
};

__device__ __forceinline__ float block_sum(float v, float* scratch) {
  v = warp_sum(v);
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  __syncthreads();
  if (lane == 0) scratch[warp] = v;
  __syncthreads();
  float t = 0.f;
  for (int i = 0; i < kThreads / 32; ++i) t += scratch[i];   // same order in every thread
  return t;
}

template <typename T, bool kCluster>
__global__ void __launch_bounds__(kThreads) bias_probe_kernel(BiasProbeParams p) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  const int D = p.head_dim, W = p.n_tokens;
  T* tile = reinterpret_cast<T*>(smem_raw);
  float* fbase = reinterpret_cast<float*>(smem_raw + ((size_t(W) * D * sizeof(T) + 15) & ~size_t(15)));
  const int R = kThreads / D;                 // row groups for column passes
  float* partial = fbase;                     // [R][D]
  float* mean_s = partial + R * D;            // [D]
  float* ivar_s = mean_s + D;                 // [D]
  float* probe_s = ivar_s + D;                // [D]
  float* red_s = probe_s + D;                 // [32]
  float* a_s = red_s + 32;                    // [W]

  const int h = blockIdx.x, unit = blockIdx.y;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const T* qbase = reinterpret_cast<const T*>(p.q) + (size_t(unit) * W * p.n_q_heads + h) * D;
  const size_t row_stride = size_t(p.n_q_heads) * D;
  constexpr int VN = Vec16<T>::N;
  const int vec_per_row = D / VN;

  // ---- 1. tile -> shared memory, one HBM pass
  for (int idx = tid; idx < W * vec_per_row; idx += kThreads) {
    const int row = idx / vec_per_row, cv = idx - row * vec_per_row;
    const uint4 v = __ldg(reinterpret_cast<const uint4*>(qbase + row * row_stride + cv * VN));
    *reinterpret_cast<uint4*>(tile + size_t(row) * D + cv * VN) = v;
  }
  __syncthreads();

  const int c = tid % D, rg = tid / D;
  const size_t hd = (size_t(unit) * p.n_q_heads + h) * D;

  if (p.do_bias) {
    // ---- 2. window mean and M2 per channel (two passes over shared memory)
    float s = 0.f;
    for (int r = rg; r < W; r += R) s += to_f32(tile[size_t(r) * D + c]);
    partial[rg * D + c] = s;
    __syncthreads();
    float wmean = 0.f;
    if (tid < D) {
      for (int i = 0; i < R; ++i) wmean += partial[i * D + tid];
      wmean /= float(W);
      mean_s[tid] = wmean;
    }
    __syncthreads();
    const float mc = mean_s[c];
    s = 0.f;
    for (int r = rg; r < W; r += R) {
      const float d = to_f32(tile[size_t(r) * D + c]) - mc;
      s = fmaf(d, d, s);
    }
    __syncthreads();
    partial[rg * D + c] = s;
    __syncthreads();
    // ---- 3. merge into the running statistics (Eq. 8 over all windows so far)
    if (tid < D) {
      double m2w = 0.0;
      for (int i = 0; i < R; ++i) m2w += double(partial[i * D + tid]);
      double mean = double(mean_s[tid]), m2 = m2w, n = double(W);
      if (p.stats_mode == ACTQKV_STATS_CUMULATIVE) {
        const double na = double(p.stats_count[size_t(unit) * p.n_q_heads + h]);
        const double mean_a = double(p.stats_mean[hd + tid]), m2_a = double(p.stats_m2[hd + tid]);
        n = na + double(W);
        const double delta = mean - mean_a;
        mean = mean_a + delta * (double(W) / n);
        m2 = m2_a + m2w + delta * delta * (na * double(W) / n);
        p.stats_mean[hd + tid] = float(mean);
        p.stats_m2[hd + tid] = float(m2);
      }
      const double var = n > 1.0 ? m2 / (n - 1.0) : 0.0;
      mean_s[tid] = float(mean);
      ivar_s[tid] = float(1.0 / fmax(var, double(p.var_eps)));
    }
    __syncthreads();
    if (tid == 0 && p.stats_mode == ACTQKV_STATS_CUMULATIVE)
      p.stats_count[size_t(unit) * p.n_q_heads + h] += W;
    // ---- 4. phi and its L1 norm per token: one warp per row
    for (int r = warp; r < W; r += kThreads / 32) {
      float acc = 0.f;
      for (int cc = lane; cc < D; cc += 32) {
        const float d = to_f32(tile[size_t(r) * D + cc]) - mean_s[cc];
        const float ph = d * d * ivar_s[cc];
        acc += ph;
        if (p.phi_full) p.phi_full[(size_t(unit) * W + r) * row_stride + size_t(h) * D + cc] = ph;
      }
      acc = warp_sum(acc);
      if (lane == 0) {
        a_s[r] = acc;
        if (p.phi_l1) p.phi_l1[(size_t(unit) * p.n_q_heads + h) * W + r] = acc;
      }
    }
  } else {
    for (int r = tid; r < W; r += kThreads) a_s[r] = p.phi_l1[(size_t(unit) * p.n_q_heads + h) * W + r];
  }
  __syncthreads();
  if (!p.do_probe) return;

  // ---- 5. weights ||phi_j||_1 / ||Phi||_1
  float part = 0.f;
  for (int r = tid; r < W; r += kThreads) part += a_s[r];
  const float total = block_sum(part, red_s);
  const bool uniform = !(total > 0.f);
  const float inv_total = uniform ? 0.f : 1.f / total;
  const float wu = 1.f / float(W);
  // ---- 6. probe = sum_j w_j q_j, column pass
  float s = 0.f;
  for (int r = rg; r < W; r += R) {
    const float w = uniform ? wu : a_s[r] * inv_total;
    s = fmaf(w, to_f32(tile[size_t(r) * D + c]), s);
  }
  __syncthreads();
  partial[rg * D + c] = s;
  __syncthreads();
  if (tid < D) {
    float pr = 0.f;
    for (int i = 0; i < R; ++i) pr += partial[i * D + tid];
    probe_s[tid] = pr;
    p.probe_qh[hd + tid] = pr;
  }
  // ---- 7. KV-head probe: mean over the G query heads of the group, via DSMEM
  if constexpr (kCluster) {
    cg::cluster_group cluster = cg::this_cluster();
    cluster.sync();
    if (cluster.block_rank() == 0 && tid < D) {
      float acc = 0.f;
      for (int r = 0; r < p.group; ++r) acc += cluster.map_shared_rank(probe_s, r)[tid];
      const int g = h / p.group;
      p.probe_kv[(size_t(unit) * p.n_kv_heads + g) * D + tid] = acc / float(p.group);
    }
    cluster.sync();
  }
}

// G = 1 (or no cluster): KV probe is the query-head probe.
__global__ void copy_probe_kernel(const float* src, float* dst, size_t n) {
  size_t i = blockIdx.x * size_t(blockDim.x) + threadIdx.x;
  if (i < n) dst[i] = src[i];
}

template <typename T>
int launch(const actqkv_config* cfg, const Batch& b, BiasProbeParams& p, cudaStream_t st) {
  const int D = cfg->head_dim, W = p.n_tokens;
  const size_t tile_bytes = (size_t(W) * D * sizeof(T) + 15) & ~size_t(15);
  const size_t smem = tile_bytes + sizeof(float) * (size_t(kThreads / D) * D + 3 * D + 32 + W);
  if (smem > 200 * 1024) return ACTQKV_ERR_SHAPE;
  const bool cluster = p.do_probe && p.group > 1;
  auto kern = cluster ? bias_probe_kernel<T, true> : bias_probe_kernel<T, false>;
  if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem)) != cudaSuccess)
    return ACTQKV_ERR_LAUNCH;
  cudaLaunchConfig_t lc = {};
  lc.gridDim = dim3(cfg->n_q_heads, b.units(), 1);
  lc.blockDim = dim3(kThreads, 1, 1);
  lc.dynamicSmemBytes = smem;
  lc.stream = st;
  cudaLaunchAttribute attr[1];
  if (cluster) {
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = p.group;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    lc.attrs = attr;
    lc.numAttrs = 1;
  }
  if (cudaLaunchKernelEx(&lc, kern, p) != cudaSuccess) return ACTQKV_ERR_LAUNCH;
  if (p.do_probe && p.group == 1) {
    const size_t n = size_t(b.units()) * cfg->n_q_heads * D;
    copy_probe_kernel<<<unsigned((n + 255) / 256), 256, 0, st>>>(p.probe_qh, p.probe_kv, n);
  }
  return launch_status();
}

int run(const actqkv_config* cfg, const actqkv_batch* batch, BiasProbeParams& p, void* stream) {
  const Batch b = get_batch(batch);
  int rc = check_config(cfg, b);
  if (rc) return rc;
  if (p.n_tokens <= 0 || p.n_tokens > cfg->window) return ACTQKV_ERR_SHAPE;
  p.n_q_heads = cfg->n_q_heads;
  p.n_kv_heads = cfg->n_kv_heads;
  p.head_dim = cfg->head_dim;
  p.group = cfg->n_q_heads / cfg->n_kv_heads;
  p.var_eps = cfg->var_eps > 0.f ? cfg->var_eps : 1e-12f;
  p.stats_mode = cfg->stats_mode;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  return cfg->dtype == ACTQKV_BF16 ? launch<__nv_bfloat16>(cfg, b, p, st) : launch<float>(cfg, b, p, st);
}

}  // namespace

extern "C" int actqkv_activation_bias(const actqkv_config* cfg, const actqkv_batch* batch, const void* q,
                                      int32_t n_tokens, int64_t* stats_count, float* stats_mean,
                                      float* stats_m2, float* phi_l1, float* phi_full, int32_t* status,
                                      void* stream) {
  if (!cfg) return ACTQKV_ERR_NULL;
  ACTQKV_REQUIRE_PTR(q);
  ACTQKV_REQUIRE_PTR(phi_l1);
  ACTQKV_OPTIONAL_PTR(phi_full);
  if (cfg->stats_mode == ACTQKV_STATS_CUMULATIVE) {
    if (!stats_count) return ACTQKV_ERR_NULL;
    ACTQKV_REQUIRE_PTR(stats_mean);
    ACTQKV_REQUIRE_PTR(stats_m2);
  }
  BiasProbeParams p = {};
  p.q = q; p.n_tokens = n_tokens;
  p.stats_count = stats_count; p.stats_mean = stats_mean; p.stats_m2 = stats_m2;
  p.phi_l1 = phi_l1; p.phi_full = phi_full;
  p.do_bias = 1; p.do_probe = 0; p.status = status;
  return run(cfg, batch, p, stream);
}

extern "C" int actqkv_probe_query(const actqkv_config* cfg, const actqkv_batch* batch, const void* q,
                                  int32_t n_tokens, const float* phi_l1, float* probe_qh, float* probe_kv,
                                  int32_t* status, void* stream) {
  if (!cfg) return ACTQKV_ERR_NULL;
  ACTQKV_REQUIRE_PTR(q);
  ACTQKV_REQUIRE_PTR(phi_l1);
  ACTQKV_REQUIRE_PTR(probe_qh);
  ACTQKV_REQUIRE_PTR(probe_kv);
  BiasProbeParams p = {};
  p.q = q; p.n_tokens = n_tokens;
  p.phi_l1 = const_cast<float*>(phi_l1);
  p.probe_qh = probe_qh; p.probe_kv = probe_kv;
  p.do_bias = 0; p.do_probe = 1; p.status = status;
  return run(cfg, batch, p, stream);
}

extern "C" int actqkv_bias_probe(const actqkv_config* cfg, const actqkv_batch* batch, const void* q,
                                 int32_t n_tokens, int64_t* stats_count, float* stats_mean, float* stats_m2,
                                 float* phi_l1, float* phi_full, float* probe_qh, float* probe_kv,
                                 int32_t* status, void* stream) {
  if (!cfg) return ACTQKV_ERR_NULL;
  ACTQKV_REQUIRE_PTR(q);
  ACTQKV_OPTIONAL_PTR(phi_l1);
  ACTQKV_OPTIONAL_PTR(phi_full);
  ACTQKV_REQUIRE_PTR(probe_qh);
  ACTQKV_REQUIRE_PTR(probe_kv);
  if (cfg->stats_mode == ACTQKV_STATS_CUMULATIVE) {
    if (!stats_count) return ACTQKV_ERR_NULL;
    ACTQKV_REQUIRE_PTR(stats_mean);
    ACTQKV_REQUIRE_PTR(stats_m2);
  }
  BiasProbeParams p = {};
  p.q = q; p.n_tokens = n_tokens;
  p.stats_count = stats_count; p.stats_mean = stats_mean; p.stats_m2 = stats_m2;
  p.phi_l1 = phi_l1; p.phi_full = phi_full;
  p.probe_qh = probe_qh; p.probe_kv = probe_kv;
  p.do_bias = 1; p.do_probe = 1; p.status = status;
  return run(cfg, batch, p, stream);
}
