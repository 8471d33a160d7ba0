// Step 4: dynamic KV cut-off (Eq. 12) and top-c block selection (Algorithm 1, last loop).
//
// Two kernels, no host round trip:
//   cutoff_chain_kernel  one CTA per sequence.  Warps evaluate (or read) the per-head
//                        information densities of every batched layer, then one thread walks
//                        the layers shallow -> deep in fp64: B^l from Eq. 12, the granted
//                        integer c^l, the running B_kv and the density history.
//   select_kernel        one CTA per (unit, KV head).  Scores become order-preserving 32-bit
//                        keys in shared memory; an MSB-first 8-bit radix select finds the c-th
//                        largest key; equal keys are admitted lowest index first; the survivors
//                        are compacted in ascending block order with block-wide scans.
#include "common.cuh"
#include "stages.cuh"

using namespace actqkv;

namespace {

constexpr int kChainThreads = 256;
constexpr int kSelThreads = 256;

struct ChainParams {
  const float* scores;
  const float* theta_in;   // NULL: compute from scores
  float* theta_out;        // written when computed here
  const int32_t* n_cand;
  double* state;
  int32_t* sel_count;
  float* budget_real;
  int n_kv_heads, n_cap, L, Lb, layer0, k_blocks, cap_blocks, thetabar_mode;
  float beta;
};

__global__ void __launch_bounds__(kChainThreads) cutoff_chain_kernel(ChainParams p) {
  extern __shared__ float theta_h[];   // [Lb][Hkv]
  const int seq = blockIdx.x;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int n = min(p.n_cand[seq], p.n_cap);
  for (int pair = warp; pair < p.Lb * p.n_kv_heads; pair += kChainThreads / 32) {
    const size_t uh = size_t(seq) * p.Lb * p.n_kv_heads + pair;
    float th;
    if (p.theta_in) {
      th = p.theta_in[uh];
    } else {
      th = warp_entropy(p.scores + uh * p.n_cap, n, p.beta);
      if (lane == 0 && p.theta_out) p.theta_out[uh] = th;
    }
    if (lane == 0) theta_h[pair] = th;
  }
  __syncthreads();
  if (threadIdx.x != 0) return;

  double* st = p.state + size_t(seq) * (1 + 2 * p.L);
  double* hist_sum = st + 1;
  double* hist_cnt = st + 1 + p.L;
  double b_rem = st[0];
  auto layer_theta = [&](int l) {
    double s = 0.0;
    for (int g = 0; g < p.n_kv_heads; ++g) s += double(theta_h[l * p.n_kv_heads + g]);
    return s / double(p.n_kv_heads);
  };
  for (int l = 0; l < p.Lb; ++l) {
    const int layer = p.layer0 + l;
    if (layer == 0) b_rem = double(p.L) * double(p.k_blocks);
    const double th = layer_theta(l);
    int c = 0;
    double real = 0.0;
    if (n > 0) {
      double rest = 0.0;
      for (int j = layer + 1; j < p.L; ++j) {
        if (p.thetabar_mode == ACTQKV_THETABAR_ALG1) {
          rest += layer_theta(j - p.layer0);
        } else if (hist_cnt[j] > 0.0) {
          rest += hist_sum[j] / hist_cnt[j];
        } else {
          rest += th;
        }
      }
      const double den = th + rest;
      real = den > 0.0 ? th / den * b_rem : b_rem / double(p.L - layer);
      const double fl = floor(real + 0.5);
      c = fl > 2.0e9 ? 2000000000 : (fl < -2.0e9 ? -2000000000 : int(fl));
      c = max(min(1, n), min(c, min(p.cap_blocks, n)));
      b_rem -= double(c);
      hist_sum[layer] += th;
      hist_cnt[layer] += 1.0;
    }
    const size_t unit = size_t(seq) * p.Lb + l;
    p.sel_count[unit] = c;
    if (p.budget_real) p.budget_real[unit] = float(real);
  }
  st[0] = b_rem;
}

// Order-preserving key: larger score <-> larger unsigned key; NaN lowest; -0 == +0.
__device__ __forceinline__ uint32_t score_key(float f) {
  if (f != f) return 0u;
  if (f == 0.f) f = 0.f;
  const uint32_t u = __float_as_uint(f);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

// Exclusive scan of one int per thread over the CTA; returns the prefix, total in *total.
__device__ __forceinline__ int block_exclusive_scan(int v, int* warp_tot, int* total) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  int inc = v;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int t = __shfl_up_sync(0xffffffffu, inc, o);
    if (lane >= o) inc += t;
  }
  __syncthreads();
  if (lane == 31) warp_tot[warp] = inc;
  __syncthreads();
  int base = 0, tot = 0;
  for (int w = 0; w < kSelThreads / 32; ++w) {
    const int t = warp_tot[w];
    if (w < warp) base += t;
    tot += t;
  }
  *total = tot;
  return base + inc - v;
}

__global__ void __launch_bounds__(kSelThreads)
select_kernel(const float* __restrict__ scores, const int32_t* __restrict__ n_cand,
              const int32_t* __restrict__ sel_count, int32_t* __restrict__ sel_idx, int n_kv_heads,
              int n_cap, int cap_blocks, int n_layers, int32_t* status) {
  extern __shared__ uint32_t keys[];           // [n_cap]
  __shared__ int hist[256];
  __shared__ int warp_tot[kSelThreads / 32];
  __shared__ uint32_t sh_prefix;
  __shared__ int sh_need;
  const int g = blockIdx.x, unit = blockIdx.y, tid = threadIdx.x;
  const int n = min(n_cand[unit / n_layers], n_cap);
  int c = sel_count[unit];
  if (c < 0 || c > min(cap_blocks, n)) {
    if (tid == 0) set_status(status, ACTQKV_DEV_BAD_SELECTION);
    c = max(0, min(c, min(cap_blocks, n)));
  }
  int32_t* out = sel_idx + (size_t(unit) * n_kv_heads + g) * cap_blocks;
  for (int i = c + tid; i < cap_blocks; i += kSelThreads) out[i] = -1;
  if (c == 0) return;
  if (c >= n) {
    for (int i = tid; i < n; i += kSelThreads) out[i] = i;
    return;
  }
  const float* s = scores + (size_t(unit) * n_kv_heads + g) * n_cap;
  for (int i = tid; i < n; i += kSelThreads) keys[i] = score_key(s[i]);
  if (tid == 0) { sh_prefix = 0u; sh_need = c; }
  __syncthreads();

  // ---- radix select of the c-th largest key
  uint32_t mask = 0u;
  for (int shift = 24; shift >= 0; shift -= 8) {
    hist[tid] = 0;                                        // kSelThreads == 256 bins
    __syncthreads();
    const uint32_t prefix = sh_prefix;
    for (int i = tid; i < n; i += kSelThreads) {
      const uint32_t k = keys[i];
      if ((k & mask) == prefix) atomicAdd(&hist[(k >> shift) & 255u], 1);
    }
    __syncthreads();
    if (tid < 32) {
      // lane l owns bins 255-8l .. 248-8l (descending)
      int loc[8], sum = 0;
#pragma unroll
      for (int j = 0; j < 8; ++j) { loc[j] = hist[255 - 8 * tid - j]; sum += loc[j]; }
      int inc = sum;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const int t = __shfl_up_sync(0xffffffffu, inc, o);
        if (tid >= o) inc += t;
      }
      int before = inc - sum;
      const int need = sh_need;
      if (before < need && need <= inc) {
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          if (before < need && need <= before + loc[j]) {
            sh_prefix = prefix | (uint32_t(255 - 8 * tid - j) << shift);
            sh_need = need - before;
            before = need;                                  // stop further matches
          } else {
            before += loc[j];
          }
        }
      }
    }
    mask |= 255u << shift;
    __syncthreads();
  }
  const uint32_t thr = sh_prefix;
  const int need_eq = sh_need;          // how many keys equal to thr are admitted (>= 1)

  // ---- admit equal keys lowest index first, compact ascending
  const int per = (n + kSelThreads - 1) / kSelThreads;
  const int i0 = min(n, tid * per), i1 = min(n, i0 + per);
  int eq = 0;
  for (int i = i0; i < i1; ++i) eq += keys[i] == thr;
  int tot;
  int eq_before = block_exclusive_scan(eq, warp_tot, &tot);
  int cnt = 0;
  {
    int e = eq_before;
    for (int i = i0; i < i1; ++i) {
      const uint32_t k = keys[i];
      if (k > thr) ++cnt;
      else if (k == thr) { if (e < need_eq) ++cnt; ++e; }
    }
  }
  int pos = block_exclusive_scan(cnt, warp_tot, &tot);
  {
    int e = eq_before;
    for (int i = i0; i < i1; ++i) {
      const uint32_t k = keys[i];
      bool take = k > thr;
      if (k == thr) { take = e < need_eq; ++e; }
      if (take && pos < cap_blocks) out[pos++] = i;
    }
  }
}

int launch_cutoff(const actqkv_config* cfg, const Batch& b, const float* scores, const float* theta_in,
                  float* theta_out, const int32_t* n_cand, void* budget_state, int32_t* sel_idx,
                  int32_t* sel_count, float* budget_real, int32_t* status, cudaStream_t st) {
  if (cfg->thetabar_mode == ACTQKV_THETABAR_ALG1 && (b.layer0 != 0 || b.n_layers != cfg->n_layers))
    return ACTQKV_ERR_UNSUPPORTED;
  if (size_t(cfg->n_cap) * 4 > 160 * 1024) return ACTQKV_ERR_SHAPE;
  ChainParams p;
  p.scores = scores; p.theta_in = theta_in; p.theta_out = theta_out; p.n_cand = n_cand;
  p.state = static_cast<double*>(budget_state);
  p.sel_count = sel_count; p.budget_real = budget_real;
  p.n_kv_heads = cfg->n_kv_heads; p.n_cap = cfg->n_cap; p.L = cfg->n_layers; p.Lb = b.n_layers;
  p.layer0 = b.layer0; p.k_blocks = cfg->k_blocks; p.cap_blocks = cfg->cap_blocks;
  p.thetabar_mode = cfg->thetabar_mode; p.beta = cfg->beta;
  const size_t sm_chain = sizeof(float) * size_t(b.n_layers) * cfg->n_kv_heads;
  if (sm_chain > 48 * 1024) return ACTQKV_ERR_SHAPE;
  cutoff_chain_kernel<<<b.n_seq, kChainThreads, sm_chain, st>>>(p);
  if (cudaGetLastError() != cudaSuccess) return ACTQKV_ERR_LAUNCH;
  if (cfg->cap_blocks == 0) return ACTQKV_OK;
  const size_t sm_sel = size_t(cfg->n_cap) * 4;
  if (sm_sel > 48 * 1024 &&
      cudaFuncSetAttribute(select_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, int(sm_sel)) != cudaSuccess)
    return ACTQKV_ERR_LAUNCH;
  select_kernel<<<dim3(cfg->n_kv_heads, b.units()), kSelThreads, sm_sel, st>>>(
      scores, n_cand, sel_count, sel_idx, cfg->n_kv_heads, cfg->n_cap, cfg->cap_blocks, b.n_layers, status);
  return launch_status();
}

}  // namespace

extern "C" int actqkv_select_cutoff(const actqkv_config* cfg, const actqkv_batch* batch, const float* scores,
                                    const float* theta, const int32_t* n_cand, void* budget_state,
                                    int32_t* sel_idx, int32_t* sel_count, float* budget_real,
                                    int32_t* status, void* stream) {
  const Batch b = get_batch(batch);
  int rc = check_config(cfg, b);
  if (rc) return rc;
  ACTQKV_REQUIRE_PTR(scores);
  if (!theta || !n_cand || !budget_state || !sel_count) return ACTQKV_ERR_NULL;
  ACTQKV_REQUIRE_PTR(sel_idx);
  return launch_cutoff(cfg, b, scores, theta, nullptr, n_cand, budget_state, sel_idx, sel_count,
                       budget_real, status, reinterpret_cast<cudaStream_t>(stream));
}

extern "C" int actqkv_score_select(const actqkv_config* cfg, const actqkv_batch* batch, const float* probe_kv,
                                   const void* repr_k, const float* repr_inv_norm, const int32_t* n_cand,
                                   void* budget_state, float* scores, float* theta, int32_t* sel_idx,
                                   int32_t* sel_count, float* budget_real, int32_t* status, void* stream) {
  const Batch b = get_batch(batch);
  int rc = check_config(cfg, b);
  if (rc) return rc;
  ACTQKV_REQUIRE_PTR(probe_kv);
  ACTQKV_REQUIRE_PTR(repr_k);
  ACTQKV_REQUIRE_PTR(repr_inv_norm);
  ACTQKV_REQUIRE_PTR(scores);
  ACTQKV_REQUIRE_PTR(sel_idx);
  if (!n_cand || !budget_state || !sel_count) return ACTQKV_ERR_NULL;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  rc = launch_scores(cfg, b, probe_kv, repr_k, repr_inv_norm, n_cand, scores, status, st);
  if (rc) return rc;
  return launch_cutoff(cfg, b, scores, nullptr, theta, n_cand, budget_state, sel_idx, sel_count,
                       budget_real, status, st);
}
