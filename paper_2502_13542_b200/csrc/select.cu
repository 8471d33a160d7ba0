// Step 4: dynamic KV cut-off (Eq. 12) and top-c block selection (Algorithm 1, last loop).
//
// No host round trip.  A call that batches several layers runs two kernels:
//   cutoff_chain_kernel  one CTA per sequence.  Warps evaluate (or read) the per-head
//                        information densities of every batched layer, then one thread walks
//                        the layers shallow -> deep in fp64: B^l from Eq. 12, the granted
//                        integer c^l, the running B_kv and the density history.
//   select_kernel        one CTA per (unit, KV head).  Scores become order-preserving 32-bit
//                        keys in shared memory; an MSB-first 8-bit radix select finds the c-th
//                        largest key; equal keys are admitted lowest index first; the survivors
//                        are compacted in ascending block order with block-wide scans.
// A call for one layer (the usual layer-by-layer use) runs select_kernel alone: the Hkv CTAs of a
// sequence form a thread-block cluster, each takes its head's density, they exchange the values
// through distributed shared memory, every CTA evaluates Eq. 12 for itself and the first one
// writes the budget state back.
#include <cooperative_groups.h>

#include "common.cuh"
#include "stages.cuh"

namespace cg = cooperative_groups;

using namespace actqkv;

namespace {

constexpr int kChainThreads = 1024;
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

// Eq. 12 for one layer with n > 0 candidates: returns the granted count c and the un-rounded
// budget; `rest` = sum over the deeper layers of their mean density (theta-bar).
struct Grant { int c; double real; };
__device__ __forceinline__ Grant grant_layer(double th, double rest, double b_rem, int layers_left, int n, int cap) {
  Grant gr;
  const double den = th + rest;
  gr.real = den > 0.0 ? th / den * b_rem : b_rem / double(layers_left);
  const double fl = floor(gr.real + 0.5);
  int c = fl > 2.0e9 ? 2000000000 : (fl < -2.0e9 ? -2000000000 : int(fl));
  gr.c = max(min(1, n), min(c, min(cap, n)));
  return gr;
}

__global__ void __launch_bounds__(kChainThreads) cutoff_chain_kernel(ChainParams p) {
  extern __shared__ float theta_h[];   // [Lb][Hkv]
  const int seq = blockIdx.x;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  grid_launch_dependents();
  grid_dependency_wait();            // scores / densities come from the stream's previous kernels
  const int n = min(p.n_cand[seq], p.n_cap);
  if (p.theta_in) {                  // one load per thread, all in flight together
    const float* src = p.theta_in + size_t(seq) * p.Lb * p.n_kv_heads;
    for (int pair = threadIdx.x; pair < p.Lb * p.n_kv_heads; pair += kChainThreads) theta_h[pair] = src[pair];
  } else {
    for (int pair = warp; pair < p.Lb * p.n_kv_heads; pair += kChainThreads / 32) {
      const size_t uh = size_t(seq) * p.Lb * p.n_kv_heads + pair;
      const float th = warp_entropy(p.scores + uh * p.n_cap, n, p.beta);
      if (lane == 0) {
        if (p.theta_out) p.theta_out[uh] = th;
        theta_h[pair] = th;
      }
    }
  }
  __syncthreads();

  // Shared work arrays after the densities: doubles [Lb] th, [L + 1] suffix of known theta-bars,
  // [L + 1] suffix count of layers without one, [Lb] ratio.
  double* th_l = reinterpret_cast<double*>(theta_h + ((p.Lb * p.n_kv_heads + 1) & ~1));
  double* suf_known = th_l + p.Lb;
  double* suf_open = suf_known + p.L + 1;
  double* ratio = suf_open + p.L + 1;
  double* st = p.state + size_t(seq) * (1 + 2 * p.L);
  double* hist_sum = st + 1;
  double* hist_cnt = st + 1 + p.L;
  const int tid = threadIdx.x;
  // ---- in parallel: each batched layer's density (mean over its KV heads, fixed order)
  if (tid < p.Lb) {
    double s = 0.0;
    for (int g = 0; g < p.n_kv_heads; ++g) s += double(theta_h[tid * p.n_kv_heads + g]);
    th_l[tid] = s / double(p.n_kv_heads);
  }
  __syncthreads();
  // ---- in parallel: theta-bar of every model layer that has one (its history mean, or this call's
  // own density in the Algorithm-1 reading); the others will take the current layer's density
  if (tid < p.L) {
    double known = 0.0, open = 0.0;
    if (p.thetabar_mode == ACTQKV_THETABAR_ALG1) known = th_l[tid - p.layer0];
    else if (hist_cnt[tid] > 0.0) known = hist_sum[tid] / hist_cnt[tid];
    else open = 1.0;
    suf_known[tid] = known;          // turned into suffix sums below
    suf_open[tid] = open;
  }
  __syncthreads();
  if (tid < 2) {                     // suffix[j] = sum over layers >= j (additions only, running sum in a register)
    double* suf = tid == 0 ? suf_known : suf_open;
    double run = 0.0;
    suf[p.L] = 0.0;
    for (int j = p.L - 1; j >= 0; --j) {
      run += suf[j];
      suf[j] = run;
    }
  }
  __syncthreads();
  // ---- in parallel: the share theta / (theta + sum of deeper theta-bars) of Eq. 12, which does
  // not depend on the running budget
  if (tid < p.Lb) {
    const int layer = p.layer0 + tid;
    const double th = th_l[tid];
    const double den = th + suf_known[layer + 1] + suf_open[layer + 1] * th;
    ratio[tid] = den > 0.0 ? th / den : -1.0;
  }
  __syncthreads();
  // ---- serial: the budget walks the layers shallow -> deep
  if (tid == 0) {
    double b_rem = st[0];
    const double lo_d = double(min(1, n)), hi_d = double(min(p.cap_blocks, n));
    for (int l = 0; l < p.Lb; ++l) {
      const int layer = p.layer0 + l;
      if (layer == 0) b_rem = double(p.L) * double(p.k_blocks);
      int c = 0;
      double real = 0.0;
      if (n > 0) {
        // The count stays a double on the path from one layer's budget to the next (the clamp
        // bounds are small integers, so clamping the double and converting gives the same count
        // as converting and clamping; a NaN budget counts as 0 before the clamp, as a conversion
        // to int would make it); the integer for the store is taken off that path.
        real = ratio[l] >= 0.0 ? ratio[l] * b_rem : b_rem / double(p.L - layer);
        const double fl = floor(real + 0.5);
        const double cd = fmax(lo_d, fmin(fl == fl ? fl : 0.0, hi_d));
        b_rem -= cd;
        c = int(cd);
      }
      const size_t unit = size_t(seq) * p.Lb + l;
      p.sel_count[unit] = c;
      if (p.budget_real) p.budget_real[unit] = float(real);
    }
    st[0] = b_rem;
  }
  if (tid < p.Lb && n > 0) {         // density history of the layers of this call
    hist_sum[p.layer0 + tid] += th_l[tid];
    hist_cnt[p.layer0 + tid] += 1.0;
  }
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

// Up to kSelThreads candidates, one per thread: the number of candidates that come before this
// thread's in the order of the selection (higher key first, equal keys by lower index).  Every
// thread counts the keys greater than its own against all of them, four per shared-memory load;
// candidates with equal keys get equal counts, which a histogram of the counts detects, and only
// those threads then add the number of their equals with a lower index.  Contains CTA barriers;
// threads past n return n.
__device__ __forceinline__ int rank_of_candidate(const float* sc, int n, uint32_t* key_s, int* rank_s, int* cnt_s) {
  const int tid = threadIdx.x;
  const uint32_t mine = tid < n ? score_key(sc[tid]) : 0u;
  key_s[tid] = mine;                            // the padding is the lowest key: never greater
  cnt_s[tid] = 0;
  __syncthreads();
  const uint4* k4 = reinterpret_cast<const uint4*>(key_s);
  const int n4 = (n + 3) >> 2;
  int r0 = 0, r1 = 0, r2 = 0, r3 = 0;
  auto count4 = [&](const uint4& v) { r0 += v.x > mine; r1 += v.y > mine; r2 += v.z > mine; r3 += v.w > mine; };
  int q = 0;
  for (; q + 4 <= n4; q += 4) {                 // four loads in flight before the first compare
    const uint4 a = k4[q], b = k4[q + 1], c = k4[q + 2], d = k4[q + 3];
    count4(a); count4(b); count4(c); count4(d);
  }
  for (; q < n4; ++q) count4(k4[q]);
  int r = (r0 + r1) + (r2 + r3);
  if (tid >= n) r = n;
  rank_s[tid] = r;
  if (tid < n) atomicAdd(&cnt_s[r], 1);
  __syncthreads();
  if (tid < n && cnt_s[r] > 1) {
    int before = 0;
    for (int j = 0; j < tid; ++j) before += rank_s[j] == r;
    r += before;
  }
  return r;
}

// kFused: the call holds one layer; the grid is launched as clusters of n_kv_heads CTAs (one
// sequence each) and the cut-off chain of that layer is evaluated here (ch), else sel_count is
// an input written by cutoff_chain_kernel.
template <bool kFused>
__global__ void __launch_bounds__(kSelThreads)
select_kernel(const float* __restrict__ scores, const int32_t* __restrict__ n_cand,
              int32_t* __restrict__ sel_count, int32_t* __restrict__ sel_idx, int n_kv_heads,
              int n_cap, int cap_blocks, int n_layers, int32_t* status, ChainParams ch) {
  extern __shared__ uint32_t sel_smem[];       // the head's scores [n_cap] (fp32), then their keys [n_cap]
  float* sc = reinterpret_cast<float*>(sel_smem);
  uint32_t* keys = sel_smem + n_cap;
  __shared__ __align__(16) uint32_t key_s[kSelThreads];
  __shared__ int rank_s[kSelThreads];
  __shared__ int hist[256];
  __shared__ int warp_tot[kSelThreads / 32];
  __shared__ uint32_t sh_prefix;
  __shared__ int sh_need;
  __shared__ float sh_thetas[8];               // the densities of the cluster's heads (written by their CTAs)
  __shared__ float red_f[3 * (kSelThreads / 32)];
  __shared__ int sh_count;
  __shared__ double sh_brem, sh_rest;
  __shared__ int sh_no_hist;
  const int g = blockIdx.x, unit = blockIdx.y, tid = threadIdx.x;
  grid_launch_dependents();
  grid_dependency_wait();            // scores / densities / counts come from the stream's previous kernels
  const int n = min(n_cand[unit / n_layers], n_cap);
  const float* s = scores + (size_t(unit) * n_kv_heads + g) * n_cap;
  // the scores are fetched once, by all threads at a time; density and selection read them from here
  for (int i = tid; i < n; i += kSelThreads) sc[i] = s[i];
  const bool small = n <= kSelThreads;      // one candidate per thread: ranked by counting
  int rank = 0;
  int c;
  if constexpr (kFused) {
    cg::cluster_group cluster = cg::this_cluster();
    const int seq = unit;                      // one layer per call: unit == sequence
    const int layer = ch.layer0;
    double* st = ch.state + size_t(seq) * (1 + 2 * ch.L);
    // The old state is read by every CTA before the cluster barrier, written by CTA 0 after it.
    // Warp 1 adds up the mean densities of the deeper layers that have a history (a lane per
    // layer, then a butterfly over the lanes) while the scores arrive.
    if (tid >= 32 && tid < 64) {
      const int lane = tid - 32;
      double part = 0.0;
      int none = 0;
      for (int j = layer + 1 + lane; j < ch.L; j += 32) {
        const double cnt = st[1 + ch.L + j];
        if (cnt > 0.0) part += st[1 + j] / cnt; else ++none;
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        part += __shfl_xor_sync(0xffffffffu, part, o);
        none += __shfl_xor_sync(0xffffffffu, none, o);
      }
      if (lane == 0) {
        sh_brem = layer == 0 ? double(ch.L) * double(ch.k_blocks) : st[0];
        sh_rest = part;
        sh_no_hist = none;
      }
    }
    __syncthreads();
    // this head's density, by the whole CTA; handed to every CTA of the cluster (one per KV head)
    // by remote stores ahead of the cluster barrier, so that nobody reads a peer's memory after it
    // and no CTA has to wait for its peers before it leaves
    {
      const size_t uh = size_t(unit) * n_kv_heads + g;
      const float th = ch.theta_in ? ch.theta_in[uh] : block_entropy<kSelThreads>(sc, n, ch.beta, red_f);
      if (tid == 0 && !ch.theta_in && ch.theta_out) ch.theta_out[uh] = th;
      if (tid < n_kv_heads) cluster.map_shared_rank(sh_thetas, unsigned(tid))[g] = th;
    }
    // arrive, rank this thread's candidate while the barrier completes (the ranks do not depend on
    // the count), then wait
    asm volatile("barrier.cluster.arrive.release;" ::: "memory");
    if (small) rank = rank_of_candidate(sc, n, key_s, rank_s, hist);
    asm volatile("barrier.cluster.wait.acquire;" ::: "memory");
    if (tid == 0) {
      float th_h[8];
#pragma unroll
      for (int h2 = 0; h2 < 8; ++h2) th_h[h2] = h2 < n_kv_heads ? sh_thetas[h2] : 0.f;
      double sum = 0.0;
#pragma unroll
      for (int h2 = 0; h2 < 8; ++h2) sum += double(th_h[h2]);
      const double th = sum / double(n_kv_heads);
      const double b_rem = sh_brem, rest_hist = sh_rest;
      const int no_hist = sh_no_hist;
      Grant gr{0, 0.0};
      if (n > 0) {
        // layers without history count with this layer's density; with every layer in the call
        // (L == 1) there is no deeper layer and both theta-bar readings coincide
        const double rest = rest_hist + double(no_hist) * th;
        gr = grant_layer(th, rest, b_rem, ch.L - layer, n, ch.cap_blocks);
        if (g == 0) {
          st[0] = b_rem - double(gr.c);
          st[1 + layer] += th;
          st[1 + ch.L + layer] += 1.0;
        }
      } else if (g == 0) {
        st[0] = b_rem;
      }
      if (g == 0) {
        sel_count[unit] = gr.c;
        if (ch.budget_real) ch.budget_real[unit] = float(gr.real);
      }
      sh_count = gr.c;
    }
    __syncthreads();
    c = sh_count;
  } else {
    if (small) rank = rank_of_candidate(sc, n, key_s, rank_s, hist);
    c = sel_count[unit];
    if (c < 0 || c > min(cap_blocks, n)) {
      if (tid == 0) set_status(status, ACTQKV_DEV_BAD_SELECTION);
      c = max(0, min(c, min(cap_blocks, n)));
    }
  }
  int32_t* out = sel_idx + (size_t(unit) * n_kv_heads + g) * cap_blocks;
  for (int i = c + tid; i < cap_blocks; i += kSelThreads) out[i] = -1;
  if (c >= n) {
    for (int i = tid; i < min(n, c); i += kSelThreads) out[i] = i;
  } else if (c > 0 && small) {
    // the c first of the order are taken and compacted in ascending index order
    const int take = tid < n && rank < c;
    int tot;
    const int pos = block_exclusive_scan(take, warp_tot, &tot);
    if (take && pos < cap_blocks) out[pos] = tid;
  } else if (c > 0) {
    for (int i = tid; i < n; i += kSelThreads) keys[i] = score_key(sc[i]);
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
}

int launch_cutoff(const actqkv_config* cfg, const Batch& b, const float* scores, const float* theta_in,
                  float* theta_out, const int32_t* n_cand, void* budget_state, int32_t* sel_idx,
                  int32_t* sel_count, float* budget_real, int32_t* status, cudaStream_t st) {
  if (cfg->thetabar_mode == ACTQKV_THETABAR_ALG1 && (b.layer0 != 0 || b.n_layers != cfg->n_layers))
    return ACTQKV_ERR_UNSUPPORTED;
  if (size_t(cfg->n_cap) * 8 > 200 * 1024) return ACTQKV_ERR_SHAPE;
  ChainParams p;
  p.scores = scores; p.theta_in = theta_in; p.theta_out = theta_out; p.n_cand = n_cand;
  p.state = static_cast<double*>(budget_state);
  p.sel_count = sel_count; p.budget_real = budget_real;
  p.n_kv_heads = cfg->n_kv_heads; p.n_cap = cfg->n_cap; p.L = cfg->n_layers; p.Lb = b.n_layers;
  p.layer0 = b.layer0; p.k_blocks = cfg->k_blocks; p.cap_blocks = cfg->cap_blocks;
  p.thetabar_mode = cfg->thetabar_mode; p.beta = cfg->beta;
  const size_t sm_sel = size_t(cfg->n_cap) * 8;        // scores and keys
  const bool fused = b.n_layers == 1 && cfg->n_kv_heads <= 8 && cfg->cap_blocks > 0;
  auto kern = fused ? select_kernel<true> : select_kernel<false>;
  if (sm_sel > 40 * 1024 &&
      cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, int(sm_sel)) != cudaSuccess)
    return ACTQKV_ERR_LAUNCH;
  if (!fused) {
    const size_t sm_chain = sizeof(float) * ((size_t(b.n_layers) * cfg->n_kv_heads + 1) & ~size_t(1)) +
                            sizeof(double) * (2 * size_t(b.n_layers) + 2 * (size_t(cfg->n_layers) + 1));
    if (sm_chain > 48 * 1024) return ACTQKV_ERR_SHAPE;
    if (!p.theta_in && theta_out && b.n_layers * cfg->n_kv_heads >= 64) {
      // many (layer, head) densities: take them with one warp each in a kernel of their own
      const int rc = launch_entropy(cfg, b, scores, n_cand, theta_out, st);
      if (rc) return rc;
      p.theta_in = theta_out;
    }
    prefer_max_shared(cutoff_chain_kernel);
    cudaLaunchConfig_t lcc = {};
    lcc.gridDim = dim3(b.n_seq, 1, 1);
    lcc.blockDim = dim3(kChainThreads, 1, 1);
    lcc.dynamicSmemBytes = sm_chain;
    lcc.stream = st;
    cudaLaunchAttribute cattr[1];
    allow_early_launch(cattr[0]);
    lcc.attrs = cattr;
    lcc.numAttrs = 1;
    if (cudaLaunchKernelEx(&lcc, cutoff_chain_kernel, p) != cudaSuccess) return ACTQKV_ERR_LAUNCH;
    if (cfg->cap_blocks == 0) return ACTQKV_OK;
  }
  prefer_max_shared(kern);
  cudaLaunchConfig_t lc = {};
  lc.gridDim = dim3(cfg->n_kv_heads, b.units(), 1);
  lc.blockDim = dim3(kSelThreads, 1, 1);
  lc.dynamicSmemBytes = sm_sel;
  lc.stream = st;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = fused ? cfg->n_kv_heads : 1;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  allow_early_launch(attr[1]);
  lc.attrs = attr;
  lc.numAttrs = 2;                  // every kernel of the chain waits for its predecessor before it reads
  if (cudaLaunchKernelEx(&lc, kern, scores, n_cand, sel_count, sel_idx, cfg->n_kv_heads, cfg->n_cap,
                         cfg->cap_blocks, b.n_layers, status, p) != cudaSuccess)
    return ACTQKV_ERR_LAUNCH;
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
