// Steps 1 and 2: Activation Bias (Eq. 7, statistics Eq. 8) and the activation-aware
// probe-query (Eq. 9).
//
// The [n_tokens x D] query tile of one (unit, query head) is split by rows over S CTAs, and the
// S x G CTAs of one KV head form a thread-block cluster (S * G <= 8).  Every CTA brings its rows from HBM into shared memory with one
// bulk asynchronous copy per row (all in flight at once) and makes three passes over them with
// 16-byte shared-memory loads:
//   1. per-channel sums of q and of (q - shift)^2, shift = the CTA's first row, which give
//      the mean and the sum of squared deviations of its rows without a second pass; the row
//      splits are merged pairwise (count, mean, M2) in a fixed order through distributed shared
//      memory and then merged into the running statistics (Eq. 8 over all windows so far);
//   2. phi and the per-token indicator ||phi_j||_1 (Eq. 7);
//   3. sum_j a_j q_j, combined with sum_j a_j by the group leaders in a fixed order (Eq. 9).
// Every reduction order is fixed, so results are bitwise reproducible.
#include <cooperative_groups.h>

#include "common.cuh"

namespace cg = cooperative_groups;
using namespace actqkv;

namespace {

constexpr int kThreads = 512;
constexpr int kMaxCluster = 8;
constexpr uint32_t kSpinLimit = 1u << 22;

struct BiasProbeParams {
  const void* q;
  int n_tokens, n_q_heads, n_kv_heads, head_dim, group;
  int split, rows_per_cta;
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

__device__ __forceinline__ uint32_t smem_addr(const void* p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

template <typename T, int D>
__global__ void __launch_bounds__(kThreads, 2) bias_probe_kernel(BiasProbeParams p) {   // 2 CTAs per SM on batched calls
  extern __shared__ __align__(128) unsigned char smem_raw[];
  cg::cluster_group cluster = cg::this_cluster();
  constexpr int VN = Vec16<T>::N;             // elements per 16-byte vector
  constexpr int VPR = D / VN;                 // vectors per row
  constexpr int RL = kThreads / VPR;          // row lanes: thread (cv, rsub) owns vector cv of rows rsub + k * RL
  constexpr int NP = kThreads / D;            // second-level slices of the row lanes
  constexpr int PER = RL / NP;
  const int W = p.n_tokens, S = p.split, RP = p.rows_per_cta;
  T* tile = reinterpret_cast<T*>(smem_raw);
  float* partial = reinterpret_cast<float*>(smem_raw + ((size_t(RP) * D * sizeof(T) + 127) & ~size_t(127)));   // [2][RL][D]
  float* level2 = partial + 2 * RL * D;       // [2][NP][D]
  // records read by other CTAs of the cluster (same offsets in every CTA)
  float* st_mean = level2 + 2 * NP * D;       // [D] mean of this CTA's rows
  float* st_m2 = st_mean + D;                 // [D] sum of squared deviations about it
  float* u_s = st_m2 + D;                     // [D] sum_j a_j q_j over this CTA's rows
  float* qsum_s = u_s + D;                    // [D] sum_j q_j over this CTA's rows
  float* scal = qsum_s + D;                   // [0] = sum_j a_j, [1] = rows held
  float* mean_s = scal + 4;                   // [D]
  float* ivar_s = mean_s + D;                 // [D]
  float* red_s = ivar_s + D;                  // [32]
  float* a_s = red_s + 32;                    // [RP]
  uint64_t* bar = reinterpret_cast<uint64_t*>(a_s + ((RP + 3) & ~3));

  const int sp = blockIdx.x, h = blockIdx.y, unit = blockIdx.z;
  const int hy = h % p.group;                 // head inside its KV group
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int r0 = min(W, sp * RP), nr = min(W, r0 + RP) - r0;      // this CTA's rows [r0, r0 + nr)
  const size_t row_stride = size_t(p.n_q_heads) * D;
  const T* qbase = reinterpret_cast<const T*>(p.q) + (size_t(unit) * W + r0) * row_stride + size_t(h) * D;
  const int cy = p.do_probe ? p.group : 1;    // cluster = (S, cy): rank of (split s, head-in-group y) = s + S * y
  const size_t hd = (size_t(unit) * p.n_q_heads + h) * D;
  const size_t uh = size_t(unit) * p.n_q_heads + h;

  grid_dependency_wait();            // q and the running statistics may come from earlier kernels of the stream
  grid_launch_dependents();
  // ---- 0. rows -> shared memory: one bulk copy per row, all in flight together
  constexpr uint32_t kRowBytes = D * sizeof(T);
  const uint32_t bar_addr = smem_addr(bar);
  if (tid == 0) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(bar_addr));
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  if (tid == 0 && nr > 0)
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar_addr), "r"(uint32_t(nr) * kRowBytes) : "memory");
  __syncthreads();
  for (int r = tid; r < nr; r += kThreads)
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(smem_addr(tile + size_t(r) * D)), "l"(qbase + size_t(r) * row_stride), "r"(kRowBytes), "r"(bar_addr)
                 : "memory");
  // running statistics of this head, fetched while the copies fly
  const bool running = p.do_bias && p.stats_mode == ACTQKV_STATS_CUMULATIVE;
  float run_mean = 0.f, run_m2 = 0.f;
  int64_t run_count = 0;
  if (running && tid < D) {
    run_mean = p.stats_mean[hd + tid];
    run_m2 = p.stats_m2[hd + tid];
    run_count = p.stats_count[uh];
  }
  if (nr > 0) {
    bool landed = false;
    for (uint32_t i = 0; i < kSpinLimit && !landed; ++i) {
      uint32_t ok;
      asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], 0;\n\tselp.b32 %0, 1, 0, p;\n\t}"
                   : "=r"(ok) : "r"(bar_addr) : "memory");
      landed = ok != 0;
    }
    if (!landed && tid == 0) set_status(p.status, ACTQKV_DEV_TIMEOUT);     // goes on with whatever arrived
  }

  const int cv = tid % VPR, rsub = tid / VPR;
  const int n_pass = (nr + RL - 1) / RL;      // same trip count in every thread
  auto load_row = [&](int r, float (&f)[VN]) { Vec16<T>::load(tile + size_t(r) * D + cv * VN, f); };
  // dst_k[D] = sum over the row lanes of acc_k, k < NA, in a fixed two-level order
  auto column_reduce2 = [&](const float (&a0)[VN], const float (&a1)[VN], float* dst0, float* dst1) {
    __syncthreads();
#pragma unroll
    for (int e = 0; e < VN; ++e) {
      partial[rsub * D + cv * VN + e] = a0[e];
      partial[RL * D + rsub * D + cv * VN + e] = a1[e];
    }
    __syncthreads();
    {
      const int ch = tid % D, part = tid / D;
      float t0 = 0.f, t1 = 0.f;
#pragma unroll
      for (int q = 0; q < PER; ++q) {
        t0 += partial[(part * PER + q) * D + ch];
        t1 += partial[RL * D + (part * PER + q) * D + ch];
      }
      level2[part * D + ch] = t0;
      level2[NP * D + part * D + ch] = t1;
    }
    __syncthreads();
    if (tid < D) {
      float t0 = 0.f, t1 = 0.f;
#pragma unroll
      for (int q = 0; q < NP; ++q) { t0 += level2[q * D + tid]; t1 += level2[NP * D + q * D + tid]; }
      dst0[tid] = t0;
      dst1[tid] = t1;
    }
    __syncthreads();
  };

  // ---- 1. shifted first and second moments of this CTA's rows
  {
    float shift[VN], s1[VN], s2[VN];
#pragma unroll
    for (int e = 0; e < VN; ++e) { s1[e] = 0.f; s2[e] = 0.f; shift[e] = 0.f; }
    if (nr > 0) load_row(0, shift);
    for (int r = rsub; r < nr; r += RL) {
      float f[VN];
      load_row(r, f);
#pragma unroll
      for (int e = 0; e < VN; ++e) { const float d = f[e] - shift[e]; s1[e] += f[e]; s2[e] = fmaf(d, d, s2[e]); }
    }
    column_reduce2(s1, s2, st_mean, st_m2);      // for now: sum q and sum (q - shift)^2
    if (tid < D) {
      const double n = double(nr), sh0 = nr > 0 ? double(to_f32(tile[tid])) : 0.0;
      const double sq = double(st_mean[tid]), b2 = double(st_m2[tid]);
      const double a = sq - n * sh0;             // sum (q - shift)
      qsum_s[tid] = st_mean[tid];
      st_mean[tid] = nr > 0 ? float(sq / n) : 0.f;
      st_m2[tid] = nr > 0 ? float(fmax(b2 - a * a / n, 0.0)) : 0.f;
    }
    if (tid == 0) scal[1] = float(nr);
  }

  if (p.do_bias) {
    cluster.sync();
    // ---- 2. merge the row splits, then the running statistics (Eq. 8 over all windows so far)
    if (tid < D) {
      float pn[kMaxCluster], pm[kMaxCluster], pm2[kMaxCluster];
#pragma unroll
      for (int s2 = 0; s2 < kMaxCluster; ++s2) {
        pn[s2] = 0.f; pm[s2] = 0.f; pm2[s2] = 0.f;
        if (s2 < S) {
          const unsigned rk = unsigned(s2 + S * (cy > 1 ? hy : 0));
          pn[s2] = cluster.map_shared_rank(scal, rk)[1];
          pm[s2] = cluster.map_shared_rank(st_mean, rk)[tid];
          pm2[s2] = cluster.map_shared_rank(st_m2, rk)[tid];
        }
      }
      double n = 0.0, mean = 0.0, m2 = 0.0;
#pragma unroll
      for (int s2 = 0; s2 < kMaxCluster; ++s2) {
        const double nb = double(pn[s2]);
        if (nb == 0.0) continue;
        const double nn = n + nb, delta = double(pm[s2]) - mean, w = nb / nn;
        mean += delta * w;
        m2 += double(pm2[s2]) + delta * delta * (n * w);
        n = nn;
      }
      if (running) {
        const double na = double(run_count), mean_a = double(run_mean), m2_a = double(run_m2);
        const double nn = na + n, delta = mean - mean_a, w = n / nn;
        mean = mean_a + delta * w;
        m2 = m2_a + m2 + delta * delta * (na * w);
        n = nn;
        if (sp == 0) {                         // every CTA took the old values at kernel start
          p.stats_mean[hd + tid] = float(mean);
          p.stats_m2[hd + tid] = float(m2);
          if (tid == 0) p.stats_count[uh] = run_count + W;
        }
      }
      const double var = n > 1.0 ? m2 / (n - 1.0) : 0.0;
      mean_s[tid] = float(mean);
      ivar_s[tid] = float(1.0 / fmax(var, double(p.var_eps)));
    }
    __syncthreads();
    // ---- 3. phi and its L1 norm per token: the VPR lanes of a row add up by shuffles
    {
      float mc[VN], iv[VN];
#pragma unroll
      for (int e = 0; e < VN; ++e) { mc[e] = mean_s[cv * VN + e]; iv[e] = ivar_s[cv * VN + e]; }
      for (int k = 0; k < n_pass; ++k) {
        const int r = rsub + k * RL;
        float part = 0.f;
        if (r < nr) {
          float f[VN], ph[VN];
          load_row(r, f);
#pragma unroll
          for (int e = 0; e < VN; ++e) { const float d = f[e] - mc[e]; ph[e] = d * d * iv[e]; part += ph[e]; }
          if (p.phi_full) {
            float* dst = p.phi_full + (size_t(unit) * W + r0 + r) * row_stride + size_t(h) * D + cv * VN;
#pragma unroll
            for (int e = 0; e < VN; e += 4) *reinterpret_cast<float4*>(dst + e) = make_float4(ph[e], ph[e + 1], ph[e + 2], ph[e + 3]);
          }
        }
#pragma unroll
        for (int o = VPR >> 1; o > 0; o >>= 1) part += __shfl_xor_sync(0xffffffffu, part, o);
        if (r < nr && cv == 0) a_s[r] = part;
      }
    }
    __syncthreads();
    if (p.phi_l1)
      for (int r = tid; r < nr; r += kThreads) p.phi_l1[uh * W + r0 + r] = a_s[r];
  } else {
    for (int r = tid; r < nr; r += kThreads) a_s[r] = p.phi_l1[uh * W + r0 + r];
    __syncthreads();
  }
  if (!p.do_probe) {
    if (p.do_bias) cluster.sync();      // peers may still be reading this CTA's record in step 2
    return;
  }

  // ---- 4. this CTA's share of ||Phi||_1 and of sum_j a_j q_j
  {
    float part = 0.f;
    for (int r = tid; r < nr; r += kThreads) part += a_s[r];
    part = warp_sum(part);
    if (lane == 0) red_s[warp] = part;
    float acc[VN], zero[VN];
#pragma unroll
    for (int e = 0; e < VN; ++e) { acc[e] = 0.f; zero[e] = 0.f; }
    for (int r = rsub; r < nr; r += RL) {
      float f[VN];
      load_row(r, f);
      const float w = a_s[r];
#pragma unroll
      for (int e = 0; e < VN; ++e) acc[e] = fmaf(w, f[e], acc[e]);
    }
    column_reduce2(acc, zero, u_s, mean_s);      // mean_s is free by now: dummy destination
    if (tid == 0) {
      float t = 0.f;
      for (int i = 0; i < kThreads / 32; ++i) t += red_s[i];
      scal[0] = t;
    }
  }
  cluster.sync();
  // ---- 5. Eq. 9 per query head, and the KV-head probe = mean over the G heads of the group.
  // The group leader repeats the per-head arithmetic in the same order, so both agree bitwise.
  if (sp == 0 && tid < D) {
    float tot[kMaxCluster], uu[kMaxCluster], qq[kMaxCluster];
    const int n_cta = S * cy;
#pragma unroll
    for (int rk = 0; rk < kMaxCluster; ++rk) {
      tot[rk] = 0.f; uu[rk] = 0.f; qq[rk] = 0.f;
      if (rk < n_cta && (hy == 0 || rk / S == hy)) {
        tot[rk] = cluster.map_shared_rank(scal, unsigned(rk))[0];
        uu[rk] = cluster.map_shared_rank(u_s, unsigned(rk))[tid];
        qq[rk] = cluster.map_shared_rank(qsum_s, unsigned(rk))[tid];
      }
    }
    auto head_probe = [&](int y) {
      float t = 0.f, u2 = 0.f, q2 = 0.f;
#pragma unroll
      for (int rk = 0; rk < kMaxCluster; ++rk)
        if (rk >= y * S && rk < (y + 1) * S) { t += tot[rk]; u2 += uu[rk]; q2 += qq[rk]; }
      return t > 0.f ? u2 / t : q2 / float(W);      // all-zero bias: uniform weights
    };
    p.probe_qh[hd + tid] = head_probe(cy > 1 ? hy : 0);
    if (hy == 0) {
      float acc = 0.f;
      for (int y = 0; y < p.group; ++y) acc += head_probe(y);
      p.probe_kv[(size_t(unit) * p.n_kv_heads + h / p.group) * D + tid] = acc / float(p.group);
    }
  }
  cluster.sync();      // peers keep their shared memory alive until the leaders have read it
}

template <typename T, int D>
int launch_d(const actqkv_config* cfg, const Batch& b, BiasProbeParams& p, cudaStream_t st) {
  const int W = p.n_tokens;
  const int cy = p.do_probe ? p.group : 1;
  auto kern = bias_probe_kernel<T, D>;
  constexpr int VN = Vec16<T>::N;
  constexpr int RL = kThreads / (D / VN), NP = kThreads / D;
  // Clusters stay within the portable size of 8: 16-CTA clusters were measured slower here (they
  // are scheduled one GPC at a time and their barrier costs more than the extra SMs bring).
  for (int max_cluster = 8; max_cluster >= 8; max_cluster >>= 1) {
    int split = max_cluster / cy;
    if (split < 1) split = 1;
    while (split > 1 && (W + split - 1) / split < 32) split >>= 1;
    p.split = split;
    p.rows_per_cta = (W + split - 1) / split;
    const size_t tile_bytes = (size_t(p.rows_per_cta) * D * sizeof(T) + 127) & ~size_t(127);
    const size_t smem = tile_bytes + sizeof(float) * (size_t(2) * RL * D + 2 * NP * D + 6 * D + 4 + 32 +
                                                       ((p.rows_per_cta + 3) & ~3)) + 16;
    if (smem > 220 * 1024) return ACTQKV_ERR_SHAPE;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem)) != cudaSuccess)
      return ACTQKV_ERR_LAUNCH;
    prefer_max_shared(kern);
    cudaLaunchConfig_t lc = {};
    lc.gridDim = dim3(split, cfg->n_q_heads, b.units());
    lc.blockDim = dim3(kThreads, 1, 1);
    lc.dynamicSmemBytes = smem;
    lc.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = split;
    attr[0].val.clusterDim.y = cy;
    attr[0].val.clusterDim.z = 1;
    allow_early_launch(attr[1]);
    lc.attrs = attr;
    lc.numAttrs = 2;
    if (cudaLaunchKernelEx(&lc, kern, p) == cudaSuccess) return launch_status();
    (void)cudaGetLastError();
  }
  return ACTQKV_ERR_LAUNCH;
}

template <typename T>
int launch(const actqkv_config* cfg, const Batch& b, BiasProbeParams& p, cudaStream_t st) {
  return cfg->head_dim == 64 ? launch_d<T, 64>(cfg, b, p, st) : launch_d<T, 128>(cfg, b, p, st);
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
