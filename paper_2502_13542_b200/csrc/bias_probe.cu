// Steps 1 and 2: Activation Bias (Eq. 7, statistics Eq. 8) and the activation-aware
// probe-query (Eq. 9).
//
// The [n_tokens x D] query tile of one (unit, query head) is split by rows over S CTAs, and the
// S x G CTAs of one KV head form a thread-block cluster (S * G <= 8).  Every CTA brings its rows
// from HBM into shared memory with tiled TMA loads of up to 256 rows each (the copy engine takes
// about as long for a 256-byte request as for a 2 KiB one, so one request per row would cost more
// than the data) and makes three passes over them with 16-byte shared-memory loads:
//   1. per-channel sums of q and of (q - shift)^2, shift = the CTA's first row, which give
//      the mean and the sum of squared deviations of its rows without a second pass; the row
//      splits are merged pairwise (count, mean, M2) in a fixed order through distributed shared
//      memory and then merged into the running statistics (Eq. 8 over all windows so far);
//   2. phi and the per-token indicator ||phi_j||_1 (Eq. 7);
//   3. sum_j a_j q_j, combined with sum_j a_j by the group leaders in a fixed order (Eq. 9).
// Every reduction order is fixed, so results are bitwise reproducible.
#include <cooperative_groups.h>

#include "tc_common.cuh"

namespace cg = cooperative_groups;
using namespace actqkv;

namespace {

constexpr int kThreads = 512;
constexpr int kMaxCluster = 8;
constexpr uint32_t kSpinLimit = 1u << 22;

struct BiasProbeParams {
  const void* q;
  int n_tokens, n_q_heads, n_kv_heads, head_dim, group;
  int split, rows_per_cta, box_rows, rows_alloc;   // rows_alloc: rows the tile holds (whole boxes)
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
  int mean_pool;  // uniform token weights (the mean-pooling probe) instead of Eq. 9's
  int32_t* status;
};

__device__ __forceinline__ uint32_t smem_addr(const void* p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

template <typename T, int D>
__global__ void __launch_bounds__(kThreads, 1) bias_probe_kernel(const __grid_constant__ CUtensorMap tm_q, BiasProbeParams p) {
  extern __shared__ __align__(128) unsigned char smem_raw[];
  cg::cluster_group cluster = cg::this_cluster();
  constexpr int VN = Vec16<T>::N;             // elements per 16-byte vector
  constexpr int VPR = D / VN;                 // vectors per row
  constexpr int RL = kThreads / VPR;          // row lanes: thread (cv, rsub) owns vector cv of rows rsub + k * RL
  constexpr int NP = kThreads / D;            // second-level slices of the row lanes
  const int W = p.n_tokens, S = p.split, RP = p.rows_per_cta;
  T* tile = reinterpret_cast<T*>(smem_raw);
  float* partial = reinterpret_cast<float*>(smem_raw + ((size_t(p.rows_alloc) * D * sizeof(T) + 127) & ~size_t(127)));   // [2][RL][D]
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
  // records that OTHER CTAs of the cluster write into this one, ahead of a cluster barrier (so
  // that nobody reads remote memory after a barrier and no CTA has to outlive its peers' reads)
  float* rec_n = a_s + ((RP + 3) & ~3);       // [kMaxCluster] rows held by split s of this head
  float* rec_mean = rec_n + kMaxCluster;      // [kMaxCluster][D] its mean
  float* rec_m2 = rec_mean + kMaxCluster * D; // [kMaxCluster][D] its sum of squared deviations
  float* prb_tot = rec_m2 + kMaxCluster * D;  // [kMaxCluster] sum_j a_j of cluster rank r (leaders only)
  float* prb_u = prb_tot + kMaxCluster;       // [kMaxCluster][D] its sum_j a_j q_j
  float* prb_q = prb_u + kMaxCluster * D;     // [kMaxCluster][D] its sum_j q_j
  uint64_t* bar = reinterpret_cast<uint64_t*>(prb_q + kMaxCluster * D);

  const int sp = blockIdx.x, h = blockIdx.y, unit = blockIdx.z;
  const int hy = h % p.group;                 // head inside its KV group
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int r0 = min(W, sp * RP), nr = min(W, r0 + RP) - r0;      // this CTA's rows [r0, r0 + nr)
  const size_t row_stride = size_t(p.n_q_heads) * D;
  const T* qbase = reinterpret_cast<const T*>(p.q) + (size_t(unit) * W + r0) * row_stride + size_t(h) * D;
  const int cy = p.do_probe ? p.group : 1;    // cluster = (S, cy): rank of (split s, head-in-group y) = s + S * y
  const size_t hd = (size_t(unit) * p.n_q_heads + h) * D;
  const size_t uh = size_t(unit) * p.n_q_heads + h;

  grid_launch_dependents();
  grid_dependency_wait();            // q and the running statistics may come from earlier kernels of the stream
  // ---- 0. rows -> shared memory
  constexpr uint32_t kRowBytes = D * sizeof(T);
  const uint32_t bar_addr = smem_addr(bar);
  if (tid == 0) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(bar_addr));
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  // q as [units * W rows][heads][D]: boxes of box_rows rows of this head.  Rows past the CTA's share
  // (or past the tensor: zero fill) land in the tile's slack and are never read.
  if (tid == 0 && nr > 0) {
    const int n_box = (nr + p.box_rows - 1) / p.box_rows;
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar_addr), "r"(uint32_t(n_box * p.box_rows) * kRowBytes) : "memory");
    for (int bx = 0; bx < n_box; ++bx)
      tc::tma_load_3d(smem_addr(tile + size_t(bx) * p.box_rows * D), &tm_q, bar_addr, 0, h, unit * W + r0 + bx * p.box_rows);
  }
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
  // dst0 / dst1 [D] = sums over the row lanes of a0 / a1, in a fixed order: the rows of a warp by
  // shuffles, then the warps in two levels through shared memory (16-byte stores, no bank conflicts)
  constexpr int NW = kThreads / 32, PERW = NW / NP;
  auto column_reduce2 = [&](float (&a0)[VN], float (&a1)[VN], float* dst0, float* dst1) {
#pragma unroll
    for (int o = VPR; o < 32; o <<= 1) {
#pragma unroll
      for (int e = 0; e < VN; ++e) {
        a0[e] += __shfl_xor_sync(0xffffffffu, a0[e], o);
        a1[e] += __shfl_xor_sync(0xffffffffu, a1[e], o);
      }
    }
    __syncthreads();
    if (lane < VPR) {
#pragma unroll
      for (int e = 0; e < VN; e += 4) {
        *reinterpret_cast<float4*>(partial + warp * D + cv * VN + e) = make_float4(a0[e], a0[e + 1], a0[e + 2], a0[e + 3]);
        *reinterpret_cast<float4*>(partial + NW * D + warp * D + cv * VN + e) = make_float4(a1[e], a1[e + 1], a1[e + 2], a1[e + 3]);
      }
    }
    __syncthreads();
    {
      const int ch = tid % D, part = tid / D;
      float t0 = 0.f, t1 = 0.f;
#pragma unroll
      for (int q = 0; q < PERW; ++q) {
        t0 += partial[(part * PERW + q) * D + ch];
        t1 += partial[NW * D + (part * PERW + q) * D + ch];
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

  float acc[VN];                       // this thread's share of sum_j a_j q_j
#pragma unroll
  for (int e = 0; e < VN; ++e) acc[e] = 0.f;
  if (p.do_bias) {
    // this CTA's record goes to every split of its head (itself included)
    if (tid < D) {
#pragma unroll
      for (int s2 = 0; s2 < kMaxCluster; ++s2) {
        if (s2 < S) {
          const unsigned rk = unsigned(s2 + S * (cy > 1 ? hy : 0));
          cluster.map_shared_rank(rec_mean, rk)[sp * D + tid] = st_mean[tid];
          cluster.map_shared_rank(rec_m2, rk)[sp * D + tid] = st_m2[tid];
          if (tid == 0) cluster.map_shared_rank(rec_n, rk)[sp] = float(nr);
        }
      }
    }
    cluster.sync();
    // ---- 2. merge the row splits, then the running statistics (Eq. 8 over all windows so far)
    if (tid < D) {
      // Rolled loops here and in step 5: these phases run once per launch, and straight-line code
      // that is executed once costs its instruction fetch (the unrolled forms took twice as long
      // inside a step as back to back with warm instructions).
      double n = 0.0, mean = 0.0, m2 = 0.0;
#pragma unroll 1
      for (int s2 = 0; s2 < S; ++s2) {
        const double nb = double(rec_n[s2]);
        if (nb == 0.0) continue;
        // the weights are ratios of token counts, the same in every thread: an fp32 division (a
        // double one is some thirty dependent instructions, five of them in a row on this path)
        const double nn = n + nb, delta = double(rec_mean[s2 * D + tid]) - mean, w = double(float(nb) / float(nn));
        mean += delta * w;
        m2 += double(rec_m2[s2 * D + tid]) + delta * delta * (n * w);
        n = nn;
      }
      if (running) {
        const double na = double(run_count), mean_a = double(run_mean), m2_a = double(run_m2);
        const double nn = na + n, delta = mean - mean_a, w = double(float(n) / float(nn));
        mean = mean_a + delta * w;
        m2 = m2_a + m2 + delta * delta * (na * w);
        n = nn;
        if (sp == 0) {                         // every CTA took the old values at kernel start
          p.stats_mean[hd + tid] = float(mean);
          p.stats_m2[hd + tid] = float(m2);
          if (tid == 0) p.stats_count[uh] = run_count + W;
        }
      }
      const float var = n > 1.0 ? float(m2) / float(n - 1.0) : 0.f;      // sigma^2 and its inverse are fp32 results
      mean_s[tid] = float(mean);
      ivar_s[tid] = 1.f / fmaxf(var, p.var_eps);
    }
    __syncthreads();
    // ---- 3. phi and its L1 norm a_j per token (the VPR lanes of a row add up by shuffles) and, with
    // the row still in registers, its term of sum_j a_j q_j
    {
      float mc[VN], iv[VN];
#pragma unroll
      for (int e = 0; e < VN; ++e) { mc[e] = mean_s[cv * VN + e]; iv[e] = ivar_s[cv * VN + e]; }
      for (int k = 0; k < n_pass; ++k) {
        const int r = rsub + k * RL;
        float part = 0.f;
        float f[VN];
#pragma unroll
        for (int e = 0; e < VN; ++e) f[e] = 0.f;
        if (r < nr) {
          float ph[VN];
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
        if (p.do_probe) {
#pragma unroll
          for (int e = 0; e < VN; ++e) acc[e] = fmaf(part, f[e], acc[e]);      // f = 0 for a row that is not there
        }
      }
    }
    __syncthreads();
    if (p.phi_l1)
      for (int r = tid; r < nr; r += kThreads) p.phi_l1[uh * W + r0 + r] = a_s[r];
  } else {
    for (int r = tid; r < nr; r += kThreads) a_s[r] = p.phi_l1[uh * W + r0 + r];
    __syncthreads();
  }
  if (!p.do_probe) return;

  // ---- 4. this CTA's share of ||Phi||_1 and of sum_j a_j q_j
  {
    float part = 0.f;
    for (int r = tid; r < nr; r += kThreads) part += a_s[r];
    part = warp_sum(part);
    if (lane == 0) red_s[warp] = part;
    float zero[VN];
#pragma unroll
    for (int e = 0; e < VN; ++e) zero[e] = 0.f;
    if (!p.do_bias) {                    // the indicator was an input: the rows have not been passed yet
      for (int r = rsub; r < nr; r += RL) {
        float f[VN];
        load_row(r, f);
        const float w = a_s[r];
#pragma unroll
        for (int e = 0; e < VN; ++e) acc[e] = fmaf(w, f[e], acc[e]);
      }
    }
    column_reduce2(acc, zero, u_s, mean_s);      // mean_s is free by now: dummy destination
    // this CTA's sums go to the leader of its head and to the leader of its KV group (rank 0)
    const unsigned me = cluster.block_rank();
    const unsigned head_leader = unsigned(S * (cy > 1 ? hy : 0));
    if (tid == 0) {
      float t = 0.f;
      for (int i = 0; i < kThreads / 32; ++i) t += red_s[i];
      cluster.map_shared_rank(prb_tot, head_leader)[me] = t;
      if (head_leader != 0) cluster.map_shared_rank(prb_tot, 0)[me] = t;
    }
    if (tid < D) {
      cluster.map_shared_rank(prb_u, head_leader)[me * D + tid] = u_s[tid];
      cluster.map_shared_rank(prb_q, head_leader)[me * D + tid] = qsum_s[tid];
      if (head_leader != 0) {
        cluster.map_shared_rank(prb_u, 0)[me * D + tid] = u_s[tid];
        cluster.map_shared_rank(prb_q, 0)[me * D + tid] = qsum_s[tid];
      }
    }
  }
  cluster.sync();
  // ---- 5. Eq. 9 per query head, and the KV-head probe = mean over the G heads of the group.
  // The group leader repeats the per-head arithmetic in the same order, so both agree bitwise.
  if (sp == 0 && tid < D) {
    auto head_probe = [&](int y) {                 // ranks y * S .. y * S + S - 1 hold head y of the group
      float t = 0.f, u2 = 0.f, q2 = 0.f;
#pragma unroll 1
      for (int rk = y * S; rk < (y + 1) * S; ++rk) { t += prb_tot[rk]; u2 += prb_u[rk * D + tid]; q2 += prb_q[rk * D + tid]; }
      return (t > 0.f && !p.mean_pool) ? u2 / t : q2 / float(W);      // all-zero bias: uniform weights
    };
    if (hy == 0) {
      float acc = 0.f, own = 0.f;
#pragma unroll 1
      for (int y = 0; y < cy; ++y) {
        const float pr = head_probe(y);
        if (y == 0) own = pr;
        acc += pr;
      }
      p.probe_qh[hd + tid] = own;
      p.probe_kv[(size_t(unit) * p.n_kv_heads + h / p.group) * D + tid] = acc / float(p.group);
    } else {
      p.probe_qh[hd + tid] = head_probe(hy);
    }
  }
}

// The N / 2 packed fp32 pairs of a 16-byte vector (element 2i in the low half of pair i).
template <typename T> struct Pairs;
template <> struct Pairs<float> {
  static constexpr int N2 = 2;
  __device__ static __forceinline__ void get(const uint4& v, uint64_t (&out)[2]) {
    asm("mov.b64 %0, {%1, %2};" : "=l"(out[0]) : "r"(v.x), "r"(v.y));
    asm("mov.b64 %0, {%1, %2};" : "=l"(out[1]) : "r"(v.z), "r"(v.w));
  }
};
template <> struct Pairs<__nv_bfloat16> {
  static constexpr int N2 = 4;
  __device__ static __forceinline__ void get(const uint4& v, uint64_t (&out)[4]) {
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) asm("mov.b64 %0, {%1, %2};" : "=l"(out[i]) : "r"(w[i] << 16), "r"(w[i] & 0xFFFF0000u));
  }
};

// q viewed as [units * W rows][heads][D] with boxes of box_rows rows of one head.
template <typename T, int D>
bool encode_q(CUtensorMap* tm, const BiasProbeParams& p, int units, int box_rows) {
  const cuuint64_t dims[3] = {cuuint64_t(D), cuuint64_t(p.n_q_heads), cuuint64_t(units) * cuuint64_t(p.n_tokens)};
  const cuuint64_t strides[2] = {cuuint64_t(D) * sizeof(T), cuuint64_t(p.n_q_heads) * D * sizeof(T)};
  const cuuint32_t box[3] = {cuuint32_t(D), 1u, cuuint32_t(box_rows)};
  return tc::encode_plain(tm, sizeof(T) == 4, p.q, 3, dims, strides, box);
}

// ---------------------------------------------------------------------------------------------
// Batched calls (many (unit, head) items, e.g. all layers of a model in one launch): a persistent
// kernel without clusters.  A CTA is small enough for TWO to share an SM -- eight consumer warps and
// one producer warp, 16 KiB chunks in a ring of four slots -- so that the reductions and barrier
// waits of one CTA's item are filled with the row passes of the other's.  An item is not kept in
// shared memory: the producer brings its chunks once for pass 1 (column sums -> statistics, Eq. 8)
// and once more for pass 2 (phi, a_j = ||phi_j||_1 and sum_j a_j q_j, Eq. 7 and 9); the second read
// is served by L2 (two items per SM are 256 KiB in flight out of 126 MB), so HBM still sees every
// query once and n_tokens is not limited by the shared memory.  Slots are handed over with
// full / empty mbarriers (the producer never takes part in a CTA barrier); every wait is bounded.
// The kernel is bound by its instruction pipes, not by memory or latency: a form that kept one whole
// item per SM in shared memory (16 warps, phases in series) took the same 57 us for 32 layers,
// three CTAs per SM are slower, and the packed fp32 and integer pipes both run at one warp
// instruction per two cycles, which the unpacking of bf16 pairs and the 24 packed operations per
// 16-byte vector fill.
constexpr int kRingThreads = 256;           // consumer threads; warp 8 is the producer
constexpr int kRingSlots = 4;
constexpr int kRingCtasPerSm = 2;           // three per SM (72 registers, 3 slots) measured slower: 87 us against 62.5
constexpr int kRingRowsPerThread = 4;       // rows of a chunk per consumer thread

__device__ __forceinline__ void consumer_barrier() { asm volatile("bar.sync 1, %0;" ::"n"(kRingThreads) : "memory"); }

template <typename T, int D>
__global__ void __launch_bounds__(kRingThreads + 32, kRingCtasPerSm)
bias_probe_ring_kernel(const __grid_constant__ CUtensorMap tm_q, BiasProbeParams p, int n_items, int n_chunks) {
  extern __shared__ __align__(128) unsigned char smem_raw[];
  constexpr int VN = Vec16<T>::N;
  constexpr int VPR = D / VN;
  constexpr int RL = kRingThreads / VPR;            // row lanes
  constexpr int NW = kRingThreads / 32;             // consumer warps
  constexpr int N2 = Pairs<T>::N2;
  constexpr int kChunkRows = RL * kRingRowsPerThread;
  constexpr uint32_t kChunkBytes = uint32_t(kChunkRows) * D * sizeof(T);      // 16 KiB for every supported shape
  const int W = p.n_tokens;
  T* ring = reinterpret_cast<T*>(smem_raw);                                   // [kRingSlots][kChunkRows][D]
  float* partial = reinterpret_cast<float*>(smem_raw + kRingSlots * kChunkBytes);   // [2][NW][D]
  float* sum_a = partial + 2 * NW * D;        // [D] first result of a column reduction
  float* sum_b = sum_a + D;                   // [D] second result
  float* mean_s = sum_b + D;                  // [D]
  float* ivar_s = mean_s + D;                 // [D]
  float* qsum_s = ivar_s + D;                 // [D] sum_j q_j of the item
  float* shift_s = qsum_s + D;                // [D] row 0 of the item (the shift of pass 1)
  float* red_s = shift_s + D;                 // [32]
  float* a_s = red_s + 32;                    // [W]
  uint64_t* bar_full = reinterpret_cast<uint64_t*>(a_s + ((W + 3) & ~3));     // [kRingSlots]
  uint64_t* bar_empty = bar_full + kRingSlots;                                // [kRingSlots]

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const bool running = p.do_bias && p.stats_mode == ACTQKV_STATS_CUMULATIVE;
  const int n_pass = p.do_bias ? 2 : 1;

  grid_launch_dependents();
  grid_dependency_wait();            // q and the running statistics may come from earlier kernels of the stream
  if (tid == 0) {
    for (int s = 0; s < kRingSlots; ++s) {
      asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(smem_addr(bar_full + s)));
      asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_addr(bar_empty + s)), "n"(NW));
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();                   // the only barrier the producer warp takes part in

  auto wait_bar = [&](uint64_t* bar, uint32_t parity) {
    const uint32_t addr = smem_addr(bar);
    bool done = false;
    for (uint32_t i = 0; i < kSpinLimit && !done; ++i) {
      uint32_t ok;
      asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.b32 %0, 1, 0, p;\n\t}"
                   : "=r"(ok) : "r"(addr), "r"(parity) : "memory");
      done = ok != 0;
    }
    if (!done && lane == 0) set_status(p.status, ACTQKV_DEV_TIMEOUT);     // goes on with whatever arrived
  };

  if (warp == NW) {
    // =========================== producer: one thread walks the load sequence ===========================
    // item by item: its chunks for pass 1, then the same chunks for pass 2.  Rows past n_tokens belong
    // to the next unit or are zero fill; they are never read.
    if (lane == 0) {
      uint32_t seq = 0;
      for (int item = blockIdx.x; item < n_items; item += gridDim.x) {
        const int unit = item / p.n_q_heads, h = item - unit * p.n_q_heads;
        for (int pass = 0; pass < n_pass; ++pass)
          for (int c = 0; c < n_chunks; ++c, ++seq) {
            const uint32_t slot = seq % kRingSlots, round = seq / kRingSlots;
            if (round > 0) wait_bar(bar_empty + slot, (round - 1) & 1);
            const uint32_t bar = smem_addr(bar_full + slot);
            asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(kChunkBytes) : "memory");
            tc::tma_load_3d(smem_addr(ring + size_t(slot) * kChunkRows * D), &tm_q, bar, 0, h, unit * W + c * kChunkRows);
          }
      }
    }
    return;
  }

  // =========================== consumers ===========================
  const int cv = tid % VPR, rsub = tid / VPR;
  const size_t row_stride = size_t(p.n_q_heads) * D;
  // dst0 / dst1 [D] = sums over the row lanes of a0 / a1 in a fixed order: the rows of a warp by
  // shuffles, then the eight warps through shared memory
  auto column_reduce2 = [&](float (&a0)[VN], float (&a1)[VN], float* dst0, float* dst1) {
#pragma unroll
    for (int o = VPR; o < 32; o <<= 1) {
#pragma unroll
      for (int e = 0; e < VN; ++e) {
        a0[e] += __shfl_xor_sync(0xffffffffu, a0[e], o);
        a1[e] += __shfl_xor_sync(0xffffffffu, a1[e], o);
      }
    }
    consumer_barrier();                              // earlier readers of `partial` are done
    if (lane < VPR) {
#pragma unroll
      for (int e = 0; e < VN; e += 4) {
        *reinterpret_cast<float4*>(partial + warp * D + cv * VN + e) = make_float4(a0[e], a0[e + 1], a0[e + 2], a0[e + 3]);
        *reinterpret_cast<float4*>(partial + NW * D + warp * D + cv * VN + e) = make_float4(a1[e], a1[e + 1], a1[e + 2], a1[e + 3]);
      }
    }
    consumer_barrier();
    for (int ch = tid; ch < 2 * D; ch += kRingThreads) {
      const float* src = partial + (ch >= D ? NW * D : 0) + (ch % D);
      float t = 0.f;
#pragma unroll
      for (int w = 0; w < NW; ++w) t += src[w * D];
      (ch >= D ? dst1 : dst0)[ch % D] = t;
    }
    consumer_barrier();
  };

  uint32_t seq = 0;
  for (int item = blockIdx.x; item < n_items; item += gridDim.x) {
    const int unit = item / p.n_q_heads, h = item - unit * p.n_q_heads;
    const size_t hd = (size_t(unit) * p.n_q_heads + h) * D;
    const size_t uh = size_t(unit) * p.n_q_heads + h;
    float run_mean = 0.f, run_m2 = 0.f;
    int64_t run_count = 0;
    if (running && tid < D) {
      run_mean = p.stats_mean[hd + tid];
      run_m2 = p.stats_m2[hd + tid];
      run_count = p.stats_count[uh];
    }
    if (p.do_bias) {
      // ---- pass 1, chunk by chunk as the rows land: sums of q and of (q - shift)^2, shift = row 0,
      // on packed pairs of channels
      uint64_t shift2[N2], s1p[N2], s2p[N2];
#pragma unroll
      for (int e = 0; e < N2; ++e) { s1p[e] = 0; s2p[e] = 0; shift2[e] = 0; }
      for (int c = 0; c < n_chunks; ++c, ++seq) {
        const uint32_t slot = seq % kRingSlots;
        wait_bar(bar_full + slot, (seq / kRingSlots) & 1);
        const T* chunk = ring + size_t(slot) * kChunkRows * D;
        if (c == 0) {
          Pairs<T>::get(*reinterpret_cast<const uint4*>(chunk + cv * VN), shift2);
          for (int ch = tid; ch < D; ch += kRingThreads) shift_s[ch] = to_f32(chunk[ch]);
        }
        const T* src = chunk + size_t(rsub) * D + cv * VN;
        const int r0 = c * kChunkRows + rsub;
        uint4 raw[kRingRowsPerThread];                 // all four loads in flight before the first use
#pragma unroll
        for (int k = 0; k < kRingRowsPerThread; ++k) raw[k] = *reinterpret_cast<const uint4*>(src + size_t(k) * RL * D);
#pragma unroll
        for (int k = 0; k < kRingRowsPerThread; ++k) {
          if (r0 + k * RL < W) {
            uint64_t x[N2];
            Pairs<T>::get(raw[k], x);
#pragma unroll
            for (int e = 0; e < N2; ++e) {
              const uint64_t d = tc::sub2(x[e], shift2[e]);
              s1p[e] = tc::add2(s1p[e], x[e]);
              s2p[e] = tc::fma2(d, d, s2p[e]);
            }
          }
        }
        __syncwarp();
        if (lane == 0) asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_addr(bar_empty + slot)) : "memory");
      }
      float s1[VN], s2[VN];
#pragma unroll
      for (int e = 0; e < N2; ++e) {
        s1[2 * e] = tc::lo2(s1p[e]); s1[2 * e + 1] = tc::hi2(s1p[e]);
        s2[2 * e] = tc::lo2(s2p[e]); s2[2 * e + 1] = tc::hi2(s2p[e]);
      }
      column_reduce2(s1, s2, sum_a, sum_b);
      // ---- statistics of the window, merged into the running ones (Eq. 8)
      if (tid < D) {
        double n = double(W);
        const double sh0 = double(shift_s[tid]);
        const double sq = double(sum_a[tid]), b2 = double(sum_b[tid]);
        const double a = sq - n * sh0;             // sum (q - shift)
        double mean = sq / n, m2 = fmax(b2 - a * a / n, 0.0);
        qsum_s[tid] = sum_a[tid];
        if (running) {
          const double na = double(run_count), mean_a = double(run_mean), m2_a = double(run_m2);
          const double nn = na + n, delta = mean - mean_a, w = n / nn;
          mean = mean_a + delta * w;
          m2 = m2_a + m2 + delta * delta * (na * w);
          n = nn;
          p.stats_mean[hd + tid] = float(mean);
          p.stats_m2[hd + tid] = float(m2);
          if (tid == 0) p.stats_count[uh] = run_count + W;
        }
        const double var = n > 1.0 ? m2 / (n - 1.0) : 0.0;
        mean_s[tid] = float(mean);
        ivar_s[tid] = float(1.0 / fmax(var, double(p.var_eps)));
      }
    } else {
      for (int r = tid; r < W; r += kRingThreads) a_s[r] = p.phi_l1[uh * W + r];
    }
    consumer_barrier();
    // ---- pass 2: phi, a_j = ||phi_j||_1 (Eq. 7) and this head's sum_j a_j q_j (and sum_j q_j when
    // pass 1 did not run), on packed pairs of channels
    uint64_t accp[N2], qsp[N2], mc2[N2], iv2[N2];
#pragma unroll
    for (int e = 0; e < N2; ++e) {
      accp[e] = 0; qsp[e] = 0;
      mc2[e] = p.do_bias ? tc::pack2(mean_s[cv * VN + 2 * e], mean_s[cv * VN + 2 * e + 1]) : 0;
      iv2[e] = p.do_bias ? tc::pack2(ivar_s[cv * VN + 2 * e], ivar_s[cv * VN + 2 * e + 1]) : 0;
    }
    float a_tot = 0.f;
    const bool four_rows = p.do_bias && p.do_probe && !p.phi_full && VPR >= 4;
    // ||phi_j||_1 is summed as sum_c q (q iv - 2 mean iv) + sum_c mean^2 iv: two packed operations per
    // pair of channels instead of three, on both paths alike (so every form of the call gives the same
    // bits); the full phi, when asked for, is written as (q - mean)^2 iv.
    uint64_t nb2[N2];
    float phi_const = 0.f;                            // this thread's channels of sum_c mean^2 iv
#pragma unroll
    for (int e = 0; e < N2; ++e) {
      const uint64_t mi = tc::mul2(mc2[e], iv2[e]);
      nb2[e] = tc::mul2(mi, tc::pack2(-2.f, -2.f));
      const uint64_t mm = tc::mul2(mi, mc2[e]);
      phi_const += tc::lo2(mm) + tc::hi2(mm);
    }
    for (int c = 0; c < n_chunks; ++c, ++seq) {
      const uint32_t slot = seq % kRingSlots;
      wait_bar(bar_full + slot, (seq / kRingSlots) & 1);
      const T* src = ring + size_t(slot) * kChunkRows * D + size_t(rsub) * D + cv * VN;
      const int r_base = c * kChunkRows + rsub;
      // the row lanes of a warp run the same passes (a warp holds whole rows; r >= W only switches
      // the row off), so the shuffles below are convergent
      if (four_rows) {
        // the thread's four rows of the chunk at once: their four sums over the VPR lanes of a row are
        // reduced together (halves swap row pairs, quarters swap rows: 3 + log2(VPR / 4) shuffles
        // instead of 4 log2(VPR)) and handed back to every lane of the row by four more
        uint64_t x[4][N2];
        float part[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const bool live = r_base + j * RL < W;
          Pairs<T>::get(live ? *reinterpret_cast<const uint4*>(src + size_t(j) * RL * D) : make_uint4(0, 0, 0, 0), x[j]);
          uint64_t part2 = 0;
#pragma unroll
          for (int e = 0; e < N2; ++e) part2 = tc::fma2(x[j][e], tc::fma2(x[j][e], iv2[e], nb2[e]), part2);
          part[j] = live ? fmaxf(tc::lo2(part2) + tc::hi2(part2) + phi_const, 0.f) : 0.f;
        }
        constexpr int H1 = VPR / 2, H2 = VPR / 4;
        const bool up1 = lane & H1, up2 = lane & H2;
        const float t0 = __shfl_xor_sync(0xffffffffu, up1 ? part[0] : part[2], H1);
        const float t1 = __shfl_xor_sync(0xffffffffu, up1 ? part[1] : part[3], H1);
        const float k0 = (up1 ? part[2] : part[0]) + t0, k1 = (up1 ? part[3] : part[1]) + t1;
        float kv = (up2 ? k1 : k0) + __shfl_xor_sync(0xffffffffu, up2 ? k0 : k1, H2);
#pragma unroll
        for (int o = H2 >> 1; o > 0; o >>= 1) kv += __shfl_xor_sync(0xffffffffu, kv, o);
        const int row_lane0 = lane & ~(VPR - 1);           // first lane of this row's lane group
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const float a = __shfl_sync(0xffffffffu, kv, row_lane0 + (j >> 1) * H1 + (j & 1) * H2);
          const int r = r_base + j * RL;
          if (r < W && cv == 0) a_s[r] = a;
          if (cv == 0) a_tot += a;
          const uint64_t a2 = tc::pack2(a, a);
#pragma unroll
          for (int e = 0; e < N2; ++e) accp[e] = tc::fma2(a2, x[j][e], accp[e]);
        }
      } else {
#pragma unroll 2
        for (int k = 0; k < kRingRowsPerThread; ++k) {
          const int r = r_base + k * RL;
          const bool live = r < W;
          uint64_t x[N2];
          Pairs<T>::get(live ? *reinterpret_cast<const uint4*>(src + size_t(k) * RL * D) : make_uint4(0, 0, 0, 0), x);
          float a;
          if (p.do_bias) {
            uint64_t part2 = 0;
            if (p.phi_full && live) {
              float* dst = p.phi_full + (size_t(unit) * W + r) * row_stride + size_t(h) * D + cv * VN;
#pragma unroll
              for (int e = 0; e < N2; ++e) {
                const uint64_t d = tc::sub2(x[e], mc2[e]);
                const uint64_t ph = tc::mul2(tc::mul2(d, d), iv2[e]);
                *reinterpret_cast<float2*>(dst + 2 * e) = make_float2(tc::lo2(ph), tc::hi2(ph));
              }
            }
#pragma unroll
            for (int e = 0; e < N2; ++e) part2 = tc::fma2(x[e], tc::fma2(x[e], iv2[e], nb2[e]), part2);   // as on the four-row path
            float part = live ? fmaxf(tc::lo2(part2) + tc::hi2(part2) + phi_const, 0.f) : 0.f;
#pragma unroll
            for (int o = VPR >> 1; o > 0; o >>= 1) part += __shfl_xor_sync(0xffffffffu, part, o);
            a = part;                                // every lane of the row holds the same sum
            if (live && cv == 0) a_s[r] = a;
          } else {
            a = live ? a_s[r] : 0.f;
          }
          if (cv == 0) a_tot += a;
          if (p.do_probe) {
            const uint64_t a2 = tc::pack2(a, a);
#pragma unroll
            for (int e = 0; e < N2; ++e) accp[e] = tc::fma2(a2, x[e], accp[e]);
            if (!p.do_bias) {
#pragma unroll
              for (int e = 0; e < N2; ++e) qsp[e] = tc::add2(qsp[e], x[e]);
            }
          }
        }
      }
      __syncwarp();
      if (lane == 0) asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_addr(bar_empty + slot)) : "memory");
    }
    float acc[VN], qs[VN];
#pragma unroll
    for (int e = 0; e < N2; ++e) {
      acc[2 * e] = tc::lo2(accp[e]); acc[2 * e + 1] = tc::hi2(accp[e]);
      qs[2 * e] = tc::lo2(qsp[e]); qs[2 * e + 1] = tc::hi2(qsp[e]);
    }
    if (p.do_probe) {
      // ---- Eq. 9 for this head
      a_tot = warp_sum(a_tot);
      if (lane == 0) red_s[warp] = a_tot;
      column_reduce2(acc, qs, sum_a, sum_b);         // its barriers also publish a_s and red_s
      if (tid < D) {
        float t = 0.f;
#pragma unroll
        for (int i = 0; i < NW; ++i) t += red_s[i];
        const float qsum = p.do_bias ? qsum_s[tid] : sum_b[tid];
        p.probe_qh[hd + tid] = (t > 0.f && !p.mean_pool) ? sum_a[tid] / t : qsum / float(W);   // all-zero bias: uniform weights
      }
    } else {
      consumer_barrier();                            // a_s is complete
    }
    if (p.do_bias && p.phi_l1)
      for (int r = tid; r < W; r += kRingThreads) p.phi_l1[uh * W + r] = a_s[r];
    consumer_barrier();                              // everything of this item has been read
  }
}

// KV-head probe = mean over the G query heads of the group (Eq. 9 under grouped-query attention).
__global__ void probe_kv_kernel(const float* probe_qh, float* probe_kv, int n_q_heads, int n_kv_heads, int group, int D) {
  const int unit = blockIdx.x / n_kv_heads, g = blockIdx.x - unit * n_kv_heads;
  for (int ch = threadIdx.x; ch < D; ch += blockDim.x) {
    float acc = 0.f;
    for (int y = 0; y < group; ++y) acc += probe_qh[(size_t(unit) * n_q_heads + g * group + y) * D + ch];
    probe_kv[(size_t(unit) * n_kv_heads + g) * D + ch] = acc / float(group);
  }
}

// A step of one token: the probe of a query head is the token's query itself, whatever the weights
// (Eq. 9 with a single term); the KV-head probe is the mean over the group.  One block per
// (unit, KV head), one thread per channel.
template <typename T>
__global__ void probe_one_token_kernel(const T* __restrict__ q, float* __restrict__ probe_qh, float* __restrict__ probe_kv,
                                       int n_q_heads, int n_kv_heads, int group) {
  grid_dependency_wait();
  const int unit = blockIdx.x / n_kv_heads, g = blockIdx.x - unit * n_kv_heads, D = blockDim.x, ch = threadIdx.x;
  float acc = 0.f;
  for (int y = 0; y < group; ++y) {
    const size_t i = (size_t(unit) * n_q_heads + g * group + y) * D + ch;
    const float x = to_f32(q[i]);
    probe_qh[i] = x;
    acc += x;
  }
  probe_kv[(size_t(unit) * n_kv_heads + g) * D + ch] = acc / float(group);
}

// The batched kernel: two CTAs per SM.  Returns 1 when the shape does not suit it (the caller takes the cluster kernel).
template <typename T, int D>
int launch_ring(const actqkv_config* cfg, const Batch& b, BiasProbeParams& p, cudaStream_t st, int n_sm) {
  constexpr int VN = Vec16<T>::N;
  constexpr int RL = kRingThreads / (D / VN), NW = kRingThreads / 32;
  constexpr int kChunkRows = RL * kRingRowsPerThread;
  const int W = p.n_tokens;
  if (kChunkRows > 256) return 1;                     // a box dimension holds at most 256
  const int n_chunks = (W + kChunkRows - 1) / kChunkRows;
  const size_t smem = size_t(kRingSlots) * kChunkRows * D * sizeof(T) +
                      sizeof(float) * (size_t(2) * NW * D + 6 * D + 32 + ((W + 3) & ~3)) + 8 * 2 * kRingSlots;
  if (smem > 227 * 1024 / kRingCtasPerSm - 1024) return 1;      // kRingCtasPerSm CTAs must fit an SM
  CUtensorMap tm_q;
  if (!encode_q<T, D>(&tm_q, p, b.units(), kChunkRows)) return ACTQKV_ERR_LAUNCH;
  auto kern = bias_probe_ring_kernel<T, D>;
  static std::atomic<bool> opted_in[kMaxDevices];
  if (!opt_in_shared_memory(kern, 227 * 1024 / kRingCtasPerSm - 1024, opted_in)) return ACTQKV_ERR_LAUNCH;
  prefer_max_shared(kern);
  const int n_items = b.units() * cfg->n_q_heads;
  cudaLaunchConfig_t lc = {};
  lc.gridDim = dim3(std::min(n_items, kRingCtasPerSm * n_sm), 1, 1);
  lc.blockDim = dim3(kRingThreads + 32, 1, 1);
  lc.dynamicSmemBytes = smem;
  lc.stream = st;
  cudaLaunchAttribute attr[1];
  allow_early_launch(attr[0]);
  lc.attrs = attr;
  lc.numAttrs = 1;
  if (cudaLaunchKernelEx(&lc, kern, tm_q, p, n_items, n_chunks) != cudaSuccess) {
    (void)cudaGetLastError();
    return ACTQKV_ERR_LAUNCH;
  }
  if (p.do_probe)
    probe_kv_kernel<<<b.units() * cfg->n_kv_heads, D, 0, st>>>(p.probe_qh, p.probe_kv, cfg->n_q_heads, cfg->n_kv_heads,
                                                                p.group, D);
  return launch_status();
}

template <typename T, int D>
int launch_d(const actqkv_config* cfg, const Batch& b, BiasProbeParams& p, cudaStream_t st) {
  const int W = p.n_tokens;
  const int cy = p.do_probe ? p.group : 1;
  // Many items: the persistent streaming kernel (throughput); few: the cluster kernel (latency).
  int dev = 0, n_sm = 0;
  if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev);
  if (n_sm > 0 && b.units() * cfg->n_q_heads >= 2 * n_sm) {
    const int rc = launch_ring<T, D>(cfg, b, p, st, n_sm);
    if (rc <= 0) return rc;
  }
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
    p.box_rows = std::min(p.rows_per_cta, 256);                          // a box dimension holds at most 256
    p.rows_alloc = (p.rows_per_cta + p.box_rows - 1) / p.box_rows * p.box_rows;
    CUtensorMap tm_q;
    if (!encode_q<T, D>(&tm_q, p, b.units(), p.box_rows)) return ACTQKV_ERR_LAUNCH;
    const size_t tile_bytes = (size_t(p.rows_alloc) * D * sizeof(T) + 127) & ~size_t(127);
    const size_t smem = tile_bytes + sizeof(float) * (size_t(2) * RL * D + 2 * NP * D + 6 * D + 4 + 32 +
                                                       ((p.rows_per_cta + 3) & ~3) + 2 * kMaxCluster +
                                                       4 * kMaxCluster * D) + 16;
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
    if (cudaLaunchKernelEx(&lc, kern, tm_q, p) == cudaSuccess) return launch_status();
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
  p.mean_pool = cfg->probe_mode == ACTQKV_PROBE_MEAN_POOL;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  if (p.n_tokens == 1 && p.do_probe && !p.do_bias) {
    // one token: every weighting gives probe_qh = q (the decode-stage probe, Sec. 4.2)
    const int n = b.units() * cfg->n_kv_heads;
    if (cfg->dtype == ACTQKV_BF16)
      probe_one_token_kernel<__nv_bfloat16><<<n, cfg->head_dim, 0, st>>>(static_cast<const __nv_bfloat16*>(p.q), p.probe_qh,
                                                                         p.probe_kv, cfg->n_q_heads, cfg->n_kv_heads, p.group);
    else
      probe_one_token_kernel<float><<<n, cfg->head_dim, 0, st>>>(static_cast<const float*>(p.q), p.probe_qh, p.probe_kv,
                                                                 cfg->n_q_heads, cfg->n_kv_heads, p.group);
    return launch_status();
  }
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
  if (n_tokens == 1) ACTQKV_OPTIONAL_PTR(phi_l1);    // a single token's weight is 1 whatever phi says
  else ACTQKV_REQUIRE_PTR(phi_l1);
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
