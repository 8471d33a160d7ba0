// Step 5, general kernel: attention of the step's queries over
//   [initial tokens | selected blocks | local past | step tokens (causal)]     (Eq. 2, Eq. 3)
// gathered from the paged cache.  fp32 accumulate on CUDA cores, any supported dtype / head
// dim / alignment; serves fp32 caches, ragged steps and single-token decode.  The bf16
// D = 128 prefill shape is served by the tcgen05 kernel instead.
//
// One CTA = 16 query rows of one query head (4 warps x 4 rows).  Keys are processed in
// chunks of 32 staged in shared memory as fp32: in the QK^T phase lane l owns key l of the
// chunk for all 4 rows of its warp; in the PV phase lane l owns channels l, l+32, ... .
// Softmax is the usual running-max / running-sum recurrence in base 2.
#include "common.cuh"
#include "stages.cuh"

using namespace actqkv;

namespace {

constexpr int kWarps = 4;
constexpr int kRows = 4;                 // query rows per warp
constexpr int kTileRows = kWarps * kRows;
constexpr int kChunk = 32;

struct SimtParams {
  AttnArgs a;
  int n_q_heads, n_kv_heads, group, block, page_tokens, n_init, n_local_prev, cap_blocks;
  int max_pages, n_phys_pages, n_layers;
  float scale_log2;
};

template <typename T, typename TO, int D>
__global__ void __launch_bounds__(kWarps * 32) attention_simt_kernel(SimtParams p) {
  __shared__ float Ks[kChunk][D + 1];
  __shared__ float Vs[kChunk][D];
  __shared__ __align__(16) float Qs[kWarps][D][kRows];

  const int tile = blockIdx.x, h = blockIdx.y, unit = blockIdx.z;
  const int g = h / p.group, seq = unit / p.n_layers, layer_local = unit - seq * p.n_layers;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int nt = p.a.n_tokens;

  const Geometry geo = make_geometry(p.a.pos0[seq], p.n_init, p.block, p.n_local_prev);
  int c = p.a.sel_count ? p.a.sel_count[unit] : 0;
  if (c < 0 || c > p.cap_blocks || c > geo.n_cand) {
    if (tid == 0) set_status(p.a.status, ACTQKV_DEV_BAD_SELECTION);
    c = max(0, min(c, min(p.cap_blocks, geo.n_cand)));
  }
  const int32_t* sel = p.a.sel_idx + (size_t(unit) * p.n_kv_heads + g) * p.cap_blocks;
  const int sel_len = c * p.block;
  const int64_t n_past = int64_t(geo.init_len) + sel_len + (geo.p0 - geo.local_start);
  const size_t page_elems = size_t(p.n_kv_heads) * p.page_tokens * D;
  const T* kp = static_cast<const T*>(p.a.k_pages) + size_t(layer_local) * p.n_phys_pages * page_elems;
  const T* vp = static_cast<const T*>(p.a.v_pages) + size_t(layer_local) * p.n_phys_pages * page_elems;
  const int32_t* pt = p.a.page_table + size_t(seq) * p.max_pages;
  const T* kw = static_cast<const T*>(p.a.k_win) + size_t(unit) * nt * p.n_kv_heads * D;
  const T* vw = static_cast<const T*>(p.a.v_win) + size_t(unit) * nt * p.n_kv_heads * D;
  const T* qb = static_cast<const T*>(p.a.q) + size_t(unit) * nt * p.n_q_heads * D;

  // queries of this warp -> Qs[warp][d][row]
  const int j0 = tile * kTileRows + warp * kRows;
  for (int idx = lane; idx < D * kRows; idx += 32) {
    const int r = idx / D, d = idx - r * D;
    const int j = j0 + r;
    Qs[warp][d][r] = j < nt ? to_f32(qb[(size_t(j) * p.n_q_heads + h) * D + d]) : 0.f;
  }

  float m[kRows], l[kRows], o[kRows][D / 32];
#pragma unroll
  for (int r = 0; r < kRows; ++r) {
    m[r] = -INFINITY; l[r] = 0.f;
#pragma unroll
    for (int i = 0; i < D / 32; ++i) o[r][i] = 0.f;
  }

  const int j_last = min(nt, (tile + 1) * kTileRows) - 1;       // last query row of the CTA
  const int64_t n_keys = n_past + j_last + 1;
  constexpr int VN = Vec16<T>::N;
  constexpr int VPR = D / VN;

  for (int64_t kc = 0; kc < n_keys; kc += kChunk) {
    __syncthreads();
    // ---- stage 32 keys / values as fp32
    for (int idx = tid; idx < kChunk * VPR; idx += kWarps * 32) {
      const int row = idx / VPR, cv = idx - row * VPR;
      const int64_t i = kc + row;
      const T *ksrc = nullptr, *vsrc = nullptr;
      if (i < n_past) {
        int64_t tok;
        bool ok = true;
        if (i < geo.init_len) {
          tok = i;
        } else if (i < geo.init_len + sel_len) {
          const int64_t r = i - geo.init_len;
          const int blk = sel[r / p.block];
          ok = blk >= 0 && blk < geo.n_cand;
          tok = int64_t(p.n_init) + int64_t(blk) * p.block + r % p.block;
          if (!ok && cv == 0) set_status(p.a.status, ACTQKV_DEV_BAD_SELECTION);
        } else {
          tok = geo.local_start + (i - geo.init_len - sel_len);
        }
        if (ok) {
          const int64_t lp = tok / p.page_tokens;
          const int phys = lp < p.max_pages ? pt[lp] : -1;
          if (phys < 0 || phys >= p.n_phys_pages) {
            if (cv == 0) set_status(p.a.status, ACTQKV_DEV_BAD_PAGE);
          } else {
            const size_t off = (size_t(phys) * p.n_kv_heads + g) * p.page_tokens * D +
                               size_t(tok % p.page_tokens) * D + cv * VN;
            ksrc = kp + off;
            vsrc = vp + off;
          }
        }
      } else if (i < n_past + nt) {
        const size_t off = (size_t(i - n_past) * p.n_kv_heads + g) * D + cv * VN;
        ksrc = kw + off;
        vsrc = vw + off;
      }
      float kf[VN], vf[VN];
      if (ksrc) {
        Vec16<T>::load_nc(ksrc, kf);
        Vec16<T>::load_nc(vsrc, vf);
      } else {
#pragma unroll
        for (int e = 0; e < VN; ++e) { kf[e] = 0.f; vf[e] = 0.f; }
      }
#pragma unroll
      for (int e = 0; e < VN; ++e) {
        Ks[row][cv * VN + e] = kf[e];
        Vs[row][cv * VN + e] = vf[e];
      }
    }
    __syncthreads();

    // ---- S = Q K^T for this warp's rows; lane = key
    float s[kRows] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll 8
    for (int d = 0; d < D; ++d) {
      const float kv = Ks[lane][d];
      const float4 q4 = *reinterpret_cast<const float4*>(&Qs[warp][d][0]);
      s[0] = fmaf(kv, q4.x, s[0]);
      s[1] = fmaf(kv, q4.y, s[1]);
      s[2] = fmaf(kv, q4.z, s[2]);
      s[3] = fmaf(kv, q4.w, s[3]);
    }
    const int64_t ki = kc + lane;
    float pr[kRows];
#pragma unroll
    for (int r = 0; r < kRows; ++r) {
      const int j = j0 + r;
      const bool valid = ki < n_past || (ki - n_past <= j && j < nt);
      const float x = valid ? s[r] * p.scale_log2 : -INFINITY;
      const float cmax = warp_max(x);
      const float m_new = fmaxf(m[r], cmax);
      float corr = 1.f, e = 0.f;
      if (m_new != -INFINITY) {
        corr = exp2f(m[r] - m_new);
        e = exp2f(x - m_new);
      }
      l[r] = l[r] * corr + warp_sum(e);
      m[r] = m_new;
      pr[r] = e;
#pragma unroll
      for (int i = 0; i < D / 32; ++i) o[r][i] *= corr;
    }
    // ---- O += P V; lane = channel (mod 32)
#pragma unroll 4
    for (int kk = 0; kk < kChunk; ++kk) {
      float vv[D / 32];
#pragma unroll
      for (int i = 0; i < D / 32; ++i) vv[i] = Vs[kk][lane + 32 * i];
#pragma unroll
      for (int r = 0; r < kRows; ++r) {
        const float pk = __shfl_sync(0xffffffffu, pr[r], kk);
#pragma unroll
        for (int i = 0; i < D / 32; ++i) o[r][i] = fmaf(pk, vv[i], o[r][i]);
      }
    }
  }

  TO* ob = static_cast<TO*>(p.a.out) + size_t(unit) * nt * p.n_q_heads * D;
#pragma unroll
  for (int r = 0; r < kRows; ++r) {
    const int j = j0 + r;
    if (j >= nt) continue;
    const float inv = l[r] > 0.f ? 1.f / l[r] : 0.f;
#pragma unroll
    for (int i = 0; i < D / 32; ++i)
      ob[(size_t(j) * p.n_q_heads + h) * D + lane + 32 * i] = from_f32<TO>(o[r][i] * inv);
    if (p.a.lse && lane == 0)
      p.a.lse[(size_t(unit) * p.n_q_heads + h) * nt + j] = (m[r] + log2f(l[r])) * 0.6931471805599453f;
  }
}

}  // namespace

namespace actqkv {

int launch_attention_simt(const actqkv_config* cfg, const Batch& b, const AttnArgs& a, cudaStream_t st) {
  SimtParams p;
  p.a = a;
  p.n_q_heads = cfg->n_q_heads; p.n_kv_heads = cfg->n_kv_heads; p.group = cfg->n_q_heads / cfg->n_kv_heads;
  p.block = cfg->block; p.page_tokens = cfg->page_tokens; p.n_init = cfg->n_init;
  p.n_local_prev = cfg->n_local_prev; p.cap_blocks = cfg->cap_blocks; p.max_pages = cfg->max_pages;
  p.n_phys_pages = cfg->n_phys_pages; p.n_layers = b.n_layers;
  const float scale = cfg->sm_scale > 0.f ? cfg->sm_scale : 1.f / sqrtf(float(cfg->head_dim));
  p.scale_log2 = scale * 1.4426950408889634f;
  dim3 grid((a.n_tokens + kTileRows - 1) / kTileRows, cfg->n_q_heads, b.units());
  const bool bf = cfg->dtype == ACTQKV_BF16, obf = cfg->out_dtype == ACTQKV_BF16;
  const int threads = kWarps * 32;
#define ACTQKV_SIMT_LAUNCH(T, TO, DD) attention_simt_kernel<T, TO, DD><<<grid, threads, 0, st>>>(p)
#define ACTQKV_SIMT_D(T, TO) \
  do { if (cfg->head_dim == 128) ACTQKV_SIMT_LAUNCH(T, TO, 128); else ACTQKV_SIMT_LAUNCH(T, TO, 64); } while (0)
  if (bf && obf) ACTQKV_SIMT_D(__nv_bfloat16, __nv_bfloat16);
  else if (bf) ACTQKV_SIMT_D(__nv_bfloat16, float);
  else if (obf) ACTQKV_SIMT_D(float, __nv_bfloat16);
  else ACTQKV_SIMT_D(float, float);
#undef ACTQKV_SIMT_D
#undef ACTQKV_SIMT_LAUNCH
  return launch_status();
}

}  // namespace actqkv
