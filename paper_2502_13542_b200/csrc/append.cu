// Step 6: cache append (Eq. 4) and representative keys of the blocks the step completes.
//
// One launch, two roles selected by blockIdx.x:
//   copy CTAs   one per (page touched, K or V): the step's rows of that page, 16-byte vectors;
//   repr CTAs   one warp per (completed block, KV head, representative): each representative is
//               the mean of B/r consecutive keys, read as 16-byte vectors, eight in flight per lane,
//               and accumulated in fp64 (exact for bf16 inputs, so the rounded table is
//               bit-reproducible), rounded to the cache dtype; the inverse norm is taken from
//               the rounded values in a fixed order.  Keys older than the step are
//               read from the pages, the step's own keys from k_win, so the two roles do not
//               depend on each other.
#include "common.cuh"

using namespace actqkv;

namespace {

constexpr int kThreads = 256;

struct AppendParams {
  const void *k_win, *v_win;
  void *k_pages, *v_pages, *repr_k;
  float* repr_inv_norm;
  const int64_t* pos0;
  const int32_t* page_table;
  int32_t* status;
  int n_tokens, n_kv_heads, D, block, n_repr, page_tokens, n_init, n_cap, max_pages, n_phys_pages;
  int n_layers, repr_mode, copy_ctas, max_new_blocks;
};

template <typename T>
__global__ void __launch_bounds__(kThreads, 3) append_kernel(AppendParams p) {
  const int unit = blockIdx.y;
  const int seq = unit / p.n_layers, layer_local = unit - seq * p.n_layers;
  const int64_t p0 = p.pos0[seq];
  const int D = p.D, tid = threadIdx.x;
  const size_t page_elems = size_t(p.n_kv_heads) * p.page_tokens * D;
  T* kp = static_cast<T*>(p.k_pages) + size_t(layer_local) * p.n_phys_pages * page_elems;
  T* vp = static_cast<T*>(p.v_pages) + size_t(layer_local) * p.n_phys_pages * page_elems;
  const int32_t* pt = p.page_table + size_t(seq) * p.max_pages;
  const T* kw = static_cast<const T*>(p.k_win) + size_t(unit) * p.n_tokens * p.n_kv_heads * D;
  const T* vw = static_cast<const T*>(p.v_win) + size_t(unit) * p.n_tokens * p.n_kv_heads * D;
  constexpr int VN = Vec16<T>::N;
  const int vpr = D / VN;

  if (int(blockIdx.x) < p.copy_ctas) {
    // ---- copy role: one CTA per (page the step touches, K or V).  The page is contiguous in the
    // cache, [head][token in page][D], and its tokens are contiguous in the window,
    // [token][head][D]: thread-linear 16-byte vectors in the page's order, eight loads in flight
    // per thread before the first store.
    const int slot = int(blockIdx.x) >> 1;
    const bool is_v = blockIdx.x & 1;
    const int pt_tok = p.page_tokens;
    const int64_t lp = p0 / pt_tok + slot;
    const int64_t page0 = lp * pt_tok;
    const int t_lo = int(max(p0, page0) - page0);
    const int t_hi = int(min(p0 + p.n_tokens, page0 + pt_tok) - page0);
    if (t_lo >= t_hi) return;
    const int phys = lp < p.max_pages ? pt[lp] : -1;
    if (phys < 0 || phys >= p.n_phys_pages) {
      if (tid == 0) set_status(p.status, ACTQKV_DEV_BAD_PAGE);
      return;
    }
    const uint4* src = reinterpret_cast<const uint4*>((is_v ? vw : kw) + size_t(page0 - p0 + t_lo) * p.n_kv_heads * D);
    uint4* dst = reinterpret_cast<uint4*>((is_v ? vp : kp) + size_t(phys) * page_elems);
    // Thread = (row lane rl, channel vector cv); a row is one token of one head.  Heads in the
    // unrolled loop, so that no index needs a division.
    const int nt = t_hi - t_lo;                              // tokens of this page in the step
    const int cv = tid % vpr, rl = tid / vpr, n_rl = kThreads / vpr;
    constexpr int kUnroll = 8;
    for (int t = rl; t < nt; t += n_rl) {
      const uint4* s_row = src + size_t(t) * p.n_kv_heads * vpr + cv;
      uint4* d_row = dst + size_t(t_lo + t) * vpr + cv;
      for (int g0 = 0; g0 < p.n_kv_heads; g0 += kUnroll) {
        uint4 val[kUnroll];
#pragma unroll
        for (int u = 0; u < kUnroll; ++u)
          if (g0 + u < p.n_kv_heads) val[u] = __ldg(s_row + (g0 + u) * vpr);
#pragma unroll
        for (int u = 0; u < kUnroll; ++u)
          if (g0 + u < p.n_kv_heads) d_row[size_t(g0 + u) * pt_tok * vpr] = val[u];
      }
    }
    // The step ends inside this page: the rows after it are zeroed, so that an attention step that
    // loads the page whole (and masks those rows) multiplies weight 0 by a finite value.
    if (p0 + p.n_tokens < page0 + pt_tok) {
      for (int t = t_hi + rl; t < pt_tok; t += n_rl)
        for (int g = 0; g < p.n_kv_heads; ++g) dst[(size_t(g) * pt_tok + t) * vpr + cv] = make_uint4(0, 0, 0, 0);
    }
    return;
  }

  // ---- repr role: one warp per (completed block, KV head, representative)
  const int warp = tid >> 5, lane = tid & 31;
  const int rid = (int(blockIdx.x) - p.copy_ctas) * (kThreads / 32) + warp;
  const int i = rid % p.n_repr;
  const int g = (rid / p.n_repr) % p.n_kv_heads, nb = rid / (p.n_repr * p.n_kv_heads);
  const int64_t p1 = p0 + p.n_tokens;
  const int64_t done0 = p0 > p.n_init ? (p0 - p.n_init) / p.block : 0;
  const int64_t done1 = p1 > p.n_init ? (p1 - p.n_init) / p.block : 0;
  const int64_t b = done0 + nb;
  if (b >= done1) return;
  if (b >= p.n_cap) {
    if (lane == 0) set_status(p.status, ACTQKV_DEV_TABLE_FULL);
    return;
  }
  // Lane = (row lane rsub, channel vector cv): it adds its vector of rows rsub, rsub + rpp, ... in
  // fp64 (exact for bf16 keys, so the rounded table does not depend on the order), then the row
  // lanes are added by shuffles in a fixed order.  vpr <= 32 lanes hold one row.
  const int rpp = 32 / vpr;                                         // rows per pass of the warp
  const int cv = lane % vpr, rsub = lane / vpr;
  const int seg = p.block / p.n_repr;
  const size_t row0 = ((size_t(unit) * p.n_kv_heads + g) * p.n_cap + size_t(b)) * p.n_repr;
  T* tab = static_cast<T*>(p.repr_k) + row0 * D;
  const int64_t blk0 = int64_t(p.n_init) + b * p.block;
  const int lo = p.repr_mode == ACTQKV_REPR_CHUNK_MEAN ? i * seg : i * seg + seg / 2;
  const int hi = p.repr_mode == ACTQKV_REPR_CHUNK_MEAN ? (i + 1) * seg : lo + 1;
  double acc[VN];
#pragma unroll
  for (int e = 0; e < VN; ++e) acc[e] = 0.0;
  constexpr int kAhead = 8;                                         // 16-byte loads in flight per lane
  for (int rb = lo + rsub; rb < hi; rb += rpp * kAhead) {
    uint4 raw[kAhead];
    bool have[kAhead];
#pragma unroll
    for (int u = 0; u < kAhead; ++u) {
      const int r = rb + u * rpp;
      have[u] = false;
      if (r < hi) {
        const int64_t tok = blk0 + r;
        const T* src = nullptr;
        if (tok >= p0) {
          src = kw + (size_t(tok - p0) * p.n_kv_heads + g) * D + cv * VN;
        } else {
          const int64_t lp = tok / p.page_tokens;
          const int phys = lp < p.max_pages ? pt[lp] : -1;
          if (phys < 0 || phys >= p.n_phys_pages) {
            if (cv == 0) set_status(p.status, ACTQKV_DEV_BAD_PAGE);
          } else {
            src = kp + (size_t(phys) * p.n_kv_heads + g) * p.page_tokens * D + size_t(tok % p.page_tokens) * D + cv * VN;
          }
        }
        if (src) {
          raw[u] = __ldg(reinterpret_cast<const uint4*>(src));
          have[u] = true;
        }
      }
    }
#pragma unroll
    for (int u = 0; u < kAhead; ++u)
      if (have[u]) {
        float kf[VN];
        Vec16<T>::unpack(raw[u], kf);
#pragma unroll
        for (int e = 0; e < VN; ++e) acc[e] += double(kf[e]);
      }
  }
  // row lanes -> row lane 0, nearest partner first
#pragma unroll
  for (int e = 0; e < VN; ++e)
    for (int o = vpr; o < 32; o <<= 1) acc[e] += __shfl_down_sync(0xffffffffu, acc[e], o);
  float sq = 0.f;
  if (rsub == 0) {
    __align__(16) T outv[VN];
#pragma unroll
    for (int e = 0; e < VN; ++e) {
      outv[e] = from_f32<T>(float(acc[e] / double(hi - lo)));          // fp64 -> fp32 -> dtype, both nearest-even
      const float stored = to_f32(outv[e]);
      sq = fmaf(stored, stored, sq);
    }
    *reinterpret_cast<uint4*>(tab + size_t(i) * D + cv * VN) = *reinterpret_cast<const uint4*>(outv);
  }
  sq = warp_sum(sq);                                                   // fixed order: per-lane sums, then a shuffle tree
  if (lane == 0) p.repr_inv_norm[row0 + i] = sq > 0.f ? rsqrtf(sq) : 0.f;
}

}  // namespace

extern "C" int actqkv_append_window(const actqkv_config* cfg, const actqkv_batch* batch, const void* k_win,
                                    const void* v_win, int32_t n_tokens, const int64_t* pos0, void* k_pages,
                                    void* v_pages, const int32_t* page_table, void* repr_k,
                                    float* repr_inv_norm, int32_t* status, void* stream) {
  const Batch b = get_batch(batch);
  int rc = check_config(cfg, b);
  if (rc) return rc;
  ACTQKV_REQUIRE_PTR(k_win);
  ACTQKV_REQUIRE_PTR(v_win);
  ACTQKV_REQUIRE_PTR(k_pages);
  ACTQKV_REQUIRE_PTR(v_pages);
  ACTQKV_REQUIRE_PTR(repr_k);
  ACTQKV_REQUIRE_PTR(repr_inv_norm);
  if (!pos0 || !page_table) return ACTQKV_ERR_NULL;
  if (n_tokens <= 0 || n_tokens > cfg->window) return ACTQKV_ERR_SHAPE;
  AppendParams p;
  p.k_win = k_win; p.v_win = v_win; p.k_pages = k_pages; p.v_pages = v_pages; p.repr_k = repr_k;
  p.repr_inv_norm = repr_inv_norm; p.pos0 = pos0; p.page_table = page_table; p.status = status;
  p.n_tokens = n_tokens; p.n_kv_heads = cfg->n_kv_heads; p.D = cfg->head_dim; p.block = cfg->block;
  p.n_repr = cfg->n_repr; p.page_tokens = cfg->page_tokens; p.n_init = cfg->n_init; p.n_cap = cfg->n_cap;
  p.max_pages = cfg->max_pages; p.n_phys_pages = cfg->n_phys_pages; p.n_layers = b.n_layers;
  p.repr_mode = cfg->repr_mode;
  const int vpr = cfg->head_dim * int(elt_size(cfg)) / 16;
  p.copy_ctas = 2 * (n_tokens / cfg->page_tokens + 2);      // K and V of every page the step can touch
  p.max_new_blocks = n_tokens / cfg->block + 2;
  const int n_reprs = p.max_new_blocks * cfg->n_kv_heads * cfg->n_repr;
  dim3 grid(p.copy_ctas + (n_reprs + kThreads / 32 - 1) / (kThreads / 32), b.units());
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  if (vpr > 32 || 32 % vpr != 0 || kThreads % vpr != 0) return ACTQKV_ERR_SHAPE;
  if (cfg->dtype == ACTQKV_BF16) append_kernel<__nv_bfloat16><<<grid, kThreads, 0, st>>>(p);
  else append_kernel<float><<<grid, kThreads, 0, st>>>(p);
  return launch_status();
}
