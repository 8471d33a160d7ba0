// Step 6: cache append (Eq. 4) and representative keys of the blocks the step completes.
//
// One launch, two roles selected by blockIdx.x:
//   copy CTAs   scatter the step's K / V rows into their pages (16-byte vectors);
//   repr CTAs   one per (completed block, KV head, representative): each representative is the
//               mean of B/r consecutive keys, read as 16-byte vectors by all threads at once
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
__global__ void __launch_bounds__(kThreads) append_kernel(AppendParams p) {
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
    // ---- copy role: one 16-byte vector of K and of V per thread iteration
    const int64_t total = int64_t(p.n_tokens) * p.n_kv_heads * vpr;
    for (int64_t idx = int64_t(blockIdx.x) * kThreads + tid; idx < total; idx += int64_t(p.copy_ctas) * kThreads) {
      const int cv = int(idx % vpr);
      const int g = int((idx / vpr) % p.n_kv_heads);
      const int j = int(idx / (int64_t(vpr) * p.n_kv_heads));
      const int64_t tok = p0 + j;
      const int64_t lp = tok / p.page_tokens;
      const int phys = lp < p.max_pages ? pt[lp] : -1;
      if (phys < 0 || phys >= p.n_phys_pages) {
        if (cv == 0) set_status(p.status, ACTQKV_DEV_BAD_PAGE);
        continue;
      }
      const size_t src = (size_t(j) * p.n_kv_heads + g) * D + cv * VN;
      const size_t dst = (size_t(phys) * p.n_kv_heads + g) * p.page_tokens * D +
                         size_t(tok % p.page_tokens) * D + cv * VN;
      *reinterpret_cast<uint4*>(kp + dst) = __ldg(reinterpret_cast<const uint4*>(kw + src));
      *reinterpret_cast<uint4*>(vp + dst) = __ldg(reinterpret_cast<const uint4*>(vw + src));
    }
    return;
  }

  // ---- repr role: one CTA per (completed block, KV head, representative)
  const int rid = blockIdx.x - p.copy_ctas;
  const int i = rid % p.n_repr;
  const int g = (rid / p.n_repr) % p.n_kv_heads, nb = rid / (p.n_repr * p.n_kv_heads);
  const int64_t p1 = p0 + p.n_tokens;
  const int64_t done0 = p0 > p.n_init ? (p0 - p.n_init) / p.block : 0;
  const int64_t done1 = p1 > p.n_init ? (p1 - p.n_init) / p.block : 0;
  const int64_t b = done0 + nb;
  if (b >= done1) return;
  if (b >= p.n_cap) {
    if (tid == 0) set_status(p.status, ACTQKV_DEV_TABLE_FULL);
    return;
  }
  // Thread t owns the 16-byte channel vector cv of rows rsub, rsub + rpp, ... of each chunk; the
  // rpp partial sums of a channel are then added in a fixed order.  fp64 throughout: exact for
  // bf16 keys, so the rounded table does not depend on the order.
  extern __shared__ __align__(16) unsigned char append_smem[];
  double* red = reinterpret_cast<double*>(append_smem);            // [rpp][D]
  float* sq_s = reinterpret_cast<float*>(red + size_t(kThreads / vpr) * D);   // [D]
  const int rpp = kThreads / vpr;                                   // rows per pass
  const int cv = tid % vpr, rsub = tid / vpr;
  const int seg = p.block / p.n_repr;
  const size_t row0 = ((size_t(unit) * p.n_kv_heads + g) * p.n_cap + size_t(b)) * p.n_repr;
  T* tab = static_cast<T*>(p.repr_k) + row0 * D;
  const int64_t blk0 = int64_t(p.n_init) + b * p.block;
  {
    const int lo = p.repr_mode == ACTQKV_REPR_CHUNK_MEAN ? i * seg : i * seg + seg / 2;
    const int hi = p.repr_mode == ACTQKV_REPR_CHUNK_MEAN ? (i + 1) * seg : lo + 1;
    double acc[VN];
#pragma unroll
    for (int e = 0; e < VN; ++e) acc[e] = 0.0;
    for (int r = lo + rsub; r < hi; r += rpp) {
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
        float kf[VN];
        Vec16<T>::load_nc(src, kf);
#pragma unroll
        for (int e = 0; e < VN; ++e) acc[e] += double(kf[e]);
      }
    }
#pragma unroll
    for (int e = 0; e < VN; ++e) red[size_t(rsub) * D + cv * VN + e] = acc[e];
    __syncthreads();
    if (tid < D) {
      double t = 0.0;
      for (int q = 0; q < rpp; ++q) t += red[size_t(q) * D + tid];
      const double mean = t / double(hi - lo);
      const T rounded = from_f32<T>(float(mean));   // fp64 -> fp32 -> dtype, both nearest-even
      tab[size_t(i) * D + tid] = rounded;
      const float stored = to_f32(rounded);
      sq_s[tid] = stored * stored;
    }
    __syncthreads();
    if (tid < 32) {                       // fixed order: lane partial sums, then a shuffle tree
      float t = 0.f;
      for (int cc = tid; cc < D; cc += 32) t += sq_s[cc];
      t = warp_sum(t);
      if (tid == 0) p.repr_inv_norm[row0 + i] = t > 0.f ? rsqrtf(t) : 0.f;
    }
  }
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
  const int64_t vecs = int64_t(n_tokens) * cfg->n_kv_heads * vpr;
  p.copy_ctas = int(std::min<int64_t>((vecs + kThreads - 1) / kThreads, 296));
  p.max_new_blocks = n_tokens / cfg->block + 2;
  dim3 grid(p.copy_ctas + p.max_new_blocks * cfg->n_kv_heads * cfg->n_repr, b.units());
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  const size_t smem = sizeof(double) * size_t(kThreads / vpr) * cfg->head_dim + sizeof(float) * cfg->head_dim;
  prefer_max_shared(append_kernel<__nv_bfloat16>);
  prefer_max_shared(append_kernel<float>);
  if (cfg->dtype == ACTQKV_BF16) append_kernel<__nv_bfloat16><<<grid, kThreads, smem, st>>>(p);
  else append_kernel<float><<<grid, kThreads, smem, st>>>(p);
  return launch_status();
}
