// Helpers of the C ABI and the dispatcher of step 5.
#include "common.cuh"
#include "stages.cuh"

using namespace actqkv;

extern "C" int actqkv_version(void) { return ACTQKV_VERSION; }

extern "C" const char* actqkv_strerror(int status) {
  switch (status) {
    case ACTQKV_OK: return "ok";
    case ACTQKV_ERR_NULL: return "a required pointer is NULL";
    case ACTQKV_ERR_ALIGN: return "a data pointer is not 16-byte aligned";
    case ACTQKV_ERR_SHAPE: return "unsupported shape or geometry";
    case ACTQKV_ERR_DTYPE: return "unsupported dtype";
    case ACTQKV_ERR_LAUNCH: return "the CUDA runtime refused the launch";
    case ACTQKV_ERR_UNSUPPORTED: return "valid request this build cannot serve";
    case ACTQKV_ERR_SCRATCH_LIMIT: return "the call needs more scratch than the library's built-in array holds";
    default: return "unknown actqkv status";
  }
}

extern "C" int64_t actqkv_budget_state_bytes(const actqkv_config* cfg) {
  return cfg ? int64_t(sizeof(double)) * (1 + 2 * int64_t(cfg->n_layers)) : 0;
}

extern "C" int32_t actqkv_n_candidates(const actqkv_config* cfg, int64_t p0) {
  if (!cfg || cfg->block <= 0) return 0;
  return make_geometry(p0, cfg->n_init, cfg->block, cfg->n_local_prev).n_cand;
}

extern "C" int actqkv_retrieval_attention(const actqkv_config* cfg, const actqkv_batch* batch, const void* q,
                                          const void* k_win, const void* v_win, int32_t n_tokens,
                                          const void* k_pages, const void* v_pages, const int32_t* page_table,
                                          const int64_t* pos0, const int32_t* sel_idx, const int32_t* sel_count,
                                          void* out, float* lse, int32_t* status, void* stream) {
  const Batch b = get_batch(batch);
  int rc = check_config(cfg, b);
  if (rc) return rc;
  ACTQKV_REQUIRE_PTR(q);
  ACTQKV_REQUIRE_PTR(k_win);
  ACTQKV_REQUIRE_PTR(v_win);
  ACTQKV_REQUIRE_PTR(k_pages);
  ACTQKV_REQUIRE_PTR(v_pages);
  ACTQKV_REQUIRE_PTR(out);
  ACTQKV_OPTIONAL_PTR(lse);
  if (!page_table || !pos0) return ACTQKV_ERR_NULL;
  if (cfg->cap_blocks > 0 && (!sel_idx || !sel_count)) return ACTQKV_ERR_NULL;
  if (n_tokens <= 0 || n_tokens > cfg->window) return ACTQKV_ERR_SHAPE;
  AttnArgs a;
  a.q = q; a.k_win = k_win; a.v_win = v_win; a.k_pages = k_pages; a.v_pages = v_pages;
  a.page_table = page_table; a.pos0 = pos0; a.sel_idx = sel_idx; a.sel_count = sel_count;
  a.out = out; a.lse = lse; a.status = status; a.n_tokens = n_tokens;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  // cfg->attention_kernel pins one kernel (for comparing kernels with each other); 0 picks by shape
  const bool simt_only = cfg->attention_kernel == ACTQKV_ATTN_GENERAL;
  const bool tc1_only = cfg->attention_kernel == ACTQKV_ATTN_SINGLE_CTA;
  if (cfg->attention_kernel == ACTQKV_ATTN_CLUSTER4 && attention_tc4_supported(cfg, n_tokens))
    return launch_attention_tc4(cfg, b, a, st);
  if (!simt_only && !tc1_only && attention_tc2_supported(cfg, n_tokens)) return launch_attention_tc2(cfg, b, a, st);
  if (!simt_only && attention_tc_supported(cfg, n_tokens)) return launch_attention_tc(cfg, b, a, st);
  if (!simt_only && attention_decode_supported(cfg, n_tokens)) return launch_attention_decode(cfg, b, a, 1, nullptr, st);
  return launch_attention_simt(cfg, b, a, st);
}

extern "C" int32_t actqkv_decode_splits(const actqkv_config* cfg, const actqkv_batch* batch) {
  const Batch b = get_batch(batch);
  if (check_config(cfg, b)) return 0;
  return attention_decode_auto_splits(cfg, b);
}

extern "C" int64_t actqkv_decode_workspace_bytes(const actqkv_config* cfg, const actqkv_batch* batch, int32_t n_tokens,
                                                 int32_t n_splits) {
  const Batch b = get_batch(batch);
  if (check_config(cfg, b) || n_tokens <= 0) return 0;
  if (n_splits <= 0) n_splits = attention_decode_auto_splits(cfg, b);
  return attention_decode_workspace_bytes(cfg, b, n_tokens, n_splits);
}

extern "C" int actqkv_decode_attention(const actqkv_config* cfg, const actqkv_batch* batch, const void* q,
                                       const void* k_win, const void* v_win, int32_t n_tokens, const void* k_pages,
                                       const void* v_pages, const int32_t* page_table, const int64_t* pos0,
                                       const int32_t* sel_idx, const int32_t* sel_count, void* out, float* lse,
                                       int32_t n_splits, void* workspace, int64_t workspace_bytes, int32_t* status,
                                       void* stream) {
  const Batch b = get_batch(batch);
  int rc = check_config(cfg, b);
  if (rc) return rc;
  ACTQKV_REQUIRE_PTR(q);
  ACTQKV_REQUIRE_PTR(k_win);
  ACTQKV_REQUIRE_PTR(v_win);
  ACTQKV_REQUIRE_PTR(k_pages);
  ACTQKV_REQUIRE_PTR(v_pages);
  ACTQKV_REQUIRE_PTR(out);
  ACTQKV_OPTIONAL_PTR(lse);
  ACTQKV_OPTIONAL_PTR(workspace);
  if (!page_table || !pos0) return ACTQKV_ERR_NULL;
  if (cfg->cap_blocks > 0 && (!sel_idx || !sel_count)) return ACTQKV_ERR_NULL;
  if (n_tokens <= 0 || n_tokens > cfg->window) return ACTQKV_ERR_SHAPE;
  if (!attention_decode_supported(cfg, n_tokens)) return ACTQKV_ERR_UNSUPPORTED;
  if (n_splits <= 0) n_splits = attention_decode_auto_splits(cfg, b);
  if (n_splits > 64) return ACTQKV_ERR_SHAPE;
  const int64_t need = attention_decode_workspace_bytes(cfg, b, n_tokens, n_splits);
  if (need > 0 && (!workspace || workspace_bytes < need)) return workspace ? ACTQKV_ERR_SHAPE : ACTQKV_ERR_NULL;
  AttnArgs a;
  a.q = q; a.k_win = k_win; a.v_win = v_win; a.k_pages = k_pages; a.v_pages = v_pages;
  a.page_table = page_table; a.pos0 = pos0; a.sel_idx = sel_idx; a.sel_count = sel_count;
  a.out = out; a.lse = lse; a.status = status; a.n_tokens = n_tokens;
  return launch_attention_decode(cfg, b, a, n_splits, workspace, reinterpret_cast<cudaStream_t>(stream));
}
