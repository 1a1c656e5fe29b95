// C ABI of the WeDLM step library: argument validation, workspace planning, kernel dispatch.
#include <atomic>

#include "common.cuh"

using namespace wedlm;

namespace {
std::atomic<unsigned long long> g_launches{0};
// One-shot profiling hook: events to record around the main attention kernel of the next
// wedlm_window_attn call made by this thread.
thread_local cudaEvent_t t_ev_before = nullptr;
thread_local cudaEvent_t t_ev_after = nullptr;
}  // namespace

namespace wedlm {
void count_launch(int n) { g_launches.fetch_add((unsigned long long)n, std::memory_order_relaxed); }

int device_sm_count() {
  constexpr int kFallbackSms = 148;
  static std::atomic<int> cached[64] = {};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); return kFallbackSms; }
  if (dev >= 0 && dev < 64) {
    const int have = cached[dev].load(std::memory_order_relaxed);
    if (have > 0) return have;
  }
  int sms = 0;
  if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms < 1) {
    cudaGetLastError();
    return kFallbackSms;
  }
  if (dev >= 0 && dev < 64) cached[dev].store(sms, std::memory_order_relaxed);
  return sms;
}
}  // namespace wedlm

namespace {

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// Checks every field a call may rely on.  `need_vocab` / `need_cache` select the groups used.
int check_config(const wedlm_config_t* c, bool need_cache, bool need_vocab) {
  if (c == nullptr) return WEDLM_ERR_INVALID_ARG;
  if (c->batch < 0 || c->window < 1 || c->window > 1024) return WEDLM_ERR_INVALID_ARG;
  if (c->dtype != WEDLM_DTYPE_BF16 && c->dtype != WEDLM_DTYPE_F32) return WEDLM_ERR_INVALID_ARG;
  if (c->commit_mode != WEDLM_COMMIT_STREAMING && c->commit_mode != WEDLM_COMMIT_BLOCK) return WEDLM_ERR_INVALID_ARG;
  if (need_cache) {
    if (c->n_q_heads < 1 || c->n_kv_heads < 1 || c->n_q_heads % c->n_kv_heads != 0) return WEDLM_ERR_INVALID_ARG;
    if (c->head_dim != 32 && c->head_dim != 64 && c->head_dim != 128 && c->head_dim != 256) return WEDLM_ERR_UNSUPPORTED;
    if (c->page_size != 8 && c->page_size != 16 && c->page_size != 32) return WEDLM_ERR_UNSUPPORTED;
    if (c->max_pages_per_seq < 1 || c->num_pages < 1) return WEDLM_ERR_INVALID_ARG;
    if (c->rope_style != 0 && c->rope_style != 1) return WEDLM_ERR_INVALID_ARG;
    if (!(c->rope_theta > 0.f) || c->softmax_scale < 0.f) return WEDLM_ERR_INVALID_ARG;
    if (c->max_prefix_len < 0) return WEDLM_ERR_INVALID_ARG;
    if ((long long)c->max_prefix_len + c->window > (long long)c->max_pages_per_seq * c->page_size) return WEDLM_ERR_INVALID_ARG;
    if (c->attn_impl < WEDLM_ATTN_AUTO || c->attn_impl > WEDLM_ATTN_TENSOR) return WEDLM_ERR_INVALID_ARG;
  }
  if (need_vocab) {
    if (c->vocab < 1) return WEDLM_ERR_INVALID_ARG;
    if (c->conf_mode != WEDLM_CONF_ENTROPY && c->conf_mode != WEDLM_CONF_MAXPROB) return WEDLM_ERR_INVALID_ARG;
    if (c->tau != c->tau || c->lambda != c->lambda || c->maxprob_thr != c->maxprob_thr) return WEDLM_ERR_INVALID_ARG;
    if (!(c->sample_temperature >= 0.f) || c->sample_temperature > 3.0e38f) return WEDLM_ERR_INVALID_ARG;
  }
  return WEDLM_OK;
}

Shape make_shape(const wedlm_config_t* c) {
  Shape s;
  s.B = c->batch; s.W = c->window; s.Hq = c->n_q_heads; s.Hkv = c->n_kv_heads; s.D = c->head_dim;
  s.G = c->n_kv_heads > 0 ? c->n_q_heads / c->n_kv_heads : 1;
  s.page = c->page_size; s.max_pages = c->max_pages_per_seq; s.num_pages = c->num_pages; s.V = c->vocab;
  s.dtype = c->dtype; s.rope_style = c->rope_style; s.theta = c->rope_theta; s.commit_mode = c->commit_mode;
  s.max_prefix = c->max_prefix_len;
  s.scale = c->softmax_scale > 0.f ? c->softmax_scale : 1.0f / sqrtf((float)c->head_dim);
  return s;
}

size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

}  // namespace

namespace wedlm {

AttnPlan plan_attention(const wedlm_config_t* c) {
  AttnPlan p{};
  const int elem = c->dtype == WEDLM_DTYPE_BF16 ? 2 : 4;
  const long long total = (long long)c->max_prefix_len + c->window;
  const bool tensor_ok = attn_tensor_supported(c);
  p.impl = (c->attn_impl == WEDLM_ATTN_GENERIC || !tensor_ok) ? WEDLM_ATTN_GENERIC : WEDLM_ATTN_TENSOR;
  long long S, chunk;
  if (p.impl == WEDLM_ATTN_TENSOR) {
    // Two CTAs per SM.  With at least one work unit (sequence, kv head, 128-row tile) per CTA slot, every CTA takes
    // one whole unit, longest first, and no partials exist at all.  With fewer units the 64-key tiles of all units
    // are cut into one equal run per slot; a unit that is cut leaves one partial per piece, at most n_splits of them
    // (the kernel keeps its runs long enough for that).
    const int G = c->n_q_heads / c->n_kv_heads;
    const long long w_t = 128 / G;
    const long long n_mtiles = (c->window + w_t - 1) / w_t;
    const long long units = (long long)c->batch * c->n_kv_heads * n_mtiles;
    const long long slots = 2LL * device_sm_count();
    S = 1;
    chunk = (total + 63) / 64 * 64;
    if (units > 0 && units < slots) {
      p.balanced = 1;
      const long long n_runs = slots / n_mtiles > 0 ? slots / n_mtiles : 1;     // a run is shared by the row tiles
      p.n_ctas = (int)(n_runs * n_mtiles);
      const long long t_max = (total + 63) / 64;
      S = n_runs / c->n_kv_heads + 3;
      if (S > t_max) S = t_max;
      if (S < 2) S = 2;
    }
  } else {
    const long long n_rb = (c->window + 15) / 16;
    const long long units = (long long)c->batch * c->n_q_heads * n_rb;
    long long want = units > 0 ? (4LL * device_sm_count() + units - 1) / units : 1;      // a few blocks per SM
    long long cap = total / 256 > 1 ? total / 256 : 1;                      // keep chunks >= 256 keys
    S = want < 1 ? 1 : (want > cap ? cap : want);
    chunk = (total + S - 1) / S;
    chunk = (chunk + c->page_size - 1) / c->page_size * c->page_size;
  }
  if (!p.balanced) S = (total + chunk - 1) / chunk;
  p.n_splits = (int)S;
  p.chunk = (int)chunk;
  p.q_rot_bytes = align_up((size_t)c->batch * c->window * c->n_q_heads * c->head_dim * elem, 256);
  if (S > 1) {
    size_t rows = (size_t)c->batch * c->n_q_heads * c->window * (size_t)S;
    p.part_o_bytes = align_up(rows * c->head_dim * sizeof(float), 256);
    p.part_ml_bytes = align_up(rows * 2 * sizeof(float), 256);
  }
  // dispatch order of the sequences (i32 per sequence), or the record of the balanced cut (i64: 2 + one per sequence)
  p.order_bytes = align_up(((size_t)c->batch + 2) * sizeof(long long), 256);
  p.total_bytes = p.q_rot_bytes + p.part_o_bytes + p.part_ml_bytes + p.order_bytes;
  return p;
}

}  // namespace wedlm

extern "C" {

const char* wedlm_strerror(int code) {
  switch (code) {
    case WEDLM_OK: return "ok";
    case WEDLM_ERR_INVALID_ARG: return "invalid argument";
    case WEDLM_ERR_UNSUPPORTED: return "unsupported configuration";
    case WEDLM_ERR_WORKSPACE_TOO_SMALL: return "workspace too small";
    case WEDLM_ERR_CUDA: return "CUDA error";
    case WEDLM_ERR_TIMEOUT: return "device wait expired";
    case WEDLM_ERR_STATIC_SCRATCH: return "problem too large for the built-in scratch array";
    default: return "unknown error code";
  }
}

int wedlm_version(void) { return 200; }

unsigned long long wedlm_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

int wedlm_selftest_wait_expiry(uint32_t max_polls, int32_t* status, void* stream) {
  if (status == nullptr || max_polls == 0 || max_polls > (1u << 24)) return WEDLM_ERR_INVALID_ARG;
  return launch_wait_expiry_selftest(max_polls, status, (cudaStream_t)stream);
}

int wedlm_profile_next_attn(void* event_before, void* event_after) {
  t_ev_before = (cudaEvent_t)event_before;
  t_ev_after = (cudaEvent_t)event_after;
  return WEDLM_OK;
}

int wedlm_reorder(const wedlm_config_t* cfg, const uint8_t* filled, const int32_t* window_tokens,
                  const int32_t* prefix_len, const int32_t* window_len, int32_t* perm, int32_t* inv_perm,
                  int32_t* pos_ids, int32_t* tokens_phys, int32_t* n_filled, int32_t* n_commit, void* stream) {
  ApiRange nvtx_range("wedlm_reorder");
  int rc = check_config(cfg, false, false);
  if (rc != WEDLM_OK) return rc;
  if (cfg->batch == 0) return WEDLM_OK;
  if (!filled || !prefix_len || !perm || !inv_perm || !pos_ids || !n_filled || !n_commit) return WEDLM_ERR_INVALID_ARG;
  if (tokens_phys && !window_tokens) return WEDLM_ERR_INVALID_ARG;
  return launch_reorder(make_shape(cfg), filled, window_tokens, prefix_len, window_len, perm, inv_perm, pos_ids,
                        tokens_phys, n_filled, n_commit, (cudaStream_t)stream);
}

size_t wedlm_window_attn_workspace_bytes(const wedlm_config_t* cfg) {
  if (check_config(cfg, true, false) != WEDLM_OK) return 0;
  size_t b = plan_attention(cfg).total_bytes;
  return b ? b : 256;
}

int wedlm_window_attn(const wedlm_config_t* cfg, const void* q, const void* k, const void* v, void* k_cache,
                      void* v_cache, const int32_t* block_table, const int32_t* prefix_len, const int32_t* pos_ids,
                      void* out, int32_t* kv_slot_idx, void* workspace, size_t workspace_bytes, int32_t* status,
                      void* stream) {
  ApiRange nvtx_range("wedlm_window_attn");
  int rc = check_config(cfg, true, false);
  if (rc != WEDLM_OK) return rc;
  if (cfg->batch == 0) return WEDLM_OK;
  if (!q || !k || !v || !k_cache || !v_cache || !block_table || !prefix_len || !pos_ids || !out || !workspace)
    return WEDLM_ERR_INVALID_ARG;
  if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(k_cache) || !aligned16(v_cache) ||
      !aligned16(out) || !aligned16(workspace))
    return WEDLM_ERR_INVALID_ARG;
  if (cfg->attn_impl == WEDLM_ATTN_TENSOR && !attn_tensor_supported(cfg)) return WEDLM_ERR_UNSUPPORTED;
  AttnPlan plan = plan_attention(cfg);
  if (workspace_bytes < plan.total_bytes) return WEDLM_ERR_WORKSPACE_TOO_SMALL;
  Shape s = make_shape(cfg);
  cudaStream_t st = (cudaStream_t)stream;
  char* ws = static_cast<char*>(workspace);
  void* q_rot = ws;
  float* part_o = reinterpret_cast<float*>(ws + plan.q_rot_bytes);
  float* part_ml = reinterpret_cast<float*>(ws + plan.q_rot_bytes + plan.part_o_bytes);
  int32_t* order = reinterpret_cast<int32_t*>(ws + plan.q_rot_bytes + plan.part_o_bytes + plan.part_ml_bytes);
  rc = launch_rope_stage(s, q, k, v, q_rot, k_cache, v_cache, block_table, prefix_len, pos_ids, nullptr, kv_slot_idx,
                         plan.impl == WEDLM_ATTN_TENSOR ? order : nullptr, status, st);
  if (rc != WEDLM_OK) return rc;
  cudaEvent_t ev0 = t_ev_before, ev1 = t_ev_after;
  t_ev_before = t_ev_after = nullptr;
  if (ev0 && cudaEventRecord(ev0, st) != cudaSuccess) return WEDLM_ERR_CUDA;
  if (plan.impl == WEDLM_ATTN_TENSOR)
    rc = launch_attn_tensor(s, plan, q_rot, k_cache, v_cache, block_table, prefix_len, order, out, part_o, part_ml, status, st);
  else
    rc = launch_attn_generic(s, plan, q_rot, k_cache, v_cache, block_table, prefix_len, out, part_o, part_ml, status, st);
  if (ev1 && cudaEventRecord(ev1, st) != cudaSuccess) return WEDLM_ERR_CUDA;
  if (rc != WEDLM_OK) return rc;
  if (plan.impl == WEDLM_ATTN_TENSOR)
    rc = launch_attn_tensor_merge(s, plan, prefix_len, order, part_o, part_ml, out, st);
  else if (plan.n_splits > 1)
    rc = launch_attn_merge(s, plan, prefix_len, part_o, part_ml, out, st);
  return rc;
}

int wedlm_kv_append(const wedlm_config_t* cfg, const void* k, const void* v, const int32_t* pos_ids, void* k_cache,
                    void* v_cache, const int32_t* block_table, const int32_t* prefix_len, const int32_t* count,
                    int32_t* kv_slot_idx, int32_t* status, void* stream) {
  ApiRange nvtx_range("wedlm_kv_append");
  int rc = check_config(cfg, true, false);
  if (rc != WEDLM_OK) return rc;
  if (cfg->batch == 0) return WEDLM_OK;
  if (!k || !v || !k_cache || !v_cache || !block_table || !prefix_len) return WEDLM_ERR_INVALID_ARG;
  if (!aligned16(k) || !aligned16(v) || !aligned16(k_cache) || !aligned16(v_cache)) return WEDLM_ERR_INVALID_ARG;
  return launch_rope_stage(make_shape(cfg), nullptr, k, v, nullptr, k_cache, v_cache, block_table, prefix_len, pos_ids,
                           count, kv_slot_idx, nullptr, status, (cudaStream_t)stream);
}

size_t wedlm_confidence_workspace_bytes(const wedlm_config_t* cfg) {
  if (check_config(cfg, false, true) != WEDLM_OK) return 0;
  size_t b = confidence_workspace_bytes(cfg);
  return b ? b : 256;
}

int wedlm_confidence_commit(const wedlm_config_t* cfg, const void* logits, const int32_t* perm,
                            const int32_t* n_filled, const int32_t* n_commit, int32_t* window_tokens,
                            uint8_t* filled, int32_t* prefix_len, int32_t* window_len, int32_t* remaining_budget,
                            int32_t* argmax, float* maxprob, float* entropy, float* lse, int32_t* committed_tokens,
                            int32_t* committed_count, int32_t* filled_count, void* workspace, size_t workspace_bytes,
                            int32_t* status, void* stream) {
  ApiRange nvtx_range("wedlm_confidence_commit");
  int rc = check_config(cfg, false, true);
  if (rc != WEDLM_OK) return rc;
  if (cfg->batch == 0) return WEDLM_OK;
  if (!logits || !perm || !n_filled || !n_commit || !window_tokens || !filled || !prefix_len || !workspace)
    return WEDLM_ERR_INVALID_ARG;
  if (!aligned16(workspace)) return WEDLM_ERR_INVALID_ARG;
  if (workspace_bytes < confidence_workspace_bytes(cfg)) return WEDLM_ERR_WORKSPACE_TOO_SMALL;
  return launch_confidence(make_shape(cfg), cfg, logits, perm, n_filled, n_commit, window_tokens, filled, prefix_len,
                           window_len, remaining_budget, argmax, maxprob, entropy, lse, committed_tokens,
                           committed_count, filled_count, workspace, status, (cudaStream_t)stream);
}

size_t wedlm_lmhead_confidence_workspace_bytes(const wedlm_config_t* cfg, int32_t hidden) {
  if (check_config(cfg, false, true) != WEDLM_OK || hidden < 64 || hidden % 64 != 0) return 0;
  return lmhead_workspace(cfg, hidden).total;
}

int wedlm_lmhead_confidence_commit(const wedlm_config_t* cfg, int32_t hidden, const void* hidden_states,
                                   const void* lm_head, const int32_t* tilt_ids, float tilt, const int32_t* perm,
                                   const int32_t* n_filled, const int32_t* n_commit, int32_t* window_tokens,
                                   uint8_t* filled, int32_t* prefix_len, int32_t* window_len, int32_t* remaining_budget,
                                   int32_t* argmax, float* maxprob, float* entropy, float* lse, int32_t* committed_tokens,
                                   int32_t* committed_count, int32_t* filled_count, void* workspace, size_t workspace_bytes,
                                   int32_t* status, void* stream) {
  ApiRange nvtx_range("wedlm_lmhead_confidence_commit");
  int rc = check_config(cfg, false, true);
  if (rc != WEDLM_OK) return rc;
  if (cfg->dtype != WEDLM_DTYPE_BF16 || hidden < 64 || hidden % 64 != 0) return WEDLM_ERR_UNSUPPORTED;
  if (cfg->sample_temperature > 0.f) return WEDLM_ERR_UNSUPPORTED;     // no stored logits to draw from
  if ((long long)cfg->batch * cfg->window >= (1ll << 31) / 2) return WEDLM_ERR_UNSUPPORTED;
  if (cfg->batch == 0) return WEDLM_OK;
  if (!hidden_states || !lm_head || !perm || !n_filled || !n_commit || !window_tokens || !filled || !prefix_len || !workspace)
    return WEDLM_ERR_INVALID_ARG;
  if (!aligned16(hidden_states) || !aligned16(lm_head) || !aligned16(workspace)) return WEDLM_ERR_INVALID_ARG;
  const LmWorkspace lw = lmhead_workspace(cfg, hidden);
  if (workspace_bytes < lw.total) return WEDLM_ERR_WORKSPACE_TOO_SMALL;
  Shape s = make_shape(cfg);
  cudaStream_t st = (cudaStream_t)stream;
  int n_tiles = 0;
  rc = launch_lmhead_conf(s, hidden, hidden_states, lm_head, tilt_ids, tilt, n_filled, window_len, workspace, lw, &n_tiles, status, st);
  if (rc != WEDLM_OK) return rc;
  return launch_conf_commit(s, cfg, n_tiles, workspace, perm, n_filled, n_commit, window_tokens, filled,
                            prefix_len, window_len, remaining_budget, argmax, maxprob, entropy, lse, committed_tokens,
                            committed_count, filled_count, st);
}

// ---------------------------------------------------------------------------------------------
// Dual-Stream Masking (Section 4.2)
// ---------------------------------------------------------------------------------------------
namespace {

struct DualPlan {
  wedlm_config_t ic;          // the batch of (sequence, stream, block) windows
  size_t pool_bytes, table_bytes, prefix_bytes, attn_bytes, total_bytes;
};

int plan_dual_stream(const wedlm_config_t* cfg, int32_t n_blocks, DualPlan* out) {
  if (cfg == nullptr || n_blocks < 1) return WEDLM_ERR_INVALID_ARG;
  if (cfg->batch < 0 || cfg->window < 1 || cfg->window > 1024) return WEDLM_ERR_INVALID_ARG;
  if (cfg->page_size < 1 || cfg->window % cfg->page_size != 0) return WEDLM_ERR_UNSUPPORTED;   // blocks own whole pages
  const long long units = (long long)cfg->batch * 2 * n_blocks;
  const long long pages_per_stream = (long long)n_blocks * (cfg->window / cfg->page_size);
  if (units > 0x7fffffffLL / 4 || units * pages_per_stream > 0x7fffffffLL || (long long)n_blocks * cfg->window > 0x7fffffffLL / 2)
    return WEDLM_ERR_UNSUPPORTED;
  DualPlan p{};
  p.ic = *cfg;
  p.ic.batch = (int32_t)units;
  p.ic.max_pages_per_seq = (int32_t)pages_per_stream;
  p.ic.num_pages = (int32_t)((long long)cfg->batch * 2 * pages_per_stream);
  p.ic.max_prefix_len = (n_blocks - 1) * cfg->window;
  p.ic.commit_mode = WEDLM_COMMIT_STREAMING;
  if (cfg->batch == 0) p.ic.num_pages = 1;
  int rc = check_config(&p.ic, true, false);
  if (rc != WEDLM_OK) return rc;
  const size_t elem = cfg->dtype == WEDLM_DTYPE_BF16 ? 2 : 4;
  p.pool_bytes = align_up((size_t)units * cfg->window * cfg->n_kv_heads * cfg->head_dim * elem, 256);
  p.table_bytes = align_up((size_t)units * pages_per_stream * sizeof(int32_t), 256);
  p.prefix_bytes = align_up((size_t)units * sizeof(int32_t), 256);
  p.attn_bytes = align_up(plan_attention(&p.ic).total_bytes, 256);
  p.total_bytes = 2 * p.pool_bytes + p.table_bytes + p.prefix_bytes + p.attn_bytes;
  *out = p;
  return WEDLM_OK;
}

}  // namespace

int wedlm_dual_stream_construct(const wedlm_config_t* cfg, int32_t n_blocks, int32_t seq_len, const int32_t* tokens,
                                const uint8_t* masked, int32_t* x_input, int32_t* p_input, uint8_t* is_mask,
                                int32_t* n_observed, void* stream) {
  ApiRange nvtx_range("wedlm_dual_stream_construct");
  if (cfg == nullptr || n_blocks < 1 || cfg->batch < 0 || cfg->window < 1 || cfg->window > 1024) return WEDLM_ERR_INVALID_ARG;
  if (seq_len < 1 || (long long)seq_len > (long long)n_blocks * cfg->window ||
      (long long)seq_len <= (long long)(n_blocks - 1) * cfg->window)
    return WEDLM_ERR_INVALID_ARG;                 // n_blocks must be ceil(seq_len / window)
  if ((long long)cfg->batch * n_blocks > 0x7fffffffLL) return WEDLM_ERR_UNSUPPORTED;
  if (cfg->batch == 0) return WEDLM_OK;
  if (!tokens || !masked || !x_input || !p_input) return WEDLM_ERR_INVALID_ARG;
  return launch_dual_stream_construct(cfg->batch, seq_len, cfg->window, n_blocks, cfg->mask_token_id, tokens, masked,
                                      x_input, p_input, is_mask, n_observed, (cudaStream_t)stream);
}

size_t wedlm_dual_stream_workspace_bytes(const wedlm_config_t* cfg, int32_t n_blocks) {
  DualPlan p;
  if (plan_dual_stream(cfg, n_blocks, &p) != WEDLM_OK) return 0;
  return p.total_bytes ? p.total_bytes : 256;
}

int wedlm_dual_stream_attn(const wedlm_config_t* cfg, int32_t n_blocks, const void* q, const void* k, const void* v,
                           const int32_t* p_input, void* out, void* workspace, size_t workspace_bytes, int32_t* status,
                           void* stream) {
  ApiRange nvtx_range("wedlm_dual_stream_attn");
  DualPlan p;
  int rc = plan_dual_stream(cfg, n_blocks, &p);
  if (rc != WEDLM_OK) return rc;
  if (cfg->batch == 0) return WEDLM_OK;
  if (!q || !k || !v || !p_input || !out || !workspace) return WEDLM_ERR_INVALID_ARG;
  if (!aligned16(workspace)) return WEDLM_ERR_INVALID_ARG;
  if (workspace_bytes < p.total_bytes) return WEDLM_ERR_WORKSPACE_TOO_SMALL;
  char* ws = static_cast<char*>(workspace);
  void* k_pool = ws;
  void* v_pool = ws + p.pool_bytes;
  int32_t* table = reinterpret_cast<int32_t*>(ws + 2 * p.pool_bytes);
  int32_t* prefix = reinterpret_cast<int32_t*>(ws + 2 * p.pool_bytes + p.table_bytes);
  void* attn_ws = ws + 2 * p.pool_bytes + p.table_bytes + p.prefix_bytes;
  rc = launch_dual_stream_tables(p.ic.batch, n_blocks, cfg->window, cfg->page_size, table, prefix, (cudaStream_t)stream);
  if (rc != WEDLM_OK) return rc;
  // every unit rotates its rows at p_input and stages them into its own pages; the attention of unit (n, s, k)
  // then walks memory pages [0, k*B) and its own block behind them
  return wedlm_window_attn(&p.ic, q, k, v, k_pool, v_pool, table, prefix, p_input, out, nullptr, attn_ws, p.attn_bytes,
                           status, stream);
}

// ---------------------------------------------------------------------------------------------
// One whole step from host buffers
// ---------------------------------------------------------------------------------------------
namespace {

struct HostStepPlan {
  size_t off_filled, off_tokens, off_prefix, off_wlen, off_budget, off_table, off_q, off_k, off_v, off_logits, off_tilt;
  size_t off_perm, off_inv, off_pos, off_tokphys, off_nfilled, off_ncommit, off_out, off_argmax, off_maxprob, off_entropy,
      off_lse, off_ctok, off_ccount, off_fcount, off_attn_ws, off_conf_ws;
  size_t attn_ws_bytes, conf_ws_bytes, total;
};

// hidden == 0: the step takes logits [B,W,V]; hidden > 0: it takes hidden states [B,W,hidden] (and per-row tilt ids)
// and the confidence pass is the fused LM-head call
int plan_host_step(const wedlm_config_t* cfg, int32_t hidden, HostStepPlan* out) {
  int rc = check_config(cfg, true, true);
  if (rc != WEDLM_OK) return rc;
  const size_t B = cfg->batch, W = cfg->window, elem = cfg->dtype == WEDLM_DTYPE_BF16 ? 2 : 4;
  HostStepPlan p{};
  size_t at = 0;
  auto take = [&](size_t bytes) { size_t o = at; at += align_up(bytes ? bytes : 1, 256); return o; };
  p.off_filled = take(B * W);
  p.off_tokens = take(B * W * 4);
  p.off_prefix = take(B * 4);
  p.off_wlen = take(B * 4);
  p.off_budget = take(B * 4);
  p.off_table = take(B * (size_t)cfg->max_pages_per_seq * 4);
  p.off_q = take(B * W * cfg->n_q_heads * cfg->head_dim * elem);
  p.off_k = take(B * W * cfg->n_kv_heads * cfg->head_dim * elem);
  p.off_v = take(B * W * cfg->n_kv_heads * cfg->head_dim * elem);
  p.off_logits = hidden > 0 ? take(B * W * (size_t)hidden * elem) : take(B * W * (size_t)cfg->vocab * elem);
  p.off_tilt = take(B * W * 4);
  p.off_perm = take(B * W * 4);
  p.off_inv = take(B * W * 4);
  p.off_pos = take(B * W * 4);
  p.off_tokphys = take(B * W * 4);
  p.off_nfilled = take(B * 4);
  p.off_ncommit = take(B * 4);
  p.off_out = take(B * W * cfg->n_q_heads * cfg->head_dim * elem);
  p.off_argmax = take(B * W * 4);
  p.off_maxprob = take(B * W * 4);
  p.off_entropy = take(B * W * 4);
  p.off_lse = take(B * W * 4);
  p.off_ctok = take(B * W * 4);
  p.off_ccount = take(B * 4);
  p.off_fcount = take(B * 4);
  p.attn_ws_bytes = plan_attention(cfg).total_bytes;
  p.conf_ws_bytes = hidden > 0 ? wedlm_lmhead_confidence_workspace_bytes(cfg, hidden) : confidence_workspace_bytes(cfg);
  p.off_attn_ws = take(p.attn_ws_bytes);
  p.off_conf_ws = take(p.conf_ws_bytes);
  p.total = at;
  *out = p;
  return WEDLM_OK;
}

}  // namespace

size_t wedlm_step_host_workspace_bytes(const wedlm_config_t* cfg) {
  HostStepPlan p;
  if (plan_host_step(cfg, 0, &p) != WEDLM_OK) return 0;
  return p.total;
}

size_t wedlm_step_host_lmhead_workspace_bytes(const wedlm_config_t* cfg, int32_t hidden) {
  HostStepPlan p;
  if (hidden < 64 || hidden % 64 != 0 || plan_host_step(cfg, hidden, &p) != WEDLM_OK) return 0;
  return p.total;
}

namespace {

// The large upload of a host step (hidden states or logits) runs on a copy stream of its own, forked from and joined
// back into the caller's stream with two events, so that it overlaps the reorder / RoPE / attention kernels instead
// of queueing behind them.  One lane per host thread and device, created on first use and kept.
struct CopyLane {
  cudaStream_t stream = nullptr;
  cudaEvent_t fork = nullptr, join = nullptr;
  bool ready = false;
};

CopyLane* copy_lane() {
  thread_local CopyLane lanes[64];
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
  CopyLane& l = lanes[dev];
  if (!l.ready) {
    if (cudaStreamCreateWithFlags(&l.stream, cudaStreamNonBlocking) != cudaSuccess) return nullptr;
    if (cudaEventCreateWithFlags(&l.fork, cudaEventDisableTiming) != cudaSuccess) return nullptr;
    if (cudaEventCreateWithFlags(&l.join, cudaEventDisableTiming) != cudaSuccess) return nullptr;
    l.ready = true;
  }
  return &l;
}

// Both host-step calls: logits from the host (h_hidden == NULL) or hidden states from the host with the output
// embedding resident on the device.
int step_host_impl(const wedlm_config_t* cfg, int32_t hidden, uint8_t* h_filled, int32_t* h_window_tokens,
                   int32_t* h_prefix_len, int32_t* h_window_len, int32_t* h_remaining_budget, const int32_t* h_block_table,
                   const void* h_q, const void* h_k, const void* h_v, const void* h_logits, const void* h_hidden,
                   const void* lm_head, const int32_t* h_tilt_ids, float tilt, void* k_cache, void* v_cache,
                   int32_t* h_committed_tokens, int32_t* h_committed_count, int32_t* h_filled_count, void* workspace,
                   size_t workspace_bytes, void** attn_out, int32_t* status, void* stream) {
  HostStepPlan p;
  int rc = plan_host_step(cfg, hidden, &p);
  if (rc != WEDLM_OK) return rc;
  if (attn_out) *attn_out = nullptr;
  if (cfg->batch == 0) return WEDLM_OK;
  const bool fused = hidden > 0;
  if (!h_filled || !h_window_tokens || !h_prefix_len || !h_block_table || !h_q || !h_k || !h_v || !k_cache ||
      !v_cache || !h_committed_tokens || !h_committed_count || !workspace)
    return WEDLM_ERR_INVALID_ARG;
  if (fused ? (!h_hidden || !lm_head) : !h_logits) return WEDLM_ERR_INVALID_ARG;
  if (!aligned16(workspace) || !aligned16(k_cache) || !aligned16(v_cache)) return WEDLM_ERR_INVALID_ARG;
  if (workspace_bytes < p.total) return WEDLM_ERR_WORKSPACE_TOO_SMALL;
  cudaStream_t st = (cudaStream_t)stream;
  char* ws = static_cast<char*>(workspace);
  const size_t B = cfg->batch, W = cfg->window, elem = cfg->dtype == WEDLM_DTYPE_BF16 ? 2 : 4;
  auto up = [&](size_t off, const void* src, size_t bytes) {
    return cudaMemcpyAsync(ws + off, src, bytes, cudaMemcpyHostToDevice, st) == cudaSuccess;
  };
  auto down = [&](void* dst, size_t off, size_t bytes) {
    return cudaMemcpyAsync(dst, ws + off, bytes, cudaMemcpyDeviceToHost, st) == cudaSuccess;
  };
  bool ok = up(p.off_filled, h_filled, B * W) && up(p.off_tokens, h_window_tokens, B * W * 4) &&
            up(p.off_prefix, h_prefix_len, B * 4) && up(p.off_table, h_block_table, B * (size_t)cfg->max_pages_per_seq * 4) &&
            up(p.off_q, h_q, B * W * cfg->n_q_heads * cfg->head_dim * elem) &&
            up(p.off_k, h_k, B * W * cfg->n_kv_heads * cfg->head_dim * elem) &&
            up(p.off_v, h_v, B * W * cfg->n_kv_heads * cfg->head_dim * elem);
  if (ok && h_window_len) ok = up(p.off_wlen, h_window_len, B * 4);
  if (ok && h_remaining_budget) ok = up(p.off_budget, h_remaining_budget, B * 4);
  if (!ok) return WEDLM_ERR_CUDA;
  // The copy lane starts after the uploads above (the copy engine serves them first: the kernels need them first)
  // and after whatever the caller's stream still had queued on this workspace.
  CopyLane* lane = copy_lane();
  if (!lane) return WEDLM_ERR_CUDA;
  if (cudaEventRecord(lane->fork, st) != cudaSuccess || cudaStreamWaitEvent(lane->stream, lane->fork, 0) != cudaSuccess)
    return WEDLM_ERR_CUDA;
  auto up_lane = [&](size_t off, const void* src, size_t bytes) {
    return cudaMemcpyAsync(ws + off, src, bytes, cudaMemcpyHostToDevice, lane->stream) == cudaSuccess;
  };
  // Whatever happens from here on, the lane is joined back into the caller's stream before this call returns: in
  // front of the confidence pass when all goes well, on the way out otherwise.
  struct Join {
    cudaStream_t st;
    CopyLane* lane;
    bool recorded = false, waited = false;
    bool wait() {
      if (waited || !recorded) return true;
      waited = true;
      return cudaStreamWaitEvent(st, lane->join, 0) == cudaSuccess;
    }
    ~Join() { wait(); }
  } join{st, lane};
  bool big_ok = true;
  if (fused) {
    // hidden states of all rows (the mask rows are gathered on the device), tilt ids if any
    big_ok = up_lane(p.off_logits, h_hidden, B * W * (size_t)hidden * elem);
    if (big_ok && h_tilt_ids) big_ok = up_lane(p.off_tilt, h_tilt_ids, B * W * 4);
  } else {
    // Logits: only the rows the confidence pass reads.  After reordering the mask rows of a sequence are the
    // physical rows [n_filled, window_len), one contiguous range, and n_filled is a count over the host's flags.
    for (size_t b = 0; big_ok && b < B; ++b) {
      long long L = h_window_len ? h_window_len[b] : (long long)W;
      L = L < 0 ? 0 : (L > (long long)W ? (long long)W : L);
      long long nf = 0;
      for (long long j = 0; j < L; ++j) nf += h_filled[b * W + j] != 0;
      if (L > nf) {
        const size_t off = (b * W + (size_t)nf) * (size_t)cfg->vocab * elem;
        big_ok = up_lane(p.off_logits + off, static_cast<const char*>(h_logits) + off, (size_t)(L - nf) * cfg->vocab * elem);
      }
    }
  }
  if (cudaEventRecord(lane->join, lane->stream) != cudaSuccess) return WEDLM_ERR_CUDA;
  join.recorded = true;
  if (!big_ok) return WEDLM_ERR_CUDA;
  uint8_t* d_filled = reinterpret_cast<uint8_t*>(ws + p.off_filled);
  int32_t* d_tokens = reinterpret_cast<int32_t*>(ws + p.off_tokens);
  int32_t* d_prefix = reinterpret_cast<int32_t*>(ws + p.off_prefix);
  int32_t* d_wlen = h_window_len ? reinterpret_cast<int32_t*>(ws + p.off_wlen) : nullptr;
  int32_t* d_budget = h_remaining_budget ? reinterpret_cast<int32_t*>(ws + p.off_budget) : nullptr;
  int32_t* d_perm = reinterpret_cast<int32_t*>(ws + p.off_perm);
  int32_t* d_pos = reinterpret_cast<int32_t*>(ws + p.off_pos);
  int32_t* d_nfilled = reinterpret_cast<int32_t*>(ws + p.off_nfilled);
  int32_t* d_ncommit = reinterpret_cast<int32_t*>(ws + p.off_ncommit);
  // reorder and attention need only the small inputs; the logits / hidden states follow
  rc = wedlm_reorder(cfg, d_filled, d_tokens, d_prefix, d_wlen, d_perm, reinterpret_cast<int32_t*>(ws + p.off_inv), d_pos,
                     reinterpret_cast<int32_t*>(ws + p.off_tokphys), d_nfilled, d_ncommit, stream);
  if (rc != WEDLM_OK) return rc;
  rc = wedlm_window_attn(cfg, ws + p.off_q, ws + p.off_k, ws + p.off_v, k_cache, v_cache,
                         reinterpret_cast<int32_t*>(ws + p.off_table), d_prefix, d_pos, ws + p.off_out, nullptr,
                         ws + p.off_attn_ws, p.attn_ws_bytes, status, stream);
  if (rc != WEDLM_OK) return rc;
  int32_t* d_argmax = reinterpret_cast<int32_t*>(ws + p.off_argmax);
  float* d_maxprob = reinterpret_cast<float*>(ws + p.off_maxprob);
  float* d_entropy = reinterpret_cast<float*>(ws + p.off_entropy);
  float* d_lse = reinterpret_cast<float*>(ws + p.off_lse);
  int32_t* d_ctok = reinterpret_cast<int32_t*>(ws + p.off_ctok);
  int32_t* d_ccount = reinterpret_cast<int32_t*>(ws + p.off_ccount);
  int32_t* d_fcount = reinterpret_cast<int32_t*>(ws + p.off_fcount);
  if (!join.wait()) return WEDLM_ERR_CUDA;             // the hidden states / logits have landed
  if (fused) {
    rc = wedlm_lmhead_confidence_commit(cfg, hidden, ws + p.off_logits, lm_head,
                                        h_tilt_ids ? reinterpret_cast<int32_t*>(ws + p.off_tilt) : nullptr, tilt, d_perm,
                                        d_nfilled, d_ncommit, d_tokens, d_filled, d_prefix, d_wlen, d_budget, d_argmax,
                                        d_maxprob, d_entropy, d_lse, d_ctok, d_ccount, d_fcount, ws + p.off_conf_ws,
                                        p.conf_ws_bytes, status, stream);
  } else {
    rc = wedlm_confidence_commit(cfg, ws + p.off_logits, d_perm, d_nfilled, d_ncommit, d_tokens, d_filled, d_prefix, d_wlen,
                                 d_budget, d_argmax, d_maxprob, d_entropy, d_lse, d_ctok, d_ccount, d_fcount,
                                 ws + p.off_conf_ws, p.conf_ws_bytes, status, stream);
  }
  if (rc != WEDLM_OK) return rc;
  ok = down(h_committed_tokens, p.off_ctok, B * W * 4) && down(h_committed_count, p.off_ccount, B * 4) &&
       down(h_filled, p.off_filled, B * W) && down(h_window_tokens, p.off_tokens, B * W * 4) &&
       down(h_prefix_len, p.off_prefix, B * 4);
  if (ok && h_filled_count) ok = down(h_filled_count, p.off_fcount, B * 4);
  if (ok && h_window_len) ok = down(h_window_len, p.off_wlen, B * 4);
  if (ok && h_remaining_budget) ok = down(h_remaining_budget, p.off_budget, B * 4);
  if (!ok) return WEDLM_ERR_CUDA;
  if (attn_out) *attn_out = ws + p.off_out;
  return WEDLM_OK;
}

}  // namespace

int wedlm_step_host(const wedlm_config_t* cfg, uint8_t* h_filled, int32_t* h_window_tokens, int32_t* h_prefix_len,
                    int32_t* h_window_len, int32_t* h_remaining_budget, const int32_t* h_block_table, const void* h_q,
                    const void* h_k, const void* h_v, const void* h_logits, void* k_cache, void* v_cache,
                    int32_t* h_committed_tokens, int32_t* h_committed_count, int32_t* h_filled_count, void* workspace,
                    size_t workspace_bytes, void** attn_out, int32_t* status, void* stream) {
  ApiRange nvtx_range("wedlm_step_host");
  return step_host_impl(cfg, 0, h_filled, h_window_tokens, h_prefix_len, h_window_len, h_remaining_budget, h_block_table, h_q,
                        h_k, h_v, h_logits, nullptr, nullptr, nullptr, 0.f, k_cache, v_cache, h_committed_tokens,
                        h_committed_count, h_filled_count, workspace, workspace_bytes, attn_out, status, stream);
}

int wedlm_step_host_lmhead(const wedlm_config_t* cfg, int32_t hidden, uint8_t* h_filled, int32_t* h_window_tokens,
                           int32_t* h_prefix_len, int32_t* h_window_len, int32_t* h_remaining_budget,
                           const int32_t* h_block_table, const void* h_q, const void* h_k, const void* h_v,
                           const void* h_hidden_states, const void* lm_head, const int32_t* h_tilt_ids, float tilt,
                           void* k_cache, void* v_cache, int32_t* h_committed_tokens, int32_t* h_committed_count,
                           int32_t* h_filled_count, void* workspace, size_t workspace_bytes, void** attn_out,
                           int32_t* status, void* stream) {
  ApiRange nvtx_range("wedlm_step_host_lmhead");
  if (cfg == nullptr || cfg->dtype != WEDLM_DTYPE_BF16 || hidden < 64 || hidden % 64 != 0) return WEDLM_ERR_UNSUPPORTED;
  return step_host_impl(cfg, hidden, h_filled, h_window_tokens, h_prefix_len, h_window_len, h_remaining_budget, h_block_table,
                        h_q, h_k, h_v, nullptr, h_hidden_states, lm_head, h_tilt_ids, tilt, k_cache, v_cache,
                        h_committed_tokens, h_committed_count, h_filled_count, workspace, workspace_bytes, attn_out, status,
                        stream);
}

int wedlm_window_refill(const wedlm_config_t* cfg, const int32_t* n_commit, int32_t* window_tokens, uint8_t* filled,
                        int32_t* prefix_len, int32_t* window_len, int32_t* remaining_budget,
                        int32_t* committed_tokens, int32_t* committed_count, void* stream) {
  ApiRange nvtx_range("wedlm_window_refill");
  int rc = check_config(cfg, false, false);
  if (rc != WEDLM_OK) return rc;
  if (cfg->batch == 0) return WEDLM_OK;
  if (!n_commit || !window_tokens || !filled || !prefix_len) return WEDLM_ERR_INVALID_ARG;
  return launch_window_refill(make_shape(cfg), cfg, n_commit, window_tokens, filled, prefix_len, window_len,
                              remaining_budget, committed_tokens, committed_count, (cudaStream_t)stream);
}

}  // extern "C"
