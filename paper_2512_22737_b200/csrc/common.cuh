// Shared device/host helpers of the WeDLM step library (sm_100a).
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <nvtx3/nvToolsExt.h>

#include "wedlm.h"

namespace wedlm {

// Launch descriptors handed from the C-ABI layer to the kernels' host launchers.
struct Shape {
  int B, W, Hq, Hkv, D, G;
  int page, max_pages, num_pages, V;
  int dtype, rope_style, commit_mode;
  int max_prefix;      // host-known bound of prefix_len[b]: the key split and the workspace are sized for it
  float theta, scale;
};

// prefix_len[b] as the attention kernels use it.  The value is device data and may have moved past the bound
// the launch was planned for (or be negative): such a value is flagged in *status by the `report` thread and
// clamped into [0, max_prefix], so that every index derived from it stays inside the planned key chunks and
// the partial buffers.  The merge kernel applies the same clamp (without reporting) and so agrees on the
// number of chunks.
__device__ __forceinline__ int checked_prefix(const int32_t* __restrict__ prefix_len, int b, int max_prefix,
                                              int32_t* status, bool report) {
  int P = prefix_len[b];
  if (P < 0 || P > max_prefix) {
    if (report && status) atomicOr(status, WEDLM_STATUS_BAD_LENGTH);
    P = P < 0 ? 0 : max_prefix;
  }
  return P;
}

__device__ __forceinline__ float ld_as_float(const float* p, size_t i) { return p[i]; }
__device__ __forceinline__ float ld_as_float(const __nv_bfloat16* p, size_t i) { return __bfloat162float(p[i]); }
__device__ __forceinline__ void st_from_float(float* p, size_t i, float x) { p[i] = x; }
__device__ __forceinline__ void st_from_float(__nv_bfloat16* p, size_t i, float x) { p[i] = __float2bfloat16_rn(x); }

// Physical cache row (page * page_size + offset) of token position t of sequence b, or -1 with a
// status bit when the block table points outside the pool.
__device__ __forceinline__ long long cache_slot(const int32_t* __restrict__ block_table, int b, int t,
                                                int page, int max_pages, int num_pages, int32_t* status) {
  int lp = t / page;
  if (t < 0 || lp >= max_pages) {
    if (status) atomicOr(status, WEDLM_STATUS_BAD_LENGTH);
    return -1;
  }
  int pp = block_table[(size_t)b * max_pages + lp];
  if (pp < 0 || pp >= num_pages) {
    if (status) atomicOr(status, WEDLM_STATUS_BAD_PAGE);
    return -1;
  }
  return (long long)pp * page + (t - lp * page);
}

// Element offset of (slot, kv head g, dim 0) in a cache laid out [num_pages][Hkv][page][D].
__device__ __forceinline__ size_t cache_offset(long long slot, int g, int page, int Hkv, int D) {
  long long pp = slot / page;
  int off = (int)(slot - pp * page);
  return (((size_t)pp * Hkv + g) * page + off) * (size_t)D;
}

// Host launchers (defined in the .cu files).
int launch_reorder(const Shape& s, const uint8_t* filled, const int32_t* window_tokens, const int32_t* prefix_len,
                   const int32_t* window_len, int32_t* perm, int32_t* inv_perm, int32_t* pos_ids,
                   int32_t* tokens_phys, int32_t* n_filled, int32_t* n_commit, cudaStream_t st);

int launch_rope_stage(const Shape& s, const void* q, const void* k, const void* v, void* q_rot, void* k_cache,
                      void* v_cache, const int32_t* block_table, const int32_t* prefix_len, const int32_t* pos_ids,
                      const int32_t* count, int32_t* kv_slot_idx, int32_t* order, int32_t* status, cudaStream_t st);

struct AttnPlan {
  int impl;            // WEDLM_ATTN_GENERIC or WEDLM_ATTN_TENSOR
  int n_splits;        // partial slots per query row: key chunks per (sequence, head), or pieces per unit (balanced)
  int chunk;           // keys per chunk (multiple of the page size; CUDA-core path)
  int balanced;        // tensor path with fewer work units than CTA slots: the tiles are cut into equal runs
  int n_ctas;          // CTAs of the balanced cut
  size_t q_rot_bytes, part_o_bytes, part_ml_bytes, order_bytes, total_bytes;
};
AttnPlan plan_attention(const wedlm_config_t* cfg);

int launch_attn_generic(const Shape& s, const AttnPlan& plan, const void* q_rot, const void* k_cache,
                        const void* v_cache, const int32_t* block_table, const int32_t* prefix_len, void* out,
                        float* part_o, float* part_ml, int32_t* status, cudaStream_t st);

bool attn_tensor_supported(const wedlm_config_t* cfg);
int launch_attn_tensor(const Shape& s, const AttnPlan& plan, const void* q_rot, const void* k_cache,
                       const void* v_cache, const int32_t* block_table, const int32_t* prefix_len,
                       const int32_t* order, void* out, float* part_o, float* part_ml, int32_t* status,
                       cudaStream_t st);

int launch_attn_tensor_merge(const Shape& s, const AttnPlan& plan, const int32_t* prefix_len, const int32_t* order,
                             const float* part_o, const float* part_ml, void* out, cudaStream_t st);

int launch_wait_expiry_selftest(uint32_t max_polls, int32_t* status, cudaStream_t st);

int launch_attn_merge(const Shape& s, const AttnPlan& plan, const int32_t* prefix_len, const float* part_o,
                      const float* part_ml, void* out, cudaStream_t st);

size_t confidence_workspace_bytes(const wedlm_config_t* cfg);
int launch_confidence(const Shape& s, const wedlm_config_t* cfg, const void* logits, const int32_t* perm,
                      const int32_t* n_filled, const int32_t* n_commit, int32_t* window_tokens, uint8_t* filled,
                      int32_t* prefix_len, int32_t* window_len, int32_t* remaining_budget, int32_t* argmax,
                      float* maxprob, float* entropy, float* lse, int32_t* committed_tokens,
                      int32_t* committed_count, int32_t* filled_count, void* workspace, int32_t* status, cudaStream_t st);

int launch_conf_commit(const Shape& s, const wedlm_config_t* cfg, int n_chunks, const void* partials, const int32_t* perm,
                       const int32_t* n_filled, const int32_t* n_commit, int32_t* window_tokens, uint8_t* filled,
                       int32_t* prefix_len, int32_t* window_len, int32_t* remaining_budget, int32_t* argmax,
                       float* maxprob, float* entropy, float* lse, int32_t* committed_tokens, int32_t* committed_count,
                       int32_t* filled_count, cudaStream_t st, void* sample_ws = nullptr);

// Fused LM head + confidence pass 1: partials [B*W][n_tiles] (n_tiles <= ceil(V/128), returned) from hidden states and the
// output embedding.  Only the mask rows are computed: they are gathered into a dense matrix in the workspace first.
struct LmWorkspace {
  size_t off_part, off_count, off_map, off_dense, total;
};
int lmhead_conf_tiles(int vocab);
LmWorkspace lmhead_workspace(const wedlm_config_t* cfg, int hidden);
int launch_lmhead_conf(const Shape& s, int hidden, const void* hidden_states, const void* lm_head, const int32_t* tilt_ids,
                       float tilt, const int32_t* n_filled, const int32_t* window_len, void* workspace,
                       const LmWorkspace& lw, int* n_tiles_out, int32_t* status, cudaStream_t st);

// Dual-Stream Masking (training forward): input construction and the per-unit page tables.
int launch_dual_stream_construct(int N, int L, int B, int K, int mask_id, const int32_t* tokens, const uint8_t* masked,
                                 int32_t* x_input, int32_t* p_input, uint8_t* is_mask, int32_t* n_observed,
                                 cudaStream_t st);
int launch_dual_stream_tables(int n_units, int K, int B, int page, int32_t* block_table, int32_t* prefix_len,
                              cudaStream_t st);

int launch_window_refill(const Shape& s, const wedlm_config_t* cfg, const int32_t* n_commit, int32_t* window_tokens,
                         uint8_t* filled, int32_t* prefix_len, int32_t* window_len, int32_t* remaining_budget,
                         int32_t* committed_tokens, int32_t* committed_count, cudaStream_t st);

inline int cuda_ok(cudaError_t e) { return e == cudaSuccess ? WEDLM_OK : WEDLM_ERR_CUDA; }

// Multiprocessor count of the current device, asked once per device ordinal; 148 (B200) when no device
// can be asked, which only happens in size queries made on a host without a GPU.
int device_sm_count();

// Number of kernels this process has launched through the library (reported by wedlm_launch_count).
void count_launch(int n = 1);

// NVTX range around a public call: shows up by name in a timeline tool, costs nothing without one attached.
struct ApiRange {
  explicit ApiRange(const char* name) { nvtxRangePushA(name); }
  ~ApiRange() { nvtxRangePop(); }
  ApiRange(const ApiRange&) = delete;
  ApiRange& operator=(const ApiRange&) = delete;
};

}  // namespace wedlm
