// Topological Reordering (Eq. 5-6): stable partition of each window by the `filled` flag with
// warp ballots, logical position ids, and the commit length of Algorithm 1.
#include "common.cuh"

namespace wedlm {

// One warp per sequence.  Slot j is "observed" iff filled[j] != 0 and j < window_len.
__global__ void __launch_bounds__(32)
reorder_kernel(int W, int commit_mode, const uint8_t* __restrict__ filled, const int32_t* __restrict__ window_tokens,
               const int32_t* __restrict__ prefix_len, const int32_t* __restrict__ window_len,
               int32_t* __restrict__ perm, int32_t* __restrict__ inv_perm, int32_t* __restrict__ pos_ids,
               int32_t* __restrict__ tokens_phys, int32_t* __restrict__ n_filled, int32_t* __restrict__ n_commit) {
  const int b = blockIdx.x;
  const int lane = threadIdx.x;
  const int L = window_len ? min(max(window_len[b], 0), W) : W;
  const int P = prefix_len[b];
  const uint8_t* f = filled + (size_t)b * W;

  // pass 1: number of observed slots and the first non-observed slot
  int total = 0;
  int first_mask = W;
  for (int base = 0; base < W; base += 32) {
    int j = base + lane;
    bool obs = (j < L) && (f[j] != 0);
    unsigned bal = __ballot_sync(0xffffffffu, obs);
    total += __popc(bal);
    unsigned valid = (W - base >= 32) ? 0xffffffffu : ((1u << (W - base)) - 1u);
    unsigned notobs = ~bal & valid;
    if (first_mask == W && notobs) first_mask = base + __ffs(notobs) - 1;
  }
  // pass 2: destinations
  int before = 0;  // observed slots in earlier chunks
  for (int base = 0; base < W; base += 32) {
    int j = base + lane;
    bool obs = (j < L) && (f[j] != 0);
    unsigned bal = __ballot_sync(0xffffffffu, obs);
    int obs_before = before + __popc(bal & ((1u << lane) - 1u));
    if (j < W) {
      int i = obs ? obs_before : total + (j - obs_before);
      size_t o = (size_t)b * W;
      perm[o + i] = j;
      inv_perm[o + j] = i;
      pos_ids[o + i] = P + j;
      if (tokens_phys && window_tokens) tokens_phys[o + i] = window_tokens[o + j];
    }
    before += __popc(bal);
  }
  if (lane == 0) {
    n_filled[b] = total;
    // streaming: the leading filled run; block-wise baseline: all active slots or nothing
    n_commit[b] = commit_mode == WEDLM_COMMIT_BLOCK ? ((total == L && L > 0) ? L : 0) : first_mask;
  }
}

int launch_reorder(const Shape& s, const uint8_t* filled, const int32_t* window_tokens, const int32_t* prefix_len,
                   const int32_t* window_len, int32_t* perm, int32_t* inv_perm, int32_t* pos_ids,
                   int32_t* tokens_phys, int32_t* n_filled, int32_t* n_commit, cudaStream_t st) {
  reorder_kernel<<<s.B, 32, 0, st>>>(s.W, s.commit_mode, filled, window_tokens, prefix_len, window_len, perm, inv_perm, pos_ids,
                                     tokens_phys, n_filled, n_commit);
  count_launch();
  return cuda_ok(cudaGetLastError());
}

}  // namespace wedlm
