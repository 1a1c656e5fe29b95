// Dual-Stream Masking (Section 4.2): construction of the two-stream training input (Eq. 8-9, block-wise
// masking and intra-block Topological Reordering) and the page tables that turn its attention pattern
// into the decoding path's "window on a cached prefix".
//
// The attention pattern says: a row of block k (either stream) sees the memory stream's rows at positions
// < k*B, plus the rows of its own block that are physically not later than itself.  That is exactly the
// decoding step's visibility with prefix = memory[0, k*B) and window = the block.  So every (sequence,
// stream, block) becomes one unit of a batch of windows of B slots with prefix length k*B, whose page table
// maps positions [0, k*B) to the memory stream's pages and [k*B, (k+1)*B) to the unit's own pages (B is a
// multiple of the page size).  RoPE, staging and the tcgen05 attention kernel then run unchanged.
#include "common.cuh"

namespace wedlm {

// One warp per (sequence, block).  Writes the block's rows of both streams:
//   memory stream      x = token, p = logical position (rows at or beyond L: mask id, p = index)
//   prediction stream  observed tokens first, masked ones last, order kept; x = token or mask id, p kept.
__global__ void __launch_bounds__(32)
dual_stream_construct_kernel(int L, int B, int K, int mask_id, const int32_t* __restrict__ tokens,
                             const uint8_t* __restrict__ masked, int32_t* __restrict__ x_input,
                             int32_t* __restrict__ p_input, uint8_t* __restrict__ is_mask, int32_t* __restrict__ n_observed) {
  const int n = blockIdx.x / K, kb = blockIdx.x - n * K;
  const int lane = threadIdx.x;
  const int Lp = K * B;
  const int lo = kb * B;
  const int len = min(B, L - lo);                 // real slots of this block (the last one may be short)
  const int32_t* tok = tokens + (size_t)n * L;
  const uint8_t* msk = masked + (size_t)n * L;
  int32_t* xm = x_input + ((size_t)n * 2 + 0) * Lp;
  int32_t* xt = x_input + ((size_t)n * 2 + 1) * Lp;
  int32_t* pm = p_input + ((size_t)n * 2 + 0) * Lp;
  int32_t* pt = p_input + ((size_t)n * 2 + 1) * Lp;

  int total = 0;                                  // observed slots of the block
  for (int base = 0; base < B; base += 32) {
    const int j = base + lane;
    const bool obs = j < len && msk[lo + j] == 0;
    total += __popc(__ballot_sync(0xffffffffu, obs));
  }
  int before = 0;
  for (int base = 0; base < B; base += 32) {
    const int j = base + lane;
    const bool real = j < len;
    const bool obs = real && msk[lo + j] == 0;
    const unsigned bal = __ballot_sync(0xffffffffu, obs);
    const int obs_before = before + __popc(bal & ((1u << lane) - 1u));
    if (j < B) {
      const int i = obs ? obs_before : total + (j - obs_before);     // padding slots sort behind the real masks
      xm[lo + j] = real ? tok[lo + j] : mask_id;
      pm[lo + j] = lo + j;
      xt[lo + i] = obs ? tok[lo + j] : mask_id;
      pt[lo + i] = lo + j;
      if (is_mask) is_mask[(size_t)n * Lp + lo + i] = (real && !obs) ? 1 : 0;
    }
    before += __popc(bal);
  }
  if (lane == 0 && n_observed) n_observed[(size_t)n * K + kb] = total;
}

// Page table and prefix length of unit u = (n*2 + s)*K + k:  positions below k*B live in the memory stream's
// pages of sequence n, everything from k*B on in the pages of stream s itself.
__global__ void dual_stream_tables_kernel(int n_units, int K, int B, int pages_per_block, int32_t* __restrict__ block_table,
                                          int32_t* __restrict__ prefix_len) {
  const int pages_per_stream = K * pages_per_block;
  const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= (long long)n_units * pages_per_stream) return;
  const int u = (int)(idx / pages_per_stream), j = (int)(idx - (long long)u * pages_per_stream);
  const int k = u % K, ns = u / K, n = ns >> 1;
  const int own_base = ns * pages_per_stream, mem_base = (n * 2) * pages_per_stream;
  block_table[idx] = (j < k * pages_per_block ? mem_base : own_base) + j;
  if (j == 0) prefix_len[u] = k * B;
}

int launch_dual_stream_construct(int N, int L, int B, int K, int mask_id, const int32_t* tokens, const uint8_t* masked,
                                 int32_t* x_input, int32_t* p_input, uint8_t* is_mask, int32_t* n_observed,
                                 cudaStream_t st) {
  dual_stream_construct_kernel<<<N * K, 32, 0, st>>>(L, B, K, mask_id, tokens, masked, x_input, p_input, is_mask, n_observed);
  count_launch();
  return cuda_ok(cudaGetLastError());
}

int launch_dual_stream_tables(int n_units, int K, int B, int page, int32_t* block_table, int32_t* prefix_len,
                              cudaStream_t st) {
  const int ppb = B / page;
  const long long total = (long long)n_units * K * ppb;
  const int threads = 256;
  dual_stream_tables_kernel<<<(unsigned)((total + threads - 1) / threads), threads, 0, st>>>(n_units, K, B, ppb, block_table,
                                                                                             prefix_len);
  count_launch();
  return cuda_ok(cudaGetLastError());
}

}  // namespace wedlm
