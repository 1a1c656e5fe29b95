// LM head fused with the vocabulary confidence reduction: the logits of the window rows are produced
// tile by tile in tensor memory and reduced there; they never reach HBM.
//
// logits[row, v] = <hidden[row, :], lm_head[v, :]>  (bf16 x bf16 -> fp32), and per mask row the same
// partials as the streaming confidence pass: m = max, a = lowest arg-max, s = sum e^(x-m),
// t = sum (x-m) e^(x-m) (entropy of Section 5.2 after the merge), one partial per vocabulary tile.
//
// Only the mask rows are computed (Algorithm 1 predicts from l_mask): a gather kernel first packs their hidden
// states into a dense matrix and records the physical row of every packed row.
//
// Work item = one vocabulary tile of tile_n <= 256 tokens x up to 256 packed rows (two 128-row accumulators
// of 256 TMEM columns each).  Items run tile-major over one persistent CTA per SM, so the row chunks of one
// vocabulary tile are in flight together: the output embedding is streamed from HBM once, whatever the number of
// rows, and the other chunks find the tile in L2.  Warp 9 feeds a 3-stage ring with TMA (hidden states
// 2 x [128 x 64], embedding [tile_n x 64] per stage, 128-byte swizzle), warp 8 issues tcgen05.mma
// (128 x tile_n x 16, 8 per stage; one elected lane, the whole warp runs the loop) and releases stages through
// tcgen05.commit, warps 0-7 read their row of the accumulators back with tcgen05.ld and reduce it.  The wide tile
// matters: every item re-reads the hidden states from L2, and with tiles of 128 (two accumulator sets, reduction
// overlapped with the next item's MMAs) the extra L2 traffic cost more than the overlap won.  Requesting the
// embedding tiles into L2 ahead of the ring, or giving them a deeper ring of their own (5 stages beside 3 for the
// hidden states), made the kernel slower; a 2-stage ring costs 22 %.  All waits are bounded.
#include <cuda.h>
#include <cudaTypedefs.h>
#include <math_constants.h>

#include "common.cuh"
#include "tc_ptx.cuh"

namespace wedlm {
namespace {

using namespace ptx;

constexpr int kLmMaxTileN = 256;              // most vocabulary entries per work item (the host picks 128..256)
constexpr int kLmTileK = 64;                  // hidden elements per stage (one 128-byte swizzle row)
constexpr int kLmStages = 3;
constexpr int kLmRows = 256;                  // window rows per work item (two 128-row accumulators)
constexpr uint32_t kLmBytesA = 128 * 128;     // one 128-row tile of hidden states per stage
constexpr uint32_t kLmStrideB = kLmMaxTileN * 128;               // room of the embedding tile per stage
constexpr uint32_t kLmOffA = 0;                                   // [stages][2][16 KB]
constexpr uint32_t kLmOffB = kLmStages * 2 * kLmBytesA;           // [stages][32 KB]
constexpr uint32_t kLmOffBar = kLmOffB + kLmStages * kLmStrideB;
constexpr uint32_t kLmSmem = kLmOffBar + 128;
constexpr int kLmThreads = 320;               // 8 reduction warps + MMA warp + TMA warp

enum LmBar { LM_FULL0 = 0, LM_FREE0 = LM_FULL0 + kLmStages, LM_ACC_FULL = LM_FREE0 + kLmStages,
             LM_ACC_FREE = LM_ACC_FULL + 1, LM_NBARS = LM_ACC_FREE + 1 };

struct LmParams {
  int W, V, H, n_tiles, tile_n;
  const int32_t* n_active;        // [1] device: number of active mask rows (the rows of the compacted hidden states)
  const int32_t* row_map;         // [n_active] physical row (b * W + i) of every compacted row
  float tilt;
  const int32_t* tilt_ids;        // [R] token whose logit gets +tilt, or NULL
  float4* part;
  int32_t* status;
};

// Persistent CTAs: work item = (row chunk, vocabulary tile), items strided over the grid.
__global__ void __launch_bounds__(kLmThreads, 1)
lmhead_conf_kernel(const __grid_constant__ CUtensorMap tm_h, const __grid_constant__ CUtensorMap tm_w, const LmParams p) {
  extern __shared__ __align__(1024) uint8_t smem[];
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int k_steps = p.H / kLmTileK;
  const int R = *p.n_active;                             // only the mask rows are computed: they were compacted
  const int n_chunks = (R + kLmRows - 1) / kLmRows;
  // items run tile-major: the row chunks of one vocabulary tile sit on neighbouring CTAs at the same time, so the
  // embedding tile comes from HBM once and from L2 for the other chunks
  const int n_items = p.n_tiles * n_chunks;
  const uint32_t sbase = smem_u32(smem);
  if ((sbase & 1023u) != 0u) return;                     // swizzled layouts need the aligned base (never expected)
  const uint32_t bars = sbase + kLmOffBar;
  auto bar = [&](int i) -> uint32_t { return bars + 8u * (uint32_t)i; };
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(smem + kLmOffBar + 8 * LM_NBARS);

  if (tid == 0) {
    for (int i = 0; i < LM_NBARS; ++i) mbar_init(bar(i), (i == LM_ACC_FREE) ? 256u : 1u);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 8) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                 ::"r"(smem_u32((const void*)tmem_slot)), "r"(512u) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  constexpr uint32_t n_stages = kLmStages;

  if (warp == 9) {
    // ------------------------------------------------------------------ TMA producer (one lane)
    if (lane == 0) {
      uint32_t kq = 0;                                   // stage uses so far, over all items
      bool ok = true;
      for (int item = blockIdx.x; ok && item < n_items; item += gridDim.x) {
        const int tile = item / n_chunks, chunk = item - tile * n_chunks;
        const int n0 = tile * p.tile_n, m0 = chunk * kLmRows;
        const int n_mt = (R - m0 > 128) ? 2 : 1;
        const uint32_t bytes = (uint32_t)n_mt * kLmBytesA + (uint32_t)p.tile_n * 128u;
        for (int k = 0; k < k_steps; ++k, ++kq) {
          const uint32_t st = kq % n_stages;
          if (kq >= n_stages && !mbar_wait(bar(LM_FREE0 + st), ((kq / n_stages) - 1u) & 1u)) { ok = false; break; }
          mbar_expect_tx(bar(LM_FULL0 + st), bytes);
          for (int mt = 0; mt < n_mt; ++mt)
            tma_load_2d(sbase + kLmOffA + (st * 2 + mt) * kLmBytesA, &tm_h, k * kLmTileK, m0 + mt * 128, bar(LM_FULL0 + st));
          tma_load_2d(sbase + kLmOffB + st * kLmStrideB, &tm_w, k * kLmTileK, n0, bar(LM_FULL0 + st));
        }
      }
      if (!ok && p.status) atomicOr(p.status, WEDLM_STATUS_WAIT_EXPIRED);
    }
  } else if (warp == 8) {
    // ------------------------------------------------------------------ MMA issue
    // all lanes run the loop and wait on the barriers, one elected lane issues (see elect_one())
    {
      const bool leader = elect_one();
      const uint32_t idesc = make_idesc(p.tile_n, false);
      uint32_t kq = 0, it = 0;
      bool ok = true;
      for (int item = blockIdx.x; ok && item < n_items; item += gridDim.x, ++it) {
        const int chunk = item % n_chunks;
        const int n_mt = (R - chunk * kLmRows > 128) ? 2 : 1;
        // the accumulators (all 512 columns) are free once the reduction warps have read the previous item
        if (it >= 1u) ok = mbar_wait(bar(LM_ACC_FREE), (it - 1u) & 1u);
        if (!ok) break;
        tc_fence_after();
        for (int k = 0; k < k_steps; ++k, ++kq) {
          const uint32_t st = kq % n_stages;
          ok = mbar_wait(bar(LM_FULL0 + st), (kq / n_stages) & 1u);
          if (!ok) break;
          tc_fence_after();
          for (int mt = 0; mt < n_mt; ++mt) {
#pragma unroll
            for (int kk = 0; kk < 4; ++kk) {
              const uint64_t ad = make_desc(sbase + kLmOffA + (st * 2 + mt) * kLmBytesA + kk * 32u, 16u, 1024u);
              const uint64_t bd = make_desc(sbase + kLmOffB + st * kLmStrideB + kk * 32u, 16u, 1024u);
              if (leader) umma(tmem_base + (uint32_t)mt * 256u, ad, bd, idesc, (k > 0) || (kk > 0));
            }
          }
          if (leader) umma_commit(bar(LM_FREE0 + st));
        }
        if (leader) umma_commit(bar(LM_ACC_FULL));            // arrives when every MMA of this item has completed
      }
      if (!ok && lane == 0 && p.status) atomicOr(p.status, WEDLM_STATUS_WAIT_EXPIRED);
    }
  } else {
    // ------------------------------------------------------------------ reduction warps: one row per thread
    const int mt = tid >> 7, r = tid & 127;
    uint32_t it = 0;
    for (int item = blockIdx.x; item < n_items; item += gridDim.x, ++it) {
      const int tile = item / n_chunks, chunk = item - tile * n_chunks;
      const int n0 = tile * p.tile_n, m0 = chunk * kLmRows;
      const int n_mt = (R - m0 > 128) ? 2 : 1;
      const int crow = m0 + mt * 128 + r;                // compacted row
      const bool active = mt < n_mt && crow < R;
      const int row = active ? p.row_map[crow] : 0;      // physical row b * W + i
      const int tilt_col = (active && p.tilt_ids) ? p.tilt_ids[row] - n0 : -1;     // column of this tile, if any
      if (!mbar_wait(bar(LM_ACC_FULL), it & 1u)) {
        if (p.status && (tid & 127) == 0) atomicOr(p.status, WEDLM_STATUS_WAIT_EXPIRED);
        break;
      }
      tc_fence_after();
      if (mt < n_mt) {
        const uint32_t taddr = tmem_base + ((uint32_t)((warp & 3) * 32) << 16) + (uint32_t)mt * 256u;
        const int n_cols = min(p.tile_n, p.V - n0);
        const int n_ch = (n_cols + 31) / 32;
        // pass 1: maximum and its lowest column
        float m = -CUDART_INF_F;
        int a = 0x7fffffff;
#pragma unroll 1
        for (int ch = 0; ch < n_ch; ++ch) {
          uint32_t o[32];
          tmem_ld32(taddr + ch * 32u, o);
          tmem_wait_ld();
#pragma unroll
          for (int e = 0; e < 32; ++e) {
            const int col = ch * 32 + e;
            float x = __uint_as_float(o[e]);
            if (col == tilt_col) x += p.tilt;
            if (col < n_cols && x > m) { m = x; a = n0 + col; }
          }
        }
        // pass 2: sums relative to the maximum (log2 domain, terms below 2^-127 are dropped)
        float s = 0.f, t = 0.f;
        const float kLog2e = 1.4426950408889634f;
        const float nm = -m * kLog2e;
#pragma unroll 1
        for (int ch = 0; ch < n_ch; ++ch) {
          uint32_t o[32];
          tmem_ld32(taddr + ch * 32u, o);
          tmem_wait_ld();
#pragma unroll
          for (int e = 0; e < 32; ++e) {
            const int col = ch * 32 + e;
            // columns at or beyond n_cols are not part of the row; beyond tile_n they were never written by this
            // item's MMAs and hold whatever the tensor memory held before (possibly inf): read them as -inf
            float x = (col < n_cols) ? __uint_as_float(o[e]) : -CUDART_INF_F;
            if (col == tilt_col) x += p.tilt;
            const float d = fmaxf(fmaf(x, kLog2e, nm), -127.f);     // -inf and NaN both end at -127, where 2^d flushes to 0
            const float ex = ex2_approx(d);
            s += ex;
            t = fmaf(d, ex, t);
          }
        }
        // every active row gets a partial for every tile: a tile without a finite logit leaves an empty one, which
        // the merge skips (the workspace is not cleared between calls)
        if (active)
          p.part[(size_t)row * p.n_tiles + tile] = (m > -CUDART_INF_F)
              ? make_float4(m, s, t * 0.6931471805599453f, __int_as_float(a))
              : make_float4(-CUDART_INF_F, 0.f, 0.f, __int_as_float(0x7fffffff));
      }
      tc_fence_before();
      mbar_arrive(bar(LM_ACC_FREE));               // this thread no longer needs the accumulators
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 8) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512u) : "memory");
  }
}

// ---------------------------------------------------------------------------------------------- row compaction
// Only mask rows need logits (Algorithm 1 predicts from l_mask).  After the reorder the mask rows of sequence b
// are the physical rows [n_filled[b], window_len[b]); their hidden states are gathered into one dense matrix so
// that the tensor-core tiles hold nothing but rows that count.  One block per physical row; every block counts the
// mask rows of the earlier sequences itself (B small integers from L2), block 0 also the total.
__device__ __forceinline__ int lm_mask_rows(int b, int W, const int32_t* n_filled, const int32_t* window_len) {
  const int L = window_len ? min(max(window_len[b], 0), W) : W;
  return L - min(max(n_filled[b], 0), L);
}

__global__ void __launch_bounds__(128)
lm_rows_gather_kernel(int B, int W, int H, const __nv_bfloat16* __restrict__ hidden, const int32_t* __restrict__ n_filled,
                      const int32_t* __restrict__ window_len, __nv_bfloat16* __restrict__ dense,
                      int32_t* __restrict__ row_map, int32_t* __restrict__ n_active) {
  __shared__ int warp_sums[4];
  const int row = blockIdx.x, b = row / W, i = row - b * W;
  const int L = window_len ? min(max(window_len[b], 0), W) : W;
  const int nf = min(max(n_filled[b], 0), L);
  const bool mask_row = i >= nf && i < L;
  if (!mask_row && row != 0) return;
  const int upto = (row == 0) ? B : b;                   // block 0 counts every sequence: the total
  int cnt = 0;
  for (int j = threadIdx.x; j < upto; j += 128) cnt += lm_mask_rows(j, W, n_filled, window_len);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) cnt += __shfl_xor_sync(0xffffffffu, cnt, o);
  if ((threadIdx.x & 31) == 0) warp_sums[threadIdx.x >> 5] = cnt;
  __syncthreads();
  const int sum = warp_sums[0] + warp_sums[1] + warp_sums[2] + warp_sums[3];
  if (row == 0 && threadIdx.x == 0) *n_active = sum;
  if (!mask_row) return;
  const int crow = (row == 0 ? 0 : sum) + (i - nf);      // row 0 belongs to sequence 0: nothing before it
  if (threadIdx.x == 0) row_map[crow] = row;
  const uint4* src = reinterpret_cast<const uint4*>(hidden + (size_t)row * H);
  uint4* dst = reinterpret_cast<uint4*>(dense + (size_t)crow * H);
  for (int v = threadIdx.x; v < H / 8; v += 128) dst[v] = src[v];
}

PFN_cuTensorMapEncodeTiled_v12000 lm_get_encode() {
  static PFN_cuTensorMapEncodeTiled_v12000 fn = nullptr;
  if (fn) return fn;
  void* ptr = nullptr;
  cudaDriverEntryPointQueryResult qres;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) != cudaSuccess ||
      qres != cudaDriverEntryPointSuccess)
    return nullptr;
  fn = reinterpret_cast<PFN_cuTensorMapEncodeTiled_v12000>(ptr);
  return fn;
}

// Vocabulary tile width: the multiple of 16 in [128, 256] that wastes the least in the last wave of
// persistent CTAs (ties go to the wider tile, which re-reads the hidden states less often).
int pick_tile_n(int vocab, int row_chunks, int sms) {
  int best_n = kLmMaxTileN;
  long long best_cost = -1;
  for (int n = kLmMaxTileN; n >= 128; n -= 16) {
    const long long items = (long long)((vocab + n - 1) / n) * row_chunks;
    const long long waves = (items + sms - 1) / sms;
    const long long cost = waves * n;
    if (best_cost < 0 || cost < best_cost) { best_cost = cost; best_n = n; }
  }
  return best_n;
}

}  // namespace

// Upper bound of the partials per row (the narrowest tile the host may pick).
int lmhead_conf_tiles(int vocab) { return (vocab + 127) / 128; }

// Workspace: [partials][n_active][row_map B W][dense hidden states B W H]
LmWorkspace lmhead_workspace(const wedlm_config_t* cfg, int hidden) {
  LmWorkspace w{};
  auto up = [](size_t x) { return (x + 255) / 256 * 256; };
  const size_t rows = (size_t)cfg->batch * cfg->window;
  w.off_part = 0;
  w.off_count = up(rows * lmhead_conf_tiles(cfg->vocab) * 16);
  w.off_map = w.off_count + 256;
  w.off_dense = w.off_map + up(rows * 4);
  w.total = w.off_dense + up(rows * (size_t)hidden * 2);
  return w;
}

int launch_lmhead_conf(const Shape& s, int hidden, const void* hidden_states, const void* lm_head, const int32_t* tilt_ids,
                       float tilt, const int32_t* n_filled, const int32_t* window_len, void* workspace,
                       const LmWorkspace& lw, int* n_tiles_out, int32_t* status, cudaStream_t st) {
  auto encode = lm_get_encode();
  if (!encode) return WEDLM_ERR_CUDA;
  const int R = s.B * s.W;
  const int sms = device_sm_count();
  {
    static bool attr_done[64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return WEDLM_ERR_CUDA;
    if (dev < 0 || dev >= 64 || !attr_done[dev]) {
      if (cudaFuncSetAttribute(lmhead_conf_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kLmSmem) != cudaSuccess)
        return WEDLM_ERR_CUDA;
      if (dev >= 0 && dev < 64) attr_done[dev] = true;
    }
  }
  char* ws = static_cast<char*>(workspace);
  int32_t* n_active = reinterpret_cast<int32_t*>(ws + lw.off_count);
  int32_t* row_map = reinterpret_cast<int32_t*>(ws + lw.off_map);
  __nv_bfloat16* dense = reinterpret_cast<__nv_bfloat16*>(ws + lw.off_dense);
  lm_rows_gather_kernel<<<R, 128, 0, st>>>(s.B, s.W, hidden, (const __nv_bfloat16*)hidden_states, n_filled, window_len, dense,
                                           row_map, n_active);
  count_launch();
  if (cudaGetLastError() != cudaSuccess) return WEDLM_ERR_CUDA;
  // the number of mask rows is device data: the tile width is picked for the most rows there can be
  const int row_chunks = (R + kLmRows - 1) / kLmRows;
  const int tile_n = pick_tile_n(s.V, row_chunks, sms);
  CUtensorMap tm_h, tm_w;
  for (int which = 0; which < 2; ++which) {
    // [rows][hidden] bf16, box = 64 hidden elements x (128 rows | tile_n tokens), 128-byte swizzle
    cuuint64_t dims[2] = {(cuuint64_t)hidden, (cuuint64_t)(which ? s.V : R)};
    cuuint64_t strides[1] = {(cuuint64_t)hidden * 2};
    cuuint32_t box[2] = {(cuuint32_t)kLmTileK, (cuuint32_t)(which ? tile_n : 128)};
    cuuint32_t estr[2] = {1, 1};
    if (encode(which ? &tm_w : &tm_h, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, which ? const_cast<void*>(lm_head) : (void*)dense,
               dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
               CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
      return WEDLM_ERR_CUDA;
  }
  LmParams p;
  p.W = s.W; p.V = s.V; p.H = hidden; p.tile_n = tile_n; p.n_tiles = (s.V + tile_n - 1) / tile_n;
  p.n_active = n_active; p.row_map = row_map;
  p.tilt = tilt; p.tilt_ids = tilt_ids;
  p.part = reinterpret_cast<float4*>(ws + lw.off_part);
  p.status = status;
  const long long max_items = (long long)p.n_tiles * row_chunks;
  const int grid = max_items < sms ? (int)max_items : sms;       // one persistent CTA per SM (the whole tensor memory each)
  lmhead_conf_kernel<<<grid, kLmThreads, kLmSmem, st>>>(tm_h, tm_w, p);
  count_launch();
  if (n_tiles_out) *n_tiles_out = p.n_tiles;
  return cuda_ok(cudaGetLastError());
}

}  // namespace wedlm
