// LM head fused with the vocabulary confidence reduction: the logits of the window rows are produced
// tile by tile in tensor memory and reduced there; they never reach HBM.
//
// logits[row, v] = <hidden[row, :], lm_head[v, :]>  (bf16 x bf16 -> fp32), and per mask row the same
// partials as the streaming confidence pass: m = max, a = lowest arg-max, s = sum e^(x-m),
// t = sum (x-m) e^(x-m) (entropy of Section 5.2 after the merge), one partial per vocabulary tile.
//
// Work item = one vocabulary tile of tile_n <= 256 tokens x up to 256 window rows (two 128-row
// accumulators of 256 TMEM columns each), so the output embedding is streamed from HBM once when
// B*W <= 256.  One persistent CTA per SM walks the items.  Warp 9 feeds a 3-stage ring with TMA (hidden
// states 2 x [128 x 64], embedding [tile_n x 64] per stage, 128-byte swizzle), warp 8 issues tcgen05.mma
// (128 x tile_n x 16, 8 per stage; one elected lane, the whole warp runs the loop) and releases stages through tcgen05.commit, warps 0-7 read their row of
// the accumulators back with tcgen05.ld and reduce it.  The wide tile matters: every item re-reads the
// hidden states from L2, and that traffic, not HBM, bounds the kernel.  All waits are bounded.
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
  int R, W, V, H, n_tiles, n_row_chunks, tile_n;
  float tilt;
  const int32_t* tilt_ids;        // [R] token whose logit gets +tilt, or NULL
  const int32_t* n_filled;
  const int32_t* window_len;
  float4* part;
  int32_t* status;
};

// Persistent CTAs: work item = (row chunk, vocabulary tile), items strided over the grid.
__global__ void __launch_bounds__(kLmThreads, 1)
lmhead_conf_kernel(const __grid_constant__ CUtensorMap tm_h, const __grid_constant__ CUtensorMap tm_w, const LmParams p) {
  extern __shared__ __align__(1024) uint8_t smem[];
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int k_steps = p.H / kLmTileK;
  const int n_items = p.n_tiles * p.n_row_chunks;
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

  if (warp == 9) {
    // ------------------------------------------------------------------ TMA producer (one lane)
    if (lane == 0) {
      uint32_t kq = 0;                                   // stage uses so far, over all items
      bool ok = true;
      for (int item = blockIdx.x; ok && item < n_items; item += gridDim.x) {
        const int chunk = item / p.n_tiles, tile = item - chunk * p.n_tiles;
        const int n0 = tile * p.tile_n, m0 = chunk * kLmRows;
        const int n_mt = (p.R - m0 > 128) ? 2 : 1;
        const uint32_t bytes = (uint32_t)n_mt * kLmBytesA + (uint32_t)p.tile_n * 128u;
        for (int k = 0; k < k_steps; ++k, ++kq) {
          const uint32_t st = kq % kLmStages;
          if (kq >= (uint32_t)kLmStages && !mbar_wait(bar(LM_FREE0 + st), ((kq / kLmStages) - 1u) & 1u)) { ok = false; break; }
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
        const int chunk = item / p.n_tiles;
        const int n_mt = (p.R - chunk * kLmRows > 128) ? 2 : 1;
        // the accumulators (all 512 columns) are free once the reduction warps have read the previous item
        if (it >= 1u) ok = mbar_wait(bar(LM_ACC_FREE), (it - 1u) & 1u);
        if (!ok) break;
        tc_fence_after();
        for (int k = 0; k < k_steps; ++k, ++kq) {
          const uint32_t st = kq % kLmStages;
          ok = mbar_wait(bar(LM_FULL0 + st), (kq / kLmStages) & 1u);
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
      const int chunk = item / p.n_tiles, tile = item - chunk * p.n_tiles;
      const int n0 = tile * p.tile_n, m0 = chunk * kLmRows;
      const int n_mt = (p.R - m0 > 128) ? 2 : 1;
      const int row = m0 + mt * 128 + r;
      bool active = false;
      if (mt < n_mt && row < p.R) {
        const int b = row / p.W, i = row - b * p.W;
        const int L = p.window_len ? min(max(p.window_len[b], 0), p.W) : p.W;
        active = i >= p.n_filled[b] && i < L;
      }
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

int launch_lmhead_conf(const Shape& s, int hidden, const void* hidden_states, const void* lm_head, const int32_t* tilt_ids,
                       float tilt, const int32_t* n_filled, const int32_t* window_len, void* partials, int* n_tiles_out,
                       int32_t* status, cudaStream_t st) {
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
  const int row_chunks = (R + kLmRows - 1) / kLmRows;
  const int tile_n = pick_tile_n(s.V, row_chunks, sms);
  CUtensorMap tm_h, tm_w;
  for (int which = 0; which < 2; ++which) {
    // [rows][hidden] bf16, box = 64 hidden elements x (128 rows | tile_n tokens), 128-byte swizzle
    cuuint64_t dims[2] = {(cuuint64_t)hidden, (cuuint64_t)(which ? s.V : R)};
    cuuint64_t strides[1] = {(cuuint64_t)hidden * 2};
    cuuint32_t box[2] = {(cuuint32_t)kLmTileK, (cuuint32_t)(which ? tile_n : 128)};
    cuuint32_t estr[2] = {1, 1};
    if (encode(which ? &tm_w : &tm_h, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(which ? lm_head : hidden_states),
               dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
               CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
      return WEDLM_ERR_CUDA;
  }
  LmParams p;
  p.R = R; p.W = s.W; p.V = s.V; p.H = hidden; p.tile_n = tile_n; p.n_tiles = (s.V + tile_n - 1) / tile_n;
  p.n_row_chunks = row_chunks;
  p.tilt = tilt; p.tilt_ids = tilt_ids; p.n_filled = n_filled; p.window_len = window_len;
  p.part = reinterpret_cast<float4*>(partials);
  p.status = status;
  const int n_items = p.n_tiles * p.n_row_chunks;
  const int grid = n_items < sms ? n_items : sms;       // one persistent CTA per SM (the whole tensor memory each)
  lmhead_conf_kernel<<<grid, kLmThreads, kLmSmem, st>>>(tm_h, tm_w, p);
  count_launch();
  if (n_tiles_out) *n_tiles_out = p.n_tiles;
  return cuda_ok(cudaGetLastError());
}

}  // namespace wedlm
