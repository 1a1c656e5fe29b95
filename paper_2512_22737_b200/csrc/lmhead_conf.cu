// LM head fused with the vocabulary confidence reduction: the logits of the window rows are produced
// tile by tile in tensor memory and reduced there; they never reach HBM.
//
// logits[row, v] = <hidden[row, :], lm_head[v, :]>  (bf16 x bf16 -> fp32), and per mask row the same
// partials as the streaming confidence pass: m = max, a = lowest arg-max, s = sum e^(x-m),
// t = sum (x-m) e^(x-m) (entropy of Section 5.2 after the merge), one partial per 128-token vocabulary tile.
//
// One CTA = one vocabulary tile of 128 tokens x up to 256 window rows (two 128-row accumulators of 128
// TMEM columns each), so the output embedding is streamed from HBM once when B*W <= 256.  Warp 9 feeds a
// 4-stage ring with TMA (hidden states 2 x [128 x 64], embedding [128 x 64] per stage, 128-byte swizzle),
// warp 8 issues tcgen05.mma (128x128x16, 8 per stage) and releases stages through tcgen05.commit, warps
// 0-7 read their row of the accumulator back with tcgen05.ld and reduce it.  All waits are bounded.
#include <cuda.h>
#include <cudaTypedefs.h>
#include <math_constants.h>

#include "common.cuh"
#include "tc_ptx.cuh"

namespace wedlm {
namespace {

using namespace ptx;

constexpr int kLmTileN = 128;                 // vocabulary entries per CTA
constexpr int kLmTileK = 64;                  // hidden elements per stage (one 128-byte swizzle row)
constexpr int kLmStages = 4;
constexpr int kLmRows = 256;                  // window rows per CTA (two accumulators)
constexpr uint32_t kLmBytesA = 128 * 128;     // one 128-row tile of hidden states per stage
constexpr uint32_t kLmBytesB = 128 * 128;     // the embedding tile per stage
constexpr uint32_t kLmOffA = 0;                                   // [stages][2][16 KB]
constexpr uint32_t kLmOffB = kLmStages * 2 * kLmBytesA;           // [stages][16 KB]
constexpr uint32_t kLmOffBar = kLmOffB + kLmStages * kLmBytesB;
constexpr uint32_t kLmSmem = kLmOffBar + 128;
constexpr int kLmThreads = 320;               // 8 reduction warps + MMA warp + TMA warp

enum LmBar { LM_FULL0 = 0, LM_FREE0 = LM_FULL0 + kLmStages, LM_ACC = LM_FREE0 + kLmStages, LM_NBARS };

struct LmParams {
  int R, W, V, H, n_tiles;
  float tilt;
  const int32_t* tilt_ids;        // [R] token whose logit gets +tilt, or NULL
  const int32_t* n_filled;
  const int32_t* window_len;
  float4* part;
};

// grid: x = vocabulary tile, y = chunk of 256 rows
__global__ void __launch_bounds__(kLmThreads, 1)
lmhead_conf_kernel(const __grid_constant__ CUtensorMap tm_h, const __grid_constant__ CUtensorMap tm_w, const LmParams p) {
  extern __shared__ __align__(1024) uint8_t smem[];
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int n0 = blockIdx.x * kLmTileN;
  const int m0 = blockIdx.y * kLmRows;
  const int n_mt = (p.R - m0 > 128) ? 2 : 1;            // 128-row tiles of this chunk that hold rows
  const int k_steps = p.H / kLmTileK;
  const uint32_t sbase = smem_u32(smem);
  if ((sbase & 1023u) != 0u) return;                     // swizzled layouts need the aligned base (never expected)
  const uint32_t bars = sbase + kLmOffBar;
  auto bar = [&](int i) -> uint32_t { return bars + 8u * (uint32_t)i; };
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(smem + kLmOffBar + 8 * LM_NBARS);

  if (tid == 0) {
    for (int i = 0; i < LM_NBARS; ++i) mbar_init(bar(i), 1u);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 8) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                 ::"r"(smem_u32((const void*)tmem_slot)), "r"(256u) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 9) {
    // ------------------------------------------------------------------ TMA producer (one lane)
    if (lane == 0) {
      const uint32_t bytes = (uint32_t)n_mt * kLmBytesA + kLmBytesB;
      for (int k = 0; k < k_steps; ++k) {
        const int st = k % kLmStages;
        if (k >= kLmStages && !mbar_wait(bar(LM_FREE0 + st), (uint32_t)((k / kLmStages) - 1) & 1u)) break;
        mbar_expect_tx(bar(LM_FULL0 + st), bytes);
        for (int mt = 0; mt < n_mt; ++mt)
          tma_load_2d(sbase + kLmOffA + (uint32_t)(st * 2 + mt) * kLmBytesA, &tm_h, k * kLmTileK, m0 + mt * 128, bar(LM_FULL0 + st));
        tma_load_2d(sbase + kLmOffB + (uint32_t)st * kLmBytesB, &tm_w, k * kLmTileK, n0, bar(LM_FULL0 + st));
      }
    }
  } else if (warp == 8) {
    // ------------------------------------------------------------------ MMA issue (one lane)
    if (lane == 0) {
      const uint32_t idesc = make_idesc(kLmTileN, false);
      bool ok = true;
      for (int k = 0; ok && k < k_steps; ++k) {
        const int st = k % kLmStages;
        ok = mbar_wait(bar(LM_FULL0 + st), (uint32_t)(k / kLmStages) & 1u);
        if (!ok) break;
        tc_fence_after();
        for (int mt = 0; mt < n_mt; ++mt) {
#pragma unroll
          for (int kk = 0; kk < 4; ++kk) {
            const uint64_t ad = make_desc(sbase + kLmOffA + (uint32_t)(st * 2 + mt) * kLmBytesA + kk * 32u, 16u, 1024u);
            const uint64_t bd = make_desc(sbase + kLmOffB + (uint32_t)st * kLmBytesB + kk * 32u, 16u, 1024u);
            umma(tmem_base + (uint32_t)mt * 128u, ad, bd, idesc, (k > 0) || (kk > 0));
          }
        }
        umma_commit(bar(LM_FREE0 + st));
      }
      umma_commit(bar(LM_ACC));        // arrives when every MMA above has completed (or at once after a give-up)
    }
  } else {
    // ------------------------------------------------------------------ reduction warps: one row per thread
    const int mt = tid >> 7, r = tid & 127;
    const int row = m0 + mt * 128 + r;
    bool active = false;
    if (mt < n_mt && row < p.R) {
      const int b = row / p.W, i = row - b * p.W;
      const int L = p.window_len ? min(max(p.window_len[b], 0), p.W) : p.W;
      active = i >= p.n_filled[b] && i < L;
    }
    const int tilt_col = (active && p.tilt_ids) ? p.tilt_ids[row] - n0 : -1;     // column of this tile, if any
    const bool ok = mbar_wait(bar(LM_ACC), 0);
    tc_fence_after();
    if (ok && mt < n_mt) {
      const uint32_t taddr = tmem_base + ((uint32_t)((warp & 3) * 32) << 16) + (uint32_t)mt * 128u;
      const int n_cols = min(kLmTileN, p.V - n0);
      // pass 1: maximum and its lowest column
      float m = -CUDART_INF_F;
      int a = 0x7fffffff;
#pragma unroll 1
      for (int ch = 0; ch < 4; ++ch) {
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
      for (int ch = 0; ch < 4; ++ch) {
        uint32_t o[32];
        tmem_ld32(taddr + ch * 32u, o);
        tmem_wait_ld();
#pragma unroll
        for (int e = 0; e < 32; ++e) {
          const int col = ch * 32 + e;
          float x = __uint_as_float(o[e]);
          if (col == tilt_col) x += p.tilt;
          const float d = fmaxf(fmaf(x, kLog2e, nm), -127.f);
          const float ex = (col < n_cols) ? ex2_approx(d) : 0.f;
          s += ex;
          t = fmaf(d, ex, t);
        }
      }
      if (active && m > -CUDART_INF_F)
        p.part[(size_t)row * p.n_tiles + blockIdx.x] = make_float4(m, s, t * 0.6931471805599453f, __int_as_float(a));
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 8) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(256u) : "memory");
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

}  // namespace

int lmhead_conf_tiles(int vocab) { return (vocab + kLmTileN - 1) / kLmTileN; }

int launch_lmhead_conf(const Shape& s, int hidden, const void* hidden_states, const void* lm_head, const int32_t* tilt_ids,
                       float tilt, const int32_t* n_filled, const int32_t* window_len, void* partials, cudaStream_t st) {
  auto encode = lm_get_encode();
  if (!encode) return WEDLM_ERR_CUDA;
  const int R = s.B * s.W;
  CUtensorMap tm_h, tm_w;
  for (int which = 0; which < 2; ++which) {
    // [rows][hidden] bf16, box = 64 hidden elements x 128 rows, 128-byte swizzle
    cuuint64_t dims[2] = {(cuuint64_t)hidden, (cuuint64_t)(which ? s.V : R)};
    cuuint64_t strides[1] = {(cuuint64_t)hidden * 2};
    cuuint32_t box[2] = {(cuuint32_t)kLmTileK, 128};
    cuuint32_t estr[2] = {1, 1};
    if (encode(which ? &tm_w : &tm_h, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(which ? lm_head : hidden_states),
               dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
               CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
      return WEDLM_ERR_CUDA;
  }
  LmParams p;
  p.R = R; p.W = s.W; p.V = s.V; p.H = hidden; p.n_tiles = lmhead_conf_tiles(s.V);
  p.tilt = tilt; p.tilt_ids = tilt_ids; p.n_filled = n_filled; p.window_len = window_len;
  p.part = reinterpret_cast<float4*>(partials);
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
  dim3 grid(p.n_tiles, (R + kLmRows - 1) / kLmRows);
  lmhead_conf_kernel<<<grid, kLmThreads, kLmSmem, st>>>(tm_h, tm_w, p);
  count_launch();
  return cuda_ok(cudaGetLastError());
}

}  // namespace wedlm
