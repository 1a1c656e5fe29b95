// Window attention on the 5th-generation tensor cores (sm_100a): TMA-staged K/V pages, tcgen05.mma
// with accumulators in tensor memory, online softmax in registers.
//
// What it computes (Section 5.2, "a causal forward over the current window conditioned on the cached
// prefix"): for one (sequence b, KV head g) the M = W_t*G query rows (W_t window slots x G grouped
// query heads, G*W_t = 128) attend to cache positions 0..P-1 and to the staged window rows P..P+i
// (physical row i sees window rows j <= i).  All keys are read from the paged cache: the window's
// rotated K and V were staged there by the RoPE/stage kernel before this kernel starts.
//
// One CTA = one (b, g, 128-row tile, key chunk).  Warps 0-3 (128 threads, one query row each) run the
// online softmax; warp 4 issues every MMA (one elected lane); warps 5 and 6 issue the TMA copies of K and V.  Per 64-key tile:
//     S[t&1] = Q K_t^T   (tcgen05.mma, 8 k-steps, fp32 in TMEM columns 0..127, double buffered)
//     softmax threads: tcgen05.ld S row -> mask -> running max (lazy rescale) -> p = 2^(s*c - m*c)
//                      -> bf16 P tile into shared memory (128-byte swizzle)
//     O += P V_t         (tcgen05.mma, 4 k-steps, V consumed MN-major straight from its page layout)
// Two CTAs fit on an SM (112 KB shared memory, 256 TMEM columns each), so one CTA's softmax overlaps
// the other's MMAs and loads.  Every wait on an mbarrier is bounded; on expiry the CTA records
// WEDLM_STATUS_WAIT_EXPIRED, drains its copies, frees its tensor memory and returns.
#include <cuda.h>
#include <cudaTypedefs.h>
#include <math_constants.h>

#include "common.cuh"
#include "tc_ptx.cuh"

namespace wedlm {
namespace {

constexpr int kTileN = 64;            // keys per tile (4 pages)
constexpr int kD = 128;               // head size
constexpr int kPage = 16;
static_assert(kTileN == 4 * kPage, "a tile is four pages");
constexpr int kThreadsT = 224;        // 4 softmax warps + MMA issue warp + two TMA producer warps
constexpr float kLazyRescaleLog2 = 8.0f;   // keep the old reference while the max grew by < 2^8

// shared memory map (bytes, base 1024-aligned)
constexpr uint32_t kOffQ = 0;                       // 2 halves x [128 rows x 128 B]
constexpr uint32_t kOffK = 32768;                   // 2 stages x 2 halves x [64 rows x 128 B]
constexpr uint32_t kOffV = 65536;                   // 2 stages x 2 halves x [64 rows x 128 B]
constexpr uint32_t kOffP = 98304;                   // [128 rows x 128 B] bf16 probabilities
constexpr uint32_t kOffBar = 114688;
constexpr uint32_t kSmemBytes = kOffBar + 256;
constexpr uint32_t kStageBytes = 16384;
constexpr uint32_t kHalfKV = 8192;
constexpr uint32_t kHalfQ = 16384;

enum Bar { Q_FULL = 0, K_FULL0, K_FULL1, V_FULL0, V_FULL1, S_FULL0, S_FULL1, O_DONE, P_READY, K_FREE0, K_FREE1,
           V_FREE0, V_FREE1, N_BARS };

struct TensorAttnParams {
  int B, W, Hq, Hkv, G, W_t, n_mtiles, n_splits, chunk, max_pages, num_pages, max_prefix;
  float scale_log2;          // softmax scale * log2(e)
  const int32_t* block_table;
  const int32_t* prefix_len;
  const int32_t* order;      // sequences by decreasing prefix length, or NULL
  __nv_bfloat16* out;
  float* part_o;
  float* part_ml;
  int32_t* status;
};

using namespace ptx;

// 1-D grid, block index = (sequence rank * Hkv + kv head) * (n_splits * n_mtiles) + split * n_mtiles + mtile
__global__ void __launch_bounds__(kThreadsT, 2)
attn_tensor_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                   const __grid_constant__ CUtensorMap tm_v, const TensorAttnParams p) {
  extern __shared__ __align__(1024) uint8_t smem[];
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int per_head = p.n_splits * p.n_mtiles;
  const int unit = (int)(blockIdx.x / (unsigned)per_head), in_head = (int)(blockIdx.x - (unsigned)unit * per_head);
  const int split = in_head / p.n_mtiles, mtile = in_head - split * p.n_mtiles;
  const int rank = unit / p.Hkv, g = unit - rank * p.Hkv;
  const int b = p.order ? p.order[rank] : rank;                      // longest sequences are dispatched first

  const int P = checked_prefix(p.prefix_len, b, p.max_prefix, p.status, tid == 0);
  const int total = P + p.W;
  const int n_valid = (total + p.chunk - 1) / p.chunk;
  if (split >= n_valid) return;
  const int slot0 = mtile * p.W_t;                          // first window slot of this row tile
  const int slot_end = min(p.W, slot0 + p.W_t);
  const int kv_begin = split * p.chunk;
  const int kv_end = min(min(kv_begin + p.chunk, total), P + slot_end);   // horizon of the last row
  const int T = kv_begin < kv_end ? (kv_end - kv_begin + kTileN - 1) / kTileN : 0;

  // this thread's query row (softmax warps only)
  const int r = tid;                                         // row of the 128-row tile
  const int i_row = slot0 + r / p.G;                         // physical window slot
  const int h = g * p.G + r % p.G;                           // query head
  const bool row_valid = (tid < 128) && (i_row < p.W);
  const float c = p.scale_log2;

  if (T == 0) {
    // nothing visible in this chunk for these rows: an empty partial (only possible when n_splits > 1)
    if (row_valid && n_valid > 1) {
      const size_t prow = (((size_t)b * p.Hq + h) * p.W + i_row) * p.n_splits + split;
      float4 z = make_float4(0.f, 0.f, 0.f, 0.f);
      float4* dst = reinterpret_cast<float4*>(p.part_o + prow * kD);
      for (int d4 = 0; d4 < kD / 4; ++d4) dst[d4] = z;
      p.part_ml[prow * 2] = -CUDART_INF_F;
      p.part_ml[prow * 2 + 1] = 0.f;
    }
    return;
  }

  const uint32_t sbase = smem_u32(smem);
  if ((sbase & 1023u) != 0u) {     // the swizzled layouts need a 1024-byte aligned base
    if (p.status && tid == 0) atomicOr(p.status, WEDLM_STATUS_WAIT_EXPIRED);
    return;
  }
  const uint32_t bars = sbase + kOffBar;
  auto bar = [&](int i) -> uint32_t { return bars + 8u * (uint32_t)i; };
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(smem + kOffBar + 112);
  volatile uint32_t* abort_flag = tmem_slot + 1;

  if (tid == 0) {
    for (int i = 0; i < N_BARS; ++i) mbar_init(bar(i), i == P_READY ? 128u : 1u);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 4) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                 ::"r"(smem_u32((const void*)tmem_slot)), "r"(256u) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  const uint32_t tmem_S = tmem_base;            // columns [0,64) and [64,128)
  const uint32_t tmem_O = tmem_base + 128u;     // columns [128,256)

  if (warp == 4) {
    // ------------------------------------------------------------------ MMA issue warp
    // All lanes run the loop and wait on the barriers; one elected lane issues (see elect_one()).  The warp
    // never waits for an MMA to finish: completion is signalled to the consumers of the result (S_FULL,
    // O_DONE) and to the producer of the operands (K_FREE, V_FREE) through tcgen05.commit.
    {
      const bool leader = elect_one();
      bool ok = true;
      const uint32_t idesc_qk = make_idesc(kTileN, false);
      const uint32_t idesc_pv = make_idesc(kD, true);
      auto issue_qk = [&](int t) {
        const uint32_t st = (uint32_t)t & 1u;
        tc_fence_after();
#pragma unroll
        for (int kk = 0; kk < 8; ++kk) {
          const uint64_t ad = make_desc(sbase + kOffQ + (kk >> 2) * kHalfQ + (kk & 3) * 32u, 16u, 1024u);
          const uint64_t bd = make_desc(sbase + kOffK + st * kStageBytes + (kk >> 2) * kHalfKV + (kk & 3) * 32u, 16u, 1024u);
          if (leader) umma(tmem_S + st * 64u, ad, bd, idesc_qk, kk > 0);
        }
        if (leader) {
          umma_commit(bar(S_FULL0 + st));
          umma_commit(bar(K_FREE0 + st));
        }
      };
      ok = mbar_wait(bar(Q_FULL), 0);
      if (ok) ok = mbar_wait(bar(K_FULL0), 0);
      if (ok) issue_qk(0);
      for (int t = 0; ok && t < T; ++t) {
        const uint32_t st = (uint32_t)t & 1u, ph = ((uint32_t)t >> 1) & 1u;
        if (t + 1 < T) {
          // S[(t+1)&1] was last read by the softmax of tile t-1, whose P_READY we saw one iteration ago
          ok = mbar_wait(bar(K_FULL0 + (st ^ 1u)), ((uint32_t)(t + 1) >> 1) & 1u);
          if (!ok) break;
          issue_qk(t + 1);
        }
        ok = mbar_wait(bar(P_READY), (uint32_t)t & 1u);
        if (!ok) break;
        ok = mbar_wait(bar(V_FULL0 + st), ph);
        if (!ok) break;
        tc_fence_after();
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const uint64_t ad = make_desc(sbase + kOffP + j * 32u, 16u, 1024u);
          const uint64_t bd = make_desc(sbase + kOffV + st * kStageBytes + j * 2048u, kHalfKV, 1024u);
          if (leader) umma(tmem_O, ad, bd, idesc_pv, (t > 0) || (j > 0));
        }
        if (leader) {
          umma_commit(bar(O_DONE));
          umma_commit(bar(V_FREE0 + st));
        }
      }
      if (!ok && lane == 0) {
        *abort_flag = 1;
        if (p.status) atomicOr(p.status, WEDLM_STATUS_WAIT_EXPIRED);
      }
    }
  } else if (warp >= 5) {
    // ------------------------------------------------------------------ TMA producer warps
    // Warp 5 streams the K tiles (and loads Q), warp 6 the V tiles; each refills a stage as soon as the
    // MMAs that read it have completed.  A tile is 8 copies of 2 KB (4 pages x 2 column halves): lanes
    // 0..7 each look up their page and issue their copy, so a tile leaves in one warp instruction.
    const bool is_k = (warp == 5);
    bool ok = true;
    const int oob_row = p.num_pages * p.Hkv * kPage;        // a row coordinate past the end: zero fill
    const int pg = (lane >> 1) & 3, half = lane & 1;
    const uint32_t lane_dst = (uint32_t)pg * 2048u + (uint32_t)half * kHalfKV;
    // TMA row coordinate of this lane's page of tile t (same for K and V)
    auto page_row = [&](int t) -> int {
      const int key0 = kv_begin + t * kTileN + pg * kPage;
      const int lp = key0 / kPage;
      int pp = -1;
      if (lp < p.max_pages) pp = p.block_table[(size_t)b * p.max_pages + lp];
      if (pp < 0 || pp >= p.num_pages) {
        if (is_k && key0 < kv_end && p.status) atomicOr(p.status, lp < p.max_pages ? WEDLM_STATUS_BAD_PAGE : WEDLM_STATUS_BAD_LENGTH);
        return oob_row;
      }
      return (pp * p.Hkv + g) * kPage;
    };
    auto wait_all = [&](uint32_t barrier, uint32_t parity) -> bool {      // lane 0 waits, the warp follows
      int good = 1;
      if (lane == 0) good = mbar_wait(barrier, parity) ? 1 : 0;
      return __shfl_sync(0xffffffffu, good, 0) != 0;
    };
    if (is_k && lane == 0) {
      // Q tile: two 64-element halves of [W_t slots x G heads] rows
      const int q_slots = min(p.W_t, p.W);        // box height along the window dimension
      mbar_expect_tx(bar(Q_FULL), (uint32_t)(2 * 64 * p.G * q_slots * 2));
      tma_load_4d(sbase + kOffQ, &tm_q, 0, g * p.G, slot0, b, bar(Q_FULL));
      tma_load_4d(sbase + kOffQ + kHalfQ, &tm_q, 64, g * p.G, slot0, b, bar(Q_FULL));
    }
    const CUtensorMap* map = is_k ? &tm_k : &tm_v;
    const uint32_t stage0 = sbase + (is_k ? kOffK : kOffV);
    const int full0 = is_k ? K_FULL0 : V_FULL0, free0 = is_k ? K_FREE0 : V_FREE0;
    int y_next = page_row(0);
    for (int t = 0; ok && t < T; ++t) {
      const uint32_t st = (uint32_t)t & 1u;
      const int y = y_next;
      if (t + 1 < T) y_next = page_row(t + 1);              // table entry of the next tile, used one iteration later
      if (t >= 2) ok = wait_all(bar(free0 + st), ((uint32_t)(t - 2) >> 1) & 1u);
      if (!ok) break;
      if (lane == 0) mbar_expect_tx(bar(full0 + st), kStageBytes);
      __syncwarp();
      if (lane < 8) tma_load_2d(stage0 + st * kStageBytes + lane_dst, map, half * 64, y, bar(full0 + st));
    }
    if (!ok && lane == 0) {
      *abort_flag = 1;
      if (p.status) atomicOr(p.status, WEDLM_STATUS_WAIT_EXPIRED);
    }
  } else {
    // ------------------------------------------------------------------ softmax warps: one row per thread
    const uint32_t lane_sel = (uint32_t)(warp * 32) << 16;
    const int limit = row_valid ? P + i_row : -1;           // last visible key index (inclusive)
    float m_ref = -CUDART_INF_F;                            // reference maximum (raw score units)
    float l = 0.f;
    bool ok = true;
    for (int t = 0; t < T; ++t) {
      const uint32_t st = (uint32_t)t & 1u, ph = ((uint32_t)t >> 1) & 1u;
      ok = mbar_wait(bar(S_FULL0 + st), ph);
      if (!ok) break;
      tc_fence_after();
      uint32_t raw[64];
      {
        uint32_t (&lo)[32] = *reinterpret_cast<uint32_t (*)[32]>(&raw[0]);
        uint32_t (&hi)[32] = *reinterpret_cast<uint32_t (*)[32]>(&raw[32]);
        tmem_ld32(tmem_S + lane_sel + st * 64u, lo);
        tmem_ld32(tmem_S + lane_sel + st * 64u + 32u, hi);
        tmem_wait_ld();
      }
      const int tile0 = kv_begin + t * kTileN;
      const bool need_mask = tile0 + kTileN > min(P + slot0 + 1, kv_end);   // block-uniform
      float m_tile;
      if (need_mask) {
        m_tile = -CUDART_INF_F;
#pragma unroll
        for (int cc = 0; cc < 64; ++cc) {
          const int key = tile0 + cc;
          float x = __uint_as_float(raw[cc]);
          x = (key <= limit && key < kv_end) ? x : -CUDART_INF_F;
          raw[cc] = __float_as_uint(x);
          m_tile = fmaxf(m_tile, x);
        }
      } else {
        float m4[4] = {-CUDART_INF_F, -CUDART_INF_F, -CUDART_INF_F, -CUDART_INF_F};
#pragma unroll
        for (int cc = 0; cc < 64; cc += 8) {
          m4[0] = max3(m4[0], __uint_as_float(raw[cc + 0]), __uint_as_float(raw[cc + 1]));
          m4[1] = max3(m4[1], __uint_as_float(raw[cc + 2]), __uint_as_float(raw[cc + 3]));
          m4[2] = max3(m4[2], __uint_as_float(raw[cc + 4]), __uint_as_float(raw[cc + 5]));
          m4[3] = max3(m4[3], __uint_as_float(raw[cc + 6]), __uint_as_float(raw[cc + 7]));
        }
        m_tile = fmaxf(fmaxf(m4[0], m4[1]), fmaxf(m4[2], m4[3]));
      }
      // lazy reference: only move it when the maximum grew by more than 2^kLazyRescaleLog2
      float alpha = 1.f;
      bool moved = false;
      if (m_tile > -CUDART_INF_F && (m_ref == -CUDART_INF_F || (m_tile - m_ref) * c > kLazyRescaleLog2)) {
        alpha = (m_ref == -CUDART_INF_F) ? 0.f : exp2f((m_ref - m_tile) * c);
        m_ref = m_tile;
        moved = true;
      }
      const float neg_mc = (m_ref == -CUDART_INF_F) ? 0.f : -m_ref * c;
      // p = 2^(s*c - m*c): the scale and the reference are folded into one packed FMA per two scores
      const unsigned long long C2 = pack2(c, c), NM2 = pack2(neg_mc, neg_mc);
      unsigned long long sumA = pack2(0.f, 0.f), sumB = sumA;
      uint32_t pk[32];
#pragma unroll
      for (int cc = 0; cc < 64; cc += 4) {
        float a0, a1, b0, b1;
        unpack2(fma2(pack2(__uint_as_float(raw[cc]), __uint_as_float(raw[cc + 1])), C2, NM2), a0, a1);
        unpack2(fma2(pack2(__uint_as_float(raw[cc + 2]), __uint_as_float(raw[cc + 3])), C2, NM2), b0, b1);
        const float p0 = ex2_approx(a0), p1 = ex2_approx(a1), p2 = ex2_approx(b0), p3 = ex2_approx(b1);
        sumA = add2(sumA, pack2(p0, p1));
        sumB = add2(sumB, pack2(p2, p3));
        pk[cc >> 1] = pack_bf16(p0, p1);
        pk[(cc >> 1) + 1] = pack_bf16(p2, p3);
      }
      float sum, sum2;
      {
        float x0, x1;
        unpack2(add2(sumA, sumB), x0, x1);
        sum = x0;
        sum2 = x1;
      }
      l = l * alpha + (sum + sum2);
      // P buffer and O are free / stable once P V_{t-1} has completed
      if (t > 0) {
        ok = mbar_wait(bar(O_DONE), (uint32_t)(t - 1) & 1u);
        if (!ok) break;
        tc_fence_after();
        if (__any_sync(0xffffffffu, moved)) {
#pragma unroll 1
          for (int ch = 0; ch < 4; ++ch) {
            uint32_t o[32];
            tmem_ld32(tmem_O + lane_sel + ch * 32u, o);
            tmem_wait_ld();
#pragma unroll
            for (int e = 0; e < 32; ++e) o[e] = __float_as_uint(__uint_as_float(o[e]) * alpha);
            tmem_st32(tmem_O + lane_sel + ch * 32u, o);
          }
          tmem_wait_st();
        }
      }
      // bf16 P row into the 128-byte-swizzled K-major tile: 16-byte chunk j of row r sits at j ^ (r & 7)
      {
        uint8_t* prow = smem + kOffP + r * 128;
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          uint4 v = make_uint4(pk[4 * j], pk[4 * j + 1], pk[4 * j + 2], pk[4 * j + 3]);
          *reinterpret_cast<uint4*>(prow + ((j ^ (r & 7)) << 4)) = v;
        }
      }
      // last tile: V rows of keys beyond the horizon may hold anything (0 * NaN = NaN): zero them
      if (t == T - 1 && kv_end - tile0 < kTileN) {
        ok = mbar_wait(bar(V_FULL0 + st), ph);
        if (!ok) break;
        const int first_bad = kv_end - tile0;
        uint8_t* vst = smem + kOffV + st * kStageBytes;
        for (int idx = tid; idx < (kTileN - first_bad) * 16; idx += 128) {      // 16 x 16-byte chunks per key row
          const int row = first_bad + idx / 16, ch = idx % 16;
          *reinterpret_cast<uint4*>(vst + (ch >> 3) * kHalfKV + row * 128 + ((ch & 7) << 4)) = make_uint4(0, 0, 0, 0);
        }
      }
      fence_async_smem();
      tc_fence_before();
      mbar_arrive(bar(P_READY));
    }
    if (ok) ok = mbar_wait(bar(O_DONE), (uint32_t)(T - 1) & 1u);
    if (!ok) {
      *abort_flag = 1;
      if (p.status) atomicOr(p.status, WEDLM_STATUS_WAIT_EXPIRED);
    } else {
      tc_fence_after();
      const bool final_out = n_valid == 1;        // the only chunk of this sequence: write the result itself
                                                  // (n_valid <= n_splits because P is clamped to the planned bound)
      const float inv = l > 0.f ? 1.f / l : 0.f;
      const size_t orow = (((size_t)b * p.W + i_row) * p.Hq + h) * kD;
      const size_t prow = (((size_t)b * p.Hq + h) * p.W + i_row) * p.n_splits + split;
#pragma unroll 1
      for (int ch = 0; ch < 4; ++ch) {
        uint32_t o[32];
        tmem_ld32(tmem_O + lane_sel + ch * 32u, o);
        tmem_wait_ld();
        if (!row_valid) continue;
        if (final_out) {
          uint4* dst = reinterpret_cast<uint4*>(p.out + orow + ch * 32);
#pragma unroll
          for (int q4 = 0; q4 < 4; ++q4) {
            uint4 v;
            v.x = pack_bf16(__uint_as_float(o[8 * q4 + 0]) * inv, __uint_as_float(o[8 * q4 + 1]) * inv);
            v.y = pack_bf16(__uint_as_float(o[8 * q4 + 2]) * inv, __uint_as_float(o[8 * q4 + 3]) * inv);
            v.z = pack_bf16(__uint_as_float(o[8 * q4 + 4]) * inv, __uint_as_float(o[8 * q4 + 5]) * inv);
            v.w = pack_bf16(__uint_as_float(o[8 * q4 + 6]) * inv, __uint_as_float(o[8 * q4 + 7]) * inv);
            dst[q4] = v;
          }
        } else {
          uint4* dst = reinterpret_cast<uint4*>(p.part_o + prow * kD + ch * 32);
#pragma unroll
          for (int q4 = 0; q4 < 8; ++q4) dst[q4] = make_uint4(o[4 * q4], o[4 * q4 + 1], o[4 * q4 + 2], o[4 * q4 + 3]);
        }
      }
      if (row_valid && !final_out) {
        p.part_ml[prow * 2] = (m_ref == -CUDART_INF_F) ? -CUDART_INF_F : m_ref * c;     // log2 domain
        p.part_ml[prow * 2 + 1] = l;
      }
    }
  }

  // ------------------------------------------------------------------ teardown
  tc_fence_before();
  __syncthreads();
  if (*abort_flag != 0) {
    // a wait expired: give copies that may still be in flight a bounded time (about 0.2 ms) to land
    // before this CTA's shared memory is handed to another CTA
    for (int it = 0; it < 200; ++it) __nanosleep(1000);
  }
  __syncthreads();
  if (warp == 4) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(256u) : "memory");
  }
}

// ---------------------------------------------------------------------------------------------- host
PFN_cuTensorMapEncodeTiled_v12000 get_encode() {
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

// Self-test of the bounded-wait mechanism: one CTA waits on an mbarrier that nothing ever arrives at,
// with the same polling helper as the attention kernel but a caller-chosen limit, then reports the
// expiry through the status word and returns normally.
__global__ void wait_expiry_selftest_kernel(uint32_t max_polls, int32_t* status) {
  __shared__ uint64_t never;
  const uint32_t bar = smem_u32(&never);
  if (threadIdx.x == 0) {
    mbar_init(bar, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    bool done = false;
    for (uint32_t it = 0; it < max_polls && !done; ++it) done = mbar_try_wait(bar, 0);
    if (!done && status) atomicOr(status, WEDLM_STATUS_WAIT_EXPIRED);
  }
}

}  // namespace

int launch_wait_expiry_selftest(uint32_t max_polls, int32_t* status, cudaStream_t st) {
  wait_expiry_selftest_kernel<<<1, 32, 0, st>>>(max_polls, status);
  count_launch();
  return cuda_ok(cudaGetLastError());
}

bool attn_tensor_supported(const wedlm_config_t* c) {
  if (c->dtype != WEDLM_DTYPE_BF16 || c->head_dim != kD || c->page_size != kPage) return false;
  const int G = c->n_q_heads / c->n_kv_heads;
  if (G < 1 || G > 128 || (128 % G) != 0) return false;
  if ((long long)c->num_pages * c->n_kv_heads * kPage >= (1ll << 31)) return false;
  return true;
}

int launch_attn_tensor(const Shape& s, const AttnPlan& plan, const void* q_rot, const void* k_cache,
                       const void* v_cache, const int32_t* block_table, const int32_t* prefix_len,
                       const int32_t* order, void* out, float* part_o, float* part_ml, int32_t* status,
                       cudaStream_t st) {
  auto encode = get_encode();
  if (!encode) return WEDLM_ERR_CUDA;
  const int W_t = 128 / s.G;
  const int n_mtiles = (s.W + W_t - 1) / W_t;

  CUtensorMap tm_q, tm_k, tm_v;
  {
    // q_rot [B][W][Hq][D] as a 4-D tensor (D, Hq, W, B); box = (64, G, min(W_t, W), 1)
    cuuint64_t dims[4] = {(cuuint64_t)kD, (cuuint64_t)s.Hq, (cuuint64_t)s.W, (cuuint64_t)s.B};
    cuuint64_t strides[3] = {(cuuint64_t)kD * 2, (cuuint64_t)s.Hq * kD * 2, (cuuint64_t)s.W * s.Hq * kD * 2};
    cuuint32_t box[4] = {64, (cuuint32_t)s.G, (cuuint32_t)(W_t < s.W ? W_t : s.W), 1};
    cuuint32_t estr[4] = {1, 1, 1, 1};
    if (encode(&tm_q, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(q_rot), dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
      return WEDLM_ERR_CUDA;
  }
  for (int which = 0; which < 2; ++which) {
    // cache [num_pages][Hkv][16][D] as a 2-D tensor (D, rows); box = one page of one head, 64 elements wide
    cuuint64_t dims[2] = {(cuuint64_t)kD, (cuuint64_t)s.num_pages * s.Hkv * kPage};
    cuuint64_t strides[1] = {(cuuint64_t)kD * 2};
    cuuint32_t box[2] = {64, (cuuint32_t)kPage};
    cuuint32_t estr[2] = {1, 1};
    if (encode(which ? &tm_v : &tm_k, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(which ? v_cache : k_cache),
               dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
               CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
      return WEDLM_ERR_CUDA;
  }
  TensorAttnParams p;
  p.B = s.B; p.W = s.W; p.Hq = s.Hq; p.Hkv = s.Hkv; p.G = s.G; p.W_t = W_t; p.n_mtiles = n_mtiles;
  p.n_splits = plan.n_splits; p.chunk = plan.chunk; p.max_pages = s.max_pages; p.num_pages = s.num_pages;
  p.max_prefix = s.max_prefix;
  p.scale_log2 = s.scale * 1.4426950408889634f;
  p.block_table = block_table; p.prefix_len = prefix_len; p.order = order;
  p.out = (__nv_bfloat16*)out; p.part_o = part_o; p.part_ml = part_ml; p.status = status;

  // the opt-in to large dynamic shared memory is per device: done once for each device ordinal
  {
    static bool attr_done[64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return WEDLM_ERR_CUDA;
    if (dev < 0 || dev >= 64 || !attr_done[dev]) {
      if (cudaFuncSetAttribute(attn_tensor_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBytes) != cudaSuccess)
        return WEDLM_ERR_CUDA;
      if (dev >= 0 && dev < 64) attr_done[dev] = true;
    }
  }
  const long long blocks = (long long)plan.n_splits * n_mtiles * s.Hkv * s.B;
  if (blocks > 0x7fffffffLL) return WEDLM_ERR_UNSUPPORTED;
  attn_tensor_kernel<<<(unsigned)blocks, kThreadsT, kSmemBytes, st>>>(tm_q, tm_k, tm_v, p);
  count_launch();
  return cuda_ok(cudaGetLastError());
}

}  // namespace wedlm
