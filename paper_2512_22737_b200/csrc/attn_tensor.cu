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
  int B, W, Hq, Hkv, G, W_t, n_mtiles, max_pages, num_pages, max_prefix;
  int balanced;              // 1: the tiles of all work units are cut into equal runs, one per CTA (see Walk)
  int n_ctas;                // CTAs that share the tiles (balanced mode)
  int n_slots;               // partial slots per query row (balanced mode): pieces a unit may be cut into
  float scale_log2;          // softmax scale * log2(e)
  const int32_t* block_table;
  const int32_t* prefix_len;
  const int32_t* order;      // sequences by decreasing prefix length, or NULL (unit-per-CTA mode)
  __nv_bfloat16* out;
  float* part_o;
  float* part_ml;
  long long* sched;          // balanced mode: [0] tiles per run, [1] padded flag, [2 + b] linear position of sequence b's
                             // first stream; written by CTA 0 for the merge kernel
  int32_t* status;
};

using namespace ptx;

// ---------------------------------------------------------------------------------------------- work assignment
// A work unit is one (sequence b, KV head g, 128-row tile mtile); its keys are the tiles 0..Tu-1 of 64 keys up to the
// horizon of the tile's last row.  Two ways of handing units to CTAs:
//   * unit per CTA: block index = (rank of b by decreasing prefix * Hkv + g) * n_mtiles + mtile, the whole unit.
//     Used when there are at least as many units as CTA slots: the longest start first and the slots stay full.
//   * balanced: with fewer units than slots the key tiles of all (b, g) streams, laid end to end, are cut into
//     n_ctas / n_mtiles runs of L tiles; run r is taken by the n_mtiles CTAs r * n_mtiles + mtile, one per row tile,
//     which therefore read the same K/V tiles at the same time (the second reader finds them in L2).  A run may end
//     one stream and begin the next.  Every slot then carries the same number of tiles.  A unit that is cut leaves
//     one partial (m, l, O) per piece, piece j of the unit in slot j of its rows, and the merge kernel recomputes
//     the same cut to find them.
// L is also kept large enough that no unit is cut into more than n_slots pieces.  Starting a second unit costs a CTA
// a Q load and a result write-out in series with its tiles; with short runs (L < kCrossMin) that is not worth the
// perfect balance, so there every stream is padded to a multiple of L in the linear order and no run crosses from
// one stream into the next (the grid has one spare run per stream for this).
constexpr int kMinTilesPerCta = 4;
constexpr int kCrossMin = 32;

__device__ __forceinline__ int unit_tiles(const TensorAttnParams& p, int P, int mtile) {
  return (P + min(p.W, (mtile + 1) * p.W_t) + kTileN - 1) / kTileN;
}
// tiles of a (b, g) stream: those of its last row tile, which sees the most keys
__device__ __forceinline__ int stream_tiles(const TensorAttnParams& p, int P) { return (P + p.W + kTileN - 1) / kTileN; }

struct Cut {
  long long total;     // length of the linear order (tiles of all streams, padded or not)
  int L;               // tiles per run
  bool pad;            // streams padded to multiples of L
};

// length of a stream in the linear order
__device__ __forceinline__ int stream_span(const Cut& c, int ts) { return c.pad ? (ts + c.L - 1) / c.L * c.L : ts; }

__device__ __forceinline__ Cut even_cut(const TensorAttnParams& p) {
  long long total = 0;
  int tmax = 1;
  for (int b = 0; b < p.B; ++b) {
    const int ts = stream_tiles(p, checked_prefix(p.prefix_len, b, p.max_prefix, nullptr, false));
    total += (long long)p.Hkv * ts;
    tmax = max(tmax, ts);
  }
  const int n_runs = p.n_ctas / p.n_mtiles;
  long long L = (total + n_runs - 1) / n_runs;
  L = max(L, (long long)kMinTilesPerCta);
  L = max(L, (long long)((tmax + p.n_slots - 2) / (p.n_slots - 1)));     // at most n_slots pieces per unit
  Cut c;
  c.total = total;
  c.L = (int)L;
  c.pad = L < kCrossMin;
  if (c.pad) {
    total = 0;
    for (int b = 0; b < p.B; ++b)
      total += (long long)p.Hkv * stream_span(c, stream_tiles(p, checked_prefix(p.prefix_len, b, p.max_prefix, nullptr, false)));
    c.total = total;
  }
  return c;
}

// one piece of work: tiles [t0, t1) of unit (b, g, mtile)
struct Seg {
  int b, g, mtile, P, t0, t1, piece;
  bool whole;          // the piece is the whole unit: its result is final
};

struct Walk {
  int b, g, mtile, P, t0;        // where the next piece starts (mtile is fixed for the CTA)
  long long pos, end, unit_off;  // linear tile positions: next tile, end of this CTA's run, first tile of the stream
  Cut cut;
  bool balanced;
};

__device__ __forceinline__ void walk_init(Walk& w, const TensorAttnParams& p, const Cut& cut, int cta) {
  w.balanced = p.balanced != 0;
  w.cut = cut;
  if (!w.balanced) {
    w.cut.pad = false;
    const int per_seq = p.Hkv * p.n_mtiles;
    const int rank = cta / per_seq, rem = cta - rank * per_seq;
    w.b = p.order ? p.order[rank] : rank;                    // longest sequences are dispatched first
    w.g = rem / p.n_mtiles;
    w.mtile = rem - w.g * p.n_mtiles;
    w.P = checked_prefix(p.prefix_len, w.b, p.max_prefix, nullptr, false);
    w.t0 = 0;
    w.pos = 0;
    w.unit_off = 0;
    w.end = stream_tiles(p, w.P);
    return;
  }
  const int run = cta / p.n_mtiles;
  w.mtile = cta - run * p.n_mtiles;
  w.pos = (long long)run * cut.L;
  w.end = min(w.pos + cut.L, cut.total);
  w.b = w.g = w.t0 = w.P = 0;
  w.unit_off = 0;
  if (w.pos >= w.end) return;
  long long cum = 0;
  for (int b = 0; b < p.B; ++b) {
    const int P = checked_prefix(p.prefix_len, b, p.max_prefix, nullptr, false);
    const int ts = stream_span(cut, stream_tiles(p, P));
    const long long seq = (long long)p.Hkv * ts;
    if (w.pos < cum + seq) {
      const int local = (int)(w.pos - cum);
      w.b = b;
      w.P = P;
      w.g = local / ts;
      w.t0 = local - w.g * ts;
      w.unit_off = w.pos - w.t0;
      return;
    }
    cum += seq;
  }
  w.end = w.pos;       // unreachable when cut.total is the sum above
}

__device__ __forceinline__ bool walk_next(Walk& w, const TensorAttnParams& p, Seg& sg) {
  while (w.pos < w.end) {
    const int ts = stream_span(w.cut, stream_tiles(p, w.P)), tu = unit_tiles(p, w.P, w.mtile);
    const int s1 = (int)min((long long)ts, (long long)w.t0 + (w.end - w.pos));      // end of the run inside this stream
    sg.b = w.b; sg.g = w.g; sg.mtile = w.mtile; sg.P = w.P;
    sg.t0 = w.t0;
    sg.t1 = min(s1, tu);                                     // this row tile's horizon may end before the stream's
    sg.whole = sg.t0 == 0 && sg.t1 == tu;
    sg.piece = w.balanced ? (int)(w.pos / w.cut.L) - (int)(w.unit_off / w.cut.L) : 0;
    w.pos += s1 - w.t0;
    if (s1 == ts) {                        // on to the next stream
      w.unit_off += ts;
      w.t0 = 0;
      if (++w.g == p.Hkv) {
        w.g = 0;
        ++w.b;
        if (w.b < p.B && w.pos < w.end) w.P = checked_prefix(p.prefix_len, w.b, p.max_prefix, nullptr, false);
      }
    } else {
      w.t0 = s1;
    }
    if (sg.t1 > sg.t0) return true;        // (else the run only touched tiles beyond this row tile's horizon)
  }
  return false;
}

__global__ void __launch_bounds__(kThreadsT, 2)
attn_tensor_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                   const __grid_constant__ CUtensorMap tm_v, const TensorAttnParams p) {
  extern __shared__ __align__(1024) uint8_t smem[];
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  Cut cut;
  cut.total = 0;
  cut.L = 0;
  cut.pad = false;
  if (p.balanced) {
    cut = even_cut(p);
    if (blockIdx.x == 0 && tid == 0) {
      // the cut, for the merge kernel
      p.sched[0] = cut.L;
      p.sched[1] = cut.pad ? 1 : 0;
      long long cum = 0;
      for (int b = 0; b < p.B; ++b) {
        p.sched[2 + b] = cum;
        cum += (long long)p.Hkv * stream_span(cut, stream_tiles(p, checked_prefix(p.prefix_len, b, p.max_prefix, nullptr, false)));
      }
    }
    if ((long long)(blockIdx.x / p.n_mtiles) * cut.L >= cut.total) return;          // more CTAs than runs
  }
  const float c = p.scale_log2;

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

  // Every role walks the same list of pieces.  Tiles are numbered through all pieces of the CTA (tt): the stage
  // rings and the barrier phases run on without a break from one piece to the next.
  Walk w;
  walk_init(w, p, cut, (int)blockIdx.x);
  Seg sg;

  if (warp == 4) {
    // ------------------------------------------------------------------ MMA issue warp
    // All lanes run the loop and wait on the barriers; one elected lane issues (see elect_one()).  The warp
    // never waits for an MMA to finish: completion is signalled to the consumers of the result (S_FULL,
    // O_DONE) and to the producer of the operands (K_FREE, V_FREE) through tcgen05.commit.
    const bool leader = elect_one();
    bool ok = true;
    const uint32_t idesc_qk = make_idesc(kTileN, false);
    const uint32_t idesc_pv = make_idesc(kD, true);
    auto issue_qk = [&](uint32_t tt) {
      const uint32_t st = tt & 1u;
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
    uint32_t gt = 0, n_seg = 0;
    while (ok && walk_next(w, p, sg)) {
      const int T = sg.t1 - sg.t0;
      ok = mbar_wait(bar(Q_FULL), n_seg & 1u);
      if (ok) ok = mbar_wait(bar(K_FULL0 + (gt & 1u)), (gt >> 1) & 1u);
      if (ok) issue_qk(gt);
      for (int t = 0; ok && t < T; ++t) {
        const uint32_t tt = gt + (uint32_t)t, st = tt & 1u, ph = (tt >> 1) & 1u;
        if (t + 1 < T) {
          // S[(tt+1)&1] was last read by the softmax of tile tt-1, whose P_READY we saw one iteration ago
          ok = mbar_wait(bar(K_FULL0 + (st ^ 1u)), ((tt + 1u) >> 1) & 1u);
          if (!ok) break;
          issue_qk(tt + 1u);
        }
        ok = mbar_wait(bar(P_READY), tt & 1u);
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
      gt += (uint32_t)T;
      ++n_seg;
    }
    if (!ok && lane == 0) {
      *abort_flag = 1;
      if (p.status) atomicOr(p.status, WEDLM_STATUS_WAIT_EXPIRED);
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
    auto wait_all = [&](uint32_t barrier, uint32_t parity) -> bool {      // lane 0 waits, the warp follows
      int good = 1;
      if (lane == 0) good = mbar_wait(barrier, parity) ? 1 : 0;
      return __shfl_sync(0xffffffffu, good, 0) != 0;
    };
    const CUtensorMap* map = is_k ? &tm_k : &tm_v;
    const uint32_t stage0 = sbase + (is_k ? kOffK : kOffV);
    const int full0 = is_k ? K_FULL0 : V_FULL0, free0 = is_k ? K_FREE0 : V_FREE0;
    uint32_t gt = 0, n_seg = 0;
    while (ok && walk_next(w, p, sg)) {
      const int T = sg.t1 - sg.t0;
      const int slot0 = sg.mtile * p.W_t;
      const int kv_end = sg.P + min(p.W, slot0 + p.W_t);                  // horizon of the tile's last row
      // TMA row coordinate of this lane's page of tile t of the unit (same for K and V)
      auto page_row = [&](int t) -> int {
        const int key0 = t * kTileN + pg * kPage;
        const int lp = key0 / kPage;
        int pp = -1;
        if (lp < p.max_pages) pp = p.block_table[(size_t)sg.b * p.max_pages + lp];
        if (pp < 0 || pp >= p.num_pages) {
          if (is_k && key0 < kv_end && p.status) atomicOr(p.status, lp < p.max_pages ? WEDLM_STATUS_BAD_PAGE : WEDLM_STATUS_BAD_LENGTH);
          return oob_row;
        }
        return (pp * p.Hkv + sg.g) * kPage;
      };
      if (is_k) {
        // the Q tile may only be replaced once every Q K^T of the previous piece has completed
        if (n_seg > 0) ok = wait_all(bar(K_FREE0 + ((gt - 1u) & 1u)), ((gt - 1u) >> 1) & 1u);
        if (!ok) break;
        if (lane == 0) {
          // Q tile: two 64-element halves of [W_t slots x G heads] rows
          const int q_slots = min(p.W_t, p.W);        // box height along the window dimension
          mbar_expect_tx(bar(Q_FULL), (uint32_t)(2 * 64 * p.G * q_slots * 2));
          tma_load_4d(sbase + kOffQ, &tm_q, 0, sg.g * p.G, slot0, sg.b, bar(Q_FULL));
          tma_load_4d(sbase + kOffQ + kHalfQ, &tm_q, 64, sg.g * p.G, slot0, sg.b, bar(Q_FULL));
        }
      }
      int y_next = page_row(sg.t0);
      for (int t = 0; ok && t < T; ++t) {
        const uint32_t tt = gt + (uint32_t)t, st = tt & 1u;
        const int y = y_next;
        if (t + 1 < T) y_next = page_row(sg.t0 + t + 1);      // table entry of the next tile, used one iteration later
        if (tt >= 2u) ok = wait_all(bar(free0 + st), ((tt - 2u) >> 1) & 1u);
        if (!ok) break;
        if (lane == 0) mbar_expect_tx(bar(full0 + st), kStageBytes);
        __syncwarp();
        if (lane < 8) tma_load_2d(stage0 + st * kStageBytes + lane_dst, map, half * 64, y, bar(full0 + st));
      }
      gt += (uint32_t)T;
      ++n_seg;
    }
    if (!ok && lane == 0) {
      *abort_flag = 1;
      if (p.status) atomicOr(p.status, WEDLM_STATUS_WAIT_EXPIRED);
    }
  } else {
    // ------------------------------------------------------------------ softmax warps: one row per thread
    const uint32_t lane_sel = (uint32_t)(warp * 32) << 16;
    const int r = tid;                                         // row of the 128-row tile
    bool ok = true;
    uint32_t gt = 0;
    while (ok && walk_next(w, p, sg)) {
      const int T = sg.t1 - sg.t0;
      const int b = sg.b, P = sg.P;
      if (tid == 0) (void)checked_prefix(p.prefix_len, b, p.max_prefix, p.status, true);    // report a bad length once
      const int slot0 = sg.mtile * p.W_t;                      // first window slot of this row tile
      const int kv_end = P + min(p.W, slot0 + p.W_t);          // horizon of the tile's last row
      const int i_row = slot0 + r / p.G;                       // physical window slot
      const int h = sg.g * p.G + r % p.G;                      // query head
      const bool row_valid = i_row < p.W;
      const int limit = row_valid ? P + i_row : -1;            // last visible key index (inclusive)
      float m_ref = -CUDART_INF_F;                             // reference maximum (raw score units)
      float l = 0.f;
      for (int t = 0; t < T; ++t) {
        const uint32_t tt = gt + (uint32_t)t, st = tt & 1u, ph = (tt >> 1) & 1u;
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
        const int tile0 = (sg.t0 + t) * kTileN;
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
        // P buffer and O are free / stable once P V of the previous tile has completed (at the first tile of a
        // later piece that was waited for when the previous piece's result was read)
        if (t > 0) {
          ok = mbar_wait(bar(O_DONE), (tt - 1u) & 1u);
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
        // last tile of the unit: V rows of keys beyond the horizon may hold anything (0 * NaN = NaN): zero them
        if (kv_end - tile0 < kTileN) {
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
      if (!ok) break;
      gt += (uint32_t)T;
      ok = mbar_wait(bar(O_DONE), (gt - 1u) & 1u);
      if (!ok) break;
      tc_fence_after();
      const float inv = l > 0.f ? 1.f / l : 0.f;
      const size_t orow = (((size_t)b * p.W + i_row) * p.Hq + h) * kD;
      const size_t prow = (((size_t)b * p.Hq + h) * p.W + i_row) * p.n_slots + sg.piece;
#pragma unroll 1
      for (int ch = 0; ch < 4; ++ch) {
        uint32_t o[32];
        tmem_ld32(tmem_O + lane_sel + ch * 32u, o);
        tmem_wait_ld();
        if (!row_valid) continue;
        if (sg.whole) {
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
      if (row_valid && !sg.whole) {
        p.part_ml[prow * 2] = (m_ref == -CUDART_INF_F) ? -CUDART_INF_F : m_ref * c;     // log2 domain
        p.part_ml[prow * 2 + 1] = l;
      }
      // the accumulator has been read: order those loads before the next piece's first P V overwrites it
      tc_fence_before();
    }
    if (!ok) {
      *abort_flag = 1;
      if (p.status) atomicOr(p.status, WEDLM_STATUS_WAIT_EXPIRED);
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

// Combines the pieces of every unit the balanced cut went through.  One warp per query row (b, h, i); from the cut
// the attention kernel left behind the warp finds how many runs shared its unit (piece j sits in slot j of the row)
// and writes the result.
// m is in the log2 domain.
__global__ void __launch_bounds__(256)
attn_merge_balanced_kernel(const TensorAttnParams p) {
  const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
  const int rows_per_seq = p.Hq * p.W;
  if (warp >= p.B * rows_per_seq) return;
  const int b = warp / rows_per_seq, rem = warp - b * rows_per_seq;
  const int h = rem / p.W, i = rem - h * p.W;                       // partial rows are ordered (b, h, i)
  Cut cut;
  cut.total = 0;
  cut.L = (int)p.sched[0];
  cut.pad = p.sched[1] != 0;
  const int P = checked_prefix(p.prefix_len, b, p.max_prefix, nullptr, false);
  const int g = h / p.G, mtile = i / p.W_t;
  const long long unit_off = p.sched[2 + b] + (long long)g * stream_span(cut, stream_tiles(p, P));
  const int tu = unit_tiles(p, P, mtile);
  const int n_pieces = (int)((unit_off + tu - 1) / cut.L) - (int)(unit_off / cut.L) + 1;
  if (n_pieces <= 1) return;                                         // written directly by the CTA that held the unit
  const size_t prow = (size_t)warp * p.n_slots;
  const size_t orow = (((size_t)b * p.W + i) * p.Hq + h) * kD;
  const int d = lane * 4;
  float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
  float l = 0.f;
  // pieces in groups of 32: lane sp holds (m, l) of piece sp, the weights travel by shuffle
  float m = -CUDART_INF_F;
  for (int sp = lane; sp < n_pieces; sp += 32) m = fmaxf(m, p.part_ml[(prow + sp) * 2]);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
  for (int base = 0; base < n_pieces; base += 32) {
    const int mine = base + lane;
    float wgt = 0.f, lw = 0.f;
    if (mine < n_pieces) {
      const float2 ml = *reinterpret_cast<const float2*>(p.part_ml + (prow + mine) * 2);
      if (ml.x != -CUDART_INF_F) {
        wgt = exp2f(ml.x - m);
        lw = wgt * ml.y;
      }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) lw += __shfl_xor_sync(0xffffffffu, lw, o);
    l += lw;
    const int n_here = min(32, n_pieces - base);
    for (int sp0 = 0; sp0 < n_here; sp0 += 4) {          // four pieces at a time, so that their loads overlap
      float ws[4];
      float4 o[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        ws[u] = __shfl_sync(0xffffffffu, wgt, (sp0 + u) & 31);
        if (sp0 + u >= n_here) ws[u] = 0.f;
        o[u] = make_float4(0.f, 0.f, 0.f, 0.f);
        if (ws[u] != 0.f) o[u] = *reinterpret_cast<const float4*>(p.part_o + (prow + base + sp0 + u) * kD + d);
      }
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        acc.x += ws[u] * o[u].x; acc.y += ws[u] * o[u].y; acc.z += ws[u] * o[u].z; acc.w += ws[u] * o[u].w;
      }
    }
  }
  const float inv = l > 0.f ? 1.f / l : 0.f;
  uint2 v;
  v.x = pack_bf16(acc.x * inv, acc.y * inv);
  v.y = pack_bf16(acc.z * inv, acc.w * inv);
  *reinterpret_cast<uint2*>(p.out + orow + d) = v;
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

namespace {

TensorAttnParams make_params(const Shape& s, const AttnPlan& plan, const int32_t* block_table, const int32_t* prefix_len,
                             const int32_t* order, void* out, float* part_o, float* part_ml, int32_t* status) {
  // the cut record shares the buffer of the dispatch order, which the balanced mode does not use
  TensorAttnParams p;
  p.B = s.B; p.W = s.W; p.Hq = s.Hq; p.Hkv = s.Hkv; p.G = s.G; p.W_t = 128 / s.G;
  p.n_mtiles = (s.W + p.W_t - 1) / p.W_t;
  p.max_pages = s.max_pages; p.num_pages = s.num_pages; p.max_prefix = s.max_prefix;
  p.balanced = plan.balanced; p.n_ctas = plan.n_ctas; p.n_slots = plan.n_splits;
  p.scale_log2 = s.scale * 1.4426950408889634f;
  p.block_table = block_table; p.prefix_len = prefix_len;
  p.order = plan.balanced ? nullptr : order;
  p.sched = plan.balanced ? reinterpret_cast<long long*>(const_cast<int32_t*>(order)) : nullptr;
  p.out = (__nv_bfloat16*)out; p.part_o = part_o; p.part_ml = part_ml; p.status = status;
  return p;
}

}  // namespace

int launch_attn_tensor(const Shape& s, const AttnPlan& plan, const void* q_rot, const void* k_cache,
                       const void* v_cache, const int32_t* block_table, const int32_t* prefix_len,
                       const int32_t* order, void* out, float* part_o, float* part_ml, int32_t* status,
                       cudaStream_t st) {
  auto encode = get_encode();
  if (!encode) return WEDLM_ERR_CUDA;
  const TensorAttnParams p = make_params(s, plan, block_table, prefix_len, order, out, part_o, part_ml, status);
  const int W_t = p.W_t, n_mtiles = p.n_mtiles;

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
  // balanced: one spare run per stream, for the case that the streams are padded
  const long long blocks = plan.balanced ? (long long)plan.n_ctas + (long long)n_mtiles * s.Hkv * s.B
                                         : (long long)n_mtiles * s.Hkv * s.B;
  if (blocks > 0x7fffffffLL) return WEDLM_ERR_UNSUPPORTED;
  attn_tensor_kernel<<<(unsigned)blocks, kThreadsT, kSmemBytes, st>>>(tm_q, tm_k, tm_v, p);
  count_launch();
  return cuda_ok(cudaGetLastError());
}

int launch_attn_tensor_merge(const Shape& s, const AttnPlan& plan, const int32_t* prefix_len, const int32_t* order,
                             const float* part_o, const float* part_ml, void* out, cudaStream_t st) {
  if (!plan.balanced) return WEDLM_OK;
  const TensorAttnParams p = make_params(s, plan, nullptr, prefix_len, order, out, const_cast<float*>(part_o),
                                         const_cast<float*>(part_ml), nullptr);
  const long long warps = (long long)s.B * s.Hq * s.W;
  attn_merge_balanced_kernel<<<(unsigned)((warps * 32 + 255) / 256), 256, 0, st>>>(p);
  count_launch();
  return cuda_ok(cudaGetLastError());
}

}  // namespace wedlm
