// Per-mask-row confidence over the vocabulary (entropy of Section 5.2; max-prob), selection by the
// distance-adjusted entropy of Eq. 11, and the Commit / Predict / Refill lines of Algorithm 1.
//
// Pass 1 (conf_partial_kernel) streams the logits of the mask rows once with 16-byte loads and
// reduces each chunk of a row to (m, s, t, a):  m = max x, a = lowest index attaining it,
// s = sum e^(x-m), t = sum (x-m) e^(x-m).  Pass 2 (conf_commit_kernel, one warp per sequence)
// merges the chunks of every row in double precision, lse = m + ln s, p_max = 1/s,
// H = ln s - t/s, then runs the window update.
//
// Sample() at a temperature T > 0 (Algorithm 1, "W[i] <- Sample(l_i)") is a third pass over the rows that
// pass 2 selected, and only those: sample_fill_kernel draws token = arg-max_v (l_v - m) / T + g_v with
// Gumbel noise from a stateless hash of (seed, sequence, position, token) and overwrites the greedy token.
#include <math_constants.h>

#include "common.cuh"

namespace wedlm {

constexpr int kConfThreads = 256;
constexpr int kConfVecs = 4;    // 16-byte loads in flight per thread

template <typename T> struct VecTraits;
template <> struct VecTraits<__nv_bfloat16> { static constexpr int VL = 8; };
template <> struct VecTraits<float> { static constexpr int VL = 4; };

template <typename T>
__host__ __device__ constexpr int conf_chunk_elems() { return kConfThreads * kConfVecs * VecTraits<T>::VL; }

__device__ __forceinline__ void unpack16(const uint4& u, float (&x)[8]) {
  const uint32_t w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
  for (int e = 0; e < 4; ++e) {
    x[2 * e] = __uint_as_float(w[e] << 16);
    x[2 * e + 1] = __uint_as_float(w[e] & 0xffff0000u);
  }
}
__device__ __forceinline__ void unpack16(const uint4& u, float (&x)[4]) {
  x[0] = __uint_as_float(u.x); x[1] = __uint_as_float(u.y); x[2] = __uint_as_float(u.z); x[3] = __uint_as_float(u.w);
}

// Packed fp32x2 arithmetic of sm_100 (two lanes per instruction).
__device__ __forceinline__ unsigned long long pack2(float lo, float hi) {     // a register pair, no instruction
  return ((unsigned long long)__float_as_uint(hi) << 32) | (unsigned long long)__float_as_uint(lo);
}
__device__ __forceinline__ void unpack2(unsigned long long v, float& lo, float& hi) {
  lo = __uint_as_float((unsigned)(v & 0xffffffffull));
  hi = __uint_as_float((unsigned)(v >> 32));
}
__device__ __forceinline__ unsigned long long fma2(unsigned long long a, unsigned long long b, unsigned long long c) {
  unsigned long long d;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
  return d;
}
__device__ __forceinline__ unsigned long long add2(unsigned long long a, unsigned long long b) {
  unsigned long long d;
  asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}
__device__ __forceinline__ float ex2_ftz(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ uint32_t bf162_max(uint32_t a, uint32_t b) {
  __nv_bfloat162 r = __hmax2(*reinterpret_cast<__nv_bfloat162*>(&a), *reinterpret_cast<__nv_bfloat162*>(&b));
  return *reinterpret_cast<uint32_t*>(&r);
}

// (value, index) arg-max combine: larger value wins, equal values keep the lower index.
__device__ __forceinline__ void argmax_combine(float& v, int& i, float ov, int oi) {
  if (ov > v || (ov == v && oi < i)) { v = ov; i = oi; }
}

// 1-D grid over (row, chunk) with the chunk index fastest; rows that are not active masks exit.
template <typename T, bool VEC>
__global__ void __launch_bounds__(kConfThreads)
conf_partial_kernel(int W, int V, int n_chunks, const T* __restrict__ logits, const int32_t* __restrict__ n_filled,
                    const int32_t* __restrict__ window_len, float4* __restrict__ part) {
  constexpr int VL = VecTraits<T>::VL;
  constexpr int EPT = kConfVecs * VL;
  constexpr int CHUNK = conf_chunk_elems<T>();
  const int row = blockIdx.x / n_chunks, chunk = blockIdx.x - row * n_chunks;
  const int b = row / W, i = row - b * W;
  const int L = window_len ? min(max(window_len[b], 0), W) : W;
  if (i < n_filled[b] || i >= L) return;
  const int tid = threadIdx.x;
  const int base = chunk * CHUNK;
  const T* src = logits + (size_t)row * V;

  float x[EPT];
  if (VEC) {
    uint4 raw[kConfVecs];
#pragma unroll
    for (int k = 0; k < kConfVecs; ++k) {
      int e0 = base + (k * kConfThreads + tid) * VL;
      if (e0 < V) raw[k] = __ldcs(reinterpret_cast<const uint4*>(src + e0));   // V % VL == 0 on this path
    }
#pragma unroll
    for (int k = 0; k < kConfVecs; ++k) {
      int e0 = base + (k * kConfThreads + tid) * VL;
      float xv[VL];
      if (e0 < V) unpack16(raw[k], xv);
#pragma unroll
      for (int e = 0; e < VL; ++e) x[k * VL + e] = (e0 < V) ? xv[e] : -CUDART_INF_F;
    }
  } else {
#pragma unroll
    for (int k = 0; k < kConfVecs; ++k)
#pragma unroll
      for (int e = 0; e < VL; ++e) {
        int idx = base + (k * kConfThreads + tid) * VL + e;
        x[k * VL + e] = idx < V ? ld_as_float(src, idx) : -CUDART_INF_F;
      }
  }
  // chunk maximum: values only (tree for ILP), then one shuffle reduction and one shared-memory hop
  float mt[4] = {-CUDART_INF_F, -CUDART_INF_F, -CUDART_INF_F, -CUDART_INF_F};
#pragma unroll
  for (int k = 0; k < EPT; k += 4) {
    mt[0] = fmaxf(mt[0], x[k]);
    mt[1] = fmaxf(mt[1], x[k + 1]);
    mt[2] = fmaxf(mt[2], x[k + 2]);
    mt[3] = fmaxf(mt[3], x[k + 3]);
  }
  const float m_thread = fmaxf(fmaxf(mt[0], mt[1]), fmaxf(mt[2], mt[3]));
  float m = m_thread;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
  __shared__ float sm_m[kConfThreads / 32];
  __shared__ float sm_s[kConfThreads / 32];
  __shared__ float sm_t[kConfThreads / 32];
  __shared__ int sm_a;
  const int warp = tid >> 5, lane = tid & 31;
  if (lane == 0) sm_m[warp] = m;
  if (tid == 0) sm_a = 0x7fffffff;
  __syncthreads();
  m = sm_m[0];
#pragma unroll
  for (int w = 1; w < kConfThreads / 32; ++w) m = fmaxf(m, sm_m[w]);
  // lowest index attaining the maximum: only the few threads that hold it look for it
  if (m_thread == m) {
    int a = 0x7fffffff;
#pragma unroll
    for (int k = kConfVecs - 1; k >= 0; --k)
#pragma unroll
      for (int e = VL - 1; e >= 0; --e)
        if (x[k * VL + e] == m) a = base + (k * kConfThreads + tid) * VL + e;     // descending scan keeps the lowest
    atomicMin(&sm_a, a);
  }

  // sums relative to the chunk maximum in the log2 domain: d = (x - m) log2(e), e = 2^d,
  // s = sum e, t = ln2 * sum d e.  d is clamped at -127, where e has already flushed to zero, so that
  // -inf logits (and the padding) add exactly 0 instead of inf * 0.
  float s0 = 0.f, s1 = 0.f, t0 = 0.f, t1 = 0.f;
  if (m > -CUDART_INF_F) {
    const float kLog2e = 1.4426950408889634f;
    const float nm = -m * kLog2e;
#pragma unroll
    for (int k = 0; k < EPT; k += 2) {
      const float d0 = fmaxf(fmaf(x[k], kLog2e, nm), -127.f);
      const float d1 = fmaxf(fmaf(x[k + 1], kLog2e, nm), -127.f);
      float e0, e1;
      asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(e0) : "f"(d0));
      asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(e1) : "f"(d1));
      s0 += e0;
      s1 += e1;
      t0 = fmaf(d0, e0, t0);
      t1 = fmaf(d1, e1, t1);
    }
  }
  float s = s0 + s1, t = (t0 + t1) * 0.6931471805599453f;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    s += __shfl_xor_sync(0xffffffffu, s, o);
    t += __shfl_xor_sync(0xffffffffu, t, o);
  }
  if (lane == 0) { sm_s[warp] = s; sm_t[warp] = t; }
  __syncthreads();
  if (tid == 0) {
    float ss = 0.f, tt = 0.f;
#pragma unroll
    for (int w = 0; w < kConfThreads / 32; ++w) { ss += sm_s[w]; tt += sm_t[w]; }
    part[(size_t)row * n_chunks + chunk] = make_float4(m, ss, tt, __int_as_float(sm_a));
  }
}

// ------------------------------------------------------------------------------------------------
// Streaming variant of pass 1 for bf16 logits with 16-byte aligned rows: persistent blocks pull
// (row, chunk) items of active mask rows through a shared-memory slot filled by bulk asynchronous
// copies (one 16 KB copy per item, completion on an mbarrier).  The consumers move an item into
// registers at once and hand the slot back, so one slot per block is enough to keep a copy in
// flight while they compute, and eight blocks fit on an SM (48 registers, 16 KB).  Same chunking and
// partial layout as conf_partial_kernel.
// ------------------------------------------------------------------------------------------------
constexpr int kStreamStages = 1;                                    // slots per block; power of two (slot = n & (stages - 1))
constexpr int kStreamBlocksPerSM = 8;                               // two 16 KB slots and 6 blocks measured 2 % slower
constexpr int kStreamThreads = 128;                                 // consumer threads per block
constexpr int kStreamVecs = 8;                                      // 16-byte vectors per thread and item
constexpr int kStreamChunk = kStreamThreads * kStreamVecs * 8;      // 8192 bf16 = 16 KB, same chunking as pass 1 above
static_assert((kStreamStages & (kStreamStages - 1)) == 0, "stage index uses a mask");
static_assert(kStreamChunk == kConfThreads * kConfVecs * 8, "both pass-1 kernels must cut rows the same way");
constexpr uint32_t kStreamSpin = 1u << 22;

__device__ __forceinline__ uint32_t cs_smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ bool cs_mbar_wait(uint32_t bar, uint32_t parity) {
  for (uint32_t it = 0; it < kStreamSpin; ++it) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    if (ok) return true;
  }
  return false;
}

__device__ __forceinline__ void cs_consumer_sync() {     // the consumer threads only
  asm volatile("bar.sync 1, %0;" ::"n"(kStreamThreads) : "memory");
}

// block = 4 consumer warps + 1 producer warp (its lane 0 issues the copies)
__global__ void __launch_bounds__(kStreamThreads + 32, kStreamBlocksPerSM)
conf_stream_kernel(int W, int V, int n_chunks, long long total_items, const __nv_bfloat16* __restrict__ logits,
                   const int32_t* __restrict__ n_filled, const int32_t* __restrict__ window_len,
                   float4* __restrict__ part, int32_t* status) {
  extern __shared__ __align__(128) unsigned char cs_smem[];
  unsigned char* stage_mem = cs_smem;                                       // kStreamStages x 16 KB
  uint64_t* full = reinterpret_cast<uint64_t*>(cs_smem + kStreamStages * kStreamChunk * 2);
  uint64_t* empty = full + kStreamStages;
  volatile int2* item_of = reinterpret_cast<volatile int2*>(empty + kStreamStages);   // (row, chunk) or (-1, -1)
  __shared__ float fm[kStreamThreads / 32];
  __shared__ float fs[kStreamThreads / 32];
  __shared__ float ft[kStreamThreads / 32];
  __shared__ int fa;
  __shared__ volatile int gave_up;                   // a bounded wait expired: every consumer leaves at the next barrier
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  if (tid == 0) gave_up = 0;
  long long cursor = blockIdx.x;                     // next candidate item of this block (producer only)

  // producer: put the next active item of this block into stage st, or -1 when the block is done;
  // returns false after the end marker
  auto produce = [&](int st) -> bool {
    const uint32_t bar = cs_smem_u32(full + st);
    for (;;) {
      const long long it = cursor;
      cursor += gridDim.x;
      if (it >= total_items) {
        item_of[st].x = -1;
        asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
        return false;
      }
      const int row = (int)(it / n_chunks), chunk = (int)(it - (long long)row * n_chunks);
      const int b = row / W, i = row - b * W;
      const int L = window_len ? min(max(window_len[b], 0), W) : W;
      if (i < n_filled[b] || i >= L) continue;       // not an active mask row
      const int base = chunk * kStreamChunk;
      const uint32_t bytes = (uint32_t)min(kStreamChunk, V - base) * 2u;
      item_of[st].x = row;
      item_of[st].y = chunk;
      asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
      asm volatile(
          "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
          ::"r"(cs_smem_u32(stage_mem + (size_t)st * kStreamChunk * 2)), "l"(logits + (size_t)row * V + base), "r"(bytes), "r"(bar)
          : "memory");
      return true;
    }
  };

  if (tid == 0) {
    for (int st = 0; st < kStreamStages; ++st) {
      asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(cs_smem_u32(full + st)));
      asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(cs_smem_u32(empty + st)));
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();

  if (warp == kStreamThreads / 32) {
    // ---- producer warp: fill the ring, then refill each stage as soon as the consumers release it
    if (lane == 0) {
      bool more = true;
      for (uint32_t n = 0; more; ++n) {
        const int st = n & (kStreamStages - 1);
        if (n >= kStreamStages && !cs_mbar_wait(cs_smem_u32(empty + st), ((n / kStreamStages) - 1) & 1u)) {
          if (status) atomicOr(status, WEDLM_STATUS_WAIT_EXPIRED);
          break;
        }
        more = produce(st);
      }
    }
    return;
  }

  for (uint32_t n = 0;; ++n) {
    const int st = n & (kStreamStages - 1);
    // Bounded, never expected to expire.  A thread whose wait does expire must not leave by itself (the others
    // would wait for it at the block barrier below for ever): it raises a flag and carries on to that barrier,
    // behind which all consumers leave together.
    if (!cs_mbar_wait(cs_smem_u32(full + st), (n / kStreamStages) & 1u)) gave_up = 1;
    const int row = gave_up ? 0 : item_of[st].x, chunk = gave_up ? 0 : item_of[st].y;
    if (row < 0) break;                              // end marker: seen by all consumers alike (set before the barrier's arrival)
    const int base = chunk * kStreamChunk;
    const uint4* src = reinterpret_cast<const uint4*>(stage_mem + (size_t)st * kStreamChunk * 2);
    uint32_t w[kStreamVecs * 4];
#pragma unroll
    for (int k = 0; k < kStreamVecs; ++k) {
      const uint4 v = src[k * kStreamThreads + tid];
      w[4 * k] = v.x; w[4 * k + 1] = v.y; w[4 * k + 2] = v.z; w[4 * k + 3] = v.w;
    }
    if (base + kStreamChunk > V) {                   // last chunk of a row: words past the row end act as padding
#pragma unroll
      for (int i = 0; i < kStreamVecs * 4; ++i) {
        const int e0 = base + ((i >> 2) * kStreamThreads + tid) * 8 + (i & 3) * 2;
        if (e0 >= V) w[i] = 0xF149F149u;
      }
    }
    // -inf logits are pulled up to -1e30 (bf16 pair 0xF149F149) so that they add exactly 0 below
    uint32_t mx[4];
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      w[q] = bf162_max(w[q], 0xF149F149u);
      mx[q] = w[q];
    }
#pragma unroll
    for (int i = 4; i < kStreamVecs * 4; ++i) {
      w[i] = bf162_max(w[i], 0xF149F149u);
      mx[i & 3] = bf162_max(mx[i & 3], w[i]);
    }
    const uint32_t m2 = bf162_max(bf162_max(mx[0], mx[1]), bf162_max(mx[2], mx[3]));
    const float m_thread = fmaxf(__uint_as_float(m2 << 16), __uint_as_float(m2 & 0xffff0000u));
    float m = m_thread;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
    if (lane == 0) fm[warp] = m;
    if (tid == 0) fa = 0x7fffffff;
    cs_consumer_sync();                              // also: every consumer holds its part of stage st in registers
    if (gave_up) {
      if (tid == 0 && status) atomicOr(status, WEDLM_STATUS_WAIT_EXPIRED);
      return;
    }
    if (tid == 0) asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(cs_smem_u32(empty + st)) : "memory");
    m = fm[0];
#pragma unroll
    for (int q = 1; q < kStreamThreads / 32; ++q) m = fmaxf(m, fm[q]);
    if (m_thread == m) {                             // lowest index attaining the maximum
      // mx[q] is the maximum over the words i with (i & 3) == q: only those quarters that hold m are searched
      int a = 0x7fffffff;
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        if (__uint_as_float(mx[q] << 16) == m || __uint_as_float(mx[q] & 0xffff0000u) == m) {
#pragma unroll
          for (int k = kStreamVecs - 1; k >= 0; --k) {
            const int i = 4 * k + q;
            const int e0 = base + (k * kStreamThreads + tid) * 8 + q * 2;
            if (__uint_as_float(w[i] & 0xffff0000u) == m) a = min(a, e0 + 1);
            if (__uint_as_float(w[i] << 16) == m) a = min(a, e0);
          }
        }
      }
      atomicMin(&fa, a);
    }
    // d = (x - m) log2(e), e = 2^d, s = sum e, t = ln2 * sum d e, two logits per instruction
    const float kLog2e = 1.4426950408889634f;
    const unsigned long long L2 = pack2(kLog2e, kLog2e), NM = pack2(-m * kLog2e, -m * kLog2e);
    unsigned long long sA = pack2(0.f, 0.f), sB = sA, tA = sA, tB = sA;
#pragma unroll
    for (int i = 0; i < kStreamVecs * 4; i += 2) {
      const unsigned long long dA = fma2(pack2(__uint_as_float(w[i] << 16), __uint_as_float(w[i] & 0xffff0000u)), L2, NM);
      const unsigned long long dB = fma2(pack2(__uint_as_float(w[i + 1] << 16), __uint_as_float(w[i + 1] & 0xffff0000u)), L2, NM);
      float a0, a1, b0, b1;
      unpack2(dA, a0, a1);
      unpack2(dB, b0, b1);
      const unsigned long long eA = pack2(ex2_ftz(a0), ex2_ftz(a1));
      const unsigned long long eB = pack2(ex2_ftz(b0), ex2_ftz(b1));
      sA = add2(sA, eA);
      sB = add2(sB, eB);
      tA = fma2(dA, eA, tA);
      tB = fma2(dB, eB, tB);
    }
    float s0, s1, t0, t1;
    unpack2(add2(sA, sB), s0, s1);
    unpack2(add2(tA, tB), t0, t1);
    float ssum = s0 + s1, tsum = (t0 + t1) * 0.6931471805599453f;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      ssum += __shfl_xor_sync(0xffffffffu, ssum, o);
      tsum += __shfl_xor_sync(0xffffffffu, tsum, o);
    }
    if (lane == 0) { fs[warp] = ssum; ft[warp] = tsum; }
    cs_consumer_sync();
    if (tid == 0) {
      float ss = 0.f, tt = 0.f;
#pragma unroll
      for (int q = 0; q < kStreamThreads / 32; ++q) { ss += fs[q]; tt += ft[q]; }
      part[(size_t)row * n_chunks + chunk] = make_float4(m, ss, tt, __int_as_float(fa));
    }
  }
}

// Commit + shift + Refill of Algorithm 1 for one sequence, executed by one warp.  tok_s / fil_s hold
// the window in logical order with this step's fills already applied.
__device__ void commit_shift_refill(int b, int W, int L, int n, const int* tok_s, const uint8_t* fil_s,
                                    int mask_id, int32_t* window_tokens, uint8_t* filled, int32_t* prefix_len,
                                    int32_t* window_len, int32_t* remaining_budget, int32_t* committed_tokens,
                                    int32_t* committed_count) {
  const int lane = threadIdx.x & 31;
  const size_t o = (size_t)b * W;
  n = min(max(n, 0), L);
  int r = n;
  if (remaining_budget) r = min(n, max(remaining_budget[b], 0));
  const int new_len = L - n + r;
  for (int j = lane; j < W; j += 32) {
    if (committed_tokens) committed_tokens[o + j] = j < n ? tok_s[j] : -1;
    int src = j + n;
    bool keep = j < L - n;          // slot shifted down from position j + n
    window_tokens[o + j] = keep ? tok_s[src] : mask_id;
    filled[o + j] = keep ? fil_s[src] : (uint8_t)0;
  }
  if (lane == 0) {
    if (committed_count) committed_count[b] = n;
    prefix_len[b] += n;
    if (window_len) window_len[b] = new_len;
    if (remaining_budget) remaining_budget[b] = max(remaining_budget[b], 0) - r;
  }
}

struct ConfParams {
  int W, n_chunks, conf_mode, mask_id;
  float tau, lambda, thr;
  float temperature;            // 0: greedy
  uint32_t seed_lo, seed_hi;
};

// Scratch of the sampling pass, carved from the caller's workspace behind the chunk partials.
struct SampleWs {
  unsigned long long* best;     // [rows] packed (ordered score bits, ~token): merged with atomicMax
  float2* cm;                   // [rows] (cut-off logit below which a token cannot win, row maximum)
  int* sel_row;                 // [n_sel] rows selected in this step, any order
  uint32_t* key;                // [rows] hash key of the row
  int* dst;                     // [rows] index into window_tokens of the slot after the shift, or -1
  int* cnt;                     // [rows] chunks finished
  int* n_sel;                   // [1]
};
constexpr size_t kSampleWsPerRow = 8 + 8 + 4 + 4 + 4 + 4;
constexpr size_t kSampleWsFixed = 16;

__host__ inline SampleWs carve_sample_ws(void* base, size_t rows) {
  SampleWs w;
  unsigned char* p = reinterpret_cast<unsigned char*>(base);
  w.best = reinterpret_cast<unsigned long long*>(p); p += rows * 8;
  w.cm = reinterpret_cast<float2*>(p);               p += rows * 8;
  w.sel_row = reinterpret_cast<int*>(p);             p += rows * 4;
  w.key = reinterpret_cast<uint32_t*>(p);            p += rows * 4;
  w.dst = reinterpret_cast<int*>(p);                 p += rows * 4;
  w.cnt = reinterpret_cast<int*>(p);                 p += rows * 4;
  w.n_sel = reinterpret_cast<int*>(p);
  return w;
}

// Stateless uniforms of the sampler: a bijective 32-bit finaliser (xor-shift / odd multiply).
__device__ __forceinline__ uint32_t mix32(uint32_t x) {
  x ^= x >> 16; x *= 0x7FEB352Du;
  x ^= x >> 15; x *= 0x846CA68Bu;
  x ^= x >> 16;
  return x;
}
__device__ __forceinline__ uint32_t sample_row_key(uint32_t seed_lo, uint32_t seed_hi, uint32_t b, uint32_t pos) {
  return mix32(mix32(seed_lo + 0x9E3779B9u * b) ^ seed_hi ^ (0x85EBCA6Bu * pos));
}
// Range of the noise g = -ln(-ln u) for u = (k + 1/2) 2^-23, k < 2^23: [-2.812, 16.636].  A token can only win
// against the row's arg-max (score >= m/T - 2.812) if its logit is within (16.636 + 2.812) T of the maximum.
constexpr float kGumbelSpan = 19.6f;

// One block per sequence with up to one warp per window row.  Each warp merges the chunk partials of
// whole rows (lanes over chunks, double precision), then warp 0 runs the selection and the window update.
__global__ void __launch_bounds__(1024)
conf_commit_kernel(ConfParams p, const float4* __restrict__ part, const int32_t* __restrict__ perm,
                   const int32_t* __restrict__ n_filled, const int32_t* __restrict__ n_commit,
                   int32_t* window_tokens, uint8_t* filled, int32_t* prefix_len, int32_t* window_len,
                   int32_t* remaining_budget, int32_t* argmax, float* maxprob, float* entropy, float* lse,
                   int32_t* committed_tokens, int32_t* committed_count, int32_t* filled_count, SampleWs sw) {
  extern __shared__ unsigned char sm_raw[];
  const int W = p.W;
  double* score = reinterpret_cast<double*>(sm_raw);        // [W] per mask k
  int* am = reinterpret_cast<int*>(score + W);                // [W] arg-max per mask k
  int* tok_s = am + W;                                        // [W] logical
  float* mrow = reinterpret_cast<float*>(tok_s + W);          // [W] row maximum per mask k
  uint8_t* fil_s = reinterpret_cast<uint8_t*>(mrow + W);      // [W] logical
  uint8_t* pass = fil_s + W;                                  // [W] per mask k

  const int b = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const size_t o = (size_t)b * W;
  const int L = window_len ? min(max(window_len[b], 0), W) : W;
  const int nf = min(max(n_filled[b], 0), L);
  const int n_mask = L - nf;
  const float qnan = __int_as_float(0x7fc00000);

  for (int j = tid; j < W; j += blockDim.x) {
    tok_s[j] = window_tokens[o + j];
    fil_s[j] = (j < L && filled[o + j]) ? 1 : 0;
  }
  // rows that are not active masks carry no statistics
  for (int i = tid; i < W; i += blockDim.x) {
    if (i < nf || i >= L) {
      if (argmax) argmax[o + i] = -1;
      if (maxprob) maxprob[o + i] = qnan;
      if (entropy) entropy[o + i] = qnan;
      if (lse) lse[o + i] = qnan;
    }
  }
  const int j0 = n_mask > 0 ? perm[o + nf] : 0;
  for (int k = warp; k < n_mask; k += (int)(blockDim.x >> 5)) {
    const int i = nf + k;
    const float4* pr = part + (o + i) * p.n_chunks;
    // arg-max over the chunks: larger maximum wins, equal maxima keep the lower token index
    float m = -CUDART_INF_F;
    int a = 0x7fffffff;
    float4 v0 = make_float4(-CUDART_INF_F, 0.f, 0.f, __int_as_float(0x7fffffff));   // this lane's first chunk
    if (lane < p.n_chunks) v0 = pr[lane];
    argmax_combine(m, a, v0.x, __float_as_int(v0.w));
    for (int c = lane + 32; c < p.n_chunks; c += 32) {
      const float4 v = pr[c];
      argmax_combine(m, a, v.x, __float_as_int(v.w));
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
      const float om = __shfl_xor_sync(0xffffffffu, m, off);
      const int oa = __shfl_xor_sync(0xffffffffu, a, off);
      argmax_combine(m, a, om, oa);
    }
    double s = 0.0, t = 0.0;
    for (int c = lane; c < p.n_chunks; c += 32) {
      const float4 v = (c == lane) ? v0 : pr[c];
      if (v.x > -CUDART_INF_F) {
        const double dm = (double)v.x - (double)m;
        const double wgt = exp(dm);
        s += wgt * (double)v.y;
        t += wgt * ((double)v.z + dm * (double)v.y);
      }
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
      s += __shfl_xor_sync(0xffffffffu, s, off);
      t += __shfl_xor_sync(0xffffffffu, t, off);
    }
    if (lane == 0) {
      const double ln_s = log(s);
      const double H = ln_s - t / s;
      const double pmax = 1.0 / s;
      if (argmax) argmax[o + i] = a;
      if (maxprob) maxprob[o + i] = (float)pmax;
      if (entropy) entropy[o + i] = (float)H;
      if (lse) lse[o + i] = (float)((double)m + ln_s);
      const int j = perm[o + i];
      double sc;
      bool ok;
      if (p.conf_mode == WEDLM_CONF_ENTROPY) {
        sc = H + (double)p.lambda * (double)(j - j0);           // Eq. 11
        ok = sc <= (double)p.tau;
      } else {
        sc = -pmax;
        ok = pmax >= (double)p.thr;
      }
      score[k] = sc;
      am[k] = a;
      mrow[k] = m;
      pass[k] = ok ? 1 : 0;
    }
  }
  __syncthreads();
  if (warp != 0) return;

  int n_pass = 0;
  for (int k = lane; k < n_mask; k += 32) n_pass += pass[k];
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) n_pass += __shfl_xor_sync(0xffffffffu, n_pass, off);
  if (n_pass == 0 && n_mask > 0) {
    // nothing passed: fill the single best-scoring mask, leftmost on ties
    double best = CUDART_INF;
    int bk = 0x7fffffff;
    for (int k = lane; k < n_mask; k += 32)
      if (score[k] < best || (score[k] == best && k < bk)) { best = score[k]; bk = k; }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
      double ob = __shfl_xor_sync(0xffffffffu, best, off);
      int ok_ = __shfl_xor_sync(0xffffffffu, bk, off);
      if (ob < best || (ob == best && ok_ < bk)) { best = ob; bk = ok_; }
    }
    if (bk == 0x7fffffff) bk = 0;     // every score NaN: still make progress at the leftmost mask
    if (lane == 0) pass[bk] = 1;
    n_pass = 1;
  }
  __syncwarp();
  const int P0 = prefix_len[b];                               // before the commit below moves it
  const int n_drop = min(max(n_commit[b], 0), L);
  for (int k = lane; k < n_mask; k += 32) {
    if (pass[k]) {
      const int j = perm[o + nf + k];
      tok_s[j] = am[k];
      fil_s[j] = 1;
      if (p.temperature > 0.f) {                              // hand the row to the sampling pass
        const size_t row = o + nf + k;
        sw.sel_row[atomicAdd(sw.n_sel, 1)] = (int)row;
        sw.key[row] = sample_row_key(p.seed_lo, p.seed_hi, (uint32_t)b, (uint32_t)(P0 + j));
        sw.dst[row] = j >= n_drop ? (int)(o + j - n_drop) : -1;
        sw.cm[row] = make_float2(mrow[k] - p.temperature * kGumbelSpan, mrow[k]);
        sw.cnt[row] = 0;
        sw.best[row] = 0ull;
      }
    }
  }
  if (lane == 0 && filled_count) filled_count[b] = n_pass;
  __syncwarp();
  commit_shift_refill(b, W, L, n_commit[b], tok_s, fil_s, p.mask_id, window_tokens, filled, prefix_len, window_len,
                      remaining_budget, committed_tokens, committed_count);
}

// Sampling pass: persistent blocks over (selected row, chunk).  Every chunk offers its best perturbed score
// to the row's packed maximum; the block that finishes a row last writes the drawn token into the window.
__device__ __forceinline__ unsigned long long pack_score(float z, int idx) {
  uint32_t bits = __float_as_uint(z);
  bits = (bits & 0x80000000u) ? ~bits : (bits | 0x80000000u);          // order-preserving map to unsigned
  return ((unsigned long long)bits << 32) | (unsigned long long)(0xFFFFFFFFu - (uint32_t)idx);   // equal scores: lower token
}

template <typename T, bool VEC>
__global__ void __launch_bounds__(kConfThreads)
sample_fill_kernel(int V, int n_chunks, float inv_t, const T* __restrict__ logits, SampleWs sw,
                   int32_t* __restrict__ argmax, int32_t* __restrict__ window_tokens) {
  constexpr int VL = VecTraits<T>::VL;
  constexpr int CHUNK = conf_chunk_elems<T>();
  const int tid = threadIdx.x, lane = tid & 31;
  const long long n_items = (long long)(*sw.n_sel) * n_chunks;
  for (long long it = blockIdx.x; it < n_items; it += gridDim.x) {
    const int r = (int)(it / n_chunks), chunk = (int)(it - (long long)r * n_chunks);
    const int row = sw.sel_row[r];
    const uint32_t key = sw.key[row];
    const float2 cm = sw.cm[row];
    const T* src = logits + (size_t)row * V;
    const int base = chunk * CHUNK;
    float bz = -CUDART_INF_F;
    int bi = 0x7fffffff;
    auto consider = [&](float x, int idx) {
      if (x >= cm.x) {                                                   // few tokens get here unless T is large
        const uint32_t h = mix32(key ^ (0x9E3779B9u * (uint32_t)idx));
        const float u = ((float)(h >> 9) + 0.5f) * 1.1920928955078125e-07f;   // exact: 24 significant bits
        const float g = -logf(-logf(u));
        const float z = fmaf(x - cm.y, inv_t, g);
        if (z > bz || (z == bz && idx < bi)) { bz = z; bi = idx; }
      }
    };
#pragma unroll
    for (int k = 0; k < kConfVecs; ++k) {
      const int e0 = base + (k * kConfThreads + tid) * VL;
      if (VEC) {
        if (e0 < V) {                                                    // V % VL == 0 on this path
          const uint4 raw = __ldg(reinterpret_cast<const uint4*>(src + e0));
          float xv[VL];
          unpack16(raw, xv);
#pragma unroll
          for (int e = 0; e < VL; ++e) consider(xv[e], e0 + e);
        }
      } else {
#pragma unroll
        for (int e = 0; e < VL; ++e)
          if (e0 + e < V) consider(ld_as_float(src, e0 + e), e0 + e);
      }
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
      const float oz = __shfl_xor_sync(0xffffffffu, bz, off);
      const int oi = __shfl_xor_sync(0xffffffffu, bi, off);
      if (oz > bz || (oz == bz && oi < bi)) { bz = oz; bi = oi; }
    }
    if (lane == 0 && bi != 0x7fffffff) atomicMax(sw.best + row, pack_score(bz, bi));
    __syncthreads();                                                     // every warp has made its offer
    if (tid == 0) {
      __threadfence();
      if (atomicAdd(sw.cnt + row, 1) == n_chunks - 1) {                  // this block completes the row
        __threadfence();
        const unsigned long long bb = atomicMax(sw.best + row, 0ull);    // coherent read
        if (bb != 0ull) {
          const int tok = (int)(0xFFFFFFFFu - (uint32_t)(bb & 0xFFFFFFFFull));
          if (argmax) argmax[row] = tok;
          const int d = sw.dst[row];
          if (d >= 0) window_tokens[d] = tok;
        }
      }
    }
  }
}

__global__ void __launch_bounds__(32)
window_refill_kernel(int W, int mask_id, const int32_t* __restrict__ n_commit, int32_t* window_tokens,
                     uint8_t* filled, int32_t* prefix_len, int32_t* window_len, int32_t* remaining_budget,
                     int32_t* committed_tokens, int32_t* committed_count) {
  extern __shared__ unsigned char sm_raw[];
  int* tok_s = reinterpret_cast<int*>(sm_raw);
  uint8_t* fil_s = reinterpret_cast<uint8_t*>(tok_s + W);
  const int b = blockIdx.x, lane = threadIdx.x;
  const size_t o = (size_t)b * W;
  const int L = window_len ? min(max(window_len[b], 0), W) : W;
  for (int j = lane; j < W; j += 32) {
    tok_s[j] = window_tokens[o + j];
    fil_s[j] = (j < L && filled[o + j]) ? 1 : 0;
  }
  __syncwarp();
  commit_shift_refill(b, W, L, n_commit[b], tok_s, fil_s, mask_id, window_tokens, filled, prefix_len, window_len,
                      remaining_budget, committed_tokens, committed_count);
}

static int conf_chunks(const wedlm_config_t* cfg) {
  int ce = cfg->dtype == WEDLM_DTYPE_BF16 ? conf_chunk_elems<__nv_bfloat16>() : conf_chunk_elems<float>();
  return (cfg->vocab + ce - 1) / ce;
}

size_t confidence_workspace_bytes(const wedlm_config_t* cfg) {
  const size_t rows = (size_t)cfg->batch * cfg->window;
  size_t bytes = rows * conf_chunks(cfg) * sizeof(float4);
  if (cfg->sample_temperature > 0.f) bytes += rows * kSampleWsPerRow + kSampleWsFixed;
  return bytes;
}

int launch_confidence(const Shape& s, const wedlm_config_t* cfg, const void* logits, const int32_t* perm,
                      const int32_t* n_filled, const int32_t* n_commit, int32_t* window_tokens, uint8_t* filled,
                      int32_t* prefix_len, int32_t* window_len, int32_t* remaining_budget, int32_t* argmax,
                      float* maxprob, float* entropy, float* lse, int32_t* committed_tokens,
                      int32_t* committed_count, int32_t* filled_count, void* workspace, int32_t* status, cudaStream_t st) {
  const int n_chunks = conf_chunks(cfg);
  const long long blocks = (long long)s.B * s.W * n_chunks;
  if (blocks > 0x7fffffffLL) return WEDLM_ERR_UNSUPPORTED;
  float4* part = reinterpret_cast<float4*>(workspace);
  if (s.dtype == WEDLM_DTYPE_BF16) {
    using T = __nv_bfloat16;
    const bool vec = (s.V % VecTraits<T>::VL == 0) && ((uintptr_t)logits % 16 == 0);
    if (vec) {
      const size_t smem = (size_t)kStreamStages * kStreamChunk * 2 + kStreamStages * 24;
      static bool attr_done[64] = {};
      int dev = 0;
      if (cudaGetDevice(&dev) != cudaSuccess) return WEDLM_ERR_CUDA;
      if (dev < 0 || dev >= 64 || !attr_done[dev]) {
        if (cudaFuncSetAttribute(conf_stream_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
          return WEDLM_ERR_CUDA;
        if (dev >= 0 && dev < 64) attr_done[dev] = true;
      }
      long long grid = (long long)device_sm_count() * kStreamBlocksPerSM;
      if (grid > blocks) grid = blocks;
      conf_stream_kernel<<<(unsigned)grid, kStreamThreads + 32, smem, st>>>(s.W, s.V, n_chunks, blocks, (const T*)logits, n_filled,
                                                                      window_len, part, status);
    } else {
      conf_partial_kernel<T, false><<<(unsigned)blocks, kConfThreads, 0, st>>>(s.W, s.V, n_chunks, (const T*)logits, n_filled, window_len, part);
    }
  } else {
    using T = float;
    const bool vec = (s.V % VecTraits<T>::VL == 0) && ((uintptr_t)logits % 16 == 0);
    if (vec) conf_partial_kernel<T, true><<<(unsigned)blocks, kConfThreads, 0, st>>>(s.W, s.V, n_chunks, (const T*)logits, n_filled, window_len, part);
    else     conf_partial_kernel<T, false><<<(unsigned)blocks, kConfThreads, 0, st>>>(s.W, s.V, n_chunks, (const T*)logits, n_filled, window_len, part);
  }
  count_launch();
  if (cudaGetLastError() != cudaSuccess) return WEDLM_ERR_CUDA;
  const bool sampling = cfg->sample_temperature > 0.f;
  const size_t rows = (size_t)s.B * s.W;
  void* sample_ws = sampling ? reinterpret_cast<unsigned char*>(workspace) + rows * n_chunks * sizeof(float4) : nullptr;
  int rc = launch_conf_commit(s, cfg, n_chunks, part, perm, n_filled, n_commit, window_tokens, filled, prefix_len, window_len,
                              remaining_budget, argmax, maxprob, entropy, lse, committed_tokens, committed_count,
                              filled_count, st, sample_ws);
  if (rc != WEDLM_OK || !sampling) return rc;
  // third pass: draw the tokens of the rows selected above
  const SampleWs sw = carve_sample_ws(sample_ws, rows);
  long long grid = (long long)device_sm_count() * 8;
  if (grid > blocks) grid = blocks;
  const float inv_t = (float)(1.0 / (double)cfg->sample_temperature);
  if (s.dtype == WEDLM_DTYPE_BF16) {
    using T = __nv_bfloat16;
    const bool vec = (s.V % VecTraits<T>::VL == 0) && ((uintptr_t)logits % 16 == 0);
    if (vec) sample_fill_kernel<T, true><<<(unsigned)grid, kConfThreads, 0, st>>>(s.V, n_chunks, inv_t, (const T*)logits, sw, argmax, window_tokens);
    else     sample_fill_kernel<T, false><<<(unsigned)grid, kConfThreads, 0, st>>>(s.V, n_chunks, inv_t, (const T*)logits, sw, argmax, window_tokens);
  } else {
    using T = float;
    const bool vec = (s.V % VecTraits<T>::VL == 0) && ((uintptr_t)logits % 16 == 0);
    if (vec) sample_fill_kernel<T, true><<<(unsigned)grid, kConfThreads, 0, st>>>(s.V, n_chunks, inv_t, (const T*)logits, sw, argmax, window_tokens);
    else     sample_fill_kernel<T, false><<<(unsigned)grid, kConfThreads, 0, st>>>(s.V, n_chunks, inv_t, (const T*)logits, sw, argmax, window_tokens);
  }
  count_launch();
  return cuda_ok(cudaGetLastError());
}

// Pass 2 alone: merge `n_chunks` partials (m, s, t, argmax) per mask row, select, commit, refill.  With a
// sampling scratch it also lists the selected rows for sample_fill_kernel.
int launch_conf_commit(const Shape& s, const wedlm_config_t* cfg, int n_chunks, const void* partials, const int32_t* perm,
                       const int32_t* n_filled, const int32_t* n_commit, int32_t* window_tokens, uint8_t* filled,
                       int32_t* prefix_len, int32_t* window_len, int32_t* remaining_budget, int32_t* argmax,
                       float* maxprob, float* entropy, float* lse, int32_t* committed_tokens, int32_t* committed_count,
                       int32_t* filled_count, cudaStream_t st, void* sample_ws) {
  ConfParams p{s.W, n_chunks, cfg->conf_mode, cfg->mask_token_id, cfg->tau, cfg->lambda, cfg->maxprob_thr,
               sample_ws ? cfg->sample_temperature : 0.f, cfg->sample_seed_lo, cfg->sample_seed_hi};
  SampleWs sw{};
  if (sample_ws) {
    sw = carve_sample_ws(sample_ws, (size_t)s.B * s.W);
    if (cudaMemsetAsync(sw.n_sel, 0, sizeof(int), st) != cudaSuccess) return WEDLM_ERR_CUDA;
  }
  size_t smem = (size_t)s.W * (sizeof(double) + 2 * sizeof(int) + sizeof(float) + 2);
  int commit_threads = 32 * s.W;
  commit_threads = commit_threads < 128 ? 128 : (commit_threads > 1024 ? 1024 : commit_threads);
  conf_commit_kernel<<<s.B, commit_threads, smem, st>>>(p, reinterpret_cast<const float4*>(partials), perm, n_filled, n_commit,
                                                        window_tokens, filled, prefix_len, window_len, remaining_budget,
                                                        argmax, maxprob, entropy, lse, committed_tokens, committed_count,
                                                        filled_count, sw);
  count_launch();
  return cuda_ok(cudaGetLastError());
}

int launch_window_refill(const Shape& s, const wedlm_config_t* cfg, const int32_t* n_commit, int32_t* window_tokens,
                         uint8_t* filled, int32_t* prefix_len, int32_t* window_len, int32_t* remaining_budget,
                         int32_t* committed_tokens, int32_t* committed_count, cudaStream_t st) {
  size_t smem = (size_t)s.W * (sizeof(int) + 1);
  window_refill_kernel<<<s.B, 32, smem, st>>>(s.W, cfg->mask_token_id, n_commit, window_tokens, filled, prefix_len,
                                              window_len, remaining_budget, committed_tokens, committed_count);
  count_launch();
  return cuda_ok(cudaGetLastError());
}

}  // namespace wedlm

// ------------------------------------------------------------------------------------------------
// Allocation-free variant of wedlm_confidence_commit.
//
// Some hosts of this library may not allocate device memory once they are running: a serving
// engine that has handed practically all of HBM to its KV-cache pool at start-up (a later cudaMalloc
// can fail, and it synchronises the device), or a decode loop with a "no allocator calls after
// warm-up" rule.  For them the chunk partials live in a fixed array inside the library image.
// ------------------------------------------------------------------------------------------------
#include <mutex>

namespace {

// Lives in every GPU context that loads the library, from load until process exit.
static __device__ __align__(256) unsigned char g_conf_static_scratch[WEDLM_STATIC_SCRATCH_BYTES];

constexpr int kMaxDevices = 64;
std::mutex g_static_mu;
void* g_static_ptr[kMaxDevices] = {};   // device address of the array, per device ordinal

// In host code the array's name is only a handle; the address a kernel can use has to be asked for,
// once per device, with that device current.
int static_scratch_address(void** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return WEDLM_ERR_CUDA;
  std::lock_guard<std::mutex> lock(g_static_mu);
  if (g_static_ptr[dev] == nullptr) {
    void* p = nullptr;
    cudaError_t e = cudaGetSymbolAddress(&p, g_conf_static_scratch);
    if (e != cudaSuccess || p == nullptr) return WEDLM_ERR_CUDA;
    g_static_ptr[dev] = p;
  }
  *out = g_static_ptr[dev];
  return WEDLM_OK;
}

}  // namespace

extern "C" int wedlm_confidence_commit_static(const wedlm_config_t* cfg, const void* logits, const int32_t* perm,
                                              const int32_t* n_filled, const int32_t* n_commit,
                                              int32_t* window_tokens, uint8_t* filled, int32_t* prefix_len,
                                              int32_t* window_len, int32_t* remaining_budget, int32_t* argmax,
                                              float* maxprob, float* entropy, float* lse,
                                              int32_t* committed_tokens, int32_t* committed_count,
                                              int32_t* filled_count, int32_t* status, void* stream) {
  wedlm::ApiRange nvtx_range("wedlm_confidence_commit_static");
  const size_t need = wedlm_confidence_workspace_bytes(cfg);     // 0 for a NULL / invalid config
  if (need == 0) return WEDLM_ERR_INVALID_ARG;
  if (need > (size_t)WEDLM_STATIC_SCRATCH_BYTES) return WEDLM_ERR_STATIC_SCRATCH;
  void* scratch = nullptr;
  int rc = static_scratch_address(&scratch);
  if (rc != WEDLM_OK) return rc;
  // Every partial that pass 2 reads is written by pass 1 of the same call, so nothing in the array
  // has to start at zero and the previous call's contents are harmless.
  return wedlm_confidence_commit(cfg, logits, perm, n_filled, n_commit, window_tokens, filled, prefix_len, window_len,
                                 remaining_budget, argmax, maxprob, entropy, lse, committed_tokens, committed_count,
                                 filled_count, scratch, (size_t)WEDLM_STATIC_SCRATCH_BYTES, status, stream);
}
