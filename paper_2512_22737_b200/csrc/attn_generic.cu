// Generic (CUDA-core) window attention: fp32 arithmetic on bf16 or fp32 storage, any supported
// head size / page size.  It is the path for fp32 configurations and the on-device cross-check of
// the tensor-core kernel.  Causal attention of the reordered window over the committed prefix and
// the window itself (Section 5.2): physical row i sees cache positions 0..P-1 and the staged
// window rows P..P+i.  Online softmax per row, optional split over the keys with a merge pass.
#include <math_constants.h>

#include "common.cuh"

namespace wedlm {

constexpr int kRB = 16;         // query rows per block
constexpr int kThreads = 128;

// 1-D grid, block index = (b * Hq * n_rowblocks + h * n_rowblocks + rb) * n_splits + split
template <typename T, int D>
__global__ void __launch_bounds__(kThreads)
attn_generic_kernel(Shape s, int n_splits, int chunk, const T* __restrict__ q_rot, const T* __restrict__ k_cache,
                    const T* __restrict__ v_cache, const int32_t* __restrict__ block_table,
                    const int32_t* __restrict__ prefix_len, T* __restrict__ out, float* __restrict__ part_o,
                    float* __restrict__ part_ml, int32_t* status) {
  constexpr int CPT = (D >= kThreads) ? D / kThreads : 1;            // columns per thread
  constexpr int RSTRIDE = (D >= kThreads) ? 1 : kThreads / D;        // row interleave when D < 128
  constexpr int RPT = kRB / RSTRIDE;                                 // rows per thread
  extern __shared__ float smem[];
  const int page = s.page;
  float* Qs = smem;                       // [kRB][D]   pre-scaled by scale*log2(e)
  float* Ks = Qs + kRB * D;               // [page][D+1]
  float* Vs = Ks + page * (D + 1);        // [page][D]
  float* Ss = Vs + page * D;              // [kRB][page] scores, then probabilities
  float* al = Ss + kRB * page;            // [kRB] rescale factors
  float* ms = al + kRB;                   // [kRB] running max (log2 domain)
  float* ls = ms + kRB;                   // [kRB] running sum

  const int tid = threadIdx.x;
  const int n_rb = (s.W + kRB - 1) / kRB;
  const unsigned per_seq = (unsigned)(s.Hq * n_rb * n_splits);
  const int b = (int)(blockIdx.x / per_seq);
  const int in_seq = (int)(blockIdx.x - (unsigned)b * per_seq);
  const int split = in_seq % n_splits, hrb = in_seq / n_splits;
  const int h = hrb / n_rb, rb = hrb - h * n_rb;
  const int g = h / s.G;
  const int P = checked_prefix(prefix_len, b, s.max_prefix, status, tid == 0);
  const int total = P + s.W;
  const int n_valid = (total + chunk - 1) / chunk;
  if (split >= n_valid) return;
  const int row0 = rb * kRB;
  const int rows = min(kRB, s.W - row0);
  const int kv_begin = split * chunk;
  const int kv_end = min(min(kv_begin + chunk, total), P + row0 + rows);   // last row's horizon

  const float qscale = s.scale * 1.4426950408889634f;
  for (int idx = tid; idx < kRB * D; idx += kThreads) {
    int r = idx / D, d = idx - r * D;
    float x = 0.f;
    if (r < rows) x = ld_as_float(q_rot, (((size_t)b * s.W + row0 + r) * s.Hq + h) * D + d) * qscale;
    Qs[idx] = x;
  }
  if (tid < kRB) { ms[tid] = -CUDART_INF_F; ls[tid] = 0.f; }
  float acc[RPT][CPT];
#pragma unroll
  for (int r = 0; r < RPT; ++r)
#pragma unroll
    for (int c = 0; c < CPT; ++c) acc[r][c] = 0.f;
  const int col0 = (D >= kThreads) ? tid : tid % D;
  const int rofs = (D >= kThreads) ? 0 : tid / D;
  __syncthreads();

  for (int t0 = kv_begin; t0 < kv_end; t0 += page) {
    // kv_begin is a multiple of the page size, so a tile is exactly one page
    long long slot = cache_slot(block_table, b, t0, page, s.max_pages, s.num_pages, status);
    const int nk = min(page, kv_end - t0);
    if (slot < 0) continue;   // page outside the pool: flagged in *status, its keys are skipped (block-uniform)
    {
      size_t base = cache_offset(slot, g, page, s.Hkv, D);
      for (int idx = tid; idx < nk * D; idx += kThreads) {
        int c = idx / D, d = idx - c * D;
        Ks[c * (D + 1) + d] = ld_as_float(k_cache, base + idx);
        Vs[idx] = ld_as_float(v_cache, base + idx);
      }
    }
    __syncthreads();
    for (int idx = tid; idx < kRB * page; idx += kThreads) {
      int r = idx / page, c = idx - r * page;
      float sc = -CUDART_INF_F;
      int t = t0 + c;
      if (r < rows && c < nk && t <= P + row0 + r) {
        float dot = 0.f;
        const float* qv = Qs + r * D;
        const float* kv = Ks + c * (D + 1);
#pragma unroll 8
        for (int d = 0; d < D; ++d) dot = fmaf(qv[d], kv[d], dot);
        sc = dot;
      }
      Ss[idx] = sc;
    }
    __syncthreads();
    if (tid < kRB) {
      float m_old = ms[tid], m_new = m_old;
      for (int c = 0; c < page; ++c) m_new = fmaxf(m_new, Ss[tid * page + c]);
      float a = 1.f, sum = 0.f;
      if (m_new == -CUDART_INF_F) {
        for (int c = 0; c < page; ++c) Ss[tid * page + c] = 0.f;
      } else {
        a = exp2f(m_old - m_new);            // m_old = -inf gives 0
        for (int c = 0; c < page; ++c) {
          float p = exp2f(Ss[tid * page + c] - m_new);
          Ss[tid * page + c] = p;
          sum += p;
        }
      }
      ls[tid] = ls[tid] * a + sum;
      ms[tid] = m_new;
      al[tid] = a;
    }
    __syncthreads();
#pragma unroll
    for (int r = 0; r < RPT; ++r) {
      const int rr = r * RSTRIDE + rofs;
      const float a = al[rr];
#pragma unroll
      for (int c = 0; c < CPT; ++c) acc[r][c] *= a;
      for (int kk = 0; kk < nk; ++kk) {
        const float p = Ss[rr * page + kk];
#pragma unroll
        for (int c = 0; c < CPT; ++c) acc[r][c] = fmaf(p, Vs[kk * D + col0 + c * kThreads], acc[r][c]);
      }
    }
    __syncthreads();
  }

#pragma unroll
  for (int r = 0; r < RPT; ++r) {
    const int rr = r * RSTRIDE + rofs;
    if (rr >= rows) continue;
    const size_t qrow = ((size_t)b * s.W + row0 + rr) * s.Hq + h;       // (b, i, h)
    if (n_valid == 1) {
      const float inv = ls[rr] > 0.f ? 1.f / ls[rr] : 0.f;
#pragma unroll
      for (int c = 0; c < CPT; ++c) st_from_float(out, qrow * D + col0 + c * kThreads, acc[r][c] * inv);
    } else {
      const size_t prow = (((size_t)b * s.Hq + h) * s.W + row0 + rr) * n_splits + split;
#pragma unroll
      for (int c = 0; c < CPT; ++c) part_o[prow * D + col0 + c * kThreads] = acc[r][c];
      if (col0 == 0) { part_ml[prow * 2] = ms[rr]; part_ml[prow * 2 + 1] = ls[rr]; }
    }
  }
}

// Merge of split partials (m, l, o): m = max m_s; w_s = 2^(m_s - m); out = sum w_s o_s / sum w_s l_s.
// One warp per (b, i, h) output row; lanes stride over D with 16-byte loads.  Sequences whose keys fit
// one chunk were written directly by the attention kernel and are skipped.  m is in the log2 domain.
template <typename T>
__global__ void __launch_bounds__(256)
attn_merge_kernel(Shape s, int n_splits, int chunk, const int32_t* __restrict__ prefix_len,
                  const float* __restrict__ part_o, const float* __restrict__ part_ml, T* __restrict__ out) {
  const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
  const int rows_per_seq = s.Hq * s.W;
  if (warp >= s.B * rows_per_seq) return;
  const int b = warp / rows_per_seq, rem = warp - b * rows_per_seq;
  const int h = rem / s.W, i = rem - h * s.W;                       // partial rows are ordered (b, h, i)
  const int P = checked_prefix(prefix_len, b, s.max_prefix, nullptr, false);      // same clamp as the attention kernels
  const int n_valid = min(n_splits, (P + s.W + chunk - 1) / chunk);
  if (n_valid <= 1) return;
  const size_t prow = (size_t)warp * n_splits;
  float m = -CUDART_INF_F;
  for (int sp = 0; sp < n_valid; ++sp) m = fmaxf(m, part_ml[(prow + sp) * 2]);
  float l = 0.f;
  for (int sp = 0; sp < n_valid; ++sp) {
    const float ms = part_ml[(prow + sp) * 2];
    if (ms != -CUDART_INF_F) l += exp2f(ms - m) * part_ml[(prow + sp) * 2 + 1];
  }
  const float inv = l > 0.f ? 1.f / l : 0.f;
  const size_t orow = (((size_t)b * s.W + i) * s.Hq + h) * s.D;
  for (int d = lane * 4; d < s.D; d += 128) {
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int sp = 0; sp < n_valid; ++sp) {
      const float ms = part_ml[(prow + sp) * 2];
      if (ms == -CUDART_INF_F) continue;
      const float w = exp2f(ms - m);
      const float4 o = *reinterpret_cast<const float4*>(part_o + (prow + sp) * s.D + d);
      acc.x += w * o.x; acc.y += w * o.y; acc.z += w * o.z; acc.w += w * o.w;
    }
    st_from_float(out, orow + d, acc.x * inv);
    st_from_float(out, orow + d + 1, acc.y * inv);
    st_from_float(out, orow + d + 2, acc.z * inv);
    st_from_float(out, orow + d + 3, acc.w * inv);
  }
}

template <typename T, int D>
static int launch_generic_t(const Shape& s, const AttnPlan& plan, const void* q_rot, const void* k_cache,
                            const void* v_cache, const int32_t* block_table, const int32_t* prefix_len, void* out,
                            float* part_o, float* part_ml, int32_t* status, cudaStream_t st) {
  const int n_rb = (s.W + kRB - 1) / kRB;
  const long long blocks = (long long)plan.n_splits * s.Hq * n_rb * s.B;
  if (blocks > 0x7fffffffLL) return WEDLM_ERR_UNSUPPORTED;
  size_t smem = sizeof(float) * ((size_t)kRB * D + (size_t)s.page * (D + 1) + (size_t)s.page * D +
                                 (size_t)kRB * s.page + 3 * kRB);
  auto kern = attn_generic_kernel<T, D>;
  if (smem > 48 * 1024) {
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return WEDLM_ERR_CUDA;
  }
  kern<<<(unsigned)blocks, kThreads, smem, st>>>(s, plan.n_splits, plan.chunk, (const T*)q_rot, (const T*)k_cache,
                                     (const T*)v_cache, block_table, prefix_len, (T*)out, part_o, part_ml, status);
  count_launch();
  return cuda_ok(cudaGetLastError());
}

template <typename T>
static int launch_generic_d(const Shape& s, const AttnPlan& plan, const void* q_rot, const void* k_cache,
                            const void* v_cache, const int32_t* block_table, const int32_t* prefix_len, void* out,
                            float* part_o, float* part_ml, int32_t* status, cudaStream_t st) {
  switch (s.D) {
    case 32:  return launch_generic_t<T, 32>(s, plan, q_rot, k_cache, v_cache, block_table, prefix_len, out, part_o, part_ml, status, st);
    case 64:  return launch_generic_t<T, 64>(s, plan, q_rot, k_cache, v_cache, block_table, prefix_len, out, part_o, part_ml, status, st);
    case 128: return launch_generic_t<T, 128>(s, plan, q_rot, k_cache, v_cache, block_table, prefix_len, out, part_o, part_ml, status, st);
    case 256: return launch_generic_t<T, 256>(s, plan, q_rot, k_cache, v_cache, block_table, prefix_len, out, part_o, part_ml, status, st);
    default:  return WEDLM_ERR_UNSUPPORTED;
  }
}

int launch_attn_generic(const Shape& s, const AttnPlan& plan, const void* q_rot, const void* k_cache,
                        const void* v_cache, const int32_t* block_table, const int32_t* prefix_len, void* out,
                        float* part_o, float* part_ml, int32_t* status, cudaStream_t st) {
  if (s.dtype == WEDLM_DTYPE_BF16)
    return launch_generic_d<__nv_bfloat16>(s, plan, q_rot, k_cache, v_cache, block_table, prefix_len, out, part_o, part_ml, status, st);
  return launch_generic_d<float>(s, plan, q_rot, k_cache, v_cache, block_table, prefix_len, out, part_o, part_ml, status, st);
}

int launch_attn_merge(const Shape& s, const AttnPlan& plan, const int32_t* prefix_len, const float* part_o,
                      const float* part_ml, void* out, cudaStream_t st) {
  const long long warps = (long long)s.B * s.Hq * s.W;
  const unsigned blocks = (unsigned)((warps * 32 + 255) / 256);
  if (s.dtype == WEDLM_DTYPE_BF16)
    attn_merge_kernel<__nv_bfloat16><<<blocks, 256, 0, st>>>(s, plan.n_splits, plan.chunk, prefix_len, part_o, part_ml, (__nv_bfloat16*)out);
  else
    attn_merge_kernel<float><<<blocks, 256, 0, st>>>(s, plan.n_splits, plan.chunk, prefix_len, part_o, part_ml, (float*)out);
  count_launch();
  return cuda_ok(cudaGetLastError());
}

}  // namespace wedlm
