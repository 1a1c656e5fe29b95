// RoPE at the supplied logical position ids (Section 2.2) for the window's q and k, and staging
// of the rotated k and of v into the paged cache at positions prefix_len + i ("Extend (K, V)" of
// Algorithm 1, done for every physical row so that a commit is just prefix_len += n).
#include <cmath>

#include "common.cuh"

namespace wedlm {

// theta^(-2d/D) for d < D/2, computed on the host in double and passed by value (D <= 256).
struct InvFreq { double v[128]; };

// grid (W, B); one block per (physical row i, sequence b).  Angles are formed in double so that
// positions of tens of thousands keep full fp32 accuracy after the range reduction.
template <typename T>
__global__ void __launch_bounds__(128)
rope_stage_kernel(Shape s, const InvFreq inv_freq, const T* __restrict__ q, const T* __restrict__ k, const T* __restrict__ v,
                  T* __restrict__ q_rot, T* __restrict__ k_cache, T* __restrict__ v_cache,
                  const int32_t* __restrict__ block_table, const int32_t* __restrict__ prefix_len,
                  const int32_t* __restrict__ pos_ids, const int32_t* __restrict__ count,
                  int32_t* __restrict__ kv_slot_idx, int32_t* __restrict__ order, int32_t* status) {
  extern __shared__ float cs_sn[];  // [D/2] cos, [D/2] sin
  const int i = blockIdx.x, b = blockIdx.y, tid = threadIdx.x;
  const int D = s.D, half = D / 2;
  float* cs = cs_sn;
  float* sn = cs_sn + half;
  const bool rotate = pos_ids != nullptr;
  if (rotate) {
    const double pos = (double)pos_ids[(size_t)b * s.W + i];
    for (int d = tid; d < half; d += blockDim.x) {
      // the angle is formed and reduced to [-pi, pi] in double (positions reach tens of thousands of
      // radians), the sine and cosine of the reduced angle are then accurate in fp32
      const double ang = pos * inv_freq.v[d];
      const double red = ang - 6.283185307179586476925 * rint(ang * 0.15915494309189533577);
      float sv, cv;
      sincosf((float)red, &sv, &cv);
      cs[d] = cv;
      sn[d] = sv;
    }
  } else {
    for (int d = tid; d < half; d += blockDim.x) { cs[d] = 1.f; sn[d] = 0.f; }
  }
  __syncthreads();

  // Side job of the blocks of row 0: rank the sequences by prefix length (longest first, ties by
  // index) so that the attention kernel can start the longest work first.  order[rank] = b.
  if (order != nullptr && i == 0) {
    __shared__ int rank_acc;
    if (tid == 0) rank_acc = 0;
    __syncthreads();
    const int mine = prefix_len[b];
    int cnt = 0;
    for (int o = tid; o < s.B; o += blockDim.x) {
      const int other = prefix_len[o];
      cnt += (other > mine || (other == mine && o < b)) ? 1 : 0;
    }
    if (cnt) atomicAdd(&rank_acc, cnt);
    __syncthreads();
    if (tid == 0) order[rank_acc] = b;
  }

  const size_t row = (size_t)b * s.W + i;
  if (q != nullptr) {
    const T* src = q + row * s.Hq * D;
    T* dst = q_rot + row * s.Hq * D;
    for (int idx = tid; idx < s.Hq * half; idx += blockDim.x) {
      int h = idx / half, d = idx - h * half;
      int i0 = s.rope_style == 0 ? d : 2 * d;
      int i1 = s.rope_style == 0 ? d + half : 2 * d + 1;
      float a = ld_as_float(src, (size_t)h * D + i0), c = ld_as_float(src, (size_t)h * D + i1);
      st_from_float(dst, (size_t)h * D + i0, a * cs[d] - c * sn[d]);
      st_from_float(dst, (size_t)h * D + i1, c * cs[d] + a * sn[d]);
    }
  }

  const int n_rows = count ? count[b] : s.W;
  long long slot = -1;
  if (i < n_rows) slot = cache_slot(block_table, b, prefix_len[b] + i, s.page, s.max_pages, s.num_pages, status);
  if (kv_slot_idx && tid == 0) kv_slot_idx[row] = (int32_t)slot;
  if (slot < 0) return;
  const T* ksrc = k + row * s.Hkv * D;
  const T* vsrc = v + row * s.Hkv * D;
  for (int idx = tid; idx < s.Hkv * half; idx += blockDim.x) {
    int g = idx / half, d = idx - g * half;
    int i0 = s.rope_style == 0 ? d : 2 * d;
    int i1 = s.rope_style == 0 ? d + half : 2 * d + 1;
    float a = ld_as_float(ksrc, (size_t)g * D + i0), c = ld_as_float(ksrc, (size_t)g * D + i1);
    size_t o = cache_offset(slot, g, s.page, s.Hkv, D);
    st_from_float(k_cache, o + i0, a * cs[d] - c * sn[d]);
    st_from_float(k_cache, o + i1, c * cs[d] + a * sn[d]);
  }
  for (int idx = tid; idx < s.Hkv * D; idx += blockDim.x) {
    int g = idx / D, d = idx - g * D;
    v_cache[cache_offset(slot, g, s.page, s.Hkv, D) + d] = vsrc[(size_t)g * D + d];
  }
}

int launch_rope_stage(const Shape& s, const void* q, const void* k, const void* v, void* q_rot, void* k_cache,
                      void* v_cache, const int32_t* block_table, const int32_t* prefix_len, const int32_t* pos_ids,
                      const int32_t* count, int32_t* kv_slot_idx, int32_t* order, int32_t* status, cudaStream_t st) {
  dim3 grid(s.W, s.B);
  size_t smem = (size_t)s.D * sizeof(float);
  InvFreq inv_freq;
  for (int d = 0; d < s.D / 2; ++d) inv_freq.v[d] = pow((double)s.theta, -2.0 * (double)d / (double)s.D);
  for (int d = s.D / 2; d < 128; ++d) inv_freq.v[d] = 0.0;
  if (s.dtype == WEDLM_DTYPE_BF16) {
    using T = __nv_bfloat16;
    rope_stage_kernel<T><<<grid, 128, smem, st>>>(s, inv_freq, (const T*)q, (const T*)k, (const T*)v, (T*)q_rot, (T*)k_cache,
                                                  (T*)v_cache, block_table, prefix_len, pos_ids, count, kv_slot_idx,
                                                  order, status);
  } else {
    using T = float;
    rope_stage_kernel<T><<<grid, 128, smem, st>>>(s, inv_freq, (const T*)q, (const T*)k, (const T*)v, (T*)q_rot, (T*)k_cache,
                                                  (T*)v_cache, block_table, prefix_len, pos_ids, count, kv_slot_idx,
                                                  order, status);
  }
  count_launch();
  return cuda_ok(cudaGetLastError());
}

}  // namespace wedlm
