// RoPE at the supplied logical position ids (Section 2.2) for the window's q and k, and staging
// of the rotated k and of v into the paged cache at positions prefix_len + i ("Extend (K, V)" of
// Algorithm 1, done for every physical row so that a commit is just prefix_len += n).
#include <cmath>

#include "common.cuh"

namespace wedlm {

// theta^(-2d/D) for d < D/2, computed on the host in double and passed by value (D <= 256).
struct InvFreq { double v[128]; };

// Rotate eight bf16 pairs (a_e, c_e) held in two 16-byte vectors: a' = a cos - c sin, c' = c cos + a sin.
__device__ __forceinline__ void rotate8(const uint4& a, const uint4& c, const float* cs, const float* sn, uint4& oa,
                                        uint4& oc) {
  const uint32_t aw[4] = {a.x, a.y, a.z, a.w}, cw[4] = {c.x, c.y, c.z, c.w};
  uint32_t ra[4], rc[4];
#pragma unroll
  for (int e = 0; e < 4; ++e) {
    const float a0 = __uint_as_float(aw[e] << 16), a1 = __uint_as_float(aw[e] & 0xffff0000u);
    const float c0 = __uint_as_float(cw[e] << 16), c1 = __uint_as_float(cw[e] & 0xffff0000u);
    const float cs0 = cs[2 * e], cs1 = cs[2 * e + 1], sn0 = sn[2 * e], sn1 = sn[2 * e + 1];
    __nv_bfloat162 va = __floats2bfloat162_rn(a0 * cs0 - c0 * sn0, a1 * cs1 - c1 * sn1);
    __nv_bfloat162 vc = __floats2bfloat162_rn(c0 * cs0 + a0 * sn0, c1 * cs1 + a1 * sn1);
    ra[e] = *reinterpret_cast<uint32_t*>(&va);
    rc[e] = *reinterpret_cast<uint32_t*>(&vc);
  }
  oa = make_uint4(ra[0], ra[1], ra[2], ra[3]);
  oc = make_uint4(rc[0], rc[1], rc[2], rc[3]);
}

// grid (B, W); one block per (sequence b, physical row i).  Angles are formed in double so that
// positions of tens of thousands keep full fp32 accuracy after the range reduction.
template <typename T>
__global__ void __launch_bounds__(128)
rope_stage_kernel(Shape s, const InvFreq inv_freq, const T* __restrict__ q, const T* __restrict__ k, const T* __restrict__ v,
                  T* __restrict__ q_rot, T* __restrict__ k_cache, T* __restrict__ v_cache,
                  const int32_t* __restrict__ block_table, const int32_t* __restrict__ prefix_len,
                  const int32_t* __restrict__ pos_ids, const int32_t* __restrict__ count,
                  int32_t* __restrict__ kv_slot_idx, int32_t* __restrict__ order, int32_t* status) {
  extern __shared__ float cs_sn[];  // [D/2] cos, [D/2] sin
  const int b = blockIdx.x, i = blockIdx.y, tid = threadIdx.x;
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
  if (sizeof(T) == 2 && s.rope_style == 0 && (D % 16) == 0) {
    // bf16, rotate-half pairing: 16-byte loads of the two halves of each head, 16-byte stores
    const int vph = half / 8;                                   // vectors per half head
    if (q != nullptr) {
      const uint4* src = reinterpret_cast<const uint4*>(q + row * s.Hq * D);
      uint4* dst = reinterpret_cast<uint4*>(q_rot + row * s.Hq * D);
      for (int idx = tid; idx < s.Hq * vph; idx += blockDim.x) {
        const int h = idx / vph, j = idx - h * vph;
        uint4 oa, oc;
        rotate8(src[h * 2 * vph + j], src[h * 2 * vph + vph + j], cs + 8 * j, sn + 8 * j, oa, oc);
        dst[h * 2 * vph + j] = oa;
        dst[h * 2 * vph + vph + j] = oc;
      }
    }
    const int n_rows = count ? count[b] : s.W;
    long long slot = -1;
    if (i < n_rows) slot = cache_slot(block_table, b, prefix_len[b] + i, s.page, s.max_pages, s.num_pages, status);
    if (kv_slot_idx && tid == 0) kv_slot_idx[row] = (int32_t)slot;
    if (slot < 0) return;
    const uint4* ksrc = reinterpret_cast<const uint4*>(k + row * s.Hkv * D);
    const uint4* vsrc = reinterpret_cast<const uint4*>(v + row * s.Hkv * D);
    for (int idx = tid; idx < s.Hkv * vph; idx += blockDim.x) {
      const int g = idx / vph, j = idx - g * vph;
      uint4 oa, oc;
      rotate8(ksrc[g * 2 * vph + j], ksrc[g * 2 * vph + vph + j], cs + 8 * j, sn + 8 * j, oa, oc);
      uint4* kd = reinterpret_cast<uint4*>(k_cache + cache_offset(slot, g, s.page, s.Hkv, D));
      kd[j] = oa;
      kd[vph + j] = oc;
    }
    for (int idx = tid; idx < s.Hkv * 2 * vph; idx += blockDim.x) {
      const int g = idx / (2 * vph), j = idx - g * 2 * vph;
      reinterpret_cast<uint4*>(v_cache + cache_offset(slot, g, s.page, s.Hkv, D))[j] = vsrc[idx];
    }
    return;
  }
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
  dim3 grid(s.B, s.W);      // W <= 1024 fits gridDim.y; the batch may be large (dual-stream units)
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
