// Gate-weighted combine: out_t = sum over the kept slots of wgt[t, slot] * y[row(t, slot)]
// (outer sums of Eq. 2 / Eq. 7 / Eq. 8).  A token with no kept expert gets exact
// zeros (Section 3.3).  Slots are added in a fixed order, so the result is
// bitwise reproducible.  With the residual flag the layer input is added before
// the single rounding to the storage dtype.
#include "internal.h"

namespace moespec {

__device__ __forceinline__ float4 load4(const float *p) { return *reinterpret_cast<const float4 *>(p); }
__device__ __forceinline__ float4 load4(const __nv_bfloat16 *p) {
  uint2 raw = *reinterpret_cast<const uint2 *>(p);
  const __nv_bfloat162 *h = reinterpret_cast<const __nv_bfloat162 *>(&raw);
  float2 a = __bfloat1622float2(h[0]), b = __bfloat1622float2(h[1]);
  return make_float4(a.x, a.y, b.x, b.y);
}
__device__ __forceinline__ float4 load4(const __half *p) {
  uint2 raw = *reinterpret_cast<const uint2 *>(p);
  const __half2 *h = reinterpret_cast<const __half2 *>(&raw);
  float2 a = __half22float2(h[0]), b = __half22float2(h[1]);
  return make_float4(a.x, a.y, b.x, b.y);
}
__device__ __forceinline__ void store4(float *p, float4 v) { *reinterpret_cast<float4 *>(p) = v; }
__device__ __forceinline__ void store4(__nv_bfloat16 *p, float4 v) {
  __nv_bfloat162 lo = __floats2bfloat162_rn(v.x, v.y), hi = __floats2bfloat162_rn(v.z, v.w);
  uint2 raw;
  raw.x = *reinterpret_cast<uint32_t *>(&lo);
  raw.y = *reinterpret_cast<uint32_t *>(&hi);
  *reinterpret_cast<uint2 *>(p) = raw;
}

// Grid (M, ceil(d / 1024)): one float4 of one token per thread.  The up-to-k rows of y are all
// loaded before the first FMA (one memory round trip), then added in slot order.
__device__ __forceinline__ void store4(__half *p, float4 v) {
  __half2 lo = __floats2half2_rn(v.x, v.y), hi = __floats2half2_rn(v.z, v.w);
  uint2 raw;
  raw.x = *reinterpret_cast<uint32_t *>(&lo);
  raw.y = *reinterpret_cast<uint32_t *>(&hi);
  *reinterpret_cast<uint2 *>(p) = raw;
}

template <typename T, typename TO>
__global__ void __launch_bounds__(256) combine_kernel(const float *__restrict__ y,
                                                      const float *__restrict__ gate_w,
                                                      const int *__restrict__ tokslot2row,
                                                      const T *__restrict__ hidden, TO *__restrict__ out, int d,
                                                      int k, int residual, const int *__restrict__ assign_idx,
                                                      int res_first, int res_count) {
  const int t = blockIdx.x;
  const int c = (blockIdx.y * blockDim.x + threadIdx.x) * 4;
  __shared__ int s_row[kMaxK];
  __shared__ float s_w[kMaxK];
  pdl_trigger();
  pdl_wait();
  if (threadIdx.x < k) {
    int row = tokslot2row[(size_t)t * k + threadIdx.x];
    if (res_count > 0 && row >= 0) {      // expert-parallel shard: only the slots of resident experts
      const int e = assign_idx[(size_t)t * k + threadIdx.x];
      if (e < res_first || e >= res_first + res_count) row = -1;
    }
    s_row[threadIdx.x] = row;
    s_w[threadIdx.x] = gate_w[(size_t)t * k + threadIdx.x];
  }
  __syncthreads();
  if (c >= d) return;
  float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
  for (int s0 = 0; s0 < k; s0 += 8) {
    float4 v[8];
#pragma unroll
    for (int s = 0; s < 8; ++s) {
      const int row = s0 + s < k ? s_row[s0 + s] : -1;
      v[s] = row >= 0 ? load4(y + (size_t)row * d + c) : make_float4(0.f, 0.f, 0.f, 0.f);
    }
#pragma unroll
    for (int s = 0; s < 8; ++s) {
      if (s0 + s < k && s_row[s0 + s] >= 0) {
        const float w = s_w[s0 + s];
        acc.x = fmaf(w, v[s].x, acc.x);
        acc.y = fmaf(w, v[s].y, acc.y);
        acc.z = fmaf(w, v[s].z, acc.z);
        acc.w = fmaf(w, v[s].w, acc.w);
      }
    }
  }
  if (residual) {
    float4 h = load4(hidden + (size_t)t * d + c);
    acc.x += h.x; acc.y += h.y; acc.z += h.z; acc.w += h.w;
  }
  store4(out + (size_t)t * d + c, acc);
}

template <typename T, typename TO>
static cudaError_t launch_t(const LaunchCtx &c, const void *hidden, void *out) {
  const moespec_layer_desc &D = *c.desc;
  return launch_kernel(combine_kernel<T, TO>, dim3(c.M, (D.d + 1023) / 1024), dim3(256), 0, c.stream, (const float *)c.ws->y,
                       (const float *)c.ws->gate_w, (const int *)c.ws->tokslot2row, (const T *)hidden, (TO *)out, D.d,
                       c.k, D.residual, (const int *)c.ws->assign_idx, c.res_first,
                       c.res_count > 0 && c.res_count < D.n_experts ? c.res_count : 0);
}

cudaError_t launch_combine(const LaunchCtx &c, const void *hidden, void *out) {
  const moespec_layer_desc &D = *c.desc;
  const int od = D.out_dtype ? D.out_dtype : D.dtype;
  if (D.dtype == MOESPEC_BF16 && od == MOESPEC_BF16) return launch_t<__nv_bfloat16, __nv_bfloat16>(c, hidden, out);
  if (D.dtype == MOESPEC_BF16) return launch_t<__nv_bfloat16, float>(c, hidden, out);
  if (D.dtype == MOESPEC_FP16 && od == MOESPEC_FP16) return launch_t<__half, __half>(c, hidden, out);
  if (D.dtype == MOESPEC_FP16) return launch_t<__half, float>(c, hidden, out);
  return launch_t<float, float>(c, hidden, out);
}

}  // namespace moespec
