// CUDA-core expert FFN: E_i(x) = W2 (silu(W1 x) * (W3 x)) on the routed rows,
// full-precision fp32 FMAs.  This is the kernel of the fp32 configuration (a
// tensor-core tf32 product would drop mantissa bits) and a slow, simple
// alternative for bf16 that shares nothing with the tensor-core kernel.
#include "internal.h"

namespace moespec {

__device__ __forceinline__ float cc_to_float(float v) { return v; }
__device__ __forceinline__ float cc_to_float(__nv_bfloat16 v) { return __bfloat162float(v); }
__device__ __forceinline__ float cc_to_float(__half v) { return __half2float(v); }
__device__ __forceinline__ void cc_store(float *p, float v) { *p = v; }
__device__ __forceinline__ void cc_store(__nv_bfloat16 *p, float v) { *p = __float2bfloat16_rn(v); }
__device__ __forceinline__ void cc_store(__half *p, float v) { *p = __float2half_rn(v); }

constexpr int kColsPerBlock = 64;

// gate/up: h_mid[r, j] = silu(w_gate[e, j, :] . x_r) * (w_up[e, j, :] . x_r)
template <typename T>
__global__ void __launch_bounds__(256) ffn_gateup_cc_kernel(const T *__restrict__ x_perm,
                                                            const T *__restrict__ w_gate,
                                                            const T *__restrict__ w_up, T *__restrict__ h_mid,
                                                            const int *__restrict__ row2expert,
                                                            const int *__restrict__ counters, int d, int f,
                                                            int res_first, int res_count) {
  extern __shared__ float xs[];
  const int r = blockIdx.x;
  pdl_trigger();
  pdl_wait();
  if (r >= counters[2]) return;
  const int e = row2expert[r] - res_first;          // index into the resident experts' weights
  if (e < 0 || e >= res_count) return;              // another GPU's expert
  const T *x = x_perm + (size_t)r * d;
  for (int j = threadIdx.x; j < d; j += blockDim.x) xs[j] = cc_to_float(x[j]);
  __syncthreads();
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
  constexpr int VEC = 16 / sizeof(T);
  for (int jj = warp; jj < kColsPerBlock; jj += nwarps) {
    const int j = blockIdx.y * kColsPerBlock + jj;
    if (j >= f) break;
    const T *g = w_gate + ((size_t)e * f + j) * d;
    const T *u = w_up + ((size_t)e * f + j) * d;
    float ag = 0.f, au = 0.f;
    for (int c = lane * VEC; c < d; c += 32 * VEC) {
      uint4 rg = *reinterpret_cast<const uint4 *>(g + c);
      uint4 ru = *reinterpret_cast<const uint4 *>(u + c);
      const T *eg = reinterpret_cast<const T *>(&rg);
      const T *eu = reinterpret_cast<const T *>(&ru);
#pragma unroll
      for (int v = 0; v < VEC; ++v) {
        ag = fmaf(cc_to_float(eg[v]), xs[c + v], ag);
        au = fmaf(cc_to_float(eu[v]), xs[c + v], au);
      }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      ag += __shfl_xor_sync(0xffffffffu, ag, o);
      au += __shfl_xor_sync(0xffffffffu, au, o);
    }
    if (lane == 0) cc_store(h_mid + (size_t)r * f + j, (ag / (1.f + expf(-ag))) * au);
  }
}

// down: y[r, c] = w_down[e, c, :] . h_mid[r, :]
template <typename T>
__global__ void __launch_bounds__(256) ffn_down_cc_kernel(const T *__restrict__ h_mid,
                                                          const T *__restrict__ w_down, float *__restrict__ y,
                                                          const int *__restrict__ row2expert,
                                                          const int *__restrict__ counters, int d, int f,
                                                          int res_first, int res_count) {
  extern __shared__ float ms[];
  const int r = blockIdx.x;
  pdl_trigger();
  pdl_wait();
  if (r >= counters[2]) return;
  const int e = row2expert[r] - res_first;          // index into the resident experts' weights
  if (e < 0 || e >= res_count) return;              // another GPU's expert
  const T *m = h_mid + (size_t)r * f;
  for (int j = threadIdx.x; j < f; j += blockDim.x) ms[j] = cc_to_float(m[j]);
  __syncthreads();
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
  constexpr int VEC = 16 / sizeof(T);
  for (int cc = warp; cc < kColsPerBlock; cc += nwarps) {
    const int c = blockIdx.y * kColsPerBlock + cc;
    if (c >= d) break;
    const T *w = w_down + ((size_t)e * d + c) * f;
    float acc = 0.f;
    for (int j = lane * VEC; j < f; j += 32 * VEC) {
      uint4 rw = *reinterpret_cast<const uint4 *>(w + j);
      const T *ew = reinterpret_cast<const T *>(&rw);
#pragma unroll
      for (int v = 0; v < VEC; ++v) acc = fmaf(cc_to_float(ew[v]), ms[j + v], acc);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
    if (lane == 0) y[(size_t)r * d + c] = acc;
  }
}

template <typename T>
static cudaError_t launch_cc(const LaunchCtx &c, int phase) {
  const moespec_layer_desc &D = *c.desc;
  const int rows = c.M * c.k;
  if (phase == 0) {
    dim3 g1(rows, (D.f + kColsPerBlock - 1) / kColsPerBlock);
    return launch_kernel(ffn_gateup_cc_kernel<T>, g1, dim3(256), D.d * sizeof(float), c.stream,
                         (const T *)c.ws->x_perm, (const T *)D.w_gate, (const T *)D.w_up, (T *)c.ws->h_mid,
                         (const int *)c.ws->row2expert, (const int *)c.ws->counters, D.d, D.f, c.res_first,
                         c.res_count > 0 ? c.res_count : D.n_experts);
  } else {
    dim3 g2(rows, (D.d + kColsPerBlock - 1) / kColsPerBlock);
    return launch_kernel(ffn_down_cc_kernel<T>, g2, dim3(256), D.f * sizeof(float), c.stream,
                         (const T *)c.ws->h_mid, (const T *)D.w_down, c.ws->y, (const int *)c.ws->row2expert,
                         (const int *)c.ws->counters, D.d, D.f, c.res_first, c.res_count > 0 ? c.res_count : D.n_experts);
  }
}

// The kernels stage one row (d or f floats) in dynamic shared memory; rows beyond 48 KB need the opt-in
// limit raised, and rows beyond the device's opt-in maximum do not fit at all (*fits = false).
template <typename T>
static cudaError_t configure_cc(size_t up_bytes, size_t down_bytes) {
  cudaError_t e = cudaSuccess;
  if (up_bytes > 48 * 1024)
    e = cudaFuncSetAttribute(ffn_gateup_cc_kernel<T>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)up_bytes);
  if (e == cudaSuccess && down_bytes > 48 * 1024)
    e = cudaFuncSetAttribute(ffn_down_cc_kernel<T>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)down_bytes);
  return e;
}

cudaError_t cc_configure(const moespec_layer_desc &D, bool *fits) {
  const size_t up_bytes = (size_t)D.d * sizeof(float), down_bytes = (size_t)D.f * sizeof(float);
  int optin = 0;
  cudaError_t e = cudaDeviceGetAttribute(&optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, D.device);
  if (e != cudaSuccess) return e;
  *fits = up_bytes <= (size_t)optin && down_bytes <= (size_t)optin;
  if (!*fits) return cudaSuccess;
  if (D.dtype == MOESPEC_BF16) return configure_cc<__nv_bfloat16>(up_bytes, down_bytes);
  if (D.dtype == MOESPEC_FP16) return configure_cc<__half>(up_bytes, down_bytes);
  return configure_cc<float>(up_bytes, down_bytes);
}

cudaError_t launch_ffn_cuda_core(const LaunchCtx &c, int phase) {
  if (c.desc->dtype == MOESPEC_BF16) return launch_cc<__nv_bfloat16>(c, phase);
  if (c.desc->dtype == MOESPEC_FP16) return launch_cc<__half>(c, phase);
  return launch_cc<float>(c, phase);
}

}  // namespace moespec
