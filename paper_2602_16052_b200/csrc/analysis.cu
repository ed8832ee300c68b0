// Analysis mode: oracle (greedy reconstruction-error) ranking of Eq. 6 and the reconstruction error
// of Section 4.5.  Both work on what an unbudgeted pass of the layer leaves in the workspace: the rows
// y[row(t, a)] = E_i(h_t) of every (token, natural top-k expert) pair, their mixing weights and the
// gather order.
//
// With c_{t,i} = g_i(h_t) E_i(h_t) the objective of Eq. 6 for a set S is
//     sum_t || sum_{j in T_k(h_t) \ S} c_{t,j} ||^2,
// so adding expert i lowers it by
//     gain_i(S) = sum_{t : i in T_k(h_t)} ( 2 * sum_{j in T_k(h_t) \ S} c_{t,j}.c_{t,i}  -  c_{t,i}.c_{t,i} ).
// Everything the greedy loop needs is therefore the k x k Gram matrix of each token's weighted rows.
// Kernel 1 forms the Gram matrices (fp32 inputs, fp64 products and sums, fixed order); kernel 2 runs
// the whole greedy loop in one CTA (fp64, ties -> lower expert index, a fixed summation order).
#include "internal.h"

namespace moespec {

namespace {

constexpr unsigned kFullMask = 0xffffffffu;

__device__ __forceinline__ float to_float(float v) { return v; }
__device__ __forceinline__ float to_float(__nv_bfloat16 v) { return __bfloat162float(v); }
__device__ __forceinline__ float to_float(__half v) { return __half2float(v); }

__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    int lo = __double2loint(v), hi = __double2hiint(v);
    lo = __shfl_xor_sync(kFullMask, lo, o);
    hi = __shfl_xor_sync(kFullMask, hi, o);
    v += __hiloint2double(hi, lo);
  }
  return v;
}

// G[t][a][b] = (w_a y_a) . (w_b y_b) for the k slots of token t; slots without a row give zeros.
// Grid M, 256 threads: the k(k+1)/2 pairs are dealt to the 8 warps, a warp walks the two rows together.
__global__ void __launch_bounds__(256) gram_kernel(const float *__restrict__ y, const float *__restrict__ gate_w,
                                                   const int *__restrict__ tokslot2row, double *__restrict__ gram,
                                                   int *__restrict__ row2slot, int d, int k) {
  const int t = blockIdx.x, lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  if (threadIdx.x < k) {
    const int row = tokslot2row[(size_t)t * k + threadIdx.x];
    if (row >= 0) row2slot[row] = threadIdx.x;
  }
  const int n_pairs = k * (k + 1) / 2;
  for (int p = warp; p < n_pairs; p += 8) {
    // pair index -> (a, b), a <= b
    int a = 0, rem = p;
    while (rem >= k - a) {
      rem -= k - a;
      ++a;
    }
    const int b = a + rem;
    const int ra = tokslot2row[(size_t)t * k + a], rb = tokslot2row[(size_t)t * k + b];
    double acc = 0.0;
    if (ra >= 0 && rb >= 0) {
      const float4 *pa = reinterpret_cast<const float4 *>(y + (size_t)ra * d);
      const float4 *pb = reinterpret_cast<const float4 *>(y + (size_t)rb * d);
      for (int c = lane; c < d / 4; c += 32) {
        const float4 u = __ldcg(pa + c), v = __ldcg(pb + c);
        acc += (double)u.x * (double)v.x;
        acc += (double)u.y * (double)v.y;
        acc += (double)u.z * (double)v.z;
        acc += (double)u.w * (double)v.w;
      }
      acc = warp_sum(acc);
      acc *= (double)gate_w[(size_t)t * k + a] * (double)gate_w[(size_t)t * k + b];
    }
    if (lane == 0) {
      gram[((size_t)t * k + a) * k + b] = acc;
      gram[((size_t)t * k + b) * k + a] = acc;
    }
  }
}

// Greedy loop of Eq. 6 in one CTA of 256 threads.  Per step: warp w computes the gain of experts
// w, w+8, ... (lanes stride the expert's rows in gather order, partial sums meet in a shuffle tree), then
// warp 0 takes the largest gain (ties -> lower index; an expert without rows has gain 0).
__global__ void __launch_bounds__(256) greedy_kernel(const double *__restrict__ gram, const int *__restrict__ assign_idx,
                                                     const int *__restrict__ offset, const int *__restrict__ perm_row2tok,
                                                     const int *__restrict__ row2slot, int M, int N, int k, int n_pick,
                                                     int *__restrict__ order, double *__restrict__ objective,
                                                     double *__restrict__ gold_energy) {
  __shared__ unsigned char s_in[kMaxExperts];
  __shared__ double s_gain[kMaxExperts];
  __shared__ double s_part[8];
  __shared__ double s_err;
  __shared__ int s_best;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  for (int i = tid; i < N; i += blockDim.x) s_in[i] = 0;
  // objective of the empty set: sum_t || O*_t ||^2 = sum_t sum_{a,b} G_t[a][b], in a fixed order
  {
    double acc = 0.0;
    const size_t n = (size_t)M * k * k;
    for (size_t i = tid; i < n; i += blockDim.x) acc += gram[i];
    acc = warp_sum(acc);
    if (lane == 0) s_part[warp] = acc;
    __syncthreads();
    if (tid == 0) {
      double tot = 0.0;
      for (int w = 0; w < 8; ++w) tot += s_part[w];
      s_err = tot;
      *gold_energy = tot;
    }
  }
  __syncthreads();
  for (int step = 0; step < n_pick; ++step) {
    for (int i = warp; i < N; i += 8) {
      double g = 0.0;
      if (!s_in[i]) {
        for (int r = offset[i] + lane; r < offset[i + 1]; r += 32) {
          const int t = perm_row2tok[r], a = row2slot[r];
          const double *G = gram + ((size_t)t * k + a) * k;
          double cross = 0.0;
          for (int b = 0; b < k; ++b) {
            const int j = assign_idx[(size_t)t * k + b];
            if (j >= 0 && !s_in[j]) cross += G[b];
          }
          g += 2.0 * cross - G[a];
        }
        g = warp_sum(g);
      }
      if (lane == 0) s_gain[i] = g;
    }
    __syncthreads();
    if (warp == 0) {
      double best = 0.0;
      int best_i = -1;
      for (int i = lane; i < N; i += 32) {
        if (s_in[i]) continue;
        if (best_i < 0 || s_gain[i] > best) {        // ascending i: an equal gain keeps the lower index
          best = s_gain[i];
          best_i = i;
        }
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        int lo = __double2loint(best), hi = __double2hiint(best);
        lo = __shfl_xor_sync(kFullMask, lo, o);
        hi = __shfl_xor_sync(kFullMask, hi, o);
        const double ob = __hiloint2double(hi, lo);
        const int oi = __shfl_xor_sync(kFullMask, best_i, o);
        if (oi >= 0 && (best_i < 0 || ob > best || (ob == best && oi < best_i))) {
          best = ob;
          best_i = oi;
        }
      }
      if (lane == 0) {
        s_best = best_i;
        s_in[best_i] = 1;
        s_err -= best;
        order[step] = best_i;
        objective[step] = s_err;
      }
    }
    __syncthreads();
  }
}

// sum (a - b)^2 and sum b^2 over n elements: every CTA reduces one contiguous slice in a fixed order,
// the partial sums are added by a one-CTA launch.
template <typename T>
__global__ void __launch_bounds__(256) sqdiff_partial_kernel(const T *__restrict__ a, const T *__restrict__ b, size_t n,
                                                             double *__restrict__ partial) {
  const size_t per = (n + gridDim.x - 1) / gridDim.x;
  const size_t lo = (size_t)blockIdx.x * per, hi = lo + per < n ? lo + per : n;
  double num = 0.0, den = 0.0;
  for (size_t i = lo + threadIdx.x; i < hi; i += blockDim.x) {
    const double x = (double)to_float(a[i]), r = (double)to_float(b[i]);
    num += (x - r) * (x - r);
    den += r * r;
  }
  __shared__ double s_n[8], s_d[8];
  num = warp_sum(num);
  den = warp_sum(den);
  if ((threadIdx.x & 31) == 0) {
    s_n[threadIdx.x >> 5] = num;
    s_d[threadIdx.x >> 5] = den;
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    double tn = 0.0, td = 0.0;
    for (int w = 0; w < 8; ++w) {
      tn += s_n[w];
      td += s_d[w];
    }
    partial[2 * blockIdx.x] = tn;
    partial[2 * blockIdx.x + 1] = td;
  }
}

__global__ void sqdiff_final_kernel(const double *__restrict__ partial, int n_parts, double *__restrict__ out) {
  if (threadIdx.x == 0) {
    double tn = 0.0, td = 0.0;
    for (int i = 0; i < n_parts; ++i) {
      tn += partial[2 * i];
      td += partial[2 * i + 1];
    }
    out[0] = tn;
    out[1] = td;
  }
}

}  // namespace

cudaError_t launch_gram(const LaunchCtx &c, double *gram, int *row2slot) {
  gram_kernel<<<c.M, 256, 0, c.stream>>>(c.ws->y, c.ws->gate_w, c.ws->tokslot2row, gram, row2slot, c.desc->d, c.k);
  return cudaGetLastError();
}

cudaError_t launch_greedy(const LaunchCtx &c, const double *gram, const int *row2slot, int n_pick, int *order,
                          double *objective, double *gold_energy) {
  greedy_kernel<<<1, 256, 0, c.stream>>>(gram, c.ws->assign_idx, c.ws->offset, c.ws->perm_row2tok, row2slot, c.M,
                                         c.desc->n_experts, c.k, n_pick, order, objective, gold_energy);
  return cudaGetLastError();
}

cudaError_t launch_sqdiff(const void *a, const void *b, size_t n, int dtype, double *partial, double *out,
                          cudaStream_t stream) {
  if (dtype == MOESPEC_FP32)
    sqdiff_partial_kernel<float><<<kSqdiffParts, 256, 0, stream>>>((const float *)a, (const float *)b, n, partial);
  else if (dtype == MOESPEC_FP16)
    sqdiff_partial_kernel<__half><<<kSqdiffParts, 256, 0, stream>>>((const __half *)a, (const __half *)b, n, partial);
  else
    sqdiff_partial_kernel<__nv_bfloat16><<<kSqdiffParts, 256, 0, stream>>>((const __nv_bfloat16 *)a,
                                                                           (const __nv_bfloat16 *)b, n, partial);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  sqdiff_final_kernel<<<1, 32, 0, stream>>>(partial, kSqdiffParts, out);
  return cudaGetLastError();
}

}  // namespace moespec
