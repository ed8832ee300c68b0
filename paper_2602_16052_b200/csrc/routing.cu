// Routing half of the layer: router projection (Eq. 1 numerator), softmax and
// natural top-k (Eq. 1, Eq. 2), union (Eq. 3), router-based scores (Eq. 5),
// top-B shortlist (Section 3.2), re-routing under substitution (Eq. 8) or
// truncation (Eq. 7) with the mixing weights of Section 3.3, and the
// per-expert gather order (Appendix C).
#include "internal.h"
#include <math_constants.h>

namespace moespec {

__device__ __forceinline__ float to_float(float v) { return v; }
__device__ __forceinline__ float to_float(__nv_bfloat16 v) { return __bfloat162float(v); }

// ---------------------------------------------------------------------------
// K1a: z[t,i] = b_i + w_i . h_t, fp32 accumulation.  One CTA per token; the
// token row is staged in shared memory as fp32, each warp takes experts
// warp, warp+8, ... and reads the router row with 16-byte loads.
// ---------------------------------------------------------------------------
template <typename T>
__global__ void __launch_bounds__(256) router_logits_kernel(const T *__restrict__ hidden,
                                                            const T *__restrict__ Wr,
                                                            const float *__restrict__ bias,
                                                            float *__restrict__ logits, int N, int d) {
  extern __shared__ float xs[];
  const int t = blockIdx.x;
  const T *h = hidden + (size_t)t * d;
  for (int j = threadIdx.x; j < d; j += blockDim.x) xs[j] = to_float(h[j]);
  __syncthreads();
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
  constexpr int VEC = 16 / sizeof(T);
  for (int i = warp; i < N; i += nwarps) {
    const T *w = Wr + (size_t)i * d;
    float acc = 0.f;
    for (int j = lane * VEC; j < d; j += 32 * VEC) {
      uint4 raw = *reinterpret_cast<const uint4 *>(w + j);
      const T *e = reinterpret_cast<const T *>(&raw);
#pragma unroll
      for (int v = 0; v < VEC; ++v) acc = fmaf(to_float(e[v]), xs[j + v], acc);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
    if (lane == 0) logits[(size_t)t * N + i] = acc + (bias ? bias[i] : 0.f);
  }
}

cudaError_t launch_router_logits(const LaunchCtx &c, const void *hidden) {
  const moespec_layer_desc &D = *c.desc;
  size_t smem = (size_t)D.d * sizeof(float);
  if (D.dtype == MOESPEC_BF16)
    router_logits_kernel<__nv_bfloat16><<<c.M, 256, smem, c.stream>>>(
        (const __nv_bfloat16 *)hidden, (const __nv_bfloat16 *)D.router_w, D.router_bias, c.ws->logits,
        D.n_experts, D.d);
  else
    router_logits_kernel<float><<<c.M, 256, smem, c.stream>>>((const float *)hidden, (const float *)D.router_w,
                                                              D.router_bias, c.ws->logits, D.n_experts, D.d);
  return cudaGetLastError();
}

// ---------------------------------------------------------------------------
// Warp-wide ranking: repeatedly take the best remaining candidate under
// (value descending, index ascending).  Lane l owns experts l, l+32, ...
// `valid` has bit s set when local slot s is still a candidate.  Returns the
// number of winners written to sel[] (warp-uniform), clears winners from valid.
// ---------------------------------------------------------------------------
__device__ __forceinline__ int warp_take_best(const float (&v)[kMaskWords], uint32_t &valid, int rounds,
                                              int *sel, int lane) {
  int n = 0;
  for (int r = 0; r < rounds; ++r) {
    float bv = -CUDART_INF_F;
    int bi = 0x7fffffff;
#pragma unroll
    for (int s = 0; s < kMaskWords; ++s) {
      if ((valid >> s) & 1u) {
        int idx = lane + 32 * s;
        if (bi == 0x7fffffff || v[s] > bv) { bv = v[s]; bi = idx; }
      }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      float ov = __shfl_xor_sync(0xffffffffu, bv, o);
      int oi = __shfl_xor_sync(0xffffffffu, bi, o);
      bool take = (oi != 0x7fffffff) && (bi == 0x7fffffff || ov > bv || (ov == bv && oi < bi));
      if (take) { bv = ov; bi = oi; }
    }
    if (bi == 0x7fffffff) break;
    if ((bi & 31) == lane) valid &= ~(1u << (bi >> 5));
    sel[n++] = bi;
  }
  return n;
}

struct RouteArgs {
  const float *logits;
  Workspace ws;
  int M, N, k, B;
  int policy, shortlist, renormalize;
  int tiles_up, tiles_down;     // f/128, d/128 (0 when the tensor-core path is not used)
  long long expert_bytes;       // 3*d*f*sizeof(dtype)
};

// ---------------------------------------------------------------------------
// K2: everything between the logits and the expert FFNs, in one CTA.  The data
// is tiny (M*N <= a few 10k values); one CTA keeps every ranking deterministic
// and needs no inter-CTA synchronisation.
// ---------------------------------------------------------------------------
__global__ void __launch_bounds__(1024) route_kernel(RouteArgs a) {
  __shared__ double s_score[kMaxExperts];
  __shared__ int s_cand[kMaxExperts];
  __shared__ int s_count[kMaxExperts];
  __shared__ int s_offset[kMaxExperts + 1];
  __shared__ int s_unit_base[kMaxExperts + 1];
  __shared__ uint32_t s_Smask[kMaskWords];
  __shared__ int s_nS, s_nactive, s_nunion;

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, nwarps = blockDim.x >> 5;
  const int M = a.M, N = a.N, k = a.k;
  const int W = kMaskWords;
  const Workspace &ws = a.ws;
  uint32_t *natmask = reinterpret_cast<uint32_t *>(ws.natmask);
  uint32_t *amask = reinterpret_cast<uint32_t *>(ws.amask);
  if (tid < W) s_Smask[tid] = 0;
  if (tid == 0) *ws.status = 0;

  // ---- phase A: softmax (Eq. 1) and natural top-k (Eq. 2), one warp per token
  for (int t = warp; t < M; t += nwarps) {
    float v[kMaskWords];
    uint32_t valid = 0;
    float mx = -CUDART_INF_F;
#pragma unroll
    for (int s = 0; s < kMaskWords; ++s) {
      int idx = lane + 32 * s;
      v[s] = -CUDART_INF_F;
      if (idx < N) {
        v[s] = a.logits[(size_t)t * N + idx];
        valid |= 1u << s;
        mx = fmaxf(mx, v[s]);
      }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
    double e[kMaskWords], sum = 0.0;
#pragma unroll
    for (int s = 0; s < kMaskWords; ++s) {
      e[s] = 0.0;
      if ((valid >> s) & 1u) { e[s] = exp((double)v[s] - (double)mx); sum += e[s]; }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
#pragma unroll
    for (int s = 0; s < kMaskWords; ++s)
      if ((valid >> s) & 1u) ws.prob[(size_t)t * N + lane + 32 * s] = e[s] / sum;

    int sel[kMaxK];
    uint32_t rem = valid;
    int n = warp_take_best(v, rem, k, sel, lane);
    uint32_t chosen = valid & ~rem;
#pragma unroll
    for (int s = 0; s < kMaskWords; ++s) {
      uint32_t word = __ballot_sync(0xffffffffu, (chosen >> s) & 1u);
      if (lane == 0) natmask[(size_t)t * W + s] = word;
    }
    if (lane == 0)
      for (int r = 0; r < k; ++r) ws.topk_idx[(size_t)t * k + r] = r < n ? sel[r] : -1;
  }
  __syncthreads();

  // ---- phase B: union (Eq. 3), scores (Eq. 5: tokens added in ascending order, fp64)
  int my_cand = 0, in_union = 0;
  if (tid < N) {
    int natcnt = 0;
    double s = 0.0;
    const int w = tid >> 5;
    const uint32_t bit = 1u << (tid & 31);
    for (int t = 0; t < M; ++t) {
      natcnt += (natmask[(size_t)t * W + w] & bit) ? 1 : 0;
      s += ws.prob[(size_t)t * N + tid];
    }
    s_score[tid] = s;
    ws.score[tid] = s;
    in_union = natcnt > 0;
    my_cand = (a.shortlist == MOESPEC_FROM_UNION) ? in_union : 1;
    s_cand[tid] = my_cand;
  }
  const int n_union = __syncthreads_count(in_union);
  const int n_cand = __syncthreads_count(my_cand);
  if (tid == 0) s_nunion = n_union;
  const int nS = min(a.B, n_cand);

  // ---- top-B shortlist: rank by counting under (score desc, index asc)
  if (tid < N && my_cand) {
    int rank = 0;
    const double si = s_score[tid];
    for (int j = 0; j < N; ++j)
      if (s_cand[j]) {
        double sj = s_score[j];
        rank += (sj > si || (sj == si && j < tid)) ? 1 : 0;
      }
    if (rank < nS) {
      ws.S_rank[rank] = tid;
      atomicOr(&s_Smask[tid >> 5], 1u << (tid & 31));
    }
  }
  if (tid == 0) s_nS = nS;
  __syncthreads();

  // ---- phase C: re-routing (Eq. 7 / Eq. 8) and mixing weights (Section 3.3), one warp per token
  for (int t = warp; t < M; t += nwarps) {
    int sel[kMaxK];
    int n = 0;
    uint32_t kept_bits = 0;   // local slots of kept experts
    if (a.policy == MOESPEC_SUBSTITUTION) {
      float v[kMaskWords];
      uint32_t valid = 0;
#pragma unroll
      for (int s = 0; s < kMaskWords; ++s) {
        int idx = lane + 32 * s;
        v[s] = -CUDART_INF_F;
        if (idx < N && ((s_Smask[s] >> lane) & 1u)) {
          v[s] = a.logits[(size_t)t * N + idx];
          valid |= 1u << s;
        }
      }
      uint32_t rem = valid;
      n = warp_take_best(v, rem, min(k, nS), sel, lane);
      kept_bits = valid & ~rem;
      for (int r = n; r < k; ++r) sel[r] = -1;
    } else {
      for (int r = 0; r < k; ++r) {
        int idx = ws.topk_idx[(size_t)t * k + r];
        bool keep = idx >= 0 && ((s_Smask[idx >> 5] >> (idx & 31)) & 1u);
        sel[r] = keep ? idx : -1;
        if (keep && (idx & 31) == lane) kept_bits |= 1u << (idx >> 5);
      }
      n = k;
    }
#pragma unroll
    for (int s = 0; s < kMaskWords; ++s) {
      uint32_t word = __ballot_sync(0xffffffffu, (kept_bits >> s) & 1u);
      if (lane == 0) amask[(size_t)t * W + s] = word;
    }
    if (lane == 0) {
      double denom = 1.0;
      if (a.renormalize) {
        denom = 0.0;
        if (a.policy == MOESPEC_SUBSTITUTION) {
          for (int r = 0; r < k; ++r)
            if (sel[r] >= 0) denom += ws.prob[(size_t)t * N + sel[r]];
        } else {            // the original top-k set, not the reduced one
          for (int r = 0; r < k; ++r) {
            int idx = ws.topk_idx[(size_t)t * k + r];
            if (idx >= 0) denom += ws.prob[(size_t)t * N + idx];
          }
        }
      }
      for (int r = 0; r < k; ++r) {
        ws.assign_idx[(size_t)t * k + r] = sel[r];
        ws.gate_w[(size_t)t * k + r] = sel[r] >= 0 ? (float)(ws.prob[(size_t)t * N + sel[r]] / denom) : 0.f;
        ws.tokslot2row[(size_t)t * k + r] = -1;
      }
    }
  }
  __syncthreads();

  // ---- phase D: rows per expert and their exclusive scan (Appendix C gather)
  if (tid < N) {
    int c = 0;
    const int w = tid >> 5;
    const uint32_t bit = 1u << (tid & 31);
    for (int t = 0; t < M; ++t) c += (amask[(size_t)t * W + w] & bit) ? 1 : 0;
    s_count[tid] = c;
    ws.count[tid] = c;
  }
  __syncthreads();
  if (tid == 0) {
    int run = 0, na = 0, ub = 0;
    for (int i = 0; i < N; ++i) {
      s_offset[i] = run;
      ws.offset[i] = run;
      s_unit_base[i] = ub;
      if (s_count[i] > 0) {
        ws.active[na++] = i;
        ub += (s_count[i] + kMaxTokChunk - 1) / kMaxTokChunk;   // token chunks of this expert
      }
      run += s_count[i];
    }
    s_offset[N] = run;
    ws.offset[N] = run;
    s_unit_base[N] = ub;
    s_nactive = na;
  }
  __syncthreads();

  // ---- phase E: rows ordered by (expert ascending, token ascending)
  if (tid < N && s_count[tid] > 0) {
    int row = s_offset[tid];
    const int w = tid >> 5;
    const uint32_t bit = 1u << (tid & 31);
    for (int t = 0; t < M; ++t) {
      if (amask[(size_t)t * W + w] & bit) {
        ws.perm_row2tok[row] = t;
        ws.row2expert[row] = tid;
        for (int r = 0; r < k; ++r)
          if (ws.assign_idx[(size_t)t * k + r] == tid) ws.tokslot2row[(size_t)t * k + r] = row;
        ++row;
      }
    }
  }

  // ---- phase F: tensor-core work units (expert, token chunk, 128-row slab)
  const int n_chunks = s_unit_base[N];
  if (a.tiles_up > 0) {
    for (int i = warp; i < N; i += nwarps) {
      const int cnt = s_count[i];
      if (cnt == 0) continue;
      const int chunks = (cnt + kMaxTokChunk - 1) / kMaxTokChunk;
      for (int c = 0; c < chunks; ++c) {
        const int row0 = s_offset[i] + c * kMaxTokChunk;
        const int rows = min(kMaxTokChunk, cnt - c * kMaxTokChunk);
        const int ci = s_unit_base[i] + c;
        for (int tl = lane; tl < a.tiles_up; tl += 32) ws.units_up[(size_t)ci * a.tiles_up + tl] = Unit{i, tl, row0, rows};
        for (int tl = lane; tl < a.tiles_down; tl += 32) ws.units_down[(size_t)ci * a.tiles_down + tl] = Unit{i, tl, row0, rows};
      }
    }
  }

  if (tid == 0) {
    const int R = s_offset[N];
    ws.counters[0] = s_nS;
    ws.counters[1] = s_nactive;
    ws.counters[2] = R;
    ws.counters[3] = n_chunks * a.tiles_up;
    ws.counters[4] = n_chunks * a.tiles_down;
    double cov = 0.0;
    for (int r = 0; r < s_nS; ++r) cov += s_score[ws.S_rank[r]];
    moespec_stats st;
    st.n_union = s_nunion;
    st.n_shortlist = s_nS;
    st.n_active = s_nactive;
    st.n_rows = R;
    st.n_dropped = M * k - R;
    st.status = 0;
    st.coverage = M > 0 ? cov / (double)M : 0.0;
    st.weight_bytes = (long long)s_nactive * a.expert_bytes;
    *ws.stats = st;
  }
}

cudaError_t launch_route(const LaunchCtx &c, const float *logits) {
  const moespec_layer_desc &D = *c.desc;
  RouteArgs a;
  a.logits = logits;
  a.ws = *c.ws;
  a.M = c.M; a.N = D.n_experts; a.k = c.k; a.B = c.B;
  a.policy = D.policy; a.shortlist = D.shortlist; a.renormalize = D.renormalize;
  const bool tc = (D.f % kTile == 0) && (D.d % kTile == 0);
  a.tiles_up = tc ? D.f / kTile : 0;
  a.tiles_down = tc ? D.d / kTile : 0;
  a.expert_bytes = 3LL * D.d * D.f * (D.dtype == MOESPEC_BF16 ? 2 : 4);
  int threads = 1024;
  route_kernel<<<1, threads, 0, c.stream>>>(a);
  return cudaGetLastError();
}

// ---------------------------------------------------------------------------
// K3: gather routed rows: x_perm[r, :] = hidden[perm_row2tok[r], :].
// ---------------------------------------------------------------------------
__global__ void __launch_bounds__(128) gather_rows_kernel(const uint4 *__restrict__ hidden,
                                                          uint4 *__restrict__ x_perm,
                                                          const int *__restrict__ perm,
                                                          const int *__restrict__ counters, int row_vec) {
  const int r = blockIdx.x;
  if (r >= counters[2]) return;
  const int t = perm[r];
  const uint4 *src = hidden + (size_t)t * row_vec;
  uint4 *dst = x_perm + (size_t)r * row_vec;
  for (int j = threadIdx.x; j < row_vec; j += blockDim.x) dst[j] = src[j];
}

cudaError_t launch_gather(const LaunchCtx &c, const void *hidden) {
  const moespec_layer_desc &D = *c.desc;
  const int row_vec = D.d * (D.dtype == MOESPEC_BF16 ? 2 : 4) / 16;
  const int rows = c.M * c.k;
  if (rows == 0) return cudaSuccess;
  gather_rows_kernel<<<rows, 128, 0, c.stream>>>((const uint4 *)hidden, (uint4 *)c.ws->x_perm,
                                                 c.ws->perm_row2tok, c.ws->counters, row_vec);
  return cudaGetLastError();
}

}  // namespace moespec
