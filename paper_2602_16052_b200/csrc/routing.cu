// Routing half of the layer: router projection (Eq. 1 numerator), softmax and
// natural top-k (Eq. 1, Eq. 2), union (Eq. 3), router-based scores (Eq. 5),
// top-B shortlist (Section 3.2), re-routing under substitution (Eq. 8) or
// truncation (Eq. 7) with the mixing weights of Section 3.3, and the
// per-expert gather order (Appendix C).
//
// Two launches:
//   router_topk_kernel   one warp per (token, expert) dot product; the CTA that
//                        finishes a token's last logit also runs that token's
//                        softmax and top-k (a counter, never a wait)
//   route_kernel         one CTA: scores, shortlist, re-routing, scan, gather
//                        order, work-unit list, statistics
// A stand-alone softmax/top-k kernel serves callers that inject logits.
#include "internal.h"
#include <math_constants.h>
#include <stdio.h>

namespace moespec {

__device__ __forceinline__ float to_float(float v) { return v; }
__device__ __forceinline__ float to_float(__nv_bfloat16 v) { return __bfloat162float(v); }

constexpr unsigned kFull = 0xffffffffu;
constexpr int kNone = 0x7fffffff;

// Monotone map float -> uint32 (larger float, larger key); -0 and +0 share a key.
__device__ __forceinline__ uint32_t order_key(float f) {
  if (f == 0.f) f = 0.f;
  const uint32_t u = __float_as_uint(f);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

// ---------------------------------------------------------------------------
// Warp-wide ranking under (value descending, expert index ascending).  Lane l
// owns experts l, l+32, ...; `valid` has bit s set while local slot s is still
// a candidate.  Each round is two warp reductions: the maximum key, then the
// lowest expert index among the lanes that hold it.  Winner r is returned in
// lane r (-1 when fewer than r+1 candidates existed); winners leave `valid`.
// ---------------------------------------------------------------------------
template <int W>
__device__ __forceinline__ int warp_take_best(const uint32_t (&key)[W], uint32_t &valid, int rounds, int lane) {
  int mine = -1;
  for (int r = 0; r < rounds; ++r) {
    uint32_t bk = 0;
    int bi = kNone;
#pragma unroll
    for (int s = 0; s < W; ++s)
      if (((valid >> s) & 1u) && (bi == kNone || key[s] > bk)) { bk = key[s]; bi = lane + 32 * s; }
    const uint32_t mk = __reduce_max_sync(kFull, bi == kNone ? 0u : bk);
    const int win = __reduce_min_sync(kFull, (bi != kNone && bk == mk) ? bi : kNone);
    if (win == kNone) break;
    if ((win & 31) == lane) valid &= ~(1u << (win >> 5));
    if (lane == r) mine = win;
  }
  return mine;
}

// Softmax (Eq. 1, fp64) and natural top-k (Eq. 2) of one token by one warp.
template <int W>
__device__ __forceinline__ void token_softmax_topk(const float *zrow, int N, int k, double *prob_row, int *topk_row,
                                                   int lane) {
  float v[W];
  uint32_t key[W];
  uint32_t valid = 0;
  float mx = -CUDART_INF_F;
#pragma unroll
  for (int s = 0; s < W; ++s) {
    const int idx = lane + 32 * s;
    v[s] = -CUDART_INF_F;
    key[s] = 0;
    if (idx < N) {
      v[s] = __ldcg(zrow + idx);          // written by other CTAs of this launch: read through L2
      key[s] = order_key(v[s]);
      valid |= 1u << s;
      mx = fmaxf(mx, v[s]);
    }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(kFull, mx, o));
  double e[W], sum = 0.0;
#pragma unroll
  for (int s = 0; s < W; ++s) {
    e[s] = 0.0;
    if ((valid >> s) & 1u) { e[s] = exp((double)v[s] - (double)mx); sum += e[s]; }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(kFull, sum, o);
#pragma unroll
  for (int s = 0; s < W; ++s)
    if ((valid >> s) & 1u) prob_row[lane + 32 * s] = e[s] / sum;
  const int mine = warp_take_best<W>(key, valid, k, lane);
  if (lane < k) topk_row[lane] = mine;
}

__device__ __forceinline__ void token_phase(const float *zrow, int N, int k, double *prob_row, int *topk_row, int lane) {
  if (N <= 32) token_softmax_topk<1>(zrow, N, k, prob_row, topk_row, lane);
  else if (N <= 64) token_softmax_topk<2>(zrow, N, k, prob_row, topk_row, lane);
  else if (N <= 128) token_softmax_topk<4>(zrow, N, k, prob_row, topk_row, lane);
  else token_softmax_topk<8>(zrow, N, k, prob_row, topk_row, lane);
}

// ---------------------------------------------------------------------------
// K1: z[t,i] = b_i + w_i . h_t with fp32 accumulation, fused with the token's
// softmax and top-k.  A CTA takes TT tokens x 8 experts; warp w owns expert w of
// the tile, keeps 2 KB chunks of its router row in registers and runs them
// against the TT token rows (shared through L1), so a router row is read once per
// token tile.  Each CTA then bumps the token tile's arrival counter; the CTA
// that sees the final count runs softmax and top-k of those TT tokens (one warp
// each) and resets the counter for the next call.  A counter, never a wait.
// ---------------------------------------------------------------------------
template <typename T, int TT>
__global__ void __launch_bounds__(256) router_topk_kernel(const T *__restrict__ hidden, const T *__restrict__ Wr,
                                                          const float *__restrict__ bias, float *logits,
                                                          double *prob, int *topk_idx, int *arrive, int M, int N,
                                                          int d, int k) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int t0 = blockIdx.y * TT;
  const int i = blockIdx.x * 8 + warp;
  __shared__ int s_last;
  pdl_trigger();
  pdl_wait();          // hidden may be the previous layer's output; the workspace is still in use until then
  if (i < N) {
    constexpr int VEC = 16 / sizeof(T);
    constexpr int U = 8;
    const T *w = Wr + (size_t)i * d;
    float acc[TT];
#pragma unroll
    for (int tt = 0; tt < TT; ++tt) acc[tt] = 0.f;
    for (int j0 = lane * VEC; j0 < d; j0 += 32 * VEC * U) {
      uint4 rw[U];
#pragma unroll
      for (int u = 0; u < U; ++u)
        if (j0 + u * 32 * VEC < d) rw[u] = *reinterpret_cast<const uint4 *>(w + j0 + u * 32 * VEC);
#pragma unroll
      for (int tt = 0; tt < TT; ++tt) {
        if (t0 + tt >= M) break;
        const T *h = hidden + (size_t)(t0 + tt) * d;
        uint4 rh[U];
#pragma unroll
        for (int u = 0; u < U; ++u)
          if (j0 + u * 32 * VEC < d) rh[u] = *reinterpret_cast<const uint4 *>(h + j0 + u * 32 * VEC);
#pragma unroll
        for (int u = 0; u < U; ++u) {
          if (j0 + u * 32 * VEC < d) {
            const T *ew = reinterpret_cast<const T *>(&rw[u]);
            const T *eh = reinterpret_cast<const T *>(&rh[u]);
#pragma unroll
            for (int v = 0; v < VEC; ++v) acc[tt] = fmaf(to_float(ew[v]), to_float(eh[v]), acc[tt]);
          }
        }
      }
    }
    const float b = bias ? bias[i] : 0.f;
#pragma unroll
    for (int tt = 0; tt < TT; ++tt) {
      float a = acc[tt];
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) a += __shfl_xor_sync(kFull, a, o);
      if (lane == 0 && t0 + tt < M) logits[(size_t)(t0 + tt) * N + i] = a + b;
    }
    if (lane == 0) __threadfence();
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    const int prev = atomicAdd(&arrive[blockIdx.y], 1);
    s_last = (prev == (int)gridDim.x - 1);
    if (s_last) {
      arrive[blockIdx.y] = 0;
      __threadfence();
    }
  }
  __syncthreads();
  if (s_last && warp < TT && t0 + warp < M) {
    const int t = t0 + warp;
    token_phase(logits + (size_t)t * N, N, k, prob + (size_t)t * N, topk_idx + (size_t)t * k, lane);
  }
}

template <typename T>
static cudaError_t launch_router_t(const LaunchCtx &c, const void *hidden) {
  const moespec_layer_desc &D = *c.desc;
  const Workspace &ws = *c.ws;
  const int ex_tiles = (D.n_experts + 7) / 8;
  if (c.M <= 64)
    return launch_kernel(router_topk_kernel<T, 4>, dim3(ex_tiles, (c.M + 3) / 4), dim3(256), 0, c.stream,
                         (const T *)hidden, (const T *)D.router_w, D.router_bias, ws.logits, ws.prob, ws.topk_idx,
                         ws.arrive, c.M, D.n_experts, D.d, c.k);
  return launch_kernel(router_topk_kernel<T, 8>, dim3(ex_tiles, (c.M + 7) / 8), dim3(256), 0, c.stream,
                       (const T *)hidden, (const T *)D.router_w, D.router_bias, ws.logits, ws.prob, ws.topk_idx,
                       ws.arrive, c.M, D.n_experts, D.d, c.k);
}

cudaError_t launch_router_logits(const LaunchCtx &c, const void *hidden) {
  return c.desc->dtype == MOESPEC_BF16 ? launch_router_t<__nv_bfloat16>(c, hidden) : launch_router_t<float>(c, hidden);
}

// Softmax and top-k from caller-supplied logits: one warp per token.
__global__ void __launch_bounds__(128) softmax_topk_kernel(const float *logits, double *prob, int *topk_idx, int M,
                                                           int N, int k) {
  const int t = blockIdx.x * 4 + (threadIdx.x >> 5);
  pdl_trigger();
  pdl_wait();
  if (t < M) token_phase(logits + (size_t)t * N, N, k, prob + (size_t)t * N, topk_idx + (size_t)t * k, threadIdx.x & 31);
}

__device__ __forceinline__ double shfl_double(double x, int src) {
  int lo = __double2loint(x), hi = __double2hiint(x);
  lo = __shfl_sync(kFull, lo, src);
  hi = __shfl_sync(kFull, hi, src);
  return __hiloint2double(hi, lo);
}
__device__ __forceinline__ double shfl_xor_double(double x, int mask) {
  int lo = __double2loint(x), hi = __double2hiint(x);
  lo = __shfl_xor_sync(kFull, lo, mask);
  hi = __shfl_xor_sync(kFull, hi, mask);
  return __hiloint2double(hi, lo);
}

struct RouteArgs {
  const float *logits;
  Workspace ws;
  int M, N, k, B;
  int policy, shortlist, renormalize;
  int tiles_up, tiles_down;     // f/128, d/128 (0 when the tensor-core path is not used)
  long long expert_bytes;       // 3*d*f*sizeof(dtype)
};

// Re-routing of one token (Eq. 7 / Eq. 8) with its mixing weights (Section 3.3); lane r owns slot r.
template <int W>
__device__ __forceinline__ void token_reroute(const RouteArgs &a, int t, int nS, const uint32_t *s_Smask,
                                              uint32_t *colmask, int mw, int lane) {
  const Workspace &ws = a.ws;
  const int N = a.N, k = a.k;
  int mine = -1;        // kept expert of slot `lane`
  int base = -1;        // expert whose probability enters the renormalisation sum at position `lane`
  if (a.policy == MOESPEC_SUBSTITUTION) {
    uint32_t key[W];
    uint32_t valid = 0;
#pragma unroll
    for (int s = 0; s < W; ++s) {
      const int idx = lane + 32 * s;
      key[s] = 0;
      if (idx < N && ((s_Smask[s] >> lane) & 1u)) {
        key[s] = order_key(a.logits[(size_t)t * N + idx]);
        valid |= 1u << s;
      }
    }
    mine = warp_take_best<W>(key, valid, min(k, nS), lane);
    base = mine;                                   // weights over the constrained selection
  } else if (lane < k) {
    const int idx = ws.topk_idx[(size_t)t * k + lane];
    const bool keep = idx >= 0 && ((s_Smask[idx >> 5] >> (idx & 31)) & 1u);
    mine = keep ? idx : -1;
    base = idx;                                    // weights over the original top-k set
  }
  const double p_mine = mine >= 0 ? ws.prob[(size_t)t * N + mine] : 0.0;
  const double p_base = base >= 0 ? (base == mine ? p_mine : ws.prob[(size_t)t * N + base]) : 0.0;
  double denom = 1.0;
  if (a.renormalize) {
    denom = 0.0;
    for (int r = 0; r < k; ++r) denom += shfl_double(p_base, r);   // rank order
  }
  if (lane < k) {
    ws.assign_idx[(size_t)t * k + lane] = mine;
    ws.gate_w[(size_t)t * k + lane] = mine >= 0 ? (float)(p_mine / denom) : 0.f;
    if (mine >= 0) atomicOr(&colmask[(size_t)mine * mw + (t >> 5)], 1u << (t & 31));
  }
}

// ---------------------------------------------------------------------------
// K2: everything between the per-token top-k and the expert FFNs, in one CTA.
// The data is tiny (M*N <= a few 10k values); one CTA keeps every ranking
// deterministic and needs no inter-CTA synchronisation.  Dynamic shared memory:
//   part[nwarps][N]  fp64 partial scores (warp w adds its tokens w, w+32, ... in
//                    ascending order; the partials are combined in a fixed tree)
//   colmask[N][mw]   bit t of row i: expert i is in A(t)
// ---------------------------------------------------------------------------
__global__ void __launch_bounds__(1024) route_kernel(RouteArgs a) {
  extern __shared__ __align__(16) unsigned char route_smem[];
  __shared__ double s_score[kMaxExperts];
  __shared__ int s_cand[kMaxExperts];
  __shared__ int s_natcnt[kMaxExperts];
  __shared__ int s_count[kMaxExperts];
  __shared__ int s_offset[kMaxExperts + 1];
  __shared__ int s_unit_base[kMaxExperts + 1];
  __shared__ int s_Srank[kMaxExperts];
  __shared__ uint32_t s_Smask[kMaskWords];
  __shared__ unsigned long long s_warp_tot[8];
  __shared__ int s_nS, s_nactive;

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, nwarps = blockDim.x >> 5;
  const int M = a.M, N = a.N, k = a.k;
  const int mw = (M + 31) >> 5;
  const Workspace &ws = a.ws;
  double *s_part = reinterpret_cast<double *>(route_smem);
  uint32_t *colmask = reinterpret_cast<uint32_t *>(route_smem + (size_t)nwarps * N * sizeof(double));

#ifdef MOESPEC_ROUTE_TIMING
  long long tmark[8];
  int nmark = 0;
#define ROUTE_MARK() do { if (tid == 0) tmark[nmark++] = clock64(); } while (0)
#else
#define ROUTE_MARK() do { } while (0)
#endif
  pdl_trigger();
  pdl_wait();
#ifdef MOESPEC_ROUTE_TIMING
  for (int rep = 0; rep < 2; ++rep) {
  nmark = 0;
  __syncthreads();
#endif
  ROUTE_MARK();
  if (tid < kMaskWords) s_Smask[tid] = 0;
  if (tid == 0) *ws.status = 0;
  for (int i = tid; i < N; i += blockDim.x) s_natcnt[i] = 0;
  for (int i = tid; i < N * mw; i += blockDim.x) colmask[i] = 0;
  __syncthreads();

  // ---- phase A: natural counts (Eq. 3) and partial scores (Eq. 5)
  for (int item = tid; item < M * k; item += blockDim.x) {
    const int e = ws.topk_idx[item];
    if (e >= 0) atomicAdd(&s_natcnt[e], 1);
  }
  {
    double part[kMaskWords];
#pragma unroll
    for (int s = 0; s < kMaskWords; ++s) part[s] = 0.0;
    for (int t = warp; t < M; t += nwarps) {
#pragma unroll
      for (int s = 0; s < kMaskWords; ++s)
        if (lane + 32 * s < N) part[s] += ws.prob[(size_t)t * N + lane + 32 * s];
    }
#pragma unroll
    for (int s = 0; s < kMaskWords; ++s)
      if (lane + 32 * s < N) s_part[(size_t)warp * N + lane + 32 * s] = part[s];
  }
  __syncthreads();
  ROUTE_MARK();

  // ---- phase B: scores (Eq. 5), union (Eq. 3), top-B shortlist by counting under (score desc, index asc)
  for (int i = warp; i < N; i += nwarps) {
    double s = lane < nwarps ? s_part[(size_t)lane * N + i] : 0.0;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) s += shfl_xor_double(s, o);
    if (lane == 0) {
      s_score[i] = s;
      ws.score[i] = s;
      s_cand[i] = (a.shortlist == MOESPEC_FROM_UNION) ? (s_natcnt[i] > 0) : 1;
    }
  }
  __syncthreads();
  const int n_union = __syncthreads_count(tid < N && s_natcnt[tid] > 0);
  const int n_cand = __syncthreads_count(tid < N && s_cand[tid]);
  const int nS = min(a.B, n_cand);
  for (int i = warp; i < N; i += nwarps) {
    if (!s_cand[i]) continue;
    const double si = s_score[i];
    int ahead = 0;
    for (int j = lane; j < N; j += 32)
      if (s_cand[j]) {
        const double sj = s_score[j];
        ahead += (sj > si || (sj == si && j < i)) ? 1 : 0;
      }
    const int rank = __reduce_add_sync(kFull, ahead);
    if (lane == 0 && rank < nS) {
      ws.S_rank[rank] = i;
      s_Srank[rank] = i;
      atomicOr(&s_Smask[i >> 5], 1u << (i & 31));
    }
  }
  if (tid == 0) s_nS = nS;
  __syncthreads();
  ROUTE_MARK();

  // ---- phase C: re-routing (Eq. 7 / Eq. 8) and mixing weights (Section 3.3), one warp per token
  for (int t = warp; t < M; t += nwarps) {
    if (N <= 32) token_reroute<1>(a, t, nS, s_Smask, colmask, mw, lane);
    else if (N <= 64) token_reroute<2>(a, t, nS, s_Smask, colmask, mw, lane);
    else if (N <= 128) token_reroute<4>(a, t, nS, s_Smask, colmask, mw, lane);
    else token_reroute<8>(a, t, nS, s_Smask, colmask, mw, lane);
  }
  __syncthreads();
  ROUTE_MARK();

  // ---- phase D: rows per expert and exclusive scans of rows, token chunks and active experts
  {
    int c = 0;
    if (tid < N)
      for (int w = 0; w < mw; ++w) c += __popc(colmask[(size_t)tid * mw + w]);
    const int chunks = (c + kMaxTokChunk - 1) / kMaxTokChunk;
    // rows in bits 0..23, chunks in bits 24..43, active flag in bits 44..
    unsigned long long v = (unsigned long long)c | ((unsigned long long)chunks << 24) |
                           ((unsigned long long)(c > 0) << 44);
    unsigned long long inc = v;
    if (tid < kMaxExperts) {
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        unsigned long long up = __shfl_up_sync(kFull, inc, o);
        if (lane >= o) inc += up;
      }
      if (lane == 31) s_warp_tot[warp] = inc;
    }
    __syncthreads();
    if (tid < kMaxExperts) {
      unsigned long long pre = inc - v;
      for (int w = 0; w < warp; ++w) pre += s_warp_tot[w];
      if (tid < N) {
        const int row0 = (int)(pre & 0xFFFFFFull), ub = (int)((pre >> 24) & 0xFFFFFull), ai = (int)(pre >> 44);
        s_count[tid] = c;
        s_offset[tid] = row0;
        s_unit_base[tid] = ub;
        ws.count[tid] = c;
        ws.offset[tid] = row0;
        if (c > 0) ws.active[ai] = tid;
        if (tid == N - 1) {
          s_offset[N] = row0 + c;
          ws.offset[N] = row0 + c;
          s_unit_base[N] = ub + chunks;
          s_nactive = ai + (c > 0);
        }
      }
    }
  }
  __syncthreads();
  ROUTE_MARK();

  // ---- phase E: rows ordered by (expert ascending, token ascending): the row of (t, e) is
  //      offset[e] + number of tokens below t that were also routed to e
  for (int item = tid; item < M * k; item += blockDim.x) {
    const int t = item / k;
    const int e = ws.assign_idx[item];
    int row = -1;
    if (e >= 0) {
      const uint32_t *cm = colmask + (size_t)e * mw;
      int below = __popc(cm[t >> 5] & ((1u << (t & 31)) - 1u));
      for (int w = 0; w < (t >> 5); ++w) below += __popc(cm[w]);
      row = s_offset[e] + below;
      ws.perm_row2tok[row] = t;
      ws.row2expert[row] = e;
    }
    ws.tokslot2row[item] = row;
  }
  ROUTE_MARK();

  // ---- phase F: tensor-core work units (expert, token chunk, 128-row slab): all gate/up units, then all
  //      down units, each group ordered by (expert, chunk, slab); ready counters and the dispenser start at 0
  const int n_chunks = s_unit_base[N];
  if (a.tiles_up > 0) {
    const int n_up = n_chunks * a.tiles_up;
    for (int i = tid; i < n_chunks; i += blockDim.x) ws.ready[i] = 0;
    if (tid == 0) *ws.unit_counter = 0;
    for (int i = warp; i < N; i += nwarps) {
      const int cnt = s_count[i];
      if (cnt == 0) continue;
      const int chunks = (cnt + kMaxTokChunk - 1) / kMaxTokChunk;
      for (int c = 0; c < chunks; ++c) {
        const int row0 = s_offset[i] + c * kMaxTokChunk;
        const int rows = min(kMaxTokChunk, cnt - c * kMaxTokChunk);
        const int ci = s_unit_base[i] + c;
        for (int tl = lane; tl < a.tiles_up; tl += 32)
          ws.units[(size_t)ci * a.tiles_up + tl] = Unit{i, tl, row0, rows, ci, 0, 0, 0};
        for (int tl = lane; tl < a.tiles_down; tl += 32)
          ws.units[(size_t)n_up + (size_t)ci * a.tiles_down + tl] = Unit{i, tl, row0, rows, ci, 1, 0, 0};
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
    for (int r = 0; r < s_nS; ++r) cov += s_score[s_Srank[r]];
    moespec_stats st;
    st.n_union = n_union;
    st.n_shortlist = s_nS;
    st.n_active = s_nactive;
    st.n_rows = R;
    st.n_dropped = M * k - R;
    st.status = 0;
    st.coverage = M > 0 ? cov / (double)M : 0.0;
    st.weight_bytes = (long long)s_nactive * a.expert_bytes;
    *ws.stats = st;
#ifdef MOESPEC_ROUTE_TIMING
    tmark[nmark++] = clock64();
    printf("route phases (cycles): A %lld B %lld C %lld D %lld E %lld F+stats %lld total %lld\n", tmark[1] - tmark[0],
           tmark[2] - tmark[1], tmark[3] - tmark[2], tmark[4] - tmark[3], tmark[5] - tmark[4], tmark[6] - tmark[5],
           tmark[6] - tmark[0]);
#endif
  }
#ifdef MOESPEC_ROUTE_TIMING
  __syncthreads();
  }
#endif
}

static cudaError_t launch_route_kernel(const LaunchCtx &c, const float *logits) {
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
  const int threads = 1024;
  const size_t smem = (size_t)(threads / 32) * a.N * sizeof(double) + (size_t)a.N * ((c.M + 31) / 32) * sizeof(uint32_t);
  if (smem > 40 * 1024) {
    cudaError_t e = cudaFuncSetAttribute(route_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
  }
  return launch_kernel(route_kernel, dim3(1), dim3(threads), smem, c.stream, a);
}

// Routing after router_topk_kernel has filled logits, prob and topk_idx.
cudaError_t launch_route_after_router(const LaunchCtx &c) { return launch_route_kernel(c, c.ws->logits); }

// Routing from caller-supplied logits: per-token softmax/top-k first (two launches).
cudaError_t launch_route(const LaunchCtx &c, const float *logits) {
  cudaError_t e = launch_kernel(softmax_topk_kernel, dim3((c.M + 3) / 4), dim3(128), 0, c.stream, logits, c.ws->prob,
                                c.ws->topk_idx, c.M, c.desc->n_experts, c.k);
  if (e != cudaSuccess) return e;
  return launch_route_kernel(c, logits);
}

// ---------------------------------------------------------------------------
// K3: gather routed rows: x_perm[r, :] = hidden[perm_row2tok[r], :].
// ---------------------------------------------------------------------------
__global__ void __launch_bounds__(128) gather_rows_kernel(const uint4 *__restrict__ hidden,
                                                          uint4 *__restrict__ x_perm,
                                                          const int *__restrict__ perm,
                                                          const int *__restrict__ counters, int row_vec) {
  const int r = blockIdx.x;
  pdl_trigger();
  pdl_wait();
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
  return launch_kernel(gather_rows_kernel, dim3(rows), dim3(128), 0, c.stream, (const uint4 *)hidden,
                       (uint4 *)c.ws->x_perm, (const int *)c.ws->perm_row2tok, (const int *)c.ws->counters, row_vec);
}

}  // namespace moespec
