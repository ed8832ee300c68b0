// Routing half of the layer: router projection (Eq. 1 numerator), softmax and
// natural top-k (Eq. 1, Eq. 2), union (Eq. 3), router-based scores (Eq. 5),
// top-B shortlist (Section 3.2), re-routing under substitution (Eq. 8) or
// truncation (Eq. 7) with the mixing weights of Section 3.3, and the
// per-expert gather order (Appendix C).
//
// Three launches:
//   router_topk_kernel   router dot products; the CTA that finishes a token
//                        tile's last logit also runs those tokens' softmax and
//                        top-k and adds their probabilities to the per-expert
//                        scores (a counter, never a wait).  router_mma_kernel is
//                        the same on the tensor cores, for larger trees.
//   route_kernel         eight tokens per CTA: every CTA ranks the scores itself
//                        (shortlist; CTA 0 publishes it for the FFN kernel),
//                        re-routes its tokens, and the CTA that finishes last
//                        does the scan, the gather order, the work-unit list and
//                        the statistics
//   gather_rows_kernel   x_perm[row] = hidden[token], for the rows that some work
//                        unit reads (rows_gather_kernel also works out the rows,
//                        for trees above 128 tokens)
// Scores are accumulated as 2^-52 fixed-point integers, so the sum does not
// depend on the order in which tokens arrive and identical experts tie exactly.
// A stand-alone softmax/top-k kernel serves callers that inject logits.
#include "internal.h"
#include <cstdlib>
#include <math_constants.h>

namespace moespec {

__device__ __forceinline__ float to_float(float v) { return v; }
__device__ __forceinline__ float to_float(__nv_bfloat16 v) { return __bfloat162float(v); }
__device__ __forceinline__ float to_float(__half v) { return __half2float(v); }

constexpr unsigned kFull = 0xffffffffu;
constexpr double kScoreScale = 4503599627370496.0;   // 2^52: scores are sums of round(p * 2^52)
constexpr unsigned long long kScoreOneMinus = (1ull << 52) - 1ull;
constexpr int kNone = 0x7fffffff;

// Monotone map float -> uint32 (larger float, larger key); -0 and +0 share a key.
__device__ __forceinline__ uint32_t order_key(float f) {
  if (f == 0.f) f = 0.f;
  const uint32_t u = __float_as_uint(f);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

// Arrival at a counter by one thread after a CTA barrier: releases the stores of every thread of the CTA that
// came before the barrier, and acquires those released by the CTAs that arrived earlier.
__device__ __forceinline__ int arrive_acq_rel(int *counter) {
  int prev;
  asm volatile("atom.acq_rel.gpu.global.add.s32 %0, [%1], 1;" : "=r"(prev) : "l"(counter) : "memory");
  return prev;
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

// Softmax of one token by one warp (Eq. 1, fp64); adds the probabilities to the per-expert scores (Eq. 5).
template <int W>
__device__ __forceinline__ void token_softmax(const float *zrow, int N, double *prob_row, unsigned long long *score_fx,
                                              int lane) {
  float v[W];
  uint32_t valid = 0;
  float mx = -CUDART_INF_F;
#pragma unroll
  for (int s = 0; s < W; ++s) {
    const int idx = lane + 32 * s;
    v[s] = -CUDART_INF_F;
    if (idx < N) {
      v[s] = __ldcg(zrow + idx);          // written by other CTAs of this launch: read through L2
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
    if ((valid >> s) & 1u) {
      const double p = e[s] / sum;
      prob_row[lane + 32 * s] = p;
      // p == 1 exactly is clamped one unit below 2^52, so that max_M = 4096 such tokens cannot wrap the sum
      atomicAdd(score_fx + lane + 32 * s, min((unsigned long long)__double2ull_rn(p * kScoreScale), kScoreOneMinus));
    }
}

// Natural top-k of one token by one warp (Eq. 2); counts the token towards its experts (Eq. 3).
template <int W>
__device__ __forceinline__ void token_topk(const float *zrow, int N, int k, int *topk_row, int *natcnt, int lane) {
  uint32_t key[W];
  uint32_t valid = 0;
#pragma unroll
  for (int s = 0; s < W; ++s) {
    const int idx = lane + 32 * s;
    key[s] = 0;
    if (idx < N) {
      key[s] = order_key(__ldcg(zrow + idx));
      valid |= 1u << s;
    }
  }
  const int mine = warp_take_best<W>(key, valid, k, lane);
  if (lane < k) {
    topk_row[lane] = mine;
    if (mine >= 0) atomicAdd(natcnt + mine, 1);
  }
}

// which: bit 0 = softmax, bit 1 = top-k
__device__ __forceinline__ void token_phase(const float *zrow, int N, int k, double *prob_row, int *topk_row,
                                            unsigned long long *score_fx, int *natcnt, int lane, int which = 3) {
  if (N <= 32) {
    if (which & 1) token_softmax<1>(zrow, N, prob_row, score_fx, lane);
    if (which & 2) token_topk<1>(zrow, N, k, topk_row, natcnt, lane);
  } else if (N <= 64) {
    if (which & 1) token_softmax<2>(zrow, N, prob_row, score_fx, lane);
    if (which & 2) token_topk<2>(zrow, N, k, topk_row, natcnt, lane);
  } else if (N <= 128) {
    if (which & 1) token_softmax<4>(zrow, N, prob_row, score_fx, lane);
    if (which & 2) token_topk<4>(zrow, N, k, topk_row, natcnt, lane);
  } else {
    if (which & 1) token_softmax<8>(zrow, N, prob_row, score_fx, lane);
    if (which & 2) token_topk<8>(zrow, N, k, topk_row, natcnt, lane);
  }
}

// Large trees leave the rows of the gather order to the row kernel (one CTA per (token, slot) pair) instead
// of the routing kernel's last CTA, which would walk them alone.  Small trees keep them in that CTA: it is
// faster there, and nothing waits for it.
static bool rows_in_row_kernel(int M) { return M > kMaxTokChunk; }

// In that mode the expert x token bit matrix outlives the routing kernel; the first kernel of the next call
// clears it (every CTA takes a slice): its last readers, the row kernel's CTAs, have long finished by then.
__device__ __forceinline__ void clear_colmask(unsigned *colmask, int words) {
  const int cta = blockIdx.y * gridDim.x + blockIdx.x, n_cta = gridDim.x * gridDim.y;
  for (int i = cta * blockDim.x + threadIdx.x; i < words; i += n_cta * blockDim.x) colmask[i] = 0u;
}

// The FFN kernel's control words must be in their initial state when its first CTA starts: the shortlist words
// at 0 (the routing kernel publishes the call's shortlist later; the FFN kernel's CTAs poll them), its unit
// dispenser and its down-unit counter at 0.  The router kernel's first CTA sets them: it runs after the
// previous call's FFN kernel has completed (it has just waited for that) and completes before this call's FFN
// kernel can start -- except with a fixed shortlist, where the FFN kernel is released right behind this kernel's
// CTAs: there the stores are performed (fence) before this CTA releases the dependents.
__device__ __forceinline__ void reset_ffn_control(int *early_flag, int n_words, int *unit_counter, int fence_reset) {
  if (!early_flag || blockIdx.x != 0 || blockIdx.y != 0) return;
  for (int i = threadIdx.x; i < n_words; i += blockDim.x) early_flag[i] = 0;
  if (threadIdx.x == 0) {
    unit_counter[0] = 0;
    unit_counter[1] = 0;
  }
  if (fence_reset) {
    __threadfence();
    __syncthreads();
  }
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
                                                          double *prob, int *topk_idx, unsigned long long *score_fx,
                                                          int *natcnt, int *arrive, int *early_flag,
                                                          int *unit_counter, int fence_reset,
                                                          unsigned *colmask, int M, int N, int d, int k) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int t0 = blockIdx.y * TT;
  const int i = blockIdx.x * 8 + warp;
  __shared__ int s_last;
  constexpr int VEC = 16 / sizeof(T);
  constexpr int U = 8;
  // The router matrix is a constant of the layer: the first pass over this warp's row (the whole row for
  // d <= 32*VEC*U) is fetched while the previous kernel in the stream is still running.
  uint4 rw[U];
  if (i < N) {
#pragma unroll
    for (int u = 0; u < U; ++u)
      if ((lane + u * 32) * VEC < d) rw[u] = *reinterpret_cast<const uint4 *>(Wr + (size_t)i * d + (lane + u * 32) * VEC);
  }
  pdl_wait();          // hidden may be the previous layer's output; the workspace is still in use until then
  reset_ffn_control(early_flag, N, unit_counter, fence_reset);
  // Dependents are released only now: with a fixed shortlist the FFN kernel of this call starts at once,
  // and it reads `hidden`, which the previous kernel in the stream may have produced.
  pdl_trigger();
  clear_colmask(colmask, N * ((M + 31) >> 5));
  if (i < N) {
    const T *w = Wr + (size_t)i * d;
    float acc[TT];
#pragma unroll
    for (int tt = 0; tt < TT; ++tt) acc[tt] = 0.f;
    for (int j0 = lane * VEC; j0 < d; j0 += 32 * VEC * U) {
      if (j0 != lane * VEC) {
#pragma unroll
        for (int u = 0; u < U; ++u)
          if (j0 + u * 32 * VEC < d) rw[u] = *reinterpret_cast<const uint4 *>(w + j0 + u * 32 * VEC);
      }
      // two tokens per pass: their loads are all issued before the first FMA
#pragma unroll
      for (int tt = 0; tt < TT; tt += 2) {
        uint4 rh[2][U];
#pragma unroll
        for (int q = 0; q < 2; ++q) {
          const int tq = min(t0 + tt + q, M - 1);           // clamp: out-of-range tokens repeat the last row
          const T *h = hidden + (size_t)tq * d;
#pragma unroll
          for (int u = 0; u < U; ++u)
            if (j0 + u * 32 * VEC < d) rh[q][u] = *reinterpret_cast<const uint4 *>(h + j0 + u * 32 * VEC);
        }
#pragma unroll
        for (int q = 0; q < 2; ++q) {
#pragma unroll
          for (int u = 0; u < U; ++u) {
            if (j0 + u * 32 * VEC < d) {
              const T *ew = reinterpret_cast<const T *>(&rw[u]);
              const T *eh = reinterpret_cast<const T *>(&rh[q][u]);
#pragma unroll
              for (int v = 0; v < VEC; ++v) acc[tt + q] = fmaf(to_float(ew[v]), to_float(eh[v]), acc[tt + q]);
            }
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
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    const int prev = arrive_acq_rel(&arrive[blockIdx.y]);
    s_last = (prev == (int)gridDim.x - 1);
    if (s_last) arrive[blockIdx.y] = 0;
  }
  __syncthreads();
  if (s_last) {
    // softmax and top-k are independent chains: with up to four tokens they run on different warps
    const bool split = 2 * TT <= 8;
    const int tt = split ? (warp % TT) : warp;
    const int which = split ? (warp < TT ? 1 : 2) : 3;
    const int t = t0 + tt;
    if (tt < TT && (split ? warp < 2 * TT : true) && t < M)
      token_phase(logits + (size_t)t * N, N, k, prob + (size_t)t * N, topk_idx + (size_t)t * k, score_fx, natcnt, lane,
                  which);
  }
}

// ---------------------------------------------------------------------------
// K1 for larger trees: the same logits, softmax and top-k, with the dot products on the tensor cores.
// A CTA takes 16 experts x 8 tokens; its NW (sixteen, or eight) warps split K, each running m16n8k16 MMAs (experts on the
// M axis, tokens on the N axis) on operands loaded straight from global memory: thread (g, tg) of a warp
// reads 16 contiguous bytes of router rows g and g+8 and of token row g at K offset 32*step + 8*tg and
// feeds them to two MMAs.  That assigns memory positions to the instruction's k slots in a permuted
// order, which is immaterial for a dot product as long as both operands use the same one.  The warps'
// partial tiles meet in shared memory and are added in warp order (a fixed order: logits are
// reproducible), then the kernel ends like router_topk_kernel: arrival counter per token tile, softmax
// and top-k by the CTA that completes the tile (with sixteen warps the two run on separate warps per token).
// The CUDA-core kernel above spends its time converting and multiplying element by element, which is what
// limits it beyond ~64 tokens.
// ---------------------------------------------------------------------------
__device__ __forceinline__ void mma_16816(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                          uint32_t b1, __nv_bfloat16) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
               : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
               : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void mma_16816(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                          uint32_t b1, __half) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
               : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
               : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

constexpr int kRmExperts = 16, kRmTokens = 8, kRmSteps = 8;     // tile of a CTA; 32-element K steps per batch

template <typename T, int NW>
__global__ void __launch_bounds__(NW * 32) router_mma_kernel(const T *__restrict__ hidden, const T *__restrict__ Wr,
                                                         const float *__restrict__ bias, float *logits, double *prob,
                                                         int *topk_idx, unsigned long long *score_fx, int *natcnt,
                                                         int *arrive, int *early_flag, int *unit_counter,
                                                         int fence_reset, unsigned *colmask, int M, int N, int d,
                                                         int k) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int g = lane >> 2, tg = lane & 3;
  const int e0 = blockIdx.x * kRmExperts, t0 = blockIdx.y * kRmTokens;
  __shared__ float s_part[NW][kRmExperts * kRmTokens];
  __shared__ int s_last;
  const int kw = d / NW;                                  // K range of this warp: [warp*kw, warp*kw + kw)
  const int ra = min(e0 + g, N - 1), rb = min(e0 + g + 8, N - 1);      // clamped: rows beyond N are never stored
  const T *wa = Wr + (size_t)ra * d + warp * kw + tg * 8;
  const T *wb = Wr + (size_t)rb * d + warp * kw + tg * 8;
  // the router matrix is a constant of the layer: the first batch of its rows is fetched before the wait
  uint4 A0[kRmSteps], A1[kRmSteps];
#pragma unroll
  for (int s = 0; s < kRmSteps; ++s) {
    if (s * 32 < kw) {
      A0[s] = *reinterpret_cast<const uint4 *>(wa + s * 32);
      A1[s] = *reinterpret_cast<const uint4 *>(wb + s * 32);
    }
  }
  pdl_wait();          // hidden may be the previous layer's output; the workspace is still in use until then
  reset_ffn_control(early_flag, N, unit_counter, fence_reset);
  pdl_trigger();       // released only now: see router_topk_kernel
  clear_colmask(colmask, N * ((M + 31) >> 5));
  const T *hb = hidden + (size_t)min(t0 + g, M - 1) * d + warp * kw + tg * 8;
  float c[4] = {0.f, 0.f, 0.f, 0.f};
  for (int k0 = 0; k0 < kw; k0 += 32 * kRmSteps) {
    uint4 Bv[kRmSteps];
#pragma unroll
    for (int s = 0; s < kRmSteps; ++s) {
      if (k0 + s * 32 < kw) {
        Bv[s] = *reinterpret_cast<const uint4 *>(hb + k0 + s * 32);
        if (k0 > 0) {
          A0[s] = *reinterpret_cast<const uint4 *>(wa + k0 + s * 32);
          A1[s] = *reinterpret_cast<const uint4 *>(wb + k0 + s * 32);
        }
      }
    }
#pragma unroll
    for (int s = 0; s < kRmSteps; ++s) {
      if (k0 + s * 32 < kw) {
        mma_16816(c, A0[s].x, A1[s].x, A0[s].y, A1[s].y, Bv[s].x, Bv[s].y, T());
        mma_16816(c, A0[s].z, A1[s].z, A0[s].w, A1[s].w, Bv[s].z, Bv[s].w, T());
      }
    }
  }
  // accumulator layout: c0,c1 = (expert g, tokens 2tg, 2tg+1); c2,c3 = (expert g+8, same tokens)
  s_part[warp][g * kRmTokens + 2 * tg] = c[0];
  s_part[warp][g * kRmTokens + 2 * tg + 1] = c[1];
  s_part[warp][(g + 8) * kRmTokens + 2 * tg] = c[2];
  s_part[warp][(g + 8) * kRmTokens + 2 * tg + 1] = c[3];
  __syncthreads();
  if (threadIdx.x < kRmExperts * kRmTokens) {
    const int el = threadIdx.x / kRmTokens, tl = threadIdx.x % kRmTokens;
    float acc = 0.f;
#pragma unroll
    for (int w = 0; w < NW; ++w) acc += s_part[w][threadIdx.x];
    if (e0 + el < N && t0 + tl < M) logits[(size_t)(t0 + tl) * N + e0 + el] = acc + (bias ? bias[e0 + el] : 0.f);
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    const int prev = arrive_acq_rel(&arrive[blockIdx.y]);
    s_last = (prev == (int)gridDim.x - 1);
    if (s_last) arrive[blockIdx.y] = 0;
  }
  __syncthreads();
  if (s_last) {
    // eight tokens: one warp each, or with sixteen warps softmax and top-k of a token on two warps
    const int t = t0 + (warp & 7);
    const int which = NW == 16 ? (warp < 8 ? 1 : 2) : 3;
    if (t < M && warp < 16)
      token_phase(logits + (size_t)t * N, N, k, prob + (size_t)t * N, topk_idx + (size_t)t * k, score_fx, natcnt, lane,
                  which);
  }
}

template <typename T, int NW = 8>
static cudaError_t launch_router_mma(const LaunchCtx &c, const void *hidden) {
  const moespec_layer_desc &D = *c.desc;
  const Workspace &ws = *c.ws;
  const dim3 grid((D.n_experts + kRmExperts - 1) / kRmExperts, (c.M + kRmTokens - 1) / kRmTokens);
  return launch_kernel(router_mma_kernel<T, NW>, grid, dim3(NW * 32), 0, c.stream, (const T *)hidden, (const T *)D.router_w,
                       D.router_bias, ws.logits, ws.prob, ws.topk_idx, ws.score_fx, ws.natcnt_acc, ws.arrive,
                       ws.early_flag, ws.unit_counter, D.shortlist == MOESPEC_STATIC ? 1 : 0, ws.colmask, c.M, D.n_experts,
                       D.d, c.k);
}
template <>
cudaError_t launch_router_mma<float, 8>(const LaunchCtx &, const void *) { return cudaErrorNotSupported; }
template <>
cudaError_t launch_router_mma<float, 16>(const LaunchCtx &, const void *) { return cudaErrorNotSupported; }

// Trees beyond 64 tokens of a 16-bit layer take the tensor-core router (d must split into eight K ranges of
// whole 32-element steps).
static bool use_router_mma(const LaunchCtx &c) {
  static const bool off = [] { const char *v = experiment_env("MOESPEC_NO_ROUTER_MMA"); return v && v[0] == '1'; }();
  static const int min_m = [] { const char *v = experiment_env("MOESPEC_ROUTER_MMA_MIN_M"); return v ? atoi(v) : 65; }();
  // (also for wide routers: with N >= 128 the tensor-core kernel wins at every tree size measured)
  return !off && is_16bit(c.desc->dtype) && (c.M >= min_m || c.desc->n_experts >= 128) && c.desc->d % 256 == 0;
}

template <typename T>
static cudaError_t launch_router_t(const LaunchCtx &c, const void *hidden) {
  // sixteen warps per CTA where K splits sixteen ways into whole 32-element steps: the eight tokens of a tile
  // then get their softmax and their top-k on separate warps (2.5 µs per layer less than eight warps at
  // 65 to 255 tokens and for 128 experts)
  if (use_router_mma(c))
    return c.desc->d % 512 == 0 ? launch_router_mma<T, 16>(c, hidden) : launch_router_mma<T, 8>(c, hidden);
  const moespec_layer_desc &D = *c.desc;
  const Workspace &ws = *c.ws;
  const int ex_tiles = (D.n_experts + 7) / 8;
  // With a fixed shortlist the FFN kernel streams while this kernel runs, but its CTAs only fit beside ONE
  // router CTA per SM (registers): more tokens per CTA keep the grid within the SM count.
  int min_tt = 2;
  if (c.early && D.shortlist == MOESPEC_STATIC) {
    const int sms = tc_grid_size(D.device);
    while (min_tt < 8 && ex_tiles * ((c.M + min_tt - 1) / min_tt) > sms) min_tt *= 2;
  }
  if (c.M <= 64 && min_tt <= 2)
    return launch_kernel(router_topk_kernel<T, 2>, dim3(ex_tiles, (c.M + 1) / 2), dim3(256), 0, c.stream,
                         (const T *)hidden, (const T *)D.router_w, D.router_bias, ws.logits, ws.prob, ws.topk_idx,
                         ws.score_fx, ws.natcnt_acc, ws.arrive, ws.early_flag, ws.unit_counter, D.shortlist == MOESPEC_STATIC ? 1 : 0,
                         ws.colmask, c.M, D.n_experts, D.d, c.k);
  if (c.M <= 128 && min_tt <= 4)
    return launch_kernel(router_topk_kernel<T, 4>, dim3(ex_tiles, (c.M + 3) / 4), dim3(256), 0, c.stream,
                         (const T *)hidden, (const T *)D.router_w, D.router_bias, ws.logits, ws.prob, ws.topk_idx,
                         ws.score_fx, ws.natcnt_acc, ws.arrive, ws.early_flag, ws.unit_counter, D.shortlist == MOESPEC_STATIC ? 1 : 0,
                         ws.colmask, c.M, D.n_experts, D.d, c.k);
  return launch_kernel(router_topk_kernel<T, 8>, dim3(ex_tiles, (c.M + 7) / 8), dim3(256), 0, c.stream,
                       (const T *)hidden, (const T *)D.router_w, D.router_bias, ws.logits, ws.prob, ws.topk_idx,
                       ws.score_fx, ws.natcnt_acc, ws.arrive, ws.early_flag, ws.unit_counter, D.shortlist == MOESPEC_STATIC ? 1 : 0,
                         ws.colmask, c.M, D.n_experts, D.d, c.k);
}

cudaError_t launch_router_logits(const LaunchCtx &c, const void *hidden) {
  if (c.desc->dtype == MOESPEC_BF16) return launch_router_t<__nv_bfloat16>(c, hidden);
  if (c.desc->dtype == MOESPEC_FP16) return launch_router_t<__half>(c, hidden);
  return launch_router_t<float>(c, hidden);
}

// Softmax and top-k from caller-supplied logits: one warp per token.
__global__ void __launch_bounds__(128) softmax_topk_kernel(const float *logits, double *prob, int *topk_idx,
                                                           unsigned long long *score_fx, int *natcnt, int *early_flag,
                                                           unsigned *colmask, int M, int N, int k) {
  const int t = blockIdx.x * 4 + (threadIdx.x >> 5);
  pdl_trigger();
  pdl_wait();
  if (early_flag && blockIdx.x == 0)
    for (int i = threadIdx.x; i < N; i += blockDim.x) early_flag[i] = 0;
  clear_colmask(colmask, N * ((M + 31) >> 5));
  if (t < M)
    token_phase(logits + (size_t)t * N, N, k, prob + (size_t)t * N, topk_idx + (size_t)t * k, score_fx, natcnt,
                threadIdx.x & 31);
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
  int tiles_up, tiles_down;     // f/RU, d/RU slabs per expert (0 when the tensor-core path is not used)
  long long expert_bytes;       // 3*d*f*sizeof(dtype)
  int early;                    // the FFN kernel starts on the shortlist before this kernel has finished
  int ffn_ctas;                 // CTAs of the FFN kernel: CTA c starts on gate/up unit c of the list
  int rows_later;               // the row of every (token, slot) pair is left to the row kernel (large trees)
  int res_first, res_count;     // experts resident on this GPU (expert-parallel shard); res_count = N: all
  int dense_all;                // gate/up units are marked "all tokens from hidden" (trees of at most 16 tokens)
};

constexpr int kRouteWarps = 8;      // tokens per CTA of route_kernel
constexpr int kColmaskCache = 1024; // words of the expert x token bit matrix the last CTA keeps in shared memory

// Probability of expert `idx` from the row a warp holds in registers (lane l owns experts l, l+32, ...).
template <int W>
__device__ __forceinline__ double row_value(const double (&p)[W], int idx) {
  const int slot = idx >> 5;
  double mine = 0.0;
#pragma unroll
  for (int s = 0; s < W; ++s) {
    const double v = shfl_double(p[s], idx & 31);   // every lane names its own source lane
    if (s == slot) mine = v;
  }
  return mine;
}

// Re-routing of one token (Eq. 7 / Eq. 8) with its mixing weights (Section 3.3); lane r owns slot r.
// key[] / p[] are the token's logit keys and probabilities, valid says which slots exist.
template <int W>
__device__ __forceinline__ void token_reroute(const RouteArgs &a, int t, int nS, const uint32_t *s_Smask,
                                              const uint32_t (&key)[W], const double (&p)[W], int nat, int lane) {
  const Workspace &ws = a.ws;
  const int k = a.k;
  const bool nat_kept = nat >= 0 && ((s_Smask[nat >> 5] >> (nat & 31)) & 1u);
  int mine = -1;        // kept expert of slot `lane`
  int base = -1;        // expert whose probability enters the renormalisation sum at position `lane`
  if (a.policy == MOESPEC_SUBSTITUTION) {
    // The surviving natural experts outrank every other member of S (they are the global top-k), so
    // top-k within S = survivors in their order, then the best of S \ T_k for the slots that are left.
    const uint32_t surv = __ballot_sync(kFull, nat_kept);
    const int n_surv = __popc(surv);
    const int want = min(k, nS);
    const unsigned src = __fns(surv, 0, lane + 1);            // lane of the (lane+1)-th survivor
    const int from_nat = __shfl_sync(kFull, nat, src < 32u ? (int)src : 0);
    if (lane < n_surv) mine = from_nat;
    if (n_surv < want) {
      // candidates: members of S that are not in the natural top-k
      uint32_t valid = 0;
#pragma unroll
      for (int s = 0; s < W; ++s)
        if ((s_Smask[s] >> lane) & 1u) valid |= 1u << s;
      for (int r = 0; r < k; ++r) {
        const int e = __shfl_sync(kFull, nat, r);
        if (e >= 0 && (e & 31) == lane) valid &= ~(1u << (e >> 5));
      }
      const int sub = warp_take_best<W>(key, valid, want - n_surv, lane);
      const int shifted = __shfl_sync(kFull, sub, (lane - n_surv) & 31);
      if (lane >= n_surv && lane < want) mine = shifted;
    }
    base = mine;                                   // weights over the constrained selection
  } else {
    mine = nat_kept ? nat : -1;
    base = nat;                                    // weights over the original top-k set
  }
  const double p_mine = row_value<W>(p, mine >= 0 ? mine : 0);
  double p_base = p_mine;
  if (a.policy != MOESPEC_SUBSTITUTION) p_base = row_value<W>(p, base >= 0 ? base : 0);   // warp-uniform branch
  double denom = 1.0;
  if (a.renormalize) {
    denom = (lane < k && base >= 0) ? p_base : 0.0;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) denom += shfl_xor_double(denom, o);
  }
  if (lane < k) {
    ws.assign_idx[(size_t)t * k + lane] = mine;
    ws.gate_w[(size_t)t * k + lane] = mine >= 0 ? (float)(p_mine / denom) : 0.f;
    if (mine >= 0) {
      atomicAdd(ws.count_acc + mine, 1);
      atomicOr(ws.colmask + (size_t)mine * ((a.M + 31) >> 5) + (t >> 5), 1u << (t & 31));
    }
  }
}

template <int W>
__device__ __forceinline__ void route_token(const RouteArgs &a, int t, int nS, const uint32_t *s_Smask,
                                            const uint32_t (&key)[W], const double (&p)[W], int nat, int lane) {
  token_reroute<W>(a, t, nS, s_Smask, key, p, nat, lane);
}

// ---------------------------------------------------------------------------
// K2: shortlist, re-routing and gather order.  Grid ceil(M/8), 256 threads: one
// warp per token.  Every CTA ranks the N scores itself (rank by counting under
// (score descending, index ascending)), which costs less than a grid-wide
// exchange.  Tokens add their kept experts to global counters and bit masks;
// the CTA that arrives last turns them into offsets, rows and work units and
// clears the accumulators for the next call.
// ---------------------------------------------------------------------------
template <int W>
__global__ void __launch_bounds__(kRouteWarps * 32) route_kernel(RouteArgs a) {
  __shared__ unsigned long long s_score[kMaxExperts];     // ranking key (score + 1, or 0 for a non-candidate)
  __shared__ unsigned long long s_fx[kMaxExperts];        // fixed-point score
  __shared__ unsigned s_colmask[kColmaskCache];
  __shared__ int s_cand[kMaxExperts];
  __shared__ int s_count[kMaxExperts];
  __shared__ int s_offset[kMaxExperts + 1];
  __shared__ int s_unit_base[kMaxExperts + 1];
  __shared__ int s_Srank[kMaxExperts];
  __shared__ uint32_t s_Smask[kMaskWords];
  __shared__ unsigned long long s_warp_tot[kRouteWarps];
  __shared__ int s_chunk_expert[kMaxExperts * 2];     // token chunk -> expert (first 2N chunks; more fall back)
  __shared__ int s_nactive, s_last, s_nchunks;
  __shared__ unsigned char s_all_dense[kMaxExperts];   // expert whose gate/up units all take every token from hidden

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int M = a.M, N = a.N, k = a.k;
  const int mw = (a.M + 31) >> 5;     // words per expert row of the bit matrix in this call
  const Workspace &ws = a.ws;
  const int t = blockIdx.x * kRouteWarps + warp;

  // With a router-based shortlist dependents are released only after the router kernel has completed:
  // the FFN kernel may then start while this kernel runs, and must find the shortlist flag already reset
  // by the router kernel.  With a fixed shortlist (Eq. 4) the FFN kernel needs nothing from the router to
  // begin streaming, so it is released at once.
  if (a.early && a.shortlist == MOESPEC_STATIC) {
    pdl_trigger();
    pdl_wait();
  } else {
    pdl_wait();
    pdl_trigger();
  }

  // ---- this warp's token: logit keys, probabilities, natural top-k (all loads issued up front)
  uint32_t key[W];
  double p[W];
  int nat = -1;
#pragma unroll
  for (int s = 0; s < W; ++s) {
    const int idx = lane + 32 * s;
    key[s] = 0;
    p[s] = 0.0;
    if (t < M && idx < N) {
      key[s] = order_key(a.logits[(size_t)t * N + idx]);
      p[s] = ws.prob[(size_t)t * N + idx];
    }
  }
  if (t < M && lane < k) nat = ws.topk_idx[(size_t)t * k + lane];

  // ---- scores (Eq. 5), union (Eq. 3), top-B shortlist
  int in_union = 0;
  if (tid < N) {
    const unsigned long long fx = __ldcg(ws.score_fx + tid);
    in_union = __ldcg(ws.natcnt_acc + tid) > 0;
    s_cand[tid] = (a.shortlist == MOESPEC_FROM_UNION) ? in_union : 1;
    s_score[tid] = s_cand[tid] ? fx + 1ull : 0ull;        // ranking key: candidates first, then by score
    s_fx[tid] = fx;
  }
  const int n_union = __syncthreads_count(in_union);
  const int n_cand = __syncthreads_count(tid < N && s_cand[tid]);
  const bool fixed = a.shortlist == MOESPEC_STATIC;
  const int nS = fixed ? min(a.B, ws.n_static) : min(a.B, n_cand);
  if (fixed) {
    // static ranking (Eq. 4): the shortlist is the first nS experts of the fixed ordering
    bool in_S = false;
    if (tid < N) {
      const int pos = ws.static_pos[tid];
      in_S = pos < nS;
      if (in_S) {
        s_Srank[pos] = tid;
        if (blockIdx.x == 0) ws.S_rank[pos] = tid;
      }
    }
    const unsigned word = __ballot_sync(kFull, in_S);
    if (lane == 0) s_Smask[warp] = word;
  } else {
    // one thread per expert; every thread walks the same j, so the shared-memory reads are broadcasts
    // Branch-free rank by counting.  s_score holds score+1 for candidates and 0 for the others, so a
    // non-candidate never outranks a candidate.
    bool in_S = false;
    if (tid < N) {
      const unsigned long long si = s_score[tid];
      int rank = 0;
#pragma unroll 16
      for (int j = 0; j < N; ++j) {
        const unsigned long long sj = s_score[j];
        rank += (int)((sj > si) | ((sj == si) & (j < tid)));
      }
      in_S = si != 0ull && rank < nS;
      if (in_S) {
        s_Srank[rank] = tid;
        if (blockIdx.x == 0) ws.S_rank[rank] = tid;
      }
    }
    const unsigned word = __ballot_sync(kFull, in_S);     // thread index = expert index: warp w owns mask word w
    if (lane == 0) s_Smask[warp] = word;
  }
  __syncthreads();
  // What the FFN kernel works on is the part of the shortlist that is resident on this GPU, in rank order
  // (all of it unless this layer is an expert-parallel shard): s_Srank / nS_l from here on.  The shortlist
  // itself stays in s_Smask (re-routing) and in ws.S_rank.
  const bool shard = a.res_count < N;
  int nS_l = nS;
  if (shard) {
    int e_r = 0;
    bool res = false;
    if (tid < nS) {
      e_r = s_Srank[tid];
      res = e_r >= a.res_first && e_r < a.res_first + a.res_count;
    }
    const unsigned bal = __ballot_sync(kFull, res);
    if (lane == 0) s_warp_tot[warp] = (unsigned long long)__popc(bal);
    __syncthreads();                         // every thread has read its entry of s_Srank
    int pos = __popc(bal & ((1u << lane) - 1u));
    for (int w = 0; w < warp; ++w) pos += (int)s_warp_tot[w];
    nS_l = 0;
    for (int w = 0; w < kRouteWarps; ++w) nS_l += (int)s_warp_tot[w];
    if (res) s_Srank[pos] = e_r;
    __syncthreads();
  }
  // publish the shortlist: the FFN kernel's CTAs start streaming the weights of its best-ranked experts while
  // the rest of the routing runs.  One word per rank (the expert, plus one; -1 beyond the last one): a CTA
  // polls the word of the rank it starts on and needs nothing else, so each word is its own payload and a
  // relaxed store suffices.
  if (blockIdx.x == 0 && ws.early_flag && tid < N)
    asm volatile("st.relaxed.gpu.global.s32 [%0], %1;" ::"l"(ws.early_flag + tid), "r"(tid < nS_l ? s_Srank[tid] + 1 : -1)
                 : "memory");

  // ---- re-routing (Eq. 7 / Eq. 8) and mixing weights (Section 3.3) of this warp's token
  if (t < M) route_token<W>(a, t, nS, s_Smask, key, p, nat, lane);

  // ---- the CTA that arrives last finishes the call
  __syncthreads();
  if (tid == 0) {
    const int prev = arrive_acq_rel(ws.arrive_route);
    s_last = (prev == (int)gridDim.x - 1);
  }
  __syncthreads();
  if (!s_last) return;
  if (tid < N) s_all_dense[tid] = 0;      // (set below, behind a barrier, for trees with early start)

  // rows per expert and exclusive scans of rows, token chunks and active experts (Appendix C gather)
  const int used_words = (M + 31) >> 5;
  const bool cm_cached = N * used_words <= kColmaskCache;
  {
    const int c = tid < N ? __ldcg(ws.count_acc + tid) : 0;
    if (cm_cached)
      for (int i = tid; i < N * used_words; i += blockDim.x) s_colmask[i] = __ldcg(ws.colmask + i);
    // work units and the active count cover the resident experts only; rows and offsets cover all
    const bool resident = tid >= a.res_first && tid < a.res_first + a.res_count;
    const int chunks = resident ? (c + kMaxTokChunk - 1) / kMaxTokChunk : 0;
    // rows in bits 0..23, chunks in bits 24..43, active flag in bits 44..
    const unsigned long long v = (unsigned long long)c | ((unsigned long long)chunks << 24) |
                                 ((unsigned long long)(c > 0 && resident) << 44);
    unsigned long long inc = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const unsigned long long up = __shfl_up_sync(kFull, inc, o);
      if (lane >= o) inc += up;
    }
    if (lane == 31) s_warp_tot[warp] = inc;
    __syncthreads();
    unsigned long long pre = inc - v;
    for (int w = 0; w < warp; ++w) pre += s_warp_tot[w];
    if (tid < N) {
      const int row0 = (int)(pre & 0xFFFFFFull), ub = (int)((pre >> 24) & 0xFFFFFull), ai = (int)(pre >> 44);
      s_count[tid] = c;
      s_offset[tid] = row0;
      s_unit_base[tid] = ub;
      s_cand[tid] = chunks;                // (the candidate flags are no longer needed: token chunks per expert)
      ws.count[tid] = c;
      ws.offset[tid] = row0;
      ws.score[tid] = (double)s_fx[tid] * (1.0 / kScoreScale);
      if (c > 0 && resident) ws.active[ai] = tid;
      for (int cc = 0; cc < chunks && ub + cc < 2 * kMaxExperts; ++cc) s_chunk_expert[ub + cc] = tid;
      if (tid == N - 1) {
        s_offset[N] = row0 + c;
        ws.offset[N] = row0 + c;
        s_unit_base[N] = ub + chunks;
        s_nchunks = ub + chunks;
        s_nactive = ai + (c > 0 && resident);
      }
    }
  }
  __syncthreads();
  if (a.early) {
    // Early start (M <= 128, so an expert has at most one token chunk): the unit list follows the
    // shortlist's rank order, and the experts whose gate/up units the FFN kernel's CTAs start on before
    // this list exists (CTA c takes unit c) keep their place even if no token was routed to them.
    // The gate/up units that CTAs may start on early (the first `ffn_ctas` of the list) are marked as taking
    // all tokens from `hidden`, whoever draws them and when; an expert all of whose gate/up units are among
    // them has no reader for its rows of the gathered copy, and they are not made.
    const int n_head = min((a.ffn_ctas + a.tiles_up - 1) / a.tiles_up, nS_l);
    bool present = false;
    int e_r = 0;
    if (tid < nS_l) {
      e_r = s_Srank[tid];
      present = s_count[e_r] > 0 || tid < n_head;
      if ((tid + 1) * a.tiles_up <= a.ffn_ctas) s_all_dense[e_r] = 1;
    }
    const unsigned bal = __ballot_sync(kFull, present);
    if (lane == 0) s_warp_tot[warp] = (unsigned long long)__popc(bal);
    __syncthreads();
    int pos = __popc(bal & ((1u << lane) - 1u));
    for (int w = 0; w < warp; ++w) pos += (int)s_warp_tot[w];
    if (present) {
      s_unit_base[e_r] = pos;
      s_chunk_expert[pos] = e_r;
    }
    if (tid == 0) {
      int tot = 0;
      for (int w = 0; w < kRouteWarps; ++w) tot += (int)s_warp_tot[w];
      s_nchunks = tot;
    }
    __syncthreads();
  } else if (a.tiles_up > 0 && M <= 2 * kMaxTokChunk) {
    // Trees of up to 256 tokens without early start: the listed experts in the shortlist's rank order too, each
    // with its one or two token chunks.  Rank order is roughly row-count order, so the units that take longest
    // (two full chunks, whose slabs are read twice) are handed out first and the list ends with cheap ones; in
    // expert-index order whatever expert came last decided how long the CTAs waited for the last of them
    // (-1 to -3 us at 129 to 255 tokens).  Larger trees keep the index order of the scan above: with three and
    // more chunks per popular expert, rank order bunches the units that live on L2 re-reads at the start of
    // the list, and the stream is slower there than with heavy and light experts interleaved (+2 % at 511
    // tokens, unbudgeted).
    int e_r = 0, ch = 0;
    if (tid < nS_l) {
      e_r = s_Srank[tid];
      ch = s_cand[e_r];
    }
    int inc = ch;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int up = __shfl_up_sync(kFull, inc, o);
      if (lane >= o) inc += up;
    }
    if (lane == 31) s_warp_tot[warp] = (unsigned long long)inc;
    __syncthreads();                       // (also: every thread is done with the index-order bases)
    int pre = inc - ch;
    for (int w = 0; w < warp; ++w) pre += (int)s_warp_tot[w];
    if (tid < nS_l) {
      s_unit_base[e_r] = pre;
      for (int cc = 0; cc < ch && pre + cc < 2 * kMaxExperts; ++cc) s_chunk_expert[pre + cc] = e_r;
    }
    __syncthreads();
  }

  // The rest is three independent jobs, each latency-bound, run side by side:
  //   warps 0-3  row of every (token, slot)       warps 4-6  work-unit list       warp 7  coverage
  const int n_chunks = s_nchunks;
  double cov = 0.0;
  if (warp < 4 && !a.rows_later) {
    // rows ordered by (expert ascending, token ascending): the row of (t, e) is
    // offset[e] + number of tokens below t that were also routed to e
    // thread -> (token, slot) with the slot count padded to a power of two (no integer division)
    int kshift = 0;
    while ((1 << kshift) < k) ++kshift;
    const int slot = tid & ((1 << kshift) - 1);
    const int tok_step = 128 >> kshift;                    // tokens covered per pass by these 128 threads
    for (int t0 = tid >> kshift; t0 < M; t0 += 4 * tok_step) {
      int e[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const int tt = t0 + u * tok_step;
        e[u] = (tt < M && slot < k) ? __ldcg(ws.assign_idx + (size_t)tt * k + slot) : -1;
      }
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const int tt = t0 + u * tok_step;
        if (tt >= M || slot >= k) continue;
        int row = -1;
        if (e[u] >= 0) {
          const unsigned *cm = cm_cached ? s_colmask + e[u] * used_words : ws.colmask + (size_t)e[u] * mw;
          int below = 0;
          if (cm_cached) {
            below = __popc(cm[tt >> 5] & ((1u << (tt & 31)) - 1u));
            for (int w = 0; w < (tt >> 5); ++w) below += __popc(cm[w]);
          } else {
            below = __popc(__ldcg(cm + (tt >> 5)) & ((1u << (tt & 31)) - 1u));
            for (int w = 0; w < (tt >> 5); ++w) below += __popc(__ldcg(cm + w));
          }
          row = s_offset[e[u]] + below;
          ws.perm_row2tok[row] = tt;
          ws.row2expert[row] = e[u];
          if (ws.gather_src) ws.gather_src[row] = s_all_dense[e[u]] ? -1 : tt;
        }
        ws.tokslot2row[(size_t)tt * k + slot] = row;
      }
    }
  } else if (warp >= 4 && warp < 7) {
    // tensor-core work units (expert, token chunk, 128-row slab): all gate/up units, then all down
    // units, each group ordered by (expert, chunk, slab); ready counters and the dispenser start at 0
    if (a.tiles_up > 0) {
      const int lt = tid - 128, nthr = 96;
      const int n_up = n_chunks * a.tiles_up, n_down = n_chunks * a.tiles_down;
      for (int i = lt; i < n_chunks; i += nthr) ws.ready[i] = 0;
      for (int u = lt; u < n_up + n_down; u += nthr) {
        const int phase = u >= n_up;
        const int tiles = phase ? a.tiles_down : a.tiles_up;
        const int v = phase ? u - n_up : u;
        const int cpos = v / tiles;           // position in chunk-prefix space: identifies the expert
        if (a.early) {                        // one chunk per listed expert, rank order
          const int e1 = s_chunk_expert[cpos];
          ws.units[u] = Unit{e1, v - cpos * tiles, s_offset[e1], s_count[e1], cpos, phase,
                             (!phase && (a.dense_all || u < a.ffn_ctas)) ? 2 : 0, 0};
          continue;
        }
        int e;
        if (cpos < 2 * kMaxExperts) {
          e = s_chunk_expert[cpos];
        } else {          // more than 2N token chunks (M far beyond 128): search the chunk bases, in rank order
          e = 0;
          for (int r = 0; r < N; ++r) {          // (whatever the order of the list: the intervals are disjoint)
            if (s_cand[r] > 0 && s_unit_base[r] <= cpos && cpos < s_unit_base[r] + s_cand[r]) { e = r; break; }
          }
        }
        // inside an expert: slab-major, token chunk innermost, so the chunks that re-read a slab are
        // handed out back to back and the second read hits L2
        const int chunks_e = s_cand[e];
        const int local = v - s_unit_base[e] * tiles;
        const int tl = local / chunks_e, c = local - tl * chunks_e;
        const int row0 = s_offset[e] + c * kMaxTokChunk;
        const int rows = min(kMaxTokChunk, s_count[e] - c * kMaxTokChunk);
        ws.units[u] = Unit{e, tl, row0, rows, s_unit_base[e] + c, phase, (a.dense_all && !phase) ? 2 : 0, 0};
      }
    }
  } else if (warp == 7) {
    for (int e = lane; e < N; e += 32)
      if ((s_Smask[e >> 5] >> (e & 31)) & 1u) cov += (double)s_fx[e];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) cov += shfl_xor_double(cov, o);
    cov *= 1.0 / kScoreScale;
  }
  if (tid == 224) {         // lane 0 of warp 7, which holds the coverage sum
    const int R = s_offset[N];
    ws.counters[0] = nS;
    ws.counters[1] = s_nactive;
    ws.counters[2] = R;
    ws.counters[3] = n_chunks * a.tiles_up;
    ws.counters[4] = n_chunks * a.tiles_down;
    moespec_stats st;
    st.n_union = n_union;
    st.n_shortlist = nS;
    st.n_active = s_nactive;
    st.n_rows = R;
    st.n_dropped = M * k - R;
    st.status = 0;
    st.coverage = M > 0 ? cov / (double)M : 0.0;
    st.weight_bytes = (long long)s_nactive * a.expert_bytes;
    *ws.stats = st;
    *ws.status = 0;
    *ws.arrive_route = 0;
  }
  __syncthreads();
  for (int i = tid; i < N; i += blockDim.x) {
    ws.score_fx[i] = 0ull;
    ws.natcnt_acc[i] = 0;
    ws.count_acc[i] = 0;
  }
  // with rows_later the bit matrix is still needed by the row kernel and is cleared by the next call's
  // first kernel instead
  if (!a.rows_later)
    for (int i = tid; i < N * used_words; i += blockDim.x) ws.colmask[i] = 0u;
}

static cudaError_t launch_route_kernel(const LaunchCtx &c, const float *logits) {
  const moespec_layer_desc &D = *c.desc;
  RouteArgs a;
  a.logits = logits;
  a.ws = *c.ws;
  a.M = c.M; a.N = D.n_experts; a.k = c.k; a.B = c.B;
  a.policy = D.policy; a.shortlist = D.shortlist; a.renormalize = D.renormalize;
  a.tiles_up = c.ru > 0 ? D.f / c.ru : 0;
  a.tiles_down = c.ru > 0 ? D.d / tc_rows_per_down_unit(c.ru) : 0;
  a.expert_bytes = 3LL * D.d * D.f * dtype_bytes(D.dtype);
  a.early = c.ru > 0 ? c.early : 0;
  a.ffn_ctas = tc_grid_size(D.device);
  a.rows_later = rows_in_row_kernel(c.M);
  a.dense_all = c.ru > 0 ? c.dense_all : 0;
  a.res_first = c.res_count > 0 ? c.res_first : 0;
  a.res_count = c.res_count > 0 ? c.res_count : D.n_experts;
  const dim3 grid((c.M + kRouteWarps - 1) / kRouteWarps), block(kRouteWarps * 32);
  if (a.N <= 32) return launch_kernel(route_kernel<1>, grid, block, 0, c.stream, a);
  if (a.N <= 64) return launch_kernel(route_kernel<2>, grid, block, 0, c.stream, a);
  if (a.N <= 128) return launch_kernel(route_kernel<4>, grid, block, 0, c.stream, a);
  return launch_kernel(route_kernel<8>, grid, block, 0, c.stream, a);
}

// Eq. 4: add the natural top-k counts of the last router launch to the calibration counters and
// clear the per-call accumulators (no routing kernel follows a calibration pass).
__global__ void __launch_bounds__(256) calib_accumulate_kernel(long long *calib, int *natcnt, unsigned long long *score_fx,
                                                               int N) {
  pdl_trigger();
  pdl_wait();
  for (int i = threadIdx.x; i < N; i += blockDim.x) {
    calib[i] += natcnt[i];
    natcnt[i] = 0;
    score_fx[i] = 0ull;
  }
}

cudaError_t launch_calib_accumulate(const LaunchCtx &c) {
  return launch_kernel(calib_accumulate_kernel, dim3(1), dim3(256), 0, c.stream, c.ws->calib_count, c.ws->natcnt_acc,
                       c.ws->score_fx, c.desc->n_experts);
}

// Routing after router_topk_kernel has filled logits, prob, topk_idx and the score accumulators.
cudaError_t launch_route_after_router(const LaunchCtx &c) { return launch_route_kernel(c, c.ws->logits); }

// Routing from caller-supplied logits: per-token softmax/top-k first (two launches).
cudaError_t launch_route(const LaunchCtx &c, const float *logits) {
  cudaError_t e = launch_kernel(softmax_topk_kernel, dim3((c.M + 3) / 4), dim3(128), 0, c.stream, logits, c.ws->prob,
                                c.ws->topk_idx, c.ws->score_fx, c.ws->natcnt_acc, c.ws->early_flag, c.ws->colmask, c.M,
                                c.desc->n_experts, c.k);
  if (e != cudaSuccess) return e;
  e = launch_route_kernel(c, logits);
  if (e != cudaSuccess || !rows_in_row_kernel(c.M)) return e;
  return launch_gather(c, nullptr);       // rows only: there is no hidden state on this path
}

// ---------------------------------------------------------------------------
// K3: gather routed rows: x_perm[r, :] = hidden[perm_row2tok[r], :] (Appendix C), one CTA per row.  `perm` is
// the gather order, or its copy in which the rows that no work unit reads are marked -1 and skipped.
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
  if (t < 0) return;                       // a row that no work unit reads
  const uint4 *src = hidden + (size_t)t * row_vec;
  uint4 *dst = x_perm + (size_t)r * row_vec;
  for (int j = threadIdx.x; j < row_vec; j += blockDim.x) dst[j] = src[j];
}

// The same for large trees, where the rows themselves are still to be worked out: one CTA per (token, slot)
// pair.  Rows are ordered by (expert ascending, token ascending): the row of (t, e) is offset[e] + the
// number of tokens below t that were also routed to e, a popcount prefix over expert e's row of the bit
// matrix.  The CTA records the row in both directions and, when `hidden` is given, copies the token's
// hidden state there.
__global__ void __launch_bounds__(128) rows_gather_kernel(const uint4 *__restrict__ hidden, uint4 *__restrict__ x_perm,
                                                          const int *__restrict__ assign_idx,
                                                          const int *__restrict__ offset,
                                                          const unsigned *__restrict__ colmask, int *perm_row2tok,
                                                          int *row2expert, int *tokslot2row, int M, int k,
                                                          int row_vec) {
  const int pair = blockIdx.x, t = pair / k;
  const int lane = threadIdx.x & 31;
  __shared__ int s_row;
  pdl_trigger();
  // The token's hidden state does not depend on the routing (it is the layer's input, valid since the router
  // kernel's wait): its first 8 KB are on their way before this kernel waits for the routing kernel, so the
  // chain behind that wait is "expert of the slot -> bit-matrix row and offset -> stores" only.
  constexpr int PRE = 4;
  const uint4 *src = hidden ? hidden + (size_t)t * row_vec : nullptr;
  uint4 pre[PRE];
#pragma unroll
  for (int u = 0; u < PRE; ++u)
    if (hidden && (int)threadIdx.x + u * 128 < row_vec) pre[u] = src[threadIdx.x + u * 128];
  pdl_wait();
  const int e = assign_idx[pair];
  if (e < 0) {                                  // dropped slot (truncation, or fewer than k experts kept)
    if (threadIdx.x == 0) tokslot2row[pair] = -1;
    return;
  }
  if (threadIdx.x < 32) {
    const unsigned *cm = colmask + (size_t)e * ((M + 31) >> 5);
    const int full = t >> 5;
    const int off = lane == 0 ? offset[e] : 0;          // in flight together with the bit-matrix words
    int below = 0;
    for (int w = lane; w < full; w += 32) below += __popc(cm[w]);
    if (lane == 0) below += __popc(cm[full] & ((1u << (t & 31)) - 1u));
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) below += __shfl_xor_sync(kFull, below, o);
    if (lane == 0) {
      const int row = off + below;
      s_row = row;
      perm_row2tok[row] = t;
      if (row2expert) row2expert[row] = e;
      tokslot2row[pair] = row;
    }
  }
  if (!hidden) return;
  __syncthreads();
  uint4 *dst = x_perm + (size_t)s_row * row_vec;
#pragma unroll
  for (int u = 0; u < PRE; ++u)
    if ((int)threadIdx.x + u * 128 < row_vec) dst[threadIdx.x + u * 128] = pre[u];
  for (int j = threadIdx.x + PRE * 128; j < row_vec; j += blockDim.x) dst[j] = src[j];
}

cudaError_t launch_gather(const LaunchCtx &c, const void *hidden) {
  const moespec_layer_desc &D = *c.desc;
  const Workspace &ws = *c.ws;
  const int row_vec = D.d * dtype_bytes(D.dtype) / 16;
  const int rows = c.M * c.k;
  if (rows == 0) return cudaSuccess;
  if (rows_in_row_kernel(c.M))
    return launch_kernel(rows_gather_kernel, dim3(rows), dim3(128), 0, c.stream, (const uint4 *)hidden,
                         (uint4 *)ws.x_perm, (const int *)ws.assign_idx, (const int *)ws.offset,
                         (const unsigned *)ws.colmask, ws.perm_row2tok, ws.row2expert, ws.tokslot2row, c.M, c.k,
                         row_vec);
  return launch_kernel(gather_rows_kernel, dim3(rows), dim3(128), 0, c.stream, (const uint4 *)hidden,
                       (uint4 *)ws.x_perm, (const int *)(ws.gather_src ? ws.gather_src : ws.perm_row2tok),
                       (const int *)ws.counters, row_vec);
}

// The FFN kernel needs nearly all of an SM's shared memory.  An SM whose L1/shared split was chosen for
// one of the small kernels above must drain before it can take such a CTA, and the small kernels sit
// resident in their dependency waits, so the FFN kernel's CTAs could not start before the gather had
// finished.  Asking for the largest shared-memory split here keeps the SMs in the configuration the FFN
// kernel needs, and its CTAs become resident next to the routing kernels' CTAs.
cudaError_t routing_configure() {
  const int pref = (int)cudaSharedmemCarveoutMaxShared;
  cudaError_t e = cudaSuccess;
  auto set = [&](const void *fn) {
    if (e == cudaSuccess) e = cudaFuncSetAttribute(fn, cudaFuncAttributePreferredSharedMemoryCarveout, pref);
  };
  set((const void *)router_topk_kernel<__nv_bfloat16, 2>);
  set((const void *)router_topk_kernel<__nv_bfloat16, 4>);
  set((const void *)router_topk_kernel<__nv_bfloat16, 8>);
  set((const void *)router_topk_kernel<__half, 2>);
  set((const void *)router_topk_kernel<__half, 4>);
  set((const void *)router_topk_kernel<__half, 8>);
  set((const void *)router_mma_kernel<__nv_bfloat16, 8>);
  set((const void *)router_mma_kernel<__half, 8>);
  set((const void *)router_mma_kernel<__nv_bfloat16, 16>);
  set((const void *)router_mma_kernel<__half, 16>);
  set((const void *)softmax_topk_kernel);
  set((const void *)route_kernel<1>);
  set((const void *)route_kernel<2>);
  set((const void *)route_kernel<4>);
  set((const void *)route_kernel<8>);
  set((const void *)gather_rows_kernel);
  set((const void *)rows_gather_kernel);
  return e;
}

}  // namespace moespec
