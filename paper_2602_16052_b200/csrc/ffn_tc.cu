// Tensor-core expert FFN for bf16 and fp16: the weight-streaming kernel of the layer.
//
// Work unit = one slab of RU (128, 64 or 32) rows of one kept expert's weight
// matrix against one chunk (<= 128) of that expert's routed rows.  RU is chosen
// per call so that there are a few units per SM even when few experts are kept
// (small budgets, small trees): an SM can only stream ~55-100 GB/s, so HBM is
// only saturated when every SM has work.  Weights are the MMA A operand (rows of
// W on the M axis; the MMA is always M = 128 and rows beyond RU are ignored),
// routed token rows are the B operand (N axis, padded to 16 or a multiple of 32),
// fp32 accumulators live in tensor memory (two buffers, so the epilogue of one
// unit overlaps the MMAs of the next).
//
//   gate/up unit:  D_g = W1[e, slab, :] X_e^T,  D_u = W3[e, slab, :] X_e^T,
//                  h_mid[row, slab] = bf16(silu(D_g) * D_u)
//   down unit:     D = W2[e, slab, :] H_e^T,     y[row, slab] = D  (fp32)
//
// One launch covers both kinds.  The unit list holds every gate/up unit, then
// every down unit; persistent CTAs (one per SM) draw EVERY unit, the first one
// included, as a ticket from a global dispenser, in list order, so the gate/up
// tail overlaps the start of the down projection.  A down unit needs all of its
// expert chunk's h_mid: each finished gate/up unit bumps a per-chunk ready
// counter (release), and the producer of a down unit waits (bounded, acquire)
// for the counter to reach the slab count.  Tickets are handed out in order to
// CTAs that are running, and gate/up units never wait, so every unit a down
// unit waits for has been drawn by a running CTA or is done: there is no
// circular wait, however the grid is placed on the SMs (a CTA that becomes
// resident late simply draws a later ticket, e.g. when another handle's kernel
// holds some of the SMs).  The dispenser and the down-unit counter are zeroed
// by the router kernel of the call, which completes before this kernel starts.
//
// Early start (trees of up to 128 tokens): the CTAs of this kernel are resident
// while the routing kernels still run.  A CTA whose first ticket c is below the
// grid size does not wait for them: as soon as the routing kernel has published
// the shortlist (a flag; at once when the shortlist is fixed) it starts on
// gate/up unit c of the rank-ordered list -- expert S_rank[c / slabs], slab
// c % slabs -- with ALL tokens of the tree as the B operand, read from `hidden`
// itself, and keeps the routed tokens' columns in the epilogue, by which time
// the gather order exists.  The routing kernel lists the units in the same
// order, so unit c of the list is that unit.
//
// Ten warps per CTA:
//   warp 0        : dispenser + TMA producer.  Lane 0 waits and draws units; all
//                   lanes issue the copies of a stage: 64-wide K chunks of the
//                   weight slab(s) (3-D tensor map, expert id is the outer
//                   coordinate: no stacking copy) and of the token rows into a
//                   ring of stages, up to 32 KB of weights per stage.
//   warp 1  lane 0: issues tcgen05.mma (kind::f16, M=128, N=n_pad, K=16) from the
//                   stage's swizzled shared memory into TMEM; tcgen05.commit frees
//                   the stage and finally publishes the accumulator.
//   warps 2-9     : epilogue.  tcgen05.ld the accumulator (a TMEM lane quarter is
//                   shared by two warps, which take alternate groups of 16
//                   columns), apply SwiGLU, store to global.
// The combine of the layer lives in this kernel too: after its last unit every
// CTA waits (bounded) until all down units are stored and then its warps produce
// their share of `out` from y, the mixing weights and tokslot2row (128 columns of
// one token per warp and step), adding slots in a fixed order.  (Fetching routed rows straight from `hidden` with one-row TMA boxes was
// measured 40 % slower than reading a gathered copy with 32-row boxes: the copy
// engine's rate for 128-byte boxes is the limit.)
// Every wait is bounded: on expiry the CTA raises an abort flag, records
// MOESPEC_ERR_TIMEOUT in the status word, drains its own copies, frees TMEM and
// returns.
#include "internal.h"
#include <cstdlib>

namespace moespec {

namespace {

constexpr int kEpiWarps = 8;                      // two warps per TMEM lane quarter, each takes every other 16 columns
constexpr int kEpiThreads = kEpiWarps * 32;
constexpr int kThreads = 64 + kEpiThreads;       // producer warp, MMA warp, epilogue warps
constexpr int kChunkK = 64;                      // bf16 elements per 128-byte swizzle row
constexpr int kARegion = 32 * 1024;              // weight bytes per stage
constexpr int kBRegionMax = 16 * 1024;           // token-row bytes per stage: 8 KB when M <= 32, else 16 KB
constexpr int kMmaTail = 16 * 1024;              // an M=128 MMA reads 16 KB from the start of a (possibly shorter) slab
constexpr int kMaxStages = 8;
constexpr int kSmemBudget = 227 * 1024;
constexpr int kCtrlBytes = 1024;                 // barriers, unit queue, TMEM base, abort flag, token->row table
constexpr uint32_t kTmemCols = 512;
constexpr long long kSpinLimitCycles = 2000000000LL;   // default bound of every wait: ~1 s at 2 GHz

constexpr int kQueue = 4;                        // units in flight between the producer and its consumers

struct TcArgs {
  const Unit *units;
  const int *n_units;   // [0] gate/up units, [1] down units
  int *unit_counter;    // dispenser
  int *ready;           // per (expert, token chunk): finished gate/up units
  int tiles_up;         // gate/up units per chunk = value of ready[] that releases its down units
  int ru;               // weight rows per gate/up unit: 128, 64 or 32
  int ru_down;          // weight rows per down unit
  int kchunks_up;       // d / 64: K chunks of a gate/up unit
  int kchunks_down;     // f / 64: K chunks of a down unit
  int n_stages;
  int b_region;         // token-row bytes per stage
  int stage_bytes;      // kARegion + b_region
  void *h_mid;          // [R, f] bf16 or fp16
  int is_fp16;          // 16-bit format of weights, hidden and h_mid: 0 bf16, 1 fp16
  float *y;             // [R, d]
  int f, d;
  int *status;
  // combine (outer sums of Eq. 2 / 7 / 8), run by every CTA once all down units are stored
  int *down_done;       // down units whose y slab is stored; zeroed by the route kernel
  const float *gate_w;  // [M, k]
  const int *tokslot2row;
  const void *hidden;   // [M, d] bf16 (residual input)
  void *out;            // [M, d] bf16 or fp32
  int M, k, residual, out_is_fp32;
  long long spin_limit; // cycles after which any wait gives up
  // early start (see the kernel's header comment)
  int early;                 // 1: tickets below the grid size are started on before routing has finished
  const int *early_flag;     // [n_words] word r: 0 until the routing kernel has published the shortlist, then the
                             // resident expert of rank r, plus one, or -1 when there are fewer
  int n_words;
  int res_first, res_count;  // experts whose weights this GPU holds: the weight tensors start at expert res_first
  const int *assign_idx;     // [M, k] kept expert per slot (the combine of a shard skips slots of other GPUs' experts)
  const int *perm_row2tok;   // gather order: row -> token
  int tiles_real;            // f / ru: gate/up units per expert
  int static_nS;             // > 0: fixed shortlist (Eq. 4) of this size, known before any kernel of the call runs
  const int *static_order;   // the fixed ordering
};

// ------------------------------------------------------------------ PTX wrappers
__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded wait.  Returns false when the CTA is aborting or the limit expired.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int *abort_flag,
                                          long long limit = kSpinLimitCycles) {
  if (mbar_try(bar, parity)) return true;
  const long long t0 = clock64();
  for (uint32_t i = 1;; ++i) {
    if (mbar_try(bar, parity)) return true;
    if ((i & 255u) == 0u) {
      if (*abort_flag) return false;
      if (clock64() - t0 > limit) {
        *abort_flag = 1;
        return false;
      }
    }
  }
}

// Weights are read once per call: evict-first keeps them from flushing the small hot set (router
// matrix, gathered rows, h_mid, y) out of L2.
__device__ __forceinline__ uint64_t l2_evict_first_policy() {
  uint64_t p;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(p));
  return p;
}
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap *map, uint32_t bar, int c0, int c1,
                                            int c2, uint64_t policy) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%3, %4, %5}], [%2], %6;"
      ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "l"(policy)
      : "memory");
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap *map, uint32_t bar, int c0, int c1) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1)
      : "memory");
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void tc_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_mma_bf16(uint32_t tmem_d, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                            uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(tmem_d), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}
__device__ __forceinline__ void tc_ld16(uint32_t taddr, uint32_t (&r)[16]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tc_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Shared-memory matrix descriptor: K-major operand, 128-byte swizzle, rows at a
// 128-byte pitch, 8-row groups 1024 bytes apart.
__device__ __forceinline__ uint64_t smem_desc_sw128(uint32_t addr) {
  uint64_t d = 0;
  d |= (uint64_t)((addr & 0x3FFFFu) >> 4);         // start address
  d |= (uint64_t)1 << 16;                          // leading byte offset (unused for swizzled K-major)
  d |= (uint64_t)(1024 >> 4) << 32;                // stride byte offset between 8-row groups
  d |= (uint64_t)1 << 46;                          // descriptor version
  d |= (uint64_t)2 << 61;                          // SWIZZLE_128B
  return d;
}
// Instruction descriptor: D fp32, A and B bf16 (format 1) or fp16 (format 0), both K-major, M = 128, N = n.
__device__ __forceinline__ uint32_t instr_desc_16bit(int n, int is_fp16) {
  const uint32_t fmt = is_fp16 ? 0u : 1u;
  return (1u << 4) | (fmt << 7) | (fmt << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(kTile >> 4) << 24);
}

}  // namespace

// K chunks carried by one ring stage of a unit: as many as fit the 32 KB weight region (gate and up
// slabs in a gate/up unit) and the 16 KB token region (n_pad rows per chunk), a power of two that
// divides the unit's chunk count.  Producer, MMA issuer and epilogue all derive it from the unit.
__device__ __forceinline__ int chunks_per_stage(const TcArgs &a, int phase, int n_pad) {
  const int cap_a = phase == 0 ? kARegion / (2 * a.ru * 128) : kARegion / (a.ru_down * 128);
  const int cap_b = a.b_region / (n_pad * 128);
  const int cap = cap_a < cap_b ? cap_a : cap_b;
  const int kch = phase == 0 ? a.kchunks_up : a.kchunks_down;
  int p = 1;
  while (p * 2 <= cap && kch % (p * 2) == 0) p *= 2;
  return p;
}

// Token rows of a unit on the MMA's N axis: 16 for the many experts that get a handful of rows (the token
// operand is re-read by every slab of the expert and competes with the weight stream for the SM's ingest
// rate), else a multiple of 32.
__device__ __forceinline__ int pad_rows(int n_rows) {
  return n_rows <= kTokBoxSmall ? kTokBoxSmall : (n_rows + kTokBox - 1) / kTokBox * kTokBox;
}

__device__ __forceinline__ int ld_acquire(const int *p) {
  int v;
  asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
// Release increment by one thread after a CTA barrier: the stores of all threads that arrived at the barrier are
// visible to whoever acquires the new value.
__device__ __forceinline__ void red_release_add(int *p) {
  asm volatile("red.release.gpu.global.add.s32 [%0], 1;" ::"l"(p) : "memory");
}
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async;" ::: "memory"); }
__device__ __forceinline__ void epilogue_bar() { asm volatile("bar.sync 1, %0;" ::"n"(kEpiThreads) : "memory"); }

__global__ void __launch_bounds__(kThreads, 1) ffn_tc_kernel(const __grid_constant__ TcMapsCall maps, TcArgs a) {
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  // stages first (1024-byte aligned for the 128-byte swizzle), control block after
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t *smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));
  const uint32_t ctrl = smem_base + (uint32_t)a.n_stages * (uint32_t)a.stage_bytes + kMmaTail;
  uint8_t *ctrl_gen = smem_gen + (size_t)a.n_stages * a.stage_bytes + kMmaTail;
  const uint32_t bar_full = ctrl;                       // [kMaxStages]
  const uint32_t bar_empty = ctrl + 8 * kMaxStages;     // [kMaxStages]
  const uint32_t bar_acc_full = ctrl + 16 * kMaxStages; // [2]
  const uint32_t bar_acc_empty = bar_acc_full + 16;     // [2]
  const uint32_t bar_q_full = bar_acc_empty + 16;       // [kQueue]
  const uint32_t bar_q_empty = bar_q_full + 8 * kQueue; // [kQueue]
  constexpr int kMiscOff = 16 * kMaxStages + 32 + 16 * kQueue;   // 224
  volatile uint32_t *tmem_slot = reinterpret_cast<volatile uint32_t *>(ctrl_gen + kMiscOff);
  volatile int *abort_flag = reinterpret_cast<volatile int *>(ctrl_gen + kMiscOff + 4);
  Unit *q_unit = reinterpret_cast<Unit *>(ctrl_gen + 256);       // [kQueue] x 32 bytes
  int *tok2row = reinterpret_cast<int *>(ctrl_gen + 512);        // [128] token -> row of h_mid (early units)

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int n_stages = a.n_stages;
  pdl_trigger();
  // The first ticket and, with early start, the first 32 shortlist words are requested before anything else:
  // their round trips through L2 overlap the set-up below.  (The router kernel of this call left the
  // dispenser at zero and has completed, or with a fixed shortlist has at least performed that reset.)
  int t_first = 0, w_pre = 0;
  if (warp == 0) {
    if (lane == 0) t_first = atomicAdd(a.unit_counter, 1);
    if (a.early && a.static_nS == 0 && lane < a.n_words) w_pre = ld_acquire(a.early_flag + lane);
  }

  if (threadIdx.x == 0) {
    for (int s = 0; s < n_stages; ++s) {
      mbar_init(bar_full + 8 * s, 1);
      mbar_init(bar_empty + 8 * s, 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(bar_acc_full + 8 * b, 1);
      mbar_init(bar_acc_empty + 8 * b, kEpiThreads);
    }
    for (int q = 0; q < kQueue; ++q) {
      mbar_init(bar_q_full + 8 * q, 1);
      mbar_init(bar_q_empty + 8 * q, kEpiThreads + 1);      // the MMA thread and the epilogue threads
    }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(
                     smem_u32(const_cast<uint32_t *>(tmem_slot))),
                 "r"(kTmemCols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  // Everything above overlaps the tail of the previous kernel.  Without early start its results are read
  // from here on; with it each role waits at the point where it first needs them.
  if (!a.early) pdl_wait();

  if (warp == 0) {
    // ===================================================== dispenser + TMA producer
    // Lane 0 owns every wait and the queue; the copies of a stage are issued by all lanes (one box
    // each), because a single thread issuing 8-16 copies per stage would cap the SM's streaming rate.
    // Every unit, the first included, is a ticket from the dispenser.  The next unit is drawn a few
    // stages before the current one ends: early enough that the atomic and the descriptor load are
    // hidden behind the stages still in flight, late enough that no CTA sits on units others could run.
    int n_total = 0;                 // valid once `waited`
    bool waited = !a.early;          // has this warp waited for the routing kernels?
    uint32_t it = 0, qi = 0;
    int ok = 1;
    const uint64_t wpol = l2_evict_first_policy();
    Unit sentinel;
    sentinel.expert = -1; sentinel.tile = 0; sentinel.row0 = 0; sentinel.n_rows = 0; sentinel.chunk = 0;
    sentinel.phase = 0; sentinel.pad0 = 0; sentinel.pad1 = 0;
    Unit un = sentinel;
    // A list entry marked 2 is a gate/up unit that takes all tokens from `hidden`: one of the first units of the
    // list, which CTAs may have started on early, or any unit of a tree so small that no gathered copy is made.
    // It runs like an early unit, and its epilogue finds its rows in the entry.
    auto from_list = [&](int u) -> Unit {
      Unit x = a.units[u];
      if (x.pad0 == 2) {
        if (x.n_rows == 0) x.pad0 = 0;             // no rows: skipped like any other empty unit
        else { x.pad0 = 1; x.pad1 = u; x.n_rows = a.M; x.row0 = 0; }
      }
      return x;
    };
    if (a.early) {
      // The routing kernel publishes the shortlist long before the gather order exists.  Ticket c below the
      // grid size is gate/up unit c of the rank-ordered list (expert S_rank[c / tiles], slab c % tiles) and
      // is started on with ALL tokens as the MMA's N dimension, read straight from `hidden`; the epilogue
      // keeps the routed tokens only.  The routing kernel builds the unit list in the same order and keeps
      // the experts of those ranks in it even without rows, so unit c of the list is this unit.
      const int r_first = __shfl_sync(0xffffffffu, t_first, 0) / a.tiles_real;
      const int v_pre = __shfl_sync(0xffffffffu, w_pre, r_first & 31);      // that rank's word as read at entry
      if (lane == 0 && t_first < (int)gridDim.x) {
        const int r = r_first;
        int v = -1;                      // the expert of rank r, plus one
        if (a.static_nS > 0) {           // a fixed shortlist needs no publication: stream from the first cycle
          if (r < a.static_nS) v = a.static_order[r] + 1;
        } else if (r < a.n_words) {
          const long long t0 = clock64();
          v = r < 32 ? v_pre : 0;
          while (v == 0 && (v = ld_acquire(a.early_flag + r)) == 0) {
            if (*abort_flag || clock64() - t0 > a.spin_limit) { *abort_flag = 1; ok = 0; break; }
            __nanosleep(32);
          }
        }
        if (ok && v > 0) {
          un.expert = v - 1;
          un.tile = t_first - r * a.tiles_real;
          un.n_rows = a.M;
          un.pad0 = 1;                 // dense: every token, rows of `hidden`
          un.pad1 = t_first;           // its place in the unit list
        }
      }
      ok = __shfl_sync(0xffffffffu, ok, 0);
      if (ok && !__shfl_sync(0xffffffffu, un.pad0, 0)) {      // no early unit for this ticket: wait like everybody
        pdl_wait();
        waited = true;
      }
    }
    if (waited) {
      n_total = a.n_units[0] + a.n_units[1];
      if (lane == 0 && !un.pad0 && t_first < n_total) un = from_list(t_first);
    }
    while (ok) {
      Unit un_next = sentinel;
      int u_next = 0x7fffffff;
      if (lane == 0) {
        // units without rows (an expert kept in the list only because CTAs may have started on it): nothing
        // to stream; a down unit still counts as done
        while (un.expert >= 0 && un.n_rows == 0 && !un.pad0) {
          if (un.phase == 1) atomicAdd(a.down_done, 1);
          const int u2 = atomicAdd(a.unit_counter, 1);
          un = u2 < n_total ? from_list(u2) : sentinel;
        }
        const uint32_t q = qi % kQueue, qph = (qi / kQueue) & 1u;
        if (!mbar_wait(bar_q_empty + 8 * q, qph ^ 1u, abort_flag, a.spin_limit)) ok = 0;
        if (ok) {
          q_unit[q] = un;
          mbar_arrive(bar_q_full + 8 * q);          // release: the queue slot is visible to the consumers
        }
      }
      ++qi;
      ok = __shfl_sync(0xffffffffu, ok, 0);
      const int expert = __shfl_sync(0xffffffffu, un.expert, 0);
      if (!ok || expert < 0) break;
      const int tile = __shfl_sync(0xffffffffu, un.tile, 0);
      const int row0 = __shfl_sync(0xffffffffu, un.row0, 0);
      const int n_rows = __shfl_sync(0xffffffffu, un.n_rows, 0);
      const int phase = __shfl_sync(0xffffffffu, un.phase, 0);
      const int dense = __shfl_sync(0xffffffffu, un.pad0, 0);
      const int n_pad = pad_rows(n_rows);
      const int cps = chunks_per_stage(a, phase, n_pad);
      const int k_iters = (phase == 0 ? a.kchunks_up : a.kchunks_down) / cps;
      const uint32_t slab_bytes = (uint32_t)n_pad * 128u;           // one K chunk of the unit's token rows
      const int ru = phase == 0 ? a.ru : a.ru_down;
      const uint32_t sub_bytes = (uint32_t)ru * 128u;              // one K chunk of one weight slab
      const int w_boxes = (phase == 0 ? 2 : 1) * cps;              // weight copies per stage
      // Token rows arrive in as few copies as possible (the copy engine handles ~13 M boxes/s per SM,
      // so 8+ boxes per stage would cap the stream): one 128- or 64-row box when n_pad allows, else 32s.
      const int bsel = n_pad == 128 ? 2 : (n_pad % 64 == 0 ? 1 : 0);
      const bool small = n_pad == kTokBoxSmall;
      const int box_rows = small ? kTokBoxSmall : kTokBox << bsel;
      const int t_per = n_pad / box_rows;                          // token copies per K chunk
      const int n_tok_rows = n_pad;                                // rows that arrive per K chunk
      const CUtensorMap *map_b = dense ? &maps.hidden
                                 : small ? (phase == 0 ? &maps.x_perm16 : &maps.h_mid16)
                                         : (phase == 0 ? &maps.x_perm[bsel] : &maps.h_mid[bsel]);
      const uint32_t tx = (uint32_t)w_boxes * sub_bytes + (uint32_t)cps * (uint32_t)n_tok_rows * 128u;
      const int draw_at = k_iters > 6 ? k_iters - 6 : 0;
      const int chunk = __shfl_sync(0xffffffffu, un.chunk, 0);
      // A stage is armed and its weight copies issued by head(); its token-row copies by rows().  A down
      // unit reads h_mid, which is complete only when every gate/up slab of its expert has been published.
      int armed = 0;                                // stages of this unit whose barrier has been armed
      auto head = [&](int kc) {
        const uint32_t s = (it + kc) % n_stages, ph = ((it + kc) / n_stages) & 1u;
        const uint32_t full = bar_full + 8 * s;
        const uint32_t stage = smem_base + s * (uint32_t)a.stage_bytes;
        if (kc == draw_at && !waited) {        // the unit list and the gathered rows are needed from here on
          pdl_wait();
          waited = true;
          n_total = a.n_units[0] + a.n_units[1];
        }
        if (lane == 0) {
          if (kc == draw_at) u_next = atomicAdd(a.unit_counter, 1);
          if (!mbar_wait(bar_empty + 8 * s, ph ^ 1u, abort_flag, a.spin_limit)) ok = 0;
          else mbar_expect_tx(full, tx);
        }
        ok = __shfl_sync(0xffffffffu, ok, 0);
        if (!ok) return;
        ++armed;
        if (lane < w_boxes) {                       // at most 8 weight copies per stage
          const int j = phase == 0 ? (lane >> 1) : lane;
          const int col = (kc * cps + j) * kChunkK;
          const CUtensorMap *mw = phase == 0 ? ((lane & 1) ? &maps.w_up : &maps.w_gate) : &maps.w_down;
          tma_load_3d(stage + lane * sub_bytes, mw, full, col, tile * ru, expert - a.res_first, wpol);
        }
      };
      auto rows = [&](int kc) {
        const uint32_t s = (it + kc) % n_stages;
        const uint32_t full = bar_full + 8 * s;
        const uint32_t stage = smem_base + s * (uint32_t)a.stage_bytes;
        for (int tb = lane; tb < cps * t_per; tb += 32) {
          const int j = tb / t_per, r = tb - j * t_per;
          const int col = (kc * cps + j) * kChunkK;
          tma_load_2d(stage + kARegion + j * slab_bytes + r * (box_rows * 128), map_b, full, col, row0 + r * box_rows);
        }
      };
      int n_pre = 0;
      if (phase == 1) {
        // Usually the expert's slabs were published long ago.  The counter is read while the slot of the
        // first stage drains behind the previous unit; if it is complete, this unit's stages follow the
        // previous unit's without a gap, weights and rows together.  (Requesting the weights of several
        // stages first, then looking at the counter, then requesting the rows left the ring standing still
        // for two round trips at the start of every down unit.)
        int seen = 0;
        if (lane == 0) seen = ld_acquire(a.ready + chunk);
        head(0);
        int is_ready = 0;
        if (ok && lane == 0 && seen >= a.tiles_up) {
          is_ready = 1;
          fence_proxy_async();                      // order the acquire before the TMA reads of h_mid
        }
        is_ready = __shfl_sync(0xffffffffu, is_ready, 0);
        if (ok && is_ready) {
          rows(0);
          n_pre = 1;
        } else if (ok) {
          // not yet: the weights of the first stages are requested BEFORE the wait, so that a CTA that runs
          // into the dependency keeps streaming instead of idling
          n_pre = k_iters < n_stages ? k_iters : n_stages;
          for (int kc = 1; kc < n_pre && ok; ++kc) head(kc);
          if (ok && lane == 0) {
            const long long t0 = clock64();
            while (ld_acquire(a.ready + chunk) < a.tiles_up) {
              if (*abort_flag || clock64() - t0 > a.spin_limit) { *abort_flag = 1; ok = 0; break; }
              __nanosleep(64);
            }
            fence_proxy_async();
          }
          ok = __shfl_sync(0xffffffffu, ok, 0);
          // on an abort the armed stages still receive their weight copies; the drain below waits for them
          for (int kc = 0; kc < n_pre && ok; ++kc) rows(kc);
        }
      }
      for (int kc = n_pre; kc < k_iters && ok; ++kc) {
        head(kc);
        if (ok) rows(kc);
      }
      it += (uint32_t)armed;                        // == k_iters unless the CTA is aborting
      if (!ok) break;
      if (lane == 0 && u_next < n_total) un_next = from_list(u_next);
      un = un_next;
    }
    if (!ok && lane == 0) {
      // drain: wait (bounded) until every copy this warp issued has landed
      const uint32_t lo = it > (uint32_t)n_stages ? it - n_stages : 0u;
      for (uint32_t j = lo; j < it; ++j) {
        const long long t0 = clock64();
        while (!mbar_try(bar_full + 8 * (j % n_stages), (j / n_stages) & 1u))
          if (clock64() - t0 > a.spin_limit) break;
      }
    }
  } else if (warp == 1 && lane == 0) {
    // ===================================================== MMA issuer
    uint32_t it = 0, acc_it = 0, qi = 0;
    bool ok = true;
    while (ok) {
      const uint32_t q = qi % kQueue, qph = (qi / kQueue) & 1u;
      if (!mbar_wait(bar_q_full + 8 * q, qph, abort_flag, a.spin_limit)) break;
      const Unit un = q_unit[q];
      ++qi;
      if (un.expert < 0) { mbar_arrive(bar_q_empty + 8 * q); break; }
      const int n_pad = pad_rows(un.n_rows);
      const uint32_t idesc = instr_desc_16bit(n_pad, a.is_fp16);
      const uint32_t ab = acc_it & 1u, aph = (acc_it >> 1) & 1u;
      if (!mbar_wait(bar_acc_empty + 8 * ab, aph ^ 1u, abort_flag, a.spin_limit)) break;
      tc_fence_after();
      const uint32_t tmem_d = tmem_base + ab * 256u;
      const int cps = chunks_per_stage(a, un.phase, n_pad);
      const int k_iters = (un.phase == 0 ? a.kchunks_up : a.kchunks_down) / cps;
      // This one thread issues every MMA of the CTA, so its instruction count per MMA bounds the rate at
      // which stages are released.  Descriptors are therefore advanced by adding to the 16-byte-granular
      // address field instead of being rebuilt: +2 per K step of 16 elements, +sub16 per weight slab,
      // +slab16 per token slab.
      const uint64_t sub16 = (uint64_t)((un.phase == 0 ? a.ru : a.ru_down) * 128 >> 4), slab16 = (uint64_t)(n_pad * 128 >> 4);
      const uint32_t tmem_u = tmem_d + (uint32_t)n_pad;
      for (int kc = 0; kc < k_iters; ++kc, ++it) {
        const uint32_t s = it % n_stages, ph = (it / n_stages) & 1u;
        if (!mbar_wait(bar_full + 8 * s, ph, abort_flag, a.spin_limit)) { ok = false; break; }
        tc_fence_after();
        uint64_t ad = smem_desc_sw128(smem_base + s * (uint32_t)a.stage_bytes);
        uint64_t bd = ad + (uint64_t)(kARegion >> 4);
        uint32_t acc = kc > 0 ? 1u : 0u;
        if (un.phase == 0) {
          for (int j = 0; j < cps; ++j) {
#pragma unroll
            for (int kk = 0; kk < kChunkK / 16; ++kk) {
              tc_mma_bf16(tmem_d, ad + 2 * kk, bd + 2 * kk, idesc, acc);
              tc_mma_bf16(tmem_u, ad + sub16 + 2 * kk, bd + 2 * kk, idesc, acc);
              acc = 1u;
            }
            ad += 2 * sub16;
            bd += slab16;
          }
        } else {
          for (int j = 0; j < cps; ++j) {
#pragma unroll
            for (int kk = 0; kk < kChunkK / 16; ++kk) {
              tc_mma_bf16(tmem_d, ad + 2 * kk, bd + 2 * kk, idesc, acc);
              acc = 1u;
            }
            ad += sub16;
            bd += slab16;
          }
        }
        tc_commit(bar_empty + 8 * s);      // stage reusable once these MMAs have read it
      }
      if (!ok) break;
      tc_commit(bar_acc_full + 8 * ab);
      mbar_arrive(bar_q_empty + 8 * q);
      ++acc_it;
    }
  } else if (warp >= 2) {
    // ===================================================== epilogue
    const int quarter = warp & 3;           // TMEM lanes 32*quarter .. +31 belong to this warp
    const int row_in_tile = quarter * 32 + lane;
    const int c_first = ((warp - 2) >> 2) * 16;   // the quarter's two warps interleave 16-column groups
    uint32_t acc_it = 0, qi = 0;
    while (true) {
      const uint32_t q = qi % kQueue, qph = (qi / kQueue) & 1u;
      if (!mbar_wait(bar_q_full + 8 * q, qph, abort_flag, a.spin_limit)) break;
      const Unit un = q_unit[q];
      ++qi;
      if (un.expert < 0) { mbar_arrive(bar_q_empty + 8 * q); break; }
      const uint32_t ab = acc_it & 1u, aph = (acc_it >> 1) & 1u;
      const int n_pad = pad_rows(un.n_rows);
      const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + ab * 256u;
      const int ru = un.phase == 0 ? a.ru : a.ru_down;
      const int col_out = un.tile * ru + row_in_tile;       // index along f (gate/up) or d (down)
      if (un.pad0) {
        // Early unit: the accumulator holds the slab for EVERY token.  Routing has finished by now (this
        // unit alone streamed for longer than the routing kernels run); its list entry says which rows of
        // h_mid the expert owns and the gather order says which token each row is.
        pdl_wait();
        const int et = (int)threadIdx.x - 64;
        Unit real = a.units[un.pad1];
        if (real.expert != un.expert || real.tile != un.tile || real.phase != 0 || real.n_rows > kMaxTokChunk) {
          if (et == 0) atomicExch(a.status, (int)MOESPEC_ERR_INTERNAL);      // the two kernels disagree on the list
          real.n_rows = 0;
        }
        if (et < kMaxTokChunk) tok2row[et] = -1;
        epilogue_bar();
        if (et < real.n_rows) tok2row[__ldcg(a.perm_row2tok + real.row0 + et)] = real.row0 + et;
        epilogue_bar();
        if (!mbar_wait(bar_acc_full + 8 * ab, aph, abort_flag, a.spin_limit)) break;
        tc_fence_after();
        const int n_tok = quarter * 32 < ru ? un.n_rows : 0;
        for (int c0 = c_first; c0 < n_tok; c0 += 32) {
          uint32_t g[16], up[16];
          tc_ld16(taddr + c0, g);
          tc_ld16(taddr + n_pad + c0, up);
          tc_ld_wait();
          float m[16];
#pragma unroll
          for (int i = 0; i < 16; ++i) {               // independent chains first, as in the gathered case
            const float gv = __uint_as_float(g[i]);
            m[i] = __fdividef(gv, 1.f + __expf(-gv)) * __uint_as_float(up[i]);
          }
#pragma unroll
          for (int i = 0; i < 16; ++i) {
            const int row = tok2row[c0 + i];          // broadcast read; -1: token not routed to this expert
            if (row < 0) continue;
            if (a.is_fp16) reinterpret_cast<__half *>(a.h_mid)[(size_t)row * a.f + col_out] = __float2half_rn(m[i]);
            else reinterpret_cast<__nv_bfloat16 *>(a.h_mid)[(size_t)row * a.f + col_out] = __float2bfloat16_rn(m[i]);
          }
        }
        tc_fence_before();
        mbar_arrive(bar_acc_empty + 8 * ab);
        fence_proxy_async();
        epilogue_bar();
        if (threadIdx.x == 64) red_release_add(a.ready + real.chunk);
        mbar_arrive(bar_q_empty + 8 * q);
        ++acc_it;
        continue;
      }
      if (!mbar_wait(bar_acc_full + 8 * ab, aph, abort_flag, a.spin_limit)) break;
      tc_fence_after();
      const int n_live = quarter * 32 < ru ? un.n_rows : 0;     // accumulator lanes beyond the slab hold nothing
      // One warp per scheduler runs this loop, so it is latency-bound: the sixteen columns of a step are
      // computed as independent chains (approximate exp and divide: two instructions each, error far
      // below the 16-bit rounding of the result) before the first store is issued.
      if (un.phase == 0) {
        for (int c0 = c_first; c0 < n_live; c0 += 32) {
          uint32_t g[16], up[16];
          tc_ld16(taddr + c0, g);
          tc_ld16(taddr + n_pad + c0, up);
          tc_ld_wait();
          float m[16];
#pragma unroll
          for (int i = 0; i < 16; ++i) {
            const float gv = __uint_as_float(g[i]);
            m[i] = __fdividef(gv, 1.f + __expf(-gv)) * __uint_as_float(up[i]);
          }
          const int n_here = min(16, un.n_rows - c0);
          if (a.is_fp16) {
            __half *dst = reinterpret_cast<__half *>(a.h_mid) + (size_t)(un.row0 + c0) * a.f + col_out;
#pragma unroll
            for (int i = 0; i < 16; ++i)
              if (i < n_here) dst[(size_t)i * a.f] = __float2half_rn(m[i]);
          } else {
            __nv_bfloat16 *dst = reinterpret_cast<__nv_bfloat16 *>(a.h_mid) + (size_t)(un.row0 + c0) * a.f + col_out;
#pragma unroll
            for (int i = 0; i < 16; ++i)
              if (i < n_here) dst[(size_t)i * a.f] = __float2bfloat16_rn(m[i]);
          }
        }
      } else {
        for (int c0 = c_first; c0 < n_live; c0 += 32) {
          uint32_t g[16];
          tc_ld16(taddr + c0, g);
          tc_ld_wait();
          const int n_here = min(16, un.n_rows - c0);
          float *dst = a.y + (size_t)(un.row0 + c0) * a.d + col_out;
#pragma unroll
          for (int i = 0; i < 16; ++i)
            if (i < n_here) dst[(size_t)i * a.d] = __uint_as_float(g[i]);
        }
      }
      tc_fence_before();
      mbar_arrive(bar_acc_empty + 8 * ab);
      // publish the slab (h_mid for a gate/up unit, y for a down unit): every thread's stores are
      // fenced, then one thread bumps the counter the consumers of the slab watch
      if (un.phase == 0) fence_proxy_async();
      epilogue_bar();
      if (threadIdx.x == 64) red_release_add(un.phase == 0 ? a.ready + un.chunk : a.down_done);
      mbar_arrive(bar_q_empty + 8 * q);
      ++acc_it;
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
  }

  if (a.early) pdl_wait();      // threads that have not needed the routing results so far
  // ===================================================== combine
  // out_t = sum over the kept slots of wgt[t, slot] * y[row(t, slot)], slots in a fixed order; a token
  // with no kept expert gets exact zeros (Section 3.3).  Needs every down unit of the call.
  // Work item = 128 consecutive columns of one token, handled by one warp (a float4 per lane): the warps of
  // all CTAs walk the item list independently, so there is no CTA-wide barrier between items.  Lane s holds
  // row and weight of slot s (k <= 32) and the warp shuffles them around; the first item's slots are
  // fetched while the last down units are still being stored.
  const int k = a.k, d = a.d;
  const int slices = d / 128;                                // items per token
  const int n_items = a.M * slices;
  const int warp_global = (int)blockIdx.x + warp * (int)gridDim.x;      // consecutive items go to different SMs
  const int warps_total = (kThreads / 32) * (int)gridDim.x;
  int my_row = -1;
  float my_w = 0.f;
  // an expert-parallel shard adds up the slots of its resident experts only (the other rows of y are not its own)
  const bool shard = a.res_count > 0;
  auto resident_slot = [&](int t, int slot) {
    const int e = a.assign_idx[(size_t)t * k + slot];
    return e >= a.res_first && e < a.res_first + a.res_count;
  };
  if (warp_global < n_items && lane < k) {
    const int t = warp_global / slices;
    my_row = a.tokslot2row[(size_t)t * k + lane];
    my_w = a.gate_w[(size_t)t * k + lane];
    if (shard && my_row >= 0 && !resident_slot(t, lane)) my_row = -1;
  }
  if (threadIdx.x == 0 && !*abort_flag) {
    const int n_down = a.n_units[1];
    const long long t0 = clock64();
    while (ld_acquire(a.down_done) < n_down) {
      if (clock64() - t0 > a.spin_limit) { *abort_flag = 1; break; }
      __nanosleep(128);
    }
  }
  __syncthreads();
  if (*abort_flag) {
    if (threadIdx.x == 0) atomicExch(a.status, (int)MOESPEC_ERR_TIMEOUT);
    return;
  }
  for (int item = warp_global; item < n_items; item += warps_total) {
    const int t = item / slices, c = (item - t * slices) * 128 + lane * 4;
    if (item != warp_global) {                               // later items: this token's slots
      my_row = lane < k ? a.tokslot2row[(size_t)t * k + lane] : -1;
      my_w = lane < k ? a.gate_w[(size_t)t * k + lane] : 0.f;
      if (shard && my_row >= 0 && !resident_slot(t, lane)) my_row = -1;
    }
    {
      float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
      for (int s0 = 0; s0 < k; s0 += 8) {
        float4 v[8];
        float w[8];
#pragma unroll
        for (int s = 0; s < 8; ++s) {
          const int row = __shfl_sync(0xffffffffu, my_row, (s0 + s) & 31);
          const float ws = __shfl_sync(0xffffffffu, my_w, (s0 + s) & 31);
          const bool live = s0 + s < k && row >= 0;
          w[s] = live ? ws : 0.f;
          v[s] = live ? __ldcg(reinterpret_cast<const float4 *>(a.y + (size_t)row * d + c))
                      : make_float4(0.f, 0.f, 0.f, 0.f);
        }
#pragma unroll
        for (int s = 0; s < 8; ++s) {
          if (s0 + s < k && w[s] != 0.f) {
            acc.x = fmaf(w[s], v[s].x, acc.x);
            acc.y = fmaf(w[s], v[s].y, acc.y);
            acc.z = fmaf(w[s], v[s].z, acc.z);
            acc.w = fmaf(w[s], v[s].w, acc.w);
          }
        }
      }
      if (a.residual) {
        const uint2 raw = *reinterpret_cast<const uint2 *>(reinterpret_cast<const uint16_t *>(a.hidden) +
                                                            (size_t)t * d + c);
        float2 lo, hi;
        if (a.is_fp16) {
          const __half2 *h2 = reinterpret_cast<const __half2 *>(&raw);
          lo = __half22float2(h2[0]); hi = __half22float2(h2[1]);
        } else {
          const __nv_bfloat162 *h2 = reinterpret_cast<const __nv_bfloat162 *>(&raw);
          lo = __bfloat1622float2(h2[0]); hi = __bfloat1622float2(h2[1]);
        }
        acc.x += lo.x; acc.y += lo.y; acc.z += hi.x; acc.w += hi.y;
      }
      if (a.out_is_fp32) {
        *reinterpret_cast<float4 *>(reinterpret_cast<float *>(a.out) + (size_t)t * d + c) = acc;
      } else {
        uint2 raw;
        if (a.is_fp16) {
          __half2 lo = __floats2half2_rn(acc.x, acc.y), hi = __floats2half2_rn(acc.z, acc.w);
          raw.x = *reinterpret_cast<uint32_t *>(&lo);
          raw.y = *reinterpret_cast<uint32_t *>(&hi);
        } else {
          __nv_bfloat162 lo = __floats2bfloat162_rn(acc.x, acc.y), hi = __floats2bfloat162_rn(acc.z, acc.w);
          raw.x = *reinterpret_cast<uint32_t *>(&lo);
          raw.y = *reinterpret_cast<uint32_t *>(&hi);
        }
        *reinterpret_cast<uint2 *>(reinterpret_cast<uint16_t *>(a.out) + (size_t)t * d + c) = raw;
      }
    }
  }
}

// ---------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static cudaError_t get_encode_fn(EncodeTiledFn *fn) {
  static EncodeTiledFn cached = nullptr;      // the entry point does not change within a process
  if (cached) {
    *fn = cached;
    return cudaSuccess;
  }
  void *p = nullptr;
  cudaDriverEntryPointQueryResult q;
  cudaError_t e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q);
  if (e != cudaSuccess) return e;
  if (q != cudaDriverEntryPointSuccess || !p) return cudaErrorNotSupported;
  cached = reinterpret_cast<EncodeTiledFn>(p);
  *fn = cached;
  return cudaSuccess;
}

cudaError_t tc_encode_maps(const moespec_layer_desc &d, const Workspace &ws, int R_cap, TcMaps *maps, int *cu_result) {
  EncodeTiledFn enc = nullptr;
  cudaError_t e = get_encode_fn(&enc);
  if (e != cudaSuccess) return e;
  const cuuint32_t ones[3] = {1, 1, 1};
  const CUtensorMapDataType tm_dtype =
      d.dtype == MOESPEC_FP16 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT16 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16;
  auto weights = [&](CUtensorMap *m, const void *base, int rows, int K, int box_rows) -> CUresult {
    cuuint64_t dims[3] = {(cuuint64_t)K, (cuuint64_t)rows, (cuuint64_t)(d.resident_count > 0 ? d.resident_count : d.n_experts)};
    cuuint64_t strides[2] = {(cuuint64_t)K * 2, (cuuint64_t)rows * K * 2};
    cuuint32_t box[3] = {kChunkK, (cuuint32_t)box_rows, 1};
    return enc(m, tm_dtype, 3, const_cast<void *>(base), dims, strides, box, ones,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  };
  auto rows2d = [&](CUtensorMap *m, void *base, int K, int box_rows) -> CUresult {
    cuuint64_t dims[2] = {(cuuint64_t)K, (cuuint64_t)R_cap};
    cuuint64_t strides[1] = {(cuuint64_t)K * 2};
    cuuint32_t box[2] = {kChunkK, (cuuint32_t)box_rows};
    return enc(m, tm_dtype, 2, base, dims, strides, box, ones, CU_TENSOR_MAP_INTERLEAVE_NONE,
               CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  };
  CUresult r = CUDA_SUCCESS;
  for (int i = 0; i < 3 && r == CUDA_SUCCESS; ++i) {
    const int box_rows = kTile >> i;      // 128, 64, 32
    if ((r = weights(&maps->w_gate[i], d.w_gate, d.f, d.d, box_rows)) != CUDA_SUCCESS) break;
    if ((r = weights(&maps->w_up[i], d.w_up, d.f, d.d, box_rows)) != CUDA_SUCCESS) break;
    r = weights(&maps->w_down[i], d.w_down, d.d, d.f, box_rows);
  }
  for (int i = 0; i < 3 && r == CUDA_SUCCESS; ++i) {
    if ((r = rows2d(&maps->x_perm[i], ws.x_perm, d.d, kTokBox << i)) != CUDA_SUCCESS) break;
    r = rows2d(&maps->h_mid[i], ws.h_mid, d.f, kTokBox << i);
  }
  if (r == CUDA_SUCCESS) r = rows2d(&maps->x_perm16, ws.x_perm, d.d, kTokBoxSmall);
  if (r == CUDA_SUCCESS) r = rows2d(&maps->h_mid16, ws.h_mid, d.f, kTokBoxSmall);
  if (r != CUDA_SUCCESS) {
    *cu_result = (int)r;
    return cudaErrorInvalidValue;
  }
  return cudaSuccess;
}

cudaError_t tc_configure() {
  return cudaFuncSetAttribute(ffn_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBudget);
}

// Early start needs every token in one MMA (N <= 128) and is an option of the tensor-core path.
bool tc_dense_all(const moespec_layer_desc &d, int M) { return is_16bit(d.dtype) && M >= 1 && M <= kTokBoxSmall; }

bool tc_early_start(const moespec_layer_desc &d, int M) {
  static const bool off = [] { const char *v = experiment_env("MOESPEC_NO_EARLY"); return v && v[0] == '1'; }();
  return !off && is_16bit(d.dtype) && M >= 1 && M <= kMaxTokChunk;
}

static int sm_count_cached(int device) {
  static int cached[64] = {0};
  if (device < 64 && cached[device]) return cached[device];
  int n = 0;
  if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, device) != cudaSuccess || n <= 0) n = 148;
  if (device < 64) cached[device] = n;
  return n;
}

int tc_grid_size(int device) { return sm_count_cached(device); }

int tc_rows_per_unit(const moespec_layer_desc &D, int M, int k, int B) {
  // Measured on B200: 128-row slabs stream fastest (each unit re-reads its expert's token rows, so
  // shorter slabs double the L2->SM traffic per weight byte); 64-row slabs only pay off when there would
  // otherwise be fewer gate/up units than half the SMs (a handful of kept experts, e.g. M = 1).
  int active = B < D.n_experts ? B : D.n_experts;          // upper bound of kept experts that get rows
  if (D.resident_count > 0 && D.resident_count < active) active = D.resident_count;      // ... on this GPU
  if ((long long)M * k < active) active = M * k;
  static const int forced = [] { const char *v = experiment_env("MOESPEC_FORCE_RU"); return v ? atoi(v) : 0; }();
  if (forced == 128 || forced == 64 || forced == 32) return forced;     // experiments only
  return (long long)active * (D.f / kTile) * 2 < sm_count_cached(D.device) ? 64 : kTile;
}

// Down units use 128-row slabs: half-height ones would shorten the tail of the list but double the copies
// per stage, and measured 10 % slower overall.
int tc_rows_per_down_unit(int ru) {
  static const int forced = [] { const char *v = experiment_env("MOESPEC_FORCE_RU_DOWN"); return v ? atoi(v) : 0; }();
  if (forced == 128 || forced == 64 || forced == 32) return forced;     // experiments only
  (void)ru;
  return kTile;
}

cudaError_t launch_ffn_tensor_core(const LaunchCtx &c, const TcMaps *maps, const void *hidden, void *out) {
  const moespec_layer_desc &D = *c.desc;
  const int ru = c.ru;
  const int ri = ru == 128 ? 0 : ru == 64 ? 1 : 2;
  TcArgs a;
  a.ru = ru;
  a.ru_down = tc_rows_per_down_unit(ru);
  a.kchunks_up = D.d / kChunkK;
  a.kchunks_down = D.f / kChunkK;
  const int n_pad_max = c.M >= kMaxTokChunk ? kMaxTokChunk : (c.M + kTokBox - 1) / kTokBox * kTokBox;
  a.b_region = n_pad_max * 128 * 2 < kBRegionMax ? n_pad_max * 128 * 2 : kBRegionMax;
  a.stage_bytes = kARegion + a.b_region;
  int stages = (kSmemBudget - 1024 - kCtrlBytes - kMmaTail) / a.stage_bytes;
  a.n_stages = stages > kMaxStages ? kMaxStages : stages;
  a.status = c.ws->status;
  a.units = c.ws->units;
  a.n_units = c.ws->counters + 3;
  a.unit_counter = c.ws->unit_counter;
  a.ready = c.ws->ready;
  a.tiles_up = D.f / ru + c.debug_ready_bias;
  a.spin_limit = c.debug_spin_limit > 0 ? c.debug_spin_limit : kSpinLimitCycles;
  a.h_mid = c.ws->h_mid;
  a.is_fp16 = D.dtype == MOESPEC_FP16;
  a.y = c.ws->y;
  a.f = D.f;
  a.d = D.d;
  a.down_done = c.ws->unit_counter + 1;
  a.gate_w = c.ws->gate_w;
  a.tokslot2row = c.ws->tokslot2row;
  a.hidden = hidden;
  a.out = out;
  a.M = c.M;
  a.k = c.k;
  a.residual = D.residual;
  a.out_is_fp32 = (D.out_dtype ? D.out_dtype : D.dtype) == MOESPEC_FP32;
  a.early = c.early;
  a.early_flag = c.ws->early_flag;
  a.n_words = D.n_experts;
  a.res_first = c.res_first;
  a.res_count = c.res_count > 0 && c.res_count < D.n_experts ? c.res_count : 0;      // 0: not a shard
  a.assign_idx = c.ws->assign_idx;
  a.perm_row2tok = c.ws->perm_row2tok;
  a.tiles_real = D.f / ru;
  a.static_nS = 0;
  a.static_order = c.ws->static_order;
  if (a.early && D.shortlist == MOESPEC_STATIC) a.static_nS = c.B < c.ws->n_static ? c.B : c.ws->n_static;
  TcMapsCall m;
  if (a.early || c.dense_all) {
    // the call's input as a TMA tensor [M, d]: rows beyond M read as zeros
    if (maps->hidden_ptr != hidden || maps->hidden_M != c.M) {
      EncodeTiledFn enc = nullptr;
      cudaError_t e = get_encode_fn(&enc);
      if (e != cudaSuccess) return e;
      const int n_pad = c.M <= kTokBoxSmall ? kTokBoxSmall : (c.M + kTokBox - 1) / kTokBox * kTokBox;
      const int box_rows = n_pad == 128 ? 128 : (n_pad % 64 == 0 ? 64 : (n_pad == kTokBoxSmall ? kTokBoxSmall : 32));
      const cuuint64_t dims[2] = {(cuuint64_t)D.d, (cuuint64_t)c.M};
      const cuuint64_t strides[1] = {(cuuint64_t)D.d * 2};
      const cuuint32_t box[2] = {kChunkK, (cuuint32_t)box_rows};
      const cuuint32_t ones[2] = {1, 1};
      const CUresult r = enc(&maps->hidden_map, D.dtype == MOESPEC_FP16 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT16
                                                                        : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16,
                             2, const_cast<void *>(hidden), dims, strides, box, ones, CU_TENSOR_MAP_INTERLEAVE_NONE,
                             CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
      if (r != CUDA_SUCCESS) return cudaErrorInvalidValue;
      maps->hidden_ptr = hidden;
      maps->hidden_M = c.M;
    }
    m.hidden = maps->hidden_map;
  } else {
    m.hidden = maps->x_perm[0];      // unused
  }
  m.w_gate = maps->w_gate[ri];
  m.w_up = maps->w_up[ri];
  m.w_down = maps->w_down[a.ru_down == 128 ? 0 : a.ru_down == 64 ? 1 : 2];
  for (int i = 0; i < 3; ++i) {
    m.x_perm[i] = maps->x_perm[i];
    m.h_mid[i] = maps->h_mid[i];
  }
  m.x_perm16 = maps->x_perm16;
  m.h_mid16 = maps->h_mid16;
  const int grid = sm_count_cached(D.device);
  const size_t smem = (size_t)a.n_stages * a.stage_bytes + kMmaTail + 1024 + kCtrlBytes;
  return launch_kernel(ffn_tc_kernel, dim3(grid), dim3(kThreads), smem, c.stream, m, a);
}

}  // namespace moespec
