// C ABI of libmoespec: handle life cycle, argument validation, workspace, launch order.
#include "internal.h"

#include <cstdlib>
#include <limits>
#include <mutex>
#include <new>
#include <unordered_set>
#include <vector>

using namespace moespec;

constexpr int kMaxProfiled = 8;   // kernels per verify call that can be bracketed by events
constexpr int kGraphCache = 4;    // instantiated graphs kept per handle (least recently used is replaced)

// One cached instantiation of the host entry point: the step for (M, k, B, buffer pair).
struct HostGraph {
  cudaGraphExec_t exec = nullptr;
  int M = 0, k = 0, B = 0;
  const void *in = nullptr;
  void *out = nullptr;
  unsigned long long used = 0;
};

struct moespec_layer {
  unsigned long long magic;
  moespec_layer_desc desc;
  Workspace ws;
  void *arena;
  size_t arena_bytes;
  int R_cap;
  bool use_tc;
  TcMaps maps;
  int last_M, last_k;
  int last_launches;
  bool profiling;
  cudaEvent_t ev[kMaxProfiled + 1];
  // host-buffer entry point: the copy-in, the kernels and the copy-out as one instantiated graph
  cudaStream_t own_stream;
  cudaEvent_t ev_in;
  HostGraph host_graph[kGraphCache];
  unsigned long long graph_clock;
  bool graph_usable;
  long long debug_spin_limit;
  int debug_ready_bias;
  unsigned epoch;       // bumped whenever something a captured graph has baked in changes
  // analysis mode (allocated by the first moespec_oracle_ranking / moespec_reconstruction_error call)
  char *analysis;       // gram [max_M, max_k, max_k] f64 | row2slot [R_cap] | order [N] | objective [N] f64 | sums
  double *an_gram, *an_objective, *an_sums, *an_partial;
  int *an_row2slot, *an_order;
  int an_M, an_k;       // shape of the Gram matrices held
};

// L layers on one residual stream (the MoE blocks of a model, one after the other)
struct moespec_stack {
  unsigned long long magic;
  std::vector<moespec_layer *> layers;
  int device, d, dtype, max_M, max_k;
  size_t row_bytes;         // d * sizeof(dtype)
  char *arena;              // x_1 .. x_{L-1}, then the host entry point's staging buffers
  char *in_stage, *out_stage;
  bool graph_on, graph_usable;
  cudaStream_t own_stream;
  cudaEvent_t ev_in;
  struct Graph {            // one cached instantiation: (M, k, budgets, buffers, epochs)
    cudaGraphExec_t exec = nullptr;
    int M = 0, k = 0;
    std::vector<int> B;
    const void *in = nullptr;
    void *out = nullptr;
    bool host = false;
    unsigned epoch = 0;
    unsigned long long used = 0;
  } graph[kGraphCache];
  unsigned long long graph_clock;
  int last_M, last_launches;
};

namespace {

constexpr unsigned long long kMagic = 0x4d6f455370656331ULL;
thread_local int tl_cuda_error = 0;
std::mutex g_mu;
std::unordered_set<moespec_layer *> g_live;
std::unordered_set<moespec_stack *> g_live_stacks;
constexpr unsigned long long kStackMagic = 0x4d6f455370656353ULL;

int cuda_fail(cudaError_t e) {
  tl_cuda_error = (int)e;
  return e == cudaErrorMemoryAllocation ? MOESPEC_ERR_OUT_OF_MEMORY : MOESPEC_ERR_CUDA;
}

}  // namespace
namespace moespec {
void record_cuda_error(cudaError_t e) { tl_cuda_error = (int)e; }
}
namespace {

bool is_live(moespec_layer *L) {
  if (!L) return false;
  std::lock_guard<std::mutex> lk(g_mu);
  return g_live.count(L) != 0 && L->magic == kMagic;
}

bool is_live(moespec_stack *S) {
  if (!S) return false;
  std::lock_guard<std::mutex> lk(g_mu);
  return g_live_stacks.count(S) != 0 && S->magic == kStackMagic;
}

struct DeviceGuard {
  int prev = -1;
  bool changed = false;
  cudaError_t err = cudaSuccess;
  explicit DeviceGuard(int dev) {
    err = cudaGetDevice(&prev);
    if (err == cudaSuccess && prev != dev) {
      err = cudaSetDevice(dev);
      changed = err == cudaSuccess;
    }
  }
  ~DeviceGuard() {
    if (changed) cudaSetDevice(prev);
  }
};

// A captured graph has the layer's settings baked into its kernel arguments: drop them all.
void drop_host_graphs(moespec_layer *L) {
  for (HostGraph &g : L->host_graph) {
    if (g.exec) cudaGraphExecDestroy(g.exec);
    g = HostGraph();
  }
}

size_t elt_bytes(const moespec_layer_desc &d) { return dtype_bytes(d.dtype); }
size_t out_elt_bytes(const moespec_layer_desc &d) { return dtype_bytes(d.out_dtype ? d.out_dtype : d.dtype); }

struct Carver {
  size_t off = 0;
  char *base = nullptr;
  template <typename T>
  void take(T *&p, size_t count) {
    off = (off + 255) & ~(size_t)255;
    if (base) p = reinterpret_cast<T *>(base + off);
    off += count * sizeof(T);
  }
  void take_bytes(void *&p, size_t bytes) {
    off = (off + 255) & ~(size_t)255;
    if (base) p = base + off;
    off += bytes;
  }
};

size_t carve(const moespec_layer_desc &d, int R_cap, char *base, Workspace *ws) {
  Carver c;
  c.base = base;
  Workspace w{};
  const size_t N = d.n_experts, M = d.max_M, K = d.max_k, eb = elt_bytes(d);
  const size_t tiles_up = d.f / 32 + 1, tiles_down = d.d / 32 + 1;      // smallest slab height is 32 rows
  // every expert can add at most one partial token chunk beyond the full ones
  const size_t max_chunks = (size_t)R_cap / kMaxTokChunk + N;
  c.take(w.logits, M * N);
  c.take(w.prob, M * N);
  c.take(w.score, N);
  c.take(w.topk_idx, M * K);
  c.take(w.S_rank, N);
  c.take(w.assign_idx, M * K);
  c.take(w.gate_w, M * K);
  c.take(w.count, N);
  c.take(w.offset, N + 1);
  c.take(w.active, N);
  c.take(w.perm_row2tok, (size_t)R_cap);
  c.take(w.gather_src, (size_t)R_cap);
  c.take(w.row2expert, (size_t)R_cap);
  c.take(w.tokslot2row, M * K);
  w.mask_words = (int)((M + 31) / 32);
  c.take(w.score_fx, N);
  c.take(w.natcnt_acc, N);
  c.take(w.count_acc, N);
  c.take(w.colmask, N * (size_t)w.mask_words);
  c.take(w.arrive, M);
  c.take(w.arrive_route, 4);
  c.take(w.early_flag, N);
  c.take(w.calib_count, N);
  c.take(w.static_pos, N);
  c.take(w.static_order, N);
  w.n_static = 0;
  c.take(w.units, max_chunks * (tiles_up + tiles_down));
  c.take(w.ready, max_chunks);
  c.take(w.unit_counter, 4);
  c.take(w.counters, 16);
  c.take(w.stats, 1);
  c.take(w.status, 4);
  c.take_bytes(w.x_perm, (size_t)R_cap * d.d * eb);
  c.take_bytes(w.h_mid, (size_t)R_cap * d.f * eb);
  c.take(w.y, (size_t)R_cap * d.d);
  c.take_bytes(w.hidden_stage, M * d.d * eb);
  c.take_bytes(w.out_stage, M * d.d * out_elt_bytes(d));
  if (ws) *ws = w;
  return (c.off + 255) & ~(size_t)255;
}

int validate_call(moespec_layer *L, int M, int k, int B) {
  const moespec_layer_desc &d = L->desc;
  if (d.shortlist == MOESPEC_STATIC && L->ws.n_static == 0) return MOESPEC_ERR_INVALID_ARG;   // no ranking set
  if (M < 0 || M > d.max_M) return MOESPEC_ERR_INVALID_ARG;
  if (k < 1 || k > d.max_k || k > d.n_experts) return MOESPEC_ERR_INVALID_ARG;
  if (B < 1) return MOESPEC_ERR_INVALID_ARG;
  return MOESPEC_OK;
}

bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

bool zero_copy_enabled() {
  static const bool off = [] { const char *v = experiment_env("MOESPEC_NO_ZERO_COPY"); return v && v[0] == '1'; }();
  return !off;
}

bool is_pinned(const void *p) {
  cudaPointerAttributes at;
  if (cudaPointerGetAttributes(&at, p) != cudaSuccess) {
    cudaGetLastError();
    return false;
  }
  return at.type == cudaMemoryTypeHost;
}

// Device-side address of a page-locked host buffer (nullptr when the buffer is not mapped for the device).
void *mapped_device_pointer(const void *p) {
  cudaPointerAttributes at;
  if (cudaPointerGetAttributes(&at, p) != cudaSuccess) {
    cudaGetLastError();
    return nullptr;
  }
  return at.type == cudaMemoryTypeHost ? at.devicePointer : nullptr;
}

// hidden (page-locked host memory, read over the interconnect) -> the layer's staging buffer.  Every thread
// has one 16-byte load in flight, so the copy is one interconnect round trip plus the transfer time; the
// router kernel behind it is launched programmatically and overlaps its prologue.
__global__ void __launch_bounds__(256) stage_in_kernel(const uint4 *__restrict__ src, uint4 *__restrict__ dst, size_t n16) {
  pdl_trigger();
  pdl_wait();          // the staging buffer may still be read by the previous call's kernels
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n16; i += (size_t)gridDim.x * blockDim.x)
    dst[i] = src[i];
}

int run_layer(moespec_layer *L, const void *hidden, int M, int k, int B, void *out, cudaStream_t stream,
              const moespec_layer_desc *desc = nullptr) {
  if (!desc) desc = &L->desc;      // the analysis mode runs the same weights under other routing settings
  LaunchCtx c{desc, &L->ws, M, k, B > L->desc.n_experts ? L->desc.n_experts : B, L->R_cap, stream, 0};
  c.res_first = L->desc.resident_first;
  c.res_count = L->desc.resident_count;
  if (L->use_tc) {
    c.ru = tc_rows_per_unit(L->desc, M, k, c.B);
    c.early = tc_early_start(*desc, M) ? 1 : 0;
    c.dense_all = tc_dense_all(*desc, M) ? 1 : 0;
    // The early units follow the shortlist's rank order.  Router-based ranks follow the tokens' own
    // probabilities, so the leading experts have rows; a fixed ordering (Eq. 4) does not look at the tree,
    // and with few tokens most of its leading experts get none: the early units would stream unused weights.
    if (desc->shortlist == MOESPEC_STATIC) {
      const int nS = c.B < L->ws.n_static ? c.B : L->ws.n_static;
      if ((long long)M * k < 4LL * nS) c.early = 0;
    }
  }
  c.debug_spin_limit = L->debug_spin_limit;
  c.debug_ready_bias = L->debug_ready_bias;
  int launches = 0;
  cudaError_t e;
  // with profiling on, an event is recorded before the first kernel and after every kernel
  auto mark = [&](int i) -> cudaError_t {
    return (L->profiling && i <= kMaxProfiled) ? cudaEventRecord(L->ev[i], stream) : cudaSuccess;
  };
  if ((e = mark(0)) != cudaSuccess) return cuda_fail(e);
  if ((e = launch_router_logits(c, hidden)) != cudaSuccess) return cuda_fail(e);
  if ((e = mark(++launches)) != cudaSuccess) return cuda_fail(e);
  if ((e = launch_route_after_router(c)) != cudaSuccess) return cuda_fail(e);
  if ((e = mark(++launches)) != cudaSuccess) return cuda_fail(e);
  if (!c.dense_all) {      // (trees of at most 16 tokens need no gathered rows on the tensor-core path)
    if ((e = launch_gather(c, hidden)) != cudaSuccess) return cuda_fail(e);
    if ((e = mark(++launches)) != cudaSuccess) return cuda_fail(e);
  }
  if (L->use_tc) {
    // both FFN phases and the combine are one persistent kernel
    if ((e = launch_ffn_tensor_core(c, &L->maps, hidden, out)) != cudaSuccess) return cuda_fail(e);
    if ((e = mark(++launches)) != cudaSuccess) return cuda_fail(e);
  } else {
    for (int phase = 0; phase < 2; ++phase) {
      if ((e = launch_ffn_cuda_core(c, phase)) != cudaSuccess) return cuda_fail(e);
      if ((e = mark(++launches)) != cudaSuccess) return cuda_fail(e);
    }
    if ((e = launch_combine(c, hidden, out)) != cudaSuccess) return cuda_fail(e);
    if ((e = mark(++launches)) != cudaSuccess) return cuda_fail(e);
  }
  L->last_M = M;
  L->last_k = k;
  L->last_launches = launches;
  return MOESPEC_OK;
}

}  // namespace

namespace moespec {
bool pdl_enabled() {
  static const bool on = [] {
    const char *v = experiment_env("MOESPEC_NO_PDL");
    return !(v && v[0] == '1');
  }();
  return on;
}
}  // namespace moespec

extern "C" {

int moespec_layer_create(const moespec_layer_desc *desc, moespec_layer_t **out_layer) {
  if (!desc || !out_layer) return MOESPEC_ERR_NULL_POINTER;
  const moespec_layer_desc &d = *desc;
  if (!d.router_w || !d.w_gate || !d.w_up || !d.w_down) return MOESPEC_ERR_NULL_POINTER;
  if (d.dtype != MOESPEC_BF16 && d.dtype != MOESPEC_FP32 && d.dtype != MOESPEC_FP16) return MOESPEC_ERR_INVALID_ARG;
  if (d.out_dtype != 0 && d.out_dtype != MOESPEC_BF16 && d.out_dtype != MOESPEC_FP32 && d.out_dtype != MOESPEC_FP16)
    return MOESPEC_ERR_INVALID_ARG;
  // out is either the layer's dtype or fp32
  if (d.out_dtype != 0 && d.out_dtype != d.dtype && d.out_dtype != MOESPEC_FP32) return MOESPEC_ERR_UNSUPPORTED;
  if (d.policy != MOESPEC_SUBSTITUTION && d.policy != MOESPEC_TRUNCATION) return MOESPEC_ERR_INVALID_ARG;
  if (d.shortlist != MOESPEC_FROM_ALL && d.shortlist != MOESPEC_FROM_UNION && d.shortlist != MOESPEC_STATIC)
    return MOESPEC_ERR_INVALID_ARG;
  if ((d.renormalize | 1) != 1 || (d.residual | 1) != 1) return MOESPEC_ERR_INVALID_ARG;
  if (d.ffn_kernel < MOESPEC_FFN_AUTO || d.ffn_kernel > MOESPEC_FFN_TENSOR_CORE) return MOESPEC_ERR_INVALID_ARG;
  if (d.d < 64 || d.f < 64 || d.n_experts < 1 || d.max_M < 1 || d.max_k < 1 || d.device < 0)
    return MOESPEC_ERR_INVALID_ARG;
  if (d.n_experts > kMaxExperts || d.max_k > kMaxK || d.max_k > d.n_experts || d.max_M > 4096 || d.d > 16384 ||
      d.f > 65536)
    return MOESPEC_ERR_INVALID_ARG;
  if (d.d % 64 || d.f % 64) return MOESPEC_ERR_UNSUPPORTED;
  if (d.resident_count < 0 || d.resident_first < 0) return MOESPEC_ERR_INVALID_ARG;
  if (d.resident_count == 0 && d.resident_first != 0) return MOESPEC_ERR_INVALID_ARG;
  if (d.resident_count > 0 && d.resident_first + d.resident_count > d.n_experts) return MOESPEC_ERR_INVALID_ARG;
  if (d.resident_count > 0 && d.resident_count < d.n_experts && d.residual) return MOESPEC_ERR_INVALID_ARG;
  if (!aligned16(d.router_w) || !aligned16(d.w_gate) || !aligned16(d.w_up) || !aligned16(d.w_down))
    return MOESPEC_ERR_UNSUPPORTED;
  bool use_tc = d.ffn_kernel == MOESPEC_FFN_TENSOR_CORE ||
                (d.ffn_kernel == MOESPEC_FFN_AUTO && is_16bit(d.dtype));
  if (use_tc && (!is_16bit(d.dtype) || d.d % kTile || d.f % kTile)) {
    if (d.ffn_kernel == MOESPEC_FFN_TENSOR_CORE) return MOESPEC_ERR_UNSUPPORTED;
    use_tc = false;
  }

  int n_dev = 0;
  cudaError_t e = cudaGetDeviceCount(&n_dev);
  if (e != cudaSuccess) return cuda_fail(e);
  if (d.device >= n_dev) return MOESPEC_ERR_INVALID_ARG;
  DeviceGuard guard(d.device);
  if (guard.err != cudaSuccess) return cuda_fail(guard.err);

  moespec_layer *L = new (std::nothrow) moespec_layer();
  if (!L) return MOESPEC_ERR_OUT_OF_MEMORY;
  L->magic = kMagic;
  L->desc = d;
  if (L->desc.resident_count == 0) L->desc.resident_count = d.n_experts;      // all experts are resident
  L->R_cap = d.max_M * d.max_k;
  L->use_tc = use_tc;
  L->arena_bytes = carve(d, L->R_cap, nullptr, nullptr);
  e = cudaMalloc(&L->arena, L->arena_bytes);
  if (e != cudaSuccess) {
    delete L;
    cudaGetLastError();
    return cuda_fail(e);
  }
  e = cudaMemset(L->arena, 0, L->arena_bytes);
  if (e != cudaSuccess) {
    cudaFree(L->arena);
    delete L;
    return cuda_fail(e);
  }
  carve(d, L->R_cap, static_cast<char *>(L->arena), &L->ws);
  if (!use_tc) {
    // the CUDA-core FFN stages a row of d (gate/up) or f (down) floats in shared memory
    bool fits = true;
    e = cc_configure(d, &fits);
    if (e != cudaSuccess || !fits) {
      cudaFree(L->arena);
      delete L;
      return e != cudaSuccess ? cuda_fail(e) : MOESPEC_ERR_UNSUPPORTED;
    }
  }
  if (use_tc) {
    int cu_res = 0;
    e = tc_encode_maps(L->desc, L->ws, L->R_cap, &L->maps, &cu_res);
    if (e == cudaSuccess) e = tc_configure();
    if (e == cudaSuccess) e = routing_configure();
    if (e != cudaSuccess) {
      cudaFree(L->arena);
      delete L;
      tl_cuda_error = cu_res ? cu_res : (int)e;
      return MOESPEC_ERR_CUDA;
    }
  }
  L->profiling = false;
  L->debug_spin_limit = 0;
  L->debug_ready_bias = 0;
  L->epoch = 0;
  L->analysis = nullptr;
  L->an_M = L->an_k = 0;
  L->graph_clock = 0;
  L->graph_usable = cudaStreamCreateWithFlags(&L->own_stream, cudaStreamNonBlocking) == cudaSuccess &&
                    cudaEventCreateWithFlags(&L->ev_in, cudaEventDisableTiming) == cudaSuccess;
  for (int i = 0; i <= kMaxProfiled; ++i) {
    e = cudaEventCreate(&L->ev[i]);
    if (e != cudaSuccess) {
      for (int j = 0; j < i; ++j) cudaEventDestroy(L->ev[j]);
      cudaFree(L->arena);
      delete L;
      return cuda_fail(e);
    }
  }
  {
    std::lock_guard<std::mutex> lk(g_mu);
    g_live.insert(L);
  }
  *out_layer = L;
  return MOESPEC_OK;
}

int moespec_verify_layer(moespec_layer_t *L, const void *hidden, int M, int k, int B, void *out, void *stream) {
  if (!is_live(L)) return MOESPEC_ERR_BAD_HANDLE;
  int rc = validate_call(L, M, k, B);
  if (rc) return rc;
  if (M == 0) return MOESPEC_OK;
  if (!hidden || !out) return MOESPEC_ERR_NULL_POINTER;
  if (!aligned16(hidden) || !aligned16(out)) return MOESPEC_ERR_UNSUPPORTED;
  if (hidden == out) return MOESPEC_ERR_INVALID_ARG;
  DeviceGuard guard(L->desc.device);
  if (guard.err != cudaSuccess) return cuda_fail(guard.err);
  return run_layer(L, hidden, M, k, B, out, static_cast<cudaStream_t>(stream));
}

int moespec_verify_layer_host(moespec_layer_t *L, const void *hidden_host, int M, int k, int B, void *out_host,
                              void *stream) {
  if (!is_live(L)) return MOESPEC_ERR_BAD_HANDLE;
  int rc = validate_call(L, M, k, B);
  if (rc) return rc;
  if (M == 0) return MOESPEC_OK;
  if (!hidden_host || !out_host) return MOESPEC_ERR_NULL_POINTER;
  DeviceGuard guard(L->desc.device);
  if (guard.err != cudaSuccess) return cuda_fail(guard.err);
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const size_t bytes = (size_t)M * L->desc.d * elt_bytes(L->desc);
  const size_t out_bytes = (size_t)M * L->desc.d * out_elt_bytes(L->desc);
  cudaError_t e;

  // Fast path: pinned buffers.  The copy-in, the kernels and the copy-out are captured once per
  // (M, k, B, buffers) into a graph on an internal stream and replayed with a single launch.  When both
  // buffers are mapped into the device's address space (page-locked memory under unified addressing) there
  // are no copy nodes at all: a kernel pulls hidden into the staging buffer and the layer's last kernel
  // writes `out` straight to the host buffer, which saves the copy engine's hand-overs on both sides.
  void *in_dev = mapped_device_pointer(hidden_host), *out_dev = mapped_device_pointer(out_host);
  const bool zero_copy = in_dev && out_dev && aligned16(in_dev) && aligned16(out_dev) && bytes % 16 == 0 &&
                         zero_copy_enabled();
  if (L->graph_usable && !L->profiling && is_pinned(hidden_host) && is_pinned(out_host)) {
    // a few instantiations are kept (a caller may alternate between trees or buffer pairs); a miss replaces
    // the least recently used one
    HostGraph *slot = nullptr;
    for (HostGraph &g : L->host_graph)
      if (g.exec && g.M == M && g.k == k && g.B == B && g.in == hidden_host && g.out == out_host) slot = &g;
    const bool hit = slot != nullptr;
    if (!hit) {
      slot = &L->host_graph[0];
      for (HostGraph &g : L->host_graph)
        if (!g.exec || (slot->exec && g.used < slot->used)) slot = &g;
      if (slot->exec) cudaGraphExecDestroy(slot->exec);
      *slot = HostGraph();
      cudaGraph_t graph = nullptr;
      e = cudaStreamBeginCapture(L->own_stream, cudaStreamCaptureModeThreadLocal);
      if (e == cudaSuccess) {
        if (zero_copy) {
          const size_t n16 = bytes / 16;
          const unsigned grid = (unsigned)((n16 + 255) / 256 < 296 ? (n16 + 255) / 256 : 296);
          e = launch_kernel(stage_in_kernel, dim3(grid), dim3(256), 0, L->own_stream, (const uint4 *)in_dev,
                            (uint4 *)L->ws.hidden_stage, n16);
          if (e == cudaSuccess && run_layer(L, L->ws.hidden_stage, M, k, B, out_dev, L->own_stream) != MOESPEC_OK)
            e = cudaErrorUnknown;
        } else {
          e = cudaMemcpyAsync(L->ws.hidden_stage, hidden_host, bytes, cudaMemcpyHostToDevice, L->own_stream);
          if (e == cudaSuccess && run_layer(L, L->ws.hidden_stage, M, k, B, L->ws.out_stage, L->own_stream) != MOESPEC_OK)
            e = cudaErrorUnknown;
          if (e == cudaSuccess)
            e = cudaMemcpyAsync(out_host, L->ws.out_stage, out_bytes, cudaMemcpyDeviceToHost, L->own_stream);
        }
        cudaError_t e2 = cudaStreamEndCapture(L->own_stream, &graph);
        if (e == cudaSuccess) e = e2;
      }
      if (e == cudaSuccess) e = cudaGraphInstantiate(&slot->exec, graph, 0);
      if (graph) cudaGraphDestroy(graph);
      if (e != cudaSuccess) {          // graphs unavailable here: use the plain path from now on
        cudaGetLastError();
        slot->exec = nullptr;
        L->graph_usable = false;
      } else {
        slot->M = M; slot->k = k; slot->B = B; slot->in = hidden_host; slot->out = out_host;
      }
    }
    if (slot->exec) {
      slot->used = ++L->graph_clock;
      // work already queued on the caller's stream (e.g. a weight update) is waited for first; the replay
      // itself runs on the internal stream (measured faster than replaying on the legacy default stream)
      if ((e = cudaEventRecord(L->ev_in, s)) != cudaSuccess) return cuda_fail(e);
      if ((e = cudaStreamWaitEvent(L->own_stream, L->ev_in, 0)) != cudaSuccess) return cuda_fail(e);
      if ((e = cudaGraphLaunch(slot->exec, L->own_stream)) != cudaSuccess) return cuda_fail(e);
      if ((e = cudaStreamSynchronize(L->own_stream)) != cudaSuccess) return cuda_fail(e);
      return MOESPEC_OK;
    }
  }

  e = cudaMemcpyAsync(L->ws.hidden_stage, hidden_host, bytes, cudaMemcpyHostToDevice, s);
  if (e != cudaSuccess) return cuda_fail(e);
  rc = run_layer(L, L->ws.hidden_stage, M, k, B, L->ws.out_stage, s);
  if (rc) return rc;
  e = cudaMemcpyAsync(out_host, L->ws.out_stage, out_bytes, cudaMemcpyDeviceToHost, s);
  if (e != cudaSuccess) return cuda_fail(e);
  e = cudaStreamSynchronize(s);
  if (e != cudaSuccess) return cuda_fail(e);
  return MOESPEC_OK;
}

#define MOESPEC_COPY_BACK(dst, src, count)                                                         \
  do {                                                                                             \
    if ((dst) && (count) > 0) {                                                                    \
      cudaError_t e_ = cudaMemcpy((dst), (src), sizeof(*(dst)) * (size_t)(count), cudaMemcpyDeviceToHost); \
      if (e_ != cudaSuccess) return cuda_fail(e_);                                                 \
    }                                                                                              \
  } while (0)

int moespec_calibrate(moespec_layer_t *L, const void *hidden, int M, int k, void *stream) {
  if (!is_live(L)) return MOESPEC_ERR_BAD_HANDLE;
  const moespec_layer_desc &d = L->desc;
  if (M < 0 || M > d.max_M || k < 1 || k > d.max_k || k > d.n_experts) return MOESPEC_ERR_INVALID_ARG;
  if (M == 0) return MOESPEC_OK;
  if (!hidden) return MOESPEC_ERR_NULL_POINTER;
  if (!aligned16(hidden)) return MOESPEC_ERR_UNSUPPORTED;
  DeviceGuard guard(d.device);
  if (guard.err != cudaSuccess) return cuda_fail(guard.err);
  LaunchCtx c{&L->desc, &L->ws, M, k, 1, L->R_cap, static_cast<cudaStream_t>(stream), 0};
  cudaError_t e = launch_router_logits(c, hidden);
  if (e == cudaSuccess) e = launch_calib_accumulate(c);
  if (e != cudaSuccess) return cuda_fail(e);
  L->last_M = M;
  L->last_k = k;
  L->last_launches = 2;
  return MOESPEC_OK;
}

int moespec_get_static_counts(moespec_layer_t *L, long long *counts_host) {
  if (!is_live(L)) return MOESPEC_ERR_BAD_HANDLE;
  if (!counts_host) return MOESPEC_ERR_NULL_POINTER;
  DeviceGuard guard(L->desc.device);
  if (guard.err != cudaSuccess) return cuda_fail(guard.err);
  cudaError_t e = cudaDeviceSynchronize();
  if (e != cudaSuccess) return cuda_fail(e);
  MOESPEC_COPY_BACK(counts_host, L->ws.calib_count, L->desc.n_experts);
  return MOESPEC_OK;
}

int moespec_reset_calibration(moespec_layer_t *L) {
  if (!is_live(L)) return MOESPEC_ERR_BAD_HANDLE;
  DeviceGuard guard(L->desc.device);
  if (guard.err != cudaSuccess) return cuda_fail(guard.err);
  cudaError_t e = cudaDeviceSynchronize();
  if (e == cudaSuccess) e = cudaMemset(L->ws.calib_count, 0, sizeof(long long) * L->desc.n_experts);
  return e == cudaSuccess ? MOESPEC_OK : cuda_fail(e);
}

int moespec_set_static_ranking(moespec_layer_t *L, const int *ranked_host, int n) {
  if (!is_live(L)) return MOESPEC_ERR_BAD_HANDLE;
  const int N = L->desc.n_experts;
  DeviceGuard guard(L->desc.device);
  if (guard.err != cudaSuccess) return cuda_fail(guard.err);
  cudaError_t e = cudaDeviceSynchronize();
  if (e != cudaSuccess) return cuda_fail(e);
  std::vector<int> order;
  if (ranked_host) {
    if (n < 1 || n > N) return MOESPEC_ERR_INVALID_ARG;
    order.assign(ranked_host, ranked_host + n);
  } else {
    std::vector<long long> cnt(N);
    e = cudaMemcpy(cnt.data(), L->ws.calib_count, sizeof(long long) * N, cudaMemcpyDeviceToHost);
    if (e != cudaSuccess) return cuda_fail(e);
    order.resize(N);
    for (int i = 0; i < N; ++i) order[i] = i;
    // (count descending, expert index ascending); insertion sort keeps the file free of <algorithm> lambdas
    for (int i = 1; i < N; ++i) {
      const int x = order[i];
      int j = i - 1;
      while (j >= 0 && (cnt[order[j]] < cnt[x] || (cnt[order[j]] == cnt[x] && order[j] > x))) {
        order[j + 1] = order[j];
        --j;
      }
      order[j + 1] = x;
    }
  }
  std::vector<int> pos(N, 0x7fffffff);
  for (size_t r = 0; r < order.size(); ++r) {
    const int ex = order[r];
    if (ex < 0 || ex >= N || pos[ex] != 0x7fffffff) return MOESPEC_ERR_INVALID_ARG;   // out of range or repeated
    pos[ex] = (int)r;
  }
  e = cudaMemcpy(L->ws.static_pos, pos.data(), sizeof(int) * N, cudaMemcpyHostToDevice);
  if (e != cudaSuccess) return cuda_fail(e);
  e = cudaMemcpy(L->ws.static_order, order.data(), sizeof(int) * order.size(), cudaMemcpyHostToDevice);
  if (e != cudaSuccess) return cuda_fail(e);
  L->ws.n_static = (int)order.size();
  ++L->epoch;
  drop_host_graphs(L);           // a captured graph has the old ordering size baked into its arguments
  return MOESPEC_OK;
}

int moespec_route_from_logits(moespec_layer_t *L, const float *logits, int M, int k, int B, void *stream) {
  if (!is_live(L)) return MOESPEC_ERR_BAD_HANDLE;
  int rc = validate_call(L, M, k, B);
  if (rc) return rc;
  if (M == 0) return MOESPEC_OK;
  if (!logits) return MOESPEC_ERR_NULL_POINTER;
  DeviceGuard guard(L->desc.device);
  if (guard.err != cudaSuccess) return cuda_fail(guard.err);
  LaunchCtx c{&L->desc, &L->ws, M, k, B > L->desc.n_experts ? L->desc.n_experts : B, L->R_cap,
              static_cast<cudaStream_t>(stream), 0};
  if (L->use_tc) c.ru = tc_rows_per_unit(L->desc, M, k, c.B);
  c.res_first = L->desc.resident_first;
  c.res_count = L->desc.resident_count;
  cudaError_t e = launch_route(c, logits);
  if (e != cudaSuccess) return cuda_fail(e);
  L->last_M = M;
  L->last_k = k;
  L->last_launches = M > kMaxTokChunk ? 3 : 2;      // large trees add the row kernel
  return MOESPEC_OK;
}


int moespec_get_routing(moespec_layer_t *L, int *S_rank, int *n_S, int *topk_idx, int *assign_idx, float *gate_w,
                        int *count, int *offset, int *perm_row2tok, int *tokslot2row, double *score,
                        int *n_rows) {
  if (!is_live(L)) return MOESPEC_ERR_BAD_HANDLE;
  DeviceGuard guard(L->desc.device);
  if (guard.err != cudaSuccess) return cuda_fail(guard.err);
  cudaError_t e = cudaDeviceSynchronize();
  if (e != cudaSuccess) return cuda_fail(e);
  int counters[8];
  e = cudaMemcpy(counters, L->ws.counters, sizeof(counters), cudaMemcpyDeviceToHost);
  if (e != cudaSuccess) return cuda_fail(e);
  const int N = L->desc.n_experts, mk = L->last_M * L->last_k;
  if (n_S) *n_S = counters[0];
  if (n_rows) *n_rows = counters[2];
  MOESPEC_COPY_BACK(S_rank, L->ws.S_rank, counters[0]);
  MOESPEC_COPY_BACK(topk_idx, L->ws.topk_idx, mk);
  MOESPEC_COPY_BACK(assign_idx, L->ws.assign_idx, mk);
  MOESPEC_COPY_BACK(gate_w, L->ws.gate_w, mk);
  MOESPEC_COPY_BACK(count, L->ws.count, N);
  MOESPEC_COPY_BACK(offset, L->ws.offset, N + 1);
  MOESPEC_COPY_BACK(perm_row2tok, L->ws.perm_row2tok, counters[2]);
  MOESPEC_COPY_BACK(tokslot2row, L->ws.tokslot2row, mk);
  MOESPEC_COPY_BACK(score, L->ws.score, N);
  return MOESPEC_OK;
}

int moespec_get_logits(moespec_layer_t *L, float *logits_host) {
  if (!is_live(L)) return MOESPEC_ERR_BAD_HANDLE;
  if (!logits_host) return MOESPEC_ERR_NULL_POINTER;
  DeviceGuard guard(L->desc.device);
  if (guard.err != cudaSuccess) return cuda_fail(guard.err);
  cudaError_t e = cudaDeviceSynchronize();
  if (e != cudaSuccess) return cuda_fail(e);
  MOESPEC_COPY_BACK(logits_host, L->ws.logits, L->last_M * L->desc.n_experts);
  return MOESPEC_OK;
}

int moespec_get_intermediate(moespec_layer_t *L, int which, void *host_buf, long long bytes) {
  if (!is_live(L)) return MOESPEC_ERR_BAD_HANDLE;
  if (!host_buf) return MOESPEC_ERR_NULL_POINTER;
  if (which < 0 || which > 2 || bytes < 0) return MOESPEC_ERR_INVALID_ARG;
  DeviceGuard guard(L->desc.device);
  if (guard.err != cudaSuccess) return cuda_fail(guard.err);
  cudaError_t e = cudaDeviceSynchronize();
  if (e != cudaSuccess) return cuda_fail(e);
  const size_t eb = elt_bytes(L->desc), R = (size_t)L->R_cap;
  const void *src = which == 0 ? L->ws.x_perm : which == 1 ? L->ws.h_mid : (const void *)L->ws.y;
  size_t cap = which == 0 ? R * L->desc.d * eb : which == 1 ? R * L->desc.f * eb : R * L->desc.d * 4;
  size_t n = (size_t)bytes < cap ? (size_t)bytes : cap;
  if (n) {
    e = cudaMemcpy(host_buf, src, n, cudaMemcpyDeviceToHost);
    if (e != cudaSuccess) return cuda_fail(e);
  }
  return MOESPEC_OK;
}

int moespec_get_stats(moespec_layer_t *L, moespec_stats *stats) {
  if (!is_live(L)) return MOESPEC_ERR_BAD_HANDLE;
  if (!stats) return MOESPEC_ERR_NULL_POINTER;
  DeviceGuard guard(L->desc.device);
  if (guard.err != cudaSuccess) return cuda_fail(guard.err);
  cudaError_t e = cudaDeviceSynchronize();
  if (e != cudaSuccess) return cuda_fail(e);
  MOESPEC_COPY_BACK(stats, L->ws.stats, 1);
  int status = 0;
  e = cudaMemcpy(&status, L->ws.status, sizeof(int), cudaMemcpyDeviceToHost);
  if (e != cudaSuccess) return cuda_fail(e);
  stats->status = status;
  return MOESPEC_OK;
}

int moespec_debug_set_wait(moespec_layer_t *L, long long limit_cycles, int ready_bias) {
  if (!is_live(L)) return MOESPEC_ERR_BAD_HANDLE;
  if (limit_cycles < 0 || ready_bias < 0) return MOESPEC_ERR_INVALID_ARG;
  L->debug_spin_limit = limit_cycles;
  L->debug_ready_bias = ready_bias;
  ++L->epoch;
  drop_host_graphs(L);           // a captured graph has the old values baked in
  return MOESPEC_OK;
}

int moespec_set_profiling(moespec_layer_t *L, int on) {
  if (!is_live(L)) return MOESPEC_ERR_BAD_HANDLE;
  L->profiling = on != 0;
  ++L->epoch;
  return MOESPEC_OK;
}

int moespec_get_kernel_times(moespec_layer_t *L, float *ms, int capacity, int *n_kernels) {
  if (!is_live(L)) return MOESPEC_ERR_BAD_HANDLE;
  if (!ms || !n_kernels) return MOESPEC_ERR_NULL_POINTER;
  if (!L->profiling || L->last_launches <= 1) return MOESPEC_ERR_INVALID_ARG;
  DeviceGuard guard(L->desc.device);
  if (guard.err != cudaSuccess) return cuda_fail(guard.err);
  const int n = L->last_launches < kMaxProfiled ? L->last_launches : kMaxProfiled;
  cudaError_t e = cudaEventSynchronize(L->ev[n]);
  if (e != cudaSuccess) return cuda_fail(e);
  *n_kernels = n;
  for (int i = 0; i < n && i < capacity; ++i) {
    e = cudaEventElapsedTime(&ms[i], L->ev[i], L->ev[i + 1]);
    if (e != cudaSuccess) return cuda_fail(e);
  }
  return MOESPEC_OK;
}

int moespec_last_launch_count(moespec_layer_t *L) {
  if (!is_live(L)) return MOESPEC_ERR_BAD_HANDLE;
  return L->last_launches;
}

int moespec_destroy(moespec_layer_t *L) {
  if (!L) return MOESPEC_OK;
  {
    std::lock_guard<std::mutex> lk(g_mu);
    if (g_live.erase(L) == 0) return MOESPEC_ERR_BAD_HANDLE;
  }
  int rc = MOESPEC_OK;
  {
    DeviceGuard guard(L->desc.device);
    for (int i = 0; i <= kMaxProfiled; ++i) cudaEventDestroy(L->ev[i]);
    drop_host_graphs(L);
    if (L->graph_usable) {
      cudaEventDestroy(L->ev_in);
      cudaStreamDestroy(L->own_stream);
    }
    if (L->analysis) cudaFree(L->analysis);
    cudaError_t e = cudaFree(L->arena);
    if (e != cudaSuccess) rc = cuda_fail(e);
  }
  L->magic = 0;
  delete L;
  return rc;
}

const char *moespec_strerror(int status) {
  switch (status) {
    case MOESPEC_OK: return "ok";
    case MOESPEC_ERR_INVALID_ARG: return "invalid argument";
    case MOESPEC_ERR_NULL_POINTER: return "null pointer";
    case MOESPEC_ERR_UNSUPPORTED: return "unsupported shape, dtype or alignment";
    case MOESPEC_ERR_OUT_OF_MEMORY: return "out of device memory";
    case MOESPEC_ERR_CUDA: return "CUDA call failed";
    case MOESPEC_ERR_TIMEOUT: return "bounded device-side wait expired";
    case MOESPEC_ERR_INTERNAL: return "device-side consistency check failed";
    case MOESPEC_ERR_BAD_HANDLE: return "bad or destroyed handle";
    case MOESPEC_ERR_TOO_LARGE: return "size exceeds the fixed scratch capacity of moespec_route_static";
    default: return "unknown status";
  }
}

int moespec_last_cuda_error(void) { return tl_cuda_error; }
int moespec_version(void) { return 120; }

}  // extern "C"

// ------------------------------------------------------------------ residual stack
namespace {

void *stack_x(moespec_stack *S, int l, const void *in, void *out) {      // x_l of the current call
  const int L = (int)S->layers.size();
  if (l == 0) return const_cast<void *>(in);
  if (l == L) return out;
  return S->arena + (size_t)(l - 1) * S->max_M * S->row_bytes;
}

// every layer of the stack, in order, on `stream`: x_{l+1} = dtype(x_l + layer_l(x_l))
int stack_enqueue(moespec_stack *S, const void *in, int M, int k, const int *B, void *out, cudaStream_t stream) {
  const int L = (int)S->layers.size();
  int launches = 0;
  for (int l = 0; l < L; ++l) {
    int rc = run_layer(S->layers[l], stack_x(S, l, in, out), M, k, B[l], stack_x(S, l + 1, in, out), stream);
    if (rc) return rc;
    launches += S->layers[l]->last_launches;
  }
  S->last_M = M;
  S->last_launches = launches;
  return MOESPEC_OK;
}

unsigned stack_epoch(moespec_stack *S) {
  unsigned e = 0;
  for (moespec_layer *L : S->layers) e = e * 31u + L->epoch;
  return e;
}

bool stack_profiling(moespec_stack *S) {
  for (moespec_layer *L : S->layers)
    if (L->profiling) return true;
  return false;
}

int stack_validate(moespec_stack *S, int M, int k, const int *B) {
  if (!B) return MOESPEC_ERR_NULL_POINTER;
  if (M < 0 || M > S->max_M) return MOESPEC_ERR_INVALID_ARG;
  for (size_t l = 0; l < S->layers.size(); ++l) {
    if (!is_live(S->layers[l])) return MOESPEC_ERR_BAD_HANDLE;       // a layer was destroyed under the stack
    int rc = validate_call(S->layers[l], M, k, B[l]);
    if (rc) return rc;
  }
  return MOESPEC_OK;
}

// Capture (or reuse) the graph of one stack pass.  host = the copies from/to pinned host buffers are
// part of the graph.  Returns nullptr when graphs cannot be used; the caller then enqueues plainly.
cudaGraphExec_t stack_graph(moespec_stack *S, const void *in, int M, int k, const int *B, void *out, bool host) {
  const int L = (int)S->layers.size();
  const unsigned epoch = stack_epoch(S);
  for (moespec_stack::Graph &g : S->graph) {
    bool hit = g.exec && g.M == M && g.k == k && g.in == in && g.out == out && g.host == host && g.epoch == epoch;
    for (int l = 0; hit && l < L; ++l) hit = g.B[l] == B[l];
    if (hit) {
      g.used = ++S->graph_clock;
      return g.exec;
    }
  }
  // miss: replace an instantiation whose layer settings are stale, else the least recently used one
  moespec_stack::Graph *slot = &S->graph[0];
  for (moespec_stack::Graph &g : S->graph) {
    const bool g_dead = !g.exec || g.epoch != epoch, s_dead = !slot->exec || slot->epoch != epoch;
    if ((g_dead && !s_dead) || (g_dead == s_dead && g.used < slot->used)) slot = &g;
  }
  if (slot->exec) {
    cudaGraphExecDestroy(slot->exec);
    slot->exec = nullptr;
  }
  const size_t bytes = (size_t)M * S->row_bytes;
  const void *dev_in = host ? S->in_stage : in;
  void *dev_out = host ? S->out_stage : out;
  cudaGraph_t graph = nullptr;
  // host buffers mapped into the device's address space: no copy nodes (see moespec_verify_layer_host)
  void *in_map = host ? mapped_device_pointer(in) : nullptr, *out_map = host ? mapped_device_pointer(out) : nullptr;
  const bool zero_copy = in_map && out_map && aligned16(in_map) && aligned16(out_map) && bytes % 16 == 0 &&
                         zero_copy_enabled();
  cudaError_t e = cudaStreamBeginCapture(S->own_stream, cudaStreamCaptureModeThreadLocal);
  if (e == cudaSuccess) {
    if (zero_copy) {
      const size_t n16 = bytes / 16;
      const unsigned grid = (unsigned)((n16 + 255) / 256 < 296 ? (n16 + 255) / 256 : 296);
      e = launch_kernel(stage_in_kernel, dim3(grid), dim3(256), 0, S->own_stream, (const uint4 *)in_map,
                        (uint4 *)S->in_stage, n16);
      if (e == cudaSuccess && stack_enqueue(S, S->in_stage, M, k, B, out_map, S->own_stream) != MOESPEC_OK)
        e = cudaErrorUnknown;
    } else {
      if (host) e = cudaMemcpyAsync(S->in_stage, in, bytes, cudaMemcpyHostToDevice, S->own_stream);
      if (e == cudaSuccess && stack_enqueue(S, dev_in, M, k, B, dev_out, S->own_stream) != MOESPEC_OK) e = cudaErrorUnknown;
      if (e == cudaSuccess && host) e = cudaMemcpyAsync(out, S->out_stage, bytes, cudaMemcpyDeviceToHost, S->own_stream);
    }
    cudaError_t e2 = cudaStreamEndCapture(S->own_stream, &graph);
    if (e == cudaSuccess) e = e2;
  }
  if (e == cudaSuccess) e = cudaGraphInstantiate(&slot->exec, graph, 0);
  if (graph) cudaGraphDestroy(graph);
  if (e != cudaSuccess) {
    cudaGetLastError();
    slot->exec = nullptr;
    S->graph_usable = false;
    return nullptr;
  }
  slot->M = M; slot->k = k; slot->in = in; slot->out = out; slot->host = host; slot->epoch = epoch;
  slot->B.assign(B, B + L);
  slot->used = ++S->graph_clock;
  return slot->exec;
}

}  // namespace

extern "C" {

int moespec_stack_create(moespec_layer_t *const *layers, int n_layers, moespec_stack_t **out_stack) {
  if (!layers || !out_stack) return MOESPEC_ERR_NULL_POINTER;
  if (n_layers < 1 || n_layers > 1024) return MOESPEC_ERR_INVALID_ARG;
  for (int l = 0; l < n_layers; ++l)
    if (!is_live(layers[l])) return MOESPEC_ERR_BAD_HANDLE;
  const moespec_layer_desc &d0 = layers[0]->desc;
  int max_M = d0.max_M, max_k = d0.max_k;
  for (int l = 0; l < n_layers; ++l) {
    const moespec_layer_desc &d = layers[l]->desc;
    if (d.device != d0.device || d.d != d0.d || d.dtype != d0.dtype) return MOESPEC_ERR_INVALID_ARG;
    // the stream stays in the storage dtype and every layer adds its input back
    if (!d.residual || (d.out_dtype != 0 && d.out_dtype != d.dtype)) return MOESPEC_ERR_INVALID_ARG;
    for (int m = 0; m < l; ++m)
      if (layers[m] == layers[l]) return MOESPEC_ERR_INVALID_ARG;     // a layer's workspace serves one position
    if (d.max_M < max_M) max_M = d.max_M;
    if (d.max_k < max_k) max_k = d.max_k;
  }
  DeviceGuard guard(d0.device);
  if (guard.err != cudaSuccess) return cuda_fail(guard.err);
  moespec_stack *S = new (std::nothrow) moespec_stack();
  if (!S) return MOESPEC_ERR_OUT_OF_MEMORY;
  S->magic = kStackMagic;
  S->layers.assign(layers, layers + n_layers);
  S->device = d0.device;
  S->d = d0.d;
  S->dtype = d0.dtype;
  S->max_M = max_M;
  S->max_k = max_k;
  S->row_bytes = (size_t)d0.d * dtype_bytes(d0.dtype);
  const size_t slab = (size_t)max_M * S->row_bytes;          // a multiple of 256 bytes: d % 64 == 0, 2 or 4 bytes each
  void *p = nullptr;
  cudaError_t e = cudaMalloc(&p, slab * (size_t)(n_layers - 1 + 2));
  if (e != cudaSuccess) {
    delete S;
    cudaGetLastError();
    return cuda_fail(e);
  }
  S->arena = static_cast<char *>(p);
  S->in_stage = S->arena + slab * (size_t)(n_layers - 1);
  S->out_stage = S->in_stage + slab;
  S->graph_clock = 0;
  S->graph_on = true;
  S->graph_usable = cudaStreamCreateWithFlags(&S->own_stream, cudaStreamNonBlocking) == cudaSuccess &&
                    cudaEventCreateWithFlags(&S->ev_in, cudaEventDisableTiming) == cudaSuccess;
  S->last_M = 0;
  S->last_launches = 0;
  {
    std::lock_guard<std::mutex> lk(g_mu);
    g_live_stacks.insert(S);
  }
  *out_stack = S;
  return MOESPEC_OK;
}

int moespec_verify_stack(moespec_stack_t *S, const void *hidden, int M, int k, const int *B_per_layer, void *out,
                         void *stream) {
  if (!is_live(S)) return MOESPEC_ERR_BAD_HANDLE;
  int rc = stack_validate(S, M, k, B_per_layer);
  if (rc) return rc;
  if (M == 0) return MOESPEC_OK;
  if (!hidden || !out) return MOESPEC_ERR_NULL_POINTER;
  if (!aligned16(hidden) || !aligned16(out)) return MOESPEC_ERR_UNSUPPORTED;
  if (hidden == out) return MOESPEC_ERR_INVALID_ARG;
  DeviceGuard guard(S->device);
  if (guard.err != cudaSuccess) return cuda_fail(guard.err);
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (S->graph_on && S->graph_usable && !stack_profiling(S)) {
    cudaGraphExec_t g = stack_graph(S, hidden, M, k, B_per_layer, out, false);
    if (g) {
      cudaError_t e = cudaGraphLaunch(g, s);
      return e == cudaSuccess ? MOESPEC_OK : cuda_fail(e);
    }
  }
  return stack_enqueue(S, hidden, M, k, B_per_layer, out, s);
}

int moespec_verify_stack_host(moespec_stack_t *S, const void *hidden_host, int M, int k, const int *B_per_layer,
                              void *out_host, void *stream) {
  if (!is_live(S)) return MOESPEC_ERR_BAD_HANDLE;
  int rc = stack_validate(S, M, k, B_per_layer);
  if (rc) return rc;
  if (M == 0) return MOESPEC_OK;
  if (!hidden_host || !out_host) return MOESPEC_ERR_NULL_POINTER;
  DeviceGuard guard(S->device);
  if (guard.err != cudaSuccess) return cuda_fail(guard.err);
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  cudaError_t e;
  if (S->graph_on && S->graph_usable && !stack_profiling(S) && is_pinned(hidden_host) && is_pinned(out_host)) {
    cudaGraphExec_t g = stack_graph(S, hidden_host, M, k, B_per_layer, out_host, true);
    if (g) {
      if ((e = cudaEventRecord(S->ev_in, s)) != cudaSuccess) return cuda_fail(e);
      if ((e = cudaStreamWaitEvent(S->own_stream, S->ev_in, 0)) != cudaSuccess) return cuda_fail(e);
      if ((e = cudaGraphLaunch(g, S->own_stream)) != cudaSuccess) return cuda_fail(e);
      if ((e = cudaStreamSynchronize(S->own_stream)) != cudaSuccess) return cuda_fail(e);
      return MOESPEC_OK;
    }
  }
  const size_t bytes = (size_t)M * S->row_bytes;
  if ((e = cudaMemcpyAsync(S->in_stage, hidden_host, bytes, cudaMemcpyHostToDevice, s)) != cudaSuccess) return cuda_fail(e);
  rc = stack_enqueue(S, S->in_stage, M, k, B_per_layer, S->out_stage, s);
  if (rc) return rc;
  if ((e = cudaMemcpyAsync(out_host, S->out_stage, bytes, cudaMemcpyDeviceToHost, s)) != cudaSuccess) return cuda_fail(e);
  if ((e = cudaStreamSynchronize(s)) != cudaSuccess) return cuda_fail(e);
  return MOESPEC_OK;
}

int moespec_stack_get_stream(moespec_stack_t *S, int l, void *host_buf) {
  if (!is_live(S)) return MOESPEC_ERR_BAD_HANDLE;
  if (!host_buf) return MOESPEC_ERR_NULL_POINTER;
  if (l < 1 || l >= (int)S->layers.size()) return MOESPEC_ERR_INVALID_ARG;
  DeviceGuard guard(S->device);
  if (guard.err != cudaSuccess) return cuda_fail(guard.err);
  cudaError_t e = cudaDeviceSynchronize();
  if (e != cudaSuccess) return cuda_fail(e);
  if (S->last_M > 0) {
    e = cudaMemcpy(host_buf, S->arena + (size_t)(l - 1) * S->max_M * S->row_bytes, (size_t)S->last_M * S->row_bytes,
                   cudaMemcpyDeviceToHost);
    if (e != cudaSuccess) return cuda_fail(e);
  }
  return MOESPEC_OK;
}

int moespec_stack_set_graph(moespec_stack_t *S, int on) {
  if (!is_live(S)) return MOESPEC_ERR_BAD_HANDLE;
  S->graph_on = on != 0;
  return MOESPEC_OK;
}

int moespec_stack_last_launch_count(moespec_stack_t *S) {
  if (!is_live(S)) return MOESPEC_ERR_BAD_HANDLE;
  return S->last_launches;
}

int moespec_stack_destroy(moespec_stack_t *S) {
  if (!S) return MOESPEC_OK;
  {
    std::lock_guard<std::mutex> lk(g_mu);
    if (g_live_stacks.erase(S) == 0) return MOESPEC_ERR_BAD_HANDLE;
  }
  int rc = MOESPEC_OK;
  {
    DeviceGuard guard(S->device);
    for (moespec_stack::Graph &g : S->graph)
      if (g.exec) cudaGraphExecDestroy(g.exec);
    if (S->graph_usable) {
      cudaEventDestroy(S->ev_in);
      cudaStreamDestroy(S->own_stream);
    }
    cudaError_t e = cudaFree(S->arena);
    if (e != cudaSuccess) rc = cuda_fail(e);
  }
  S->magic = 0;
  delete S;
  return rc;
}

}  // extern "C"

// ------------------------------------------------------------------ analysis mode
namespace {

int analysis_alloc(moespec_layer *L) {
  if (L->analysis) return MOESPEC_OK;
  const moespec_layer_desc &d = L->desc;
  Carver c;
  auto lay = [&](char *base) {
    c = Carver();
    c.base = base;
    c.take(L->an_gram, (size_t)d.max_M * d.max_k * d.max_k);
    c.take(L->an_objective, (size_t)d.n_experts);
    c.take(L->an_sums, 4);
    c.take(L->an_partial, 2 * (size_t)kSqdiffParts);
    c.take(L->an_row2slot, (size_t)L->R_cap);
    c.take(L->an_order, (size_t)d.n_experts);
    return (c.off + 255) & ~(size_t)255;
  };
  const size_t bytes = lay(nullptr);
  void *p = nullptr;
  cudaError_t e = cudaMalloc(&p, bytes);
  if (e != cudaSuccess) {
    cudaGetLastError();
    return cuda_fail(e);
  }
  L->analysis = static_cast<char *>(p);
  lay(L->analysis);
  return MOESPEC_OK;
}

}  // namespace

extern "C" {

int moespec_oracle_ranking(moespec_layer_t *L, const void *hidden, int M, int k, int n_pick, int *order_host,
                           double *objective_host, double *gold_energy_host, void *out_star, void *stream) {
  if (!is_live(L)) return MOESPEC_ERR_BAD_HANDLE;
  const moespec_layer_desc &d = L->desc;
  if (M < 1 || M > d.max_M || k < 1 || k > d.max_k || k > d.n_experts) return MOESPEC_ERR_INVALID_ARG;
  if (n_pick < 1 || n_pick > d.n_experts) return MOESPEC_ERR_INVALID_ARG;
  if (d.resident_count < d.n_experts) return MOESPEC_ERR_UNSUPPORTED;      // the analysis needs every expert's output
  if (!hidden || !order_host) return MOESPEC_ERR_NULL_POINTER;
  if (!aligned16(hidden) || (out_star && !aligned16(out_star))) return MOESPEC_ERR_UNSUPPORTED;
  if (out_star == hidden) return MOESPEC_ERR_INVALID_ARG;
  DeviceGuard guard(d.device);
  if (guard.err != cudaSuccess) return cuda_fail(guard.err);
  int rc = analysis_alloc(L);
  if (rc) return rc;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  // the unpruned model: every token keeps its natural top-k (B = N), no residual; O* goes to out_star
  moespec_layer_desc full = d;
  full.shortlist = MOESPEC_FROM_ALL;
  full.policy = MOESPEC_SUBSTITUTION;
  full.residual = 0;
  void *dump = out_star ? out_star : L->ws.out_stage;
  rc = run_layer(L, hidden, M, k, d.n_experts, dump, s, &full);
  if (rc) return rc;
  LaunchCtx c{&L->desc, &L->ws, M, k, d.n_experts, L->R_cap, s, 0};
  cudaError_t e = launch_gram(c, L->an_gram, L->an_row2slot);
  if (e == cudaSuccess)
    e = launch_greedy(c, L->an_gram, L->an_row2slot, n_pick, L->an_order, L->an_objective, L->an_sums);
  if (e != cudaSuccess) return cuda_fail(e);
  L->an_M = M;
  L->an_k = k;
  if ((e = cudaStreamSynchronize(s)) != cudaSuccess) return cuda_fail(e);
  if ((e = cudaMemcpy(order_host, L->an_order, sizeof(int) * n_pick, cudaMemcpyDeviceToHost)) != cudaSuccess)
    return cuda_fail(e);
  if (objective_host &&
      (e = cudaMemcpy(objective_host, L->an_objective, sizeof(double) * n_pick, cudaMemcpyDeviceToHost)) != cudaSuccess)
    return cuda_fail(e);
  if (gold_energy_host &&
      (e = cudaMemcpy(gold_energy_host, L->an_sums, sizeof(double), cudaMemcpyDeviceToHost)) != cudaSuccess)
    return cuda_fail(e);
  int status = 0;
  if ((e = cudaMemcpy(&status, L->ws.status, sizeof(int), cudaMemcpyDeviceToHost)) != cudaSuccess) return cuda_fail(e);
  return status;      // 0, or the device-side status of the unbudgeted pass
}

int moespec_get_gram(moespec_layer_t *L, double *gram_host) {
  if (!is_live(L)) return MOESPEC_ERR_BAD_HANDLE;
  if (!gram_host) return MOESPEC_ERR_NULL_POINTER;
  if (!L->analysis || L->an_M == 0) return MOESPEC_ERR_INVALID_ARG;
  DeviceGuard guard(L->desc.device);
  if (guard.err != cudaSuccess) return cuda_fail(guard.err);
  cudaError_t e = cudaDeviceSynchronize();
  if (e == cudaSuccess)
    e = cudaMemcpy(gram_host, L->an_gram, sizeof(double) * (size_t)L->an_M * L->an_k * L->an_k, cudaMemcpyDeviceToHost);
  return e == cudaSuccess ? MOESPEC_OK : cuda_fail(e);
}

int moespec_reconstruction_error(moespec_layer_t *L, const void *out_S, const void *out_star, int M,
                                 double *err_host, double *sums_host, void *stream) {
  if (!is_live(L)) return MOESPEC_ERR_BAD_HANDLE;
  const moespec_layer_desc &d = L->desc;
  if (M < 1 || M > d.max_M) return MOESPEC_ERR_INVALID_ARG;
  if (!out_S || !out_star || !err_host) return MOESPEC_ERR_NULL_POINTER;
  DeviceGuard guard(d.device);
  if (guard.err != cudaSuccess) return cuda_fail(guard.err);
  int rc = analysis_alloc(L);
  if (rc) return rc;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  cudaError_t e = launch_sqdiff(out_S, out_star, (size_t)M * d.d, d.out_dtype ? d.out_dtype : d.dtype, L->an_partial,
                                L->an_sums + 2, s);
  if (e == cudaSuccess) e = cudaStreamSynchronize(s);
  double sums[2] = {0.0, 0.0};
  if (e == cudaSuccess) e = cudaMemcpy(sums, L->an_sums + 2, sizeof(sums), cudaMemcpyDeviceToHost);
  if (e != cudaSuccess) return cuda_fail(e);
  if (sums_host) {
    sums_host[0] = sums[0];
    sums_host[1] = sums[1];
  }
  // one division of the two device-side sums; a zero reference gives 0 (identical) or infinity
  *err_host = sums[1] > 0.0 ? sums[0] / sums[1] : (sums[0] == 0.0 ? 0.0 : std::numeric_limits<double>::infinity());
  return MOESPEC_OK;
}

}  // extern "C"
