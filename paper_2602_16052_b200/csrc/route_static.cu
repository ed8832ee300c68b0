// moespec_route_static: the routing step for callers that must not allocate.
//
// Some callers of this library cannot call cudaMalloc where they call us: code
// running between the begin and end of a CUDA stream capture (allocation is not
// a capturable operation), latency-critical serving loops that forbid the
// implicit device synchronisation cudaMalloc/cudaFree can cause, and processes
// whose device memory was handed out up front to another allocator.  For them
// this file offers the routing step with its scratch memory in a fixed array
// that is part of the library image.  Every GPU that loads the library holds
// that array (kRouteStaticScratchBytes) until the process exits.
//
// The array is shared by every call in the process and keeps the previous
// call's contents.  The accumulators the routing kernels add into are cleared
// on the caller's stream at the start of every call; everything else is written
// before it is read.  Two calls that overlap on the GPU (different streams, or
// different threads) would race on the array.
#include "internal.h"

#include <mutex>

namespace {

using namespace moespec;

constexpr int kStaticMaxM = MOESPEC_ROUTE_STATIC_MAX_M;
constexpr int kStaticMaxN = MOESPEC_ROUTE_STATIC_MAX_N;
constexpr int kStaticMaxK = MOESPEC_ROUTE_STATIC_MAX_K;
constexpr int kStaticMaxRows = MOESPEC_ROUTE_STATIC_MAX_ROWS;

constexpr size_t align256(size_t x) { return (x + 255) & ~(size_t)255; }
constexpr size_t kOffProb = 0;                                                              // double [M, N]
constexpr size_t kOffActive = kOffProb + align256(sizeof(double) * kStaticMaxM * kStaticMaxN);
constexpr size_t kOffRow2Exp = kOffActive + align256(sizeof(int) * kStaticMaxN);
constexpr size_t kOffStats = kOffRow2Exp + align256(sizeof(int) * kStaticMaxRows);
constexpr size_t kOffStatus = kOffStats + align256(sizeof(moespec_stats));
// accumulators that must be zero when a call starts (cleared on the stream before every call)
constexpr size_t kOffZero = kOffStatus + 256;
constexpr int kStaticMaskWords = (kStaticMaxM + 31) / 32;
constexpr size_t kOffScoreFx = kOffZero;                                                    // ull [N]
constexpr size_t kOffNatcnt = kOffScoreFx + align256(sizeof(unsigned long long) * kStaticMaxN);
constexpr size_t kOffCountAcc = kOffNatcnt + align256(sizeof(int) * kStaticMaxN);
constexpr size_t kOffColmask = kOffCountAcc + align256(sizeof(int) * kStaticMaxN);         // uint [N, mask words]
constexpr size_t kOffArrive = kOffColmask + align256(sizeof(unsigned) * kStaticMaxN * kStaticMaskWords);
constexpr size_t kRouteStaticScratchBytes = kOffArrive + 256;
constexpr size_t kZeroBytes = kRouteStaticScratchBytes - kOffZero;

// In host code this name is only a handle for cudaGetSymbolAddress; it is not a device address.
static __device__ __align__(256) unsigned char g_route_scratch[kRouteStaticScratchBytes];

constexpr int kMaxDevices = 64;
std::mutex g_setup_mu;
unsigned char *g_scratch_dev[kMaxDevices] = {nullptr};

// First call on a device: resolve the device address of the array on that device.
cudaError_t scratch_for_current_device(unsigned char **out) {
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
  std::lock_guard<std::mutex> lk(g_setup_mu);
  if (!g_scratch_dev[dev]) {
    void *p = nullptr;
    e = cudaGetSymbolAddress(&p, g_route_scratch);      // `dev` is the current device here
    if (e != cudaSuccess) return e;
    if (!p) return cudaErrorInvalidSymbol;
    g_scratch_dev[dev] = static_cast<unsigned char *>(p);
  }
  *out = g_scratch_dev[dev];
  return cudaSuccess;
}

}  // namespace

extern "C" int moespec_route_static(const float *logits, int M, int N, int k, int B, int policy, int shortlist,
                                    int renormalize, int *S_rank, int *topk_idx, int *assign_idx, float *gate_w,
                                    int *count, int *offset, int *perm_row2tok, int *tokslot2row, double *score,
                                    int *summary, void *stream) {
  if (policy != MOESPEC_SUBSTITUTION && policy != MOESPEC_TRUNCATION) return MOESPEC_ERR_INVALID_ARG;
  if (shortlist != MOESPEC_FROM_ALL && shortlist != MOESPEC_FROM_UNION) return MOESPEC_ERR_INVALID_ARG;
  if ((renormalize | 1) != 1) return MOESPEC_ERR_INVALID_ARG;
  if (M < 0 || N < 1 || k < 1 || k > N || B < 1) return MOESPEC_ERR_INVALID_ARG;
  if (M > kStaticMaxM || N > kStaticMaxN || k > kStaticMaxK || (long long)M * k > kStaticMaxRows)
    return MOESPEC_ERR_TOO_LARGE;
  if (M == 0) return MOESPEC_OK;
  if (!logits || !S_rank || !topk_idx || !assign_idx || !gate_w || !count || !offset || !perm_row2tok ||
      !tokslot2row || !score || !summary)
    return MOESPEC_ERR_NULL_POINTER;

  // a failing CUDA call is remembered for moespec_last_cuda_error(), as in the handle-based entry points
  auto cuda_fail = [](cudaError_t e) {
    record_cuda_error(e);
    return (int)MOESPEC_ERR_CUDA;
  };
  unsigned char *scratch = nullptr;
  cudaError_t e = scratch_for_current_device(&scratch);
  if (e != cudaSuccess) return cuda_fail(e);

  Workspace ws{};
  ws.prob = reinterpret_cast<double *>(scratch + kOffProb);
  ws.score_fx = reinterpret_cast<unsigned long long *>(scratch + kOffScoreFx);
  ws.natcnt_acc = reinterpret_cast<int *>(scratch + kOffNatcnt);
  ws.count_acc = reinterpret_cast<int *>(scratch + kOffCountAcc);
  ws.colmask = reinterpret_cast<unsigned *>(scratch + kOffColmask);
  ws.arrive_route = reinterpret_cast<int *>(scratch + kOffArrive);
  ws.mask_words = kStaticMaskWords;
  // the shared array keeps whatever the last call (possibly an aborted one) left: clear the accumulators
  e = cudaMemsetAsync(scratch + kOffZero, 0, kZeroBytes, static_cast<cudaStream_t>(stream));
  if (e != cudaSuccess) return cuda_fail(e);
  ws.active = reinterpret_cast<int *>(scratch + kOffActive);
  ws.row2expert = reinterpret_cast<int *>(scratch + kOffRow2Exp);
  ws.stats = reinterpret_cast<moespec_stats *>(scratch + kOffStats);
  ws.status = reinterpret_cast<int *>(scratch + kOffStatus);
  ws.score = score;
  ws.topk_idx = topk_idx;
  ws.S_rank = S_rank;
  ws.assign_idx = assign_idx;
  ws.gate_w = gate_w;
  ws.count = count;
  ws.offset = offset;
  ws.perm_row2tok = perm_row2tok;
  ws.tokslot2row = tokslot2row;
  ws.counters = summary;

  moespec_layer_desc desc{};
  desc.d = 64;            // not a multiple of the tensor-core tile: no FFN work units are written
  desc.f = 64;
  desc.n_experts = N;
  desc.dtype = MOESPEC_FP32;
  desc.policy = policy;
  desc.shortlist = shortlist;
  desc.renormalize = renormalize;
  LaunchCtx c{&desc, &ws, M, k, B > N ? N : B, M * k, static_cast<cudaStream_t>(stream), 0};
  e = launch_route(c, logits);
  return e == cudaSuccess ? (int)MOESPEC_OK : cuda_fail(e);
}
