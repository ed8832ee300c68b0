// Internal declarations shared by the translation units of libmoespec.
#pragma once
#include <cuda_runtime.h>
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <stdint.h>
#include <stdlib.h>
#include "../../include/moespec.h"

namespace moespec {

// Switches that choose between equivalent code paths (for A/B measurements) are read from the
// environment only in builds made with -DMOESPEC_EXPERIMENTS; the shipped library reads no
// behaviour from the environment.
#ifdef MOESPEC_EXPERIMENTS
inline const char *experiment_env(const char *name) { return getenv(name); }
#else
inline const char *experiment_env(const char *) { return nullptr; }
#endif

// Remember the cudaError_t of a failing call for moespec_last_cuda_error() (per thread).
void record_cuda_error(cudaError_t e);

inline bool is_16bit(int dtype) { return dtype == MOESPEC_BF16 || dtype == MOESPEC_FP16; }
inline int dtype_bytes(int dtype) { return is_16bit(dtype) ? 2 : 4; }

constexpr int kMaxExperts = 256;           // N limit: 8 experts per lane in the warp-wide rankings
constexpr int kMaskWords = kMaxExperts / 32;
constexpr int kMaxK = 32;
constexpr int kTile = 128;                 // weight rows per tensor-core work unit (MMA M)
constexpr int kTokBox = 32;                // token rows per TMA box of the B operand
constexpr int kTokBoxSmall = 16;           // ... for units of at most 16 rows (the smallest MMA N)
constexpr int kMaxTokChunk = 128;          // tokens per work unit: gate and up accumulators of two units fit TMEM

// One tensor-core work unit: a slab of RU (128, 64 or 32) rows of one expert's weight
// matrix against one chunk (<= 128) of that expert's routed rows.
struct __align__(16) Unit {
  int expert;
  int tile;       // slab index along f (gate/up phase) or d (down phase)
  int row0;       // first routed row of the chunk
  int n_rows;     // rows in the chunk (1..256)
  int chunk;      // global index of the (expert, token chunk) pair: indexes the ready counters
  int phase;      // 0 gate/up, 1 down
  int pad0, pad1;
};

// Device-resident routing state and scratch of one layer handle.
struct Workspace {
  float *logits;        // [max_M, N]
  double *prob;         // [max_M, N]
  double *score;        // [N]
  int *topk_idx;        // [max_M, max_k]
  int *S_rank;          // [N]
  int *assign_idx;      // [max_M, max_k]
  float *gate_w;        // [max_M, max_k]
  int *count;           // [N]
  int *offset;          // [N+1]
  int *active;          // [N]
  int *perm_row2tok;    // [R_cap]
  int *gather_src;      // [R_cap] token whose hidden state row r of x_perm is a copy of, or -1 when no work unit
                        // reads that row (every gate/up unit of its expert takes all tokens from hidden); may be null
  int *row2expert;      // [R_cap]
  int *tokslot2row;     // [max_M, max_k]
  // accumulators shared by the CTAs of one call; every one of them is zero between calls (the routing
  // kernel's last CTA clears what the call used)
  unsigned long long *score_fx;  // [N] sum_t g_i(h_t) in 2^-52 fixed point: exact integer adds, any order
  int *natcnt_acc;      // [N] number of tokens with expert i in T_k(h_t)
  int *count_acc;       // [N] number of tokens with expert i in A(t)
  unsigned *colmask;    // [N, ceil(max_M/32)] bit t of row i: expert i in A(t)
  int *arrive;          // [max_M] arrival counters of router_topk_kernel's token tiles
  int *arrive_route;    // [1] arrival counter of route_kernel's CTAs
  int *early_flag;      // [N] word r is 0 until the shortlist of the call is published, then (resident expert of
                        // rank r) + 1, or -1 when there are fewer (may be null)
  int mask_words;       // ceil(max_M / 32)
  long long *calib_count;   // [N] Eq. 4 calibration counts c_i
  int *static_pos;          // [N] position of expert i in the fixed ordering (INT_MAX: not listed)
  int n_static;             // experts in the fixed ordering (0: none set)
  int *static_order;        // [N] the fixed ordering itself: expert at position r (first n_static entries)
  Unit *units;          // gate/up units (expert, chunk, tile ascending) followed by the down units
  int *ready;           // [chunks] gate/up units finished per (expert, token chunk); zeroed by the route kernel
  int *unit_counter;    // [0] next unit to hand out, [1] finished down units; zeroed by the router kernel
  int *counters;        // [0]=n_S [1]=n_active [2]=R [3]=n_units_up [4]=n_units_down
  moespec_stats *stats; // device copy
  int *status;          // device status word (0 = ok)
  void *x_perm;         // [R_cap, d] dtype
  void *h_mid;          // [R_cap, f] dtype
  float *y;             // [R_cap, d] fp32
  void *hidden_stage;   // [max_M, d] dtype (host-buffer variant)
  void *out_stage;      // [max_M, d] dtype
};

struct LaunchCtx {
  const moespec_layer_desc *desc;
  const Workspace *ws;
  int M, k, B;
  int R_cap;            // max_M * max_k
  cudaStream_t stream;
  int ru;               // weight rows per tensor-core work unit for this call (0: CUDA-core path)
  int early = 0;        // 1: the FFN kernel starts on the shortlist before routing has finished (see ffn_tc.cu)
  int dense_all = 0;    // 1: every gate/up unit takes ALL tokens straight from `hidden` (trees of at most 16
                        //    tokens: the smallest MMA holds them anyway), so no gathered copy is made
  int res_first = 0, res_count = 0; // resident experts [res_first, res_first + res_count) (res_count = N: all)
  long long debug_spin_limit = 0;   // test hook: bound of device-side waits in cycles (0 = default)
  int debug_ready_bias = 0;         // test hook: extra slabs every down unit waits for (never reported)
};

// Programmatic dependent launch.  Every kernel of the layer is launched with
// programmatic stream serialisation: it may be scheduled while its predecessor
// still runs, executes pdl_trigger() at once (so that its own successor can be
// scheduled too) and calls pdl_wait() before it touches anything a predecessor
// wrote or a predecessor may still read.  pdl_wait() returns when all earlier
// kernels in the stream have completed and flushed; without the launch
// attribute both calls are no-ops.
#ifdef __CUDACC__
__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
#endif
bool pdl_enabled();   // true (an experiments build can switch programmatic launches off)

template <typename... KArgs, typename... Args>
cudaError_t launch_kernel(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream,
                          Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = pdl_enabled() ? 1 : 0;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

// routing.cu
cudaError_t launch_router_logits(const LaunchCtx &c, const void *hidden);
cudaError_t launch_route(const LaunchCtx &c, const float *logits);   // softmax/top-k kernel + route kernel
cudaError_t launch_route_after_router(const LaunchCtx &c);           // route kernel only
cudaError_t launch_calib_accumulate(const LaunchCtx &c);             // c_i += natural counts of the last router launch
cudaError_t launch_gather(const LaunchCtx &c, const void *hidden);
cudaError_t routing_configure();   // one-time function attributes of the routing kernels (tensor-core path)
// ffn_simple.cu
cudaError_t launch_ffn_cuda_core(const LaunchCtx &c, int phase);   // 0 gate/up, 1 down
cudaError_t cc_configure(const moespec_layer_desc &d, bool *fits);   // shared-memory opt-in of the CUDA-core FFN
// ffn_tc.cu
struct TcMaps {            // per handle: weight maps for slab heights 128, 64, 32
  CUtensorMap w_gate[3], w_up[3], w_down[3];
  CUtensorMap x_perm[3], h_mid[3];   // token-row boxes of 32, 64 and 128 rows
  CUtensorMap x_perm16, h_mid16;     // ... and of 16 rows
  // the last call's input tensor (early-start mode): re-encoded when the pointer or M changes
  mutable CUtensorMap hidden_map;
  mutable const void *hidden_ptr = nullptr;
  mutable int hidden_M = 0;
};
struct TcMapsCall {        // per launch: the weight maps of the chosen slab heights
  CUtensorMap w_gate, w_up, w_down;
  CUtensorMap x_perm[3], h_mid[3];
  CUtensorMap x_perm16, h_mid16;     // 16-row boxes
  CUtensorMap hidden;      // the call's [M, d] input as token-row boxes (early-start mode only)
};
int tc_rows_per_unit(const moespec_layer_desc &d, int M, int k, int B);   // gate/up slab height for a call
int tc_rows_per_down_unit(int ru);                                         // down slab height for a call
int tc_grid_size(int device);                                              // CTAs of the FFN kernel (one per SM)
bool tc_early_start(const moespec_layer_desc &d, int M);                  // does a call of M tokens use early start?
bool tc_dense_all(const moespec_layer_desc &d, int M);                    // ... and no gathered rows at all?
cudaError_t tc_encode_maps(const moespec_layer_desc &d, const Workspace &ws, int R_cap, TcMaps *maps,
                           int *cu_result);
cudaError_t tc_configure();   // one-time function attributes
// gate/up + down + combine in one launch
cudaError_t launch_ffn_tensor_core(const LaunchCtx &c, const TcMaps *maps, const void *hidden, void *out);
// combine.cu
cudaError_t launch_combine(const LaunchCtx &c, const void *hidden, void *out);
// analysis.cu (oracle ranking of Eq. 6, reconstruction error of Section 4.5)
constexpr int kSqdiffParts = 64;   // slices of the squared-difference reduction
cudaError_t launch_gram(const LaunchCtx &c, double *gram, int *row2slot);
cudaError_t launch_greedy(const LaunchCtx &c, const double *gram, const int *row2slot, int n_pick, int *order,
                          double *objective, double *gold_energy);
cudaError_t launch_sqdiff(const void *a, const void *b, size_t n, int dtype, double *partial, double *out,
                          cudaStream_t stream);

}  // namespace moespec
