/*
 * moespec.h - C ABI of the budgeted MoE verify layer (MoE-Spec, Algorithm 1).
 *
 * One call runs, for M draft-tree tokens, the whole layer the target model
 * executes while verifying a speculative draft tree:
 *   router projection and softmax (Eq. 1) -> per-token top-k (Eq. 2) ->
 *   per-expert score s_i = sum_t g_i(h_t) (Eq. 5) -> shortlist S of the B best
 *   experts (Section 3.2) -> per-token re-routing under the substitution (Eq. 8)
 *   or truncation (Eq. 7) policy with the mixing weights of Section 3.3 ->
 *   per-expert gather (Appendix C) -> SwiGLU expert FFNs over the kept experts
 *   only -> gate-weighted combine (outer sums of Eq. 7 / Eq. 8).
 * Every step runs in CUDA kernels for sm_100a.  There is no CPU path.
 *
 * Conventions
 *   - All functions return 0 on success and a negative moespec_status on error.
 *     Nothing throws, aborts or traps the device.
 *   - "device" pointers are CUDA device memory of the layer's device; "host"
 *     pointers are ordinary host memory.  The library never takes ownership of a
 *     caller's buffer.  Weight, bias, hidden and out buffers are borrowed; weights
 *     and bias must stay valid and unchanged for the lifetime of the handle.
 *   - verify/route calls only enqueue work on the given stream and return; they
 *     do not synchronise (the *_host variant and the get_* calls do).
 *   - One call in flight per handle: the handle owns one workspace.
 *   - Argument rules: 0 <= M <= max_M (M = 0 is a no-op); 1 <= k <= min(N, max_k);
 *     B >= 1, B > N is clamped to N (B = N is the unbudgeted layer); B < k is legal
 *     (substitution then gives each token min(k, |S|) experts).
 *   - Rankings everywhere order by (key descending, expert index ascending).
 *     Per-token rankings use the fp32 logit as key; the shortlist uses the fp64
 *     score.  Inputs must be finite.
 */
#ifndef MOESPEC_H_
#define MOESPEC_H_

#ifdef __cplusplus
extern "C" {
#endif

typedef struct moespec_layer moespec_layer_t; /* opaque, created and freed by the library */

typedef enum {
  MOESPEC_OK = 0,
  MOESPEC_ERR_INVALID_ARG = -1,   /* a size, enum or flag outside its documented range          */
  MOESPEC_ERR_NULL_POINTER = -2,  /* a required pointer was NULL                                 */
  MOESPEC_ERR_UNSUPPORTED = -3,   /* legal request the kernels do not cover (alignment, shapes)  */
  MOESPEC_ERR_OUT_OF_MEMORY = -4, /* workspace allocation failed                                 */
  MOESPEC_ERR_CUDA = -5,          /* a CUDA runtime/driver call failed (see moespec_last_cuda_error) */
  MOESPEC_ERR_TIMEOUT = -6,       /* a bounded device-side wait expired (reported via stats)     */
  MOESPEC_ERR_INTERNAL = -7,      /* a device-side consistency check failed (reported via stats) */
  MOESPEC_ERR_BAD_HANDLE = -8,    /* handle is NULL, was destroyed, or was never created         */
  MOESPEC_ERR_TOO_LARGE = -9      /* a size exceeds the fixed capacity of moespec_route_static   */
} moespec_status;

/* MOESPEC_FP16 is the paper's own precision (Appendix A, "All models use FP16 precision"). */
typedef enum { MOESPEC_BF16 = 1, MOESPEC_FP32 = 2, MOESPEC_FP16 = 3 } moespec_dtype_t;
/* Token policy of Section 3.3: Eq. 8 / Eq. 7. */
typedef enum { MOESPEC_SUBSTITUTION = 1, MOESPEC_TRUNCATION = 2 } moespec_policy_t;
/* Which experts compete for the shortlist.  FROM_ALL is Algorithm 1 as printed
 * (all N experts ranked by s_i, so |S| = min(B, N)).  FROM_UNION restricts the
 * candidates to the union E(D) of Eq. 3 (so |S| = min(B, |E|) and any
 * B >= |E| reproduces the unbudgeted layer). */
/* MOESPEC_STATIC: the "Static Ranking" of Section 3.2.  The shortlist is the first B
 * experts of a fixed ordering by calibration count c_i (Eq. 4), set with
 * moespec_calibrate / moespec_set_static_ranking; it does not depend on the tree. */
typedef enum { MOESPEC_FROM_ALL = 1, MOESPEC_FROM_UNION = 2, MOESPEC_STATIC = 3 } moespec_shortlist_t;
/* Expert-FFN kernel choice.  AUTO picks the tensor-core kernel for bf16 and the
 * CUDA-core kernel for fp32 (fp32 accuracy needs full-precision FMAs); fp16 is treated like bf16. */
typedef enum { MOESPEC_FFN_AUTO = 0, MOESPEC_FFN_CUDA_CORE = 1, MOESPEC_FFN_TENSOR_CORE = 2 } moespec_ffn_t;

typedef struct {
  int d;              /* model width; multiple of 64                                             */
  int n_experts;      /* N, 1..256                                                               */
  int f;              /* expert FFN width; multiple of 64 (128 for the tensor-core kernel)        */
  int max_M;          /* largest M any call will pass (sizes the workspace), 1..4096              */
  int max_k;          /* largest k any call will pass, 1..min(N, 32)                              */
  int dtype;          /* moespec_dtype_t of weights and hidden; accumulation is always fp32       */
  int out_dtype;      /* moespec_dtype_t of out; 0 = same as dtype.  MOESPEC_FP32 with 16-bit weights
                         returns the fp32 accumulators unrounded; other mixes are unsupported    */
  int policy;         /* moespec_policy_t; 0 is invalid: the caller must choose                   */
  int shortlist;      /* moespec_shortlist_t; 0 is invalid: the caller must choose                */
  int renormalize;    /* 1: mixing weights are renormalised (Section 2.1, "OLMoE renormalizes"); 0: raw g_i */
  int residual;       /* 1: out = hidden + MoE(hidden) rounded once to dtype; 0: out = MoE(hidden) */
  int ffn_kernel;     /* moespec_ffn_t                                                            */
  int device;         /* CUDA device ordinal                                                      */
  const void *router_w;      /* device [N, d] row-major, dtype                                    */
  const float *router_bias;  /* device [N] fp32, or NULL for the bias-free router of Eq. 1         */
  const void *w_gate;        /* device [N, f, d], d contiguous, 16-byte aligned (W1 of SwiGLU)    */
  const void *w_up;          /* device [N, f, d], d contiguous, 16-byte aligned (W3)              */
  const void *w_down;        /* device [N, d, f], f contiguous, 16-byte aligned (W2)              */
  /* Expert-parallel shard (the paper ran its largest model on 2 GPUs, Table 3; the experts are the natural
   * unit to split).  resident_count = 0: this GPU holds all N experts (the default).  Otherwise it holds the
   * experts resident_first .. resident_first + resident_count - 1 only, and w_gate / w_up / w_down point to
   * THOSE experts' weights: [resident_count, f, d], [resident_count, f, d], [resident_count, d, f].  The
   * router (router_w, router_bias) is always the whole [N, d] matrix, so every shard takes the same routing
   * decisions from the same hidden states without any exchange; a shard runs the expert FFNs of its resident
   * kept experts only and returns the PARTIAL sum  out_t = sum_{i in A(t), i resident} wgt[t,i] E_i(h_t)
   * (zeros for a token none of whose kept experts is resident).  The layer output is the sum of the shards'
   * partial outputs (one all-reduce of [M, d]); out_dtype = MOESPEC_FP32 keeps that sum unrounded.
   * residual must be 0 on a shard (the caller adds the residual once, after the reduction).               */
  int resident_first;
  int resident_count;
} moespec_layer_desc;

typedef struct {
  int n_union;        /* |E(D)|, Eq. 3                                                            */
  int n_shortlist;    /* |S|                                                                      */
  int n_active;       /* resident experts with at least one routed row (what is streamed from HBM) */
  int n_rows;         /* R = sum_t |A(t)| routed (token, expert) pairs                            */
  int n_dropped;      /* M*k - R slots that received no expert                                    */
  int status;         /* 0, MOESPEC_ERR_TIMEOUT or MOESPEC_ERR_INTERNAL from the last call        */
  double coverage;    /* sum_{i in S} s_i / M, the routing mass kept by the shortlist (Section 4.6) */
  long long weight_bytes; /* n_active * 3*d*f*sizeof(dtype): expert bytes the call had to read     */
} moespec_stats;

/* Create a layer (Section 2.1: router W_gate and N experts; k and renormalisation
 * are properties of the architecture).  Validates the description, records the
 * borrowed weight pointers, builds TMA descriptors and allocates the workspace
 * for max_M tokens on desc->device.  *out_layer is written only on success.
 * Errors: NULL_POINTER, INVALID_ARG, UNSUPPORTED, OUT_OF_MEMORY, CUDA. */
int moespec_layer_create(const moespec_layer_desc *desc, moespec_layer_t **out_layer);

/* Algorithm 1 for one layer.  hidden: device [M, d] row-major, dtype, 16-byte
 * aligned.  out: device [M, d] in out_dtype, fully overwritten (exact zeros for a token with
 * no kept expert when residual = 0).  out must not alias hidden.
 * stream: a cudaStream_t (NULL = default stream).  Enqueues and returns.
 * A handle owns one workspace: calls on the same handle must be ordered (same
 * stream, or synchronised by the caller); different handles are independent and
 * their calls may overlap on the GPU (no kernel of the layer needs its whole grid
 * to be resident at once).
 * The call may be captured into a CUDA graph by the caller (it allocates nothing
 * and only enqueues kernels).
 * Errors: BAD_HANDLE, NULL_POINTER, INVALID_ARG, CUDA (launch failure). */
int moespec_verify_layer(moespec_layer_t *layer, const void *hidden, int M, int k, int B,
                         void *out, void *stream);

/* Same computation with HOST buffers: brings hidden (host [M, d]) to the device,
 * runs the layer, delivers the result in out (host [M, d], out_dtype) and synchronises
 * before returning.  With pinned (page-locked) buffers the whole step is captured
 * once per (M, k, B, buffer pair) into a CUDA graph and replayed with one launch on
 * an internal stream, after the work already queued on `stream`; the handle keeps the
 * four most recently used instantiations, so a caller may alternate between a few
 * trees or buffer pairs without re-capturing.  When the pinned buffers
 * are mapped into the device's address space (the default under unified addressing)
 * the graph has no copy nodes: a kernel pulls hidden over the interconnect into a
 * staging buffer and the layer's last kernel writes out directly to the host buffer.
 * Pageable buffers take a plain copy-launch-copy path on `stream`.  out_host is
 * written only by this call and is complete when it returns. */
int moespec_verify_layer_host(moespec_layer_t *layer, const void *hidden_host, int M, int k, int B,
                              void *out_host, void *stream);

/* Static ranking, Eq. 4: c_i = number of calibration tokens whose natural top-k contains
 * expert i.  moespec_calibrate runs the router, softmax and top-k on hidden (device
 * [M, d], dtype) and adds each token's top-k to the layer's counters (device, 64-bit);
 * call it as often as there is calibration data.  It enqueues on `stream` and returns.
 * moespec_get_static_counts copies c[N] to a HOST buffer (synchronises).
 * moespec_set_static_ranking fixes the ordering a MOESPEC_STATIC layer uses: `ranked`
 * is a HOST array of n distinct expert ids, best first; NULL means "order the experts
 * by (c_i descending, index ascending)" (synchronises to read the counters).  A verify
 * call on a MOESPEC_STATIC layer without a ranking returns INVALID_ARG.
 * moespec_reset_calibration zeroes the counters. */
int moespec_calibrate(moespec_layer_t *layer, const void *hidden, int M, int k, void *stream);
int moespec_get_static_counts(moespec_layer_t *layer, long long *counts_host);
int moespec_set_static_ranking(moespec_layer_t *layer, const int *ranked_host, int n);
int moespec_reset_calibration(moespec_layer_t *layer);

/* Steps after the router projection only (softmax, top-k, Eq. 5 scores,
 * shortlist, Eq. 7 / Eq. 8 re-routing, Appendix C gather order), from caller-
 * supplied fp32 logits: device [M, N] row-major.  Results stay in the workspace
 * for moespec_get_routing.  This is the hook the integer half of the layer is
 * checked through: fed the same fp32 logits, selection is exact. */
int moespec_route_from_logits(moespec_layer_t *layer, const float *logits, int M, int k, int B,
                              void *stream);

/* The routing step for callers that cannot allocate device memory.
 * (The paper has no counterpart: this entry point exists for deployment reasons only.)
 *
 * Who needs it: code that runs while a CUDA stream is being captured (allocation
 * cannot be captured), serving loops that must avoid the implicit device-wide
 * synchronisation of cudaMalloc/cudaFree, and processes whose device memory is
 * wholly owned by another allocator.  Such callers cannot use
 * moespec_layer_create, which allocates a workspace.
 *
 * What it does: exactly the computation of moespec_route_from_logits (softmax,
 * top-k, Eq. 5 scores, shortlist, Eq. 7 / Eq. 8 re-routing, Appendix C gather
 * order), without a handle.  Its scratch memory is a fixed array inside the
 * library image, about 1.1 MB, held by every GPU that loads the library until
 * the process exits.  It calls no cudaMalloc, cudaFree or other allocating routine.
 *
 * Limits: M <= MOESPEC_ROUTE_STATIC_MAX_M, N <= MOESPEC_ROUTE_STATIC_MAX_N,
 * k <= MOESPEC_ROUTE_STATIC_MAX_K, M*k <= MOESPEC_ROUTE_STATIC_MAX_ROWS; anything
 * larger returns MOESPEC_ERR_TOO_LARGE and launches nothing.
 *
 * Arguments: logits is device [M, N] fp32 on the calling thread's CURRENT
 * device; every output is a device buffer on that device, owned by the caller,
 * with the meaning and size given for moespec_get_routing (S_rank[N],
 * topk_idx/assign_idx/gate_w/tokslot2row[M*k], count[N], offset[N+1],
 * perm_row2tok[M*k], score[N]); summary is device int[8]: [0] = |S|,
 * [1] = experts with rows, [2] = R.  policy / shortlist / renormalize are the
 * fields of moespec_layer_desc.  Enqueues on `stream` and returns.
 *
 * Sharing: all calls in the process use the same scratch array, which keeps the
 * previous call's contents; each call first clears, on its stream, the part the
 * kernels accumulate into.  Two calls that overlap on the GPU (different streams
 * or threads) race on the array.  Serialise them.
 *
 * First call: the first call on each device looks up the array's device address
 * (cudaGetSymbolAddress) with that device current; make that first call before
 * starting any stream capture. */
#define MOESPEC_ROUTE_STATIC_MAX_M 512
#define MOESPEC_ROUTE_STATIC_MAX_N 256
#define MOESPEC_ROUTE_STATIC_MAX_K 32
#define MOESPEC_ROUTE_STATIC_MAX_ROWS 8192
int moespec_route_static(const float *logits, int M, int N, int k, int B, int policy, int shortlist,
                         int renormalize, int *S_rank, int *topk_idx, int *assign_idx, float *gate_w,
                         int *count, int *offset, int *perm_row2tok, int *tokslot2row, double *score,
                         int *summary, void *stream);

/* Copy the routing state of the last verify/route call into HOST buffers (any
 * may be NULL to skip it).  Synchronises the device.
 *   S_rank[N]        shortlist in rank order (first *n_S entries valid)
 *   topk_idx[M*k]    natural top-k per token, rank order
 *   assign_idx[M*k]  kept expert per slot, -1 for a dropped slot.  Substitution
 *                    fills slots 0..min(k,|S|)-1 in rank order; truncation keeps
 *                    slot r of the natural top-k or drops it
 *   gate_w[M*k]      mixing weight per slot (0 for a dropped slot)
 *   count[N], offset[N+1]   rows per expert and their exclusive scan
 *   perm_row2tok[R]  token index of each routed row; rows are ordered by
 *                    (expert ascending, token ascending)
 *   tokslot2row[M*k] row of each slot, -1 for a dropped slot
 *   score[N]         fp64 s_i of Eq. 5
 * M and k are those of the last call. */
int moespec_get_routing(moespec_layer_t *layer, int *S_rank, int *n_S, int *topk_idx, int *assign_idx,
                        float *gate_w, int *count, int *offset, int *perm_row2tok, int *tokslot2row,
                        double *score, int *n_rows);

/* Copy the fp32 router logits [M, N] of the last verify call to a HOST buffer.  Synchronises. */
int moespec_get_logits(moespec_layer_t *layer, float *logits_host);

/* Copy an intermediate of the last verify call to a HOST buffer of `bytes` bytes
 * (clipped to the buffer's size in the workspace).  which: 0 = gathered rows
 * x_perm [R, d] in dtype (Appendix C gather; on the tensor-core path not made for
 * trees of at most 16 tokens, and for trees of at most 128 tokens made only for
 * the experts some of whose gate/up work reads it: the best-ranked experts'
 * rows are taken straight from hidden), 1 = h_mid [R, f] in dtype
 * (silu(W1 x) * (W3 x) of the expert FFN), 2 = y [R, d] fp32 (expert outputs
 * before the gate-weighted sum).  Rows follow perm_row2tok.  Synchronises. */
int moespec_get_intermediate(moespec_layer_t *layer, int which, void *host_buf, long long bytes);

/* Statistics of the last call.  Synchronises the device. */
int moespec_get_stats(moespec_layer_t *layer, moespec_stats *stats);

/* Test hook for the bounded device-side waits (no fault, trap or hang is involved).
 * limit_cycles > 0 replaces the default bound (about one second of SM cycles) of every
 * wait in the expert-FFN kernel; ready_bias > 0 makes every down-projection unit wait
 * for that many extra gate/up slabs, which are never reported.  With both set, the
 * waits run out after limit_cycles: each CTA raises its abort flag, lets its copies
 * land, frees tensor memory and returns; `out` is then undefined and the next
 * moespec_get_stats reports status = MOESPEC_ERR_TIMEOUT.  Calling with (0, 0) restores
 * normal operation; the next verify call works as usual. */
int moespec_debug_set_wait(moespec_layer_t *layer, long long limit_cycles, int ready_bias);

/* Per-kernel timing.  With profiling on, verify calls record a CUDA event on the
 * stream before the first kernel and after every kernel (do not enable it while
 * the stream is being captured into a graph).  get_kernel_times waits for the
 * last verify call and writes the duration in milliseconds of each of its
 * kernels, in launch order, into ms[0 .. min(capacity, *n_kernels)).  bf16 tensor-core
 * layers launch four kernels (router + softmax + top-k; routing; gather; expert FFN +
 * combine), three for trees of at most 16 tokens (no gather: every gate/up unit then
 * takes all tokens straight from hidden); CUDA-core layers launch six (router, routing, gather, FFN gate/up, FFN
 * down, combine). */
int moespec_set_profiling(moespec_layer_t *layer, int on);
int moespec_get_kernel_times(moespec_layer_t *layer, float *ms, int capacity, int *n_kernels);

/* Number of kernels the last verify call launched (host-side count). */
int moespec_last_launch_count(moespec_layer_t *layer);

/* Free the workspace and the handle.  NULL is accepted.  Borrowed buffers are untouched. */
int moespec_destroy(moespec_layer_t *layer);

/* ---- Residual stack of budgeted MoE layers ---------------------------------
 * The method enforces the expert budget at every MoE layer of the model
 * (abstract; Section 4 runs 16-, 48- and 32-layer models) and names a per-layer
 * budget as an open extension (Limitations section).  A stack chains L existing layers on
 * one residual stream:
 *     x_0 = hidden,   x_{l+1} = dtype( x_l + layer_l(x_l ; B_l) ),   out = x_L.
 * Only the MoE blocks are on this path (attention and normalisation between them
 * are not part of the method).  Every layer must have been created with
 * residual = 1 and out_dtype equal to its dtype, on one device, with equal d and
 * dtype; a layer may appear once.  The stack borrows the layer handles (they
 * must outlive it, and must not run in another stream at the same time: each
 * layer's workspace is used by its position in the pass) and owns the L-1
 * intermediate streams, each [max_M, d] with max_M the smallest of the layers'.
 *
 * One pass is enqueued as ONE CUDA graph launch: the 4L kernels are captured once
 * per (M, k, budgets, buffer pair) on an internal stream with programmatic
 * dependent launch edges, so that each kernel's prologue (barrier set-up, tensor
 * memory allocation, the router-matrix prefetch of the next layer) overlaps the
 * tail of its predecessor; the four most recently used instantiations are kept, and
 * one is re-made when a layer setting (static ranking, profiling, wait bounds)
 * changes.  The first call with new arguments therefore allocates (graph
 * instantiation); later calls do not.  moespec_stack_set_graph(stack, 0) enqueues the kernels one by one
 * instead (same results). */
typedef struct moespec_stack moespec_stack_t;

/* layers: host array of n_layers (1..1024) live layer handles, first layer first.
 * Errors: NULL_POINTER, BAD_HANDLE (a dead layer), INVALID_ARG (mismatched d,
 * dtype, device; residual = 0; fp32 output on a 16-bit layer; repeated layer),
 * OUT_OF_MEMORY, CUDA. */
int moespec_stack_create(moespec_layer_t *const *layers, int n_layers, moespec_stack_t **out_stack);

/* One pass.  hidden, out: device [M, d] in the layers' dtype, 16-byte aligned, not
 * aliased.  B_per_layer: HOST array of n_layers budgets (read before returning).
 * k as in moespec_verify_layer.  Enqueues on `stream` and returns.
 * Errors: BAD_HANDLE (also when a member layer was destroyed), NULL_POINTER,
 * INVALID_ARG, UNSUPPORTED (alignment), CUDA. */
int moespec_verify_stack(moespec_stack_t *stack, const void *hidden, int M, int k, const int *B_per_layer,
                         void *out, void *stream);

/* Same pass with HOST buffers [M, d] (dtype): copy in, L layers, copy out, then
 * synchronise.  Pinned buffers: copies and kernels are one graph launch on the
 * internal stream, after the work already queued on `stream`. */
int moespec_verify_stack_host(moespec_stack_t *stack, const void *hidden_host, int M, int k,
                              const int *B_per_layer, void *out_host, void *stream);

/* Copy x_l of the last pass (1 <= l <= n_layers-1; x_0 and x_L are the caller's
 * buffers) to host_buf [M, d].  Synchronises the device.  Per-layer routing and
 * statistics of the pass are read from the layer handles as usual. */
int moespec_stack_get_stream(moespec_stack_t *stack, int l, void *host_buf);

int moespec_stack_set_graph(moespec_stack_t *stack, int on);
/* Kernels of the last pass (sum over its layers; one graph launch carries them all). */
int moespec_stack_last_launch_count(moespec_stack_t *stack);
/* Frees the intermediate streams and the graph; the layers stay alive.  NULL is accepted. */
int moespec_stack_destroy(moespec_stack_t *stack);

/* ---- Analysis mode: oracle ranking (Eq. 6) and reconstruction error (Section 4.5) ----
 * Not part of the verification hot path: the paper uses the oracle as an upper
 * bound on selection quality ("requires running all experts and is impractical
 * for speedup").
 *
 * moespec_oracle_ranking runs the layer unpruned on hidden [M, d] (every token
 * keeps its natural top-k with the architecture's mixing weights, whatever the
 * layer's policy and shortlist mode), which leaves every term
 * c_{t,i} = g_i(h_t) E_i(h_t) of the gold output O*_t = sum_{i in T_k(h_t)} c_{t,i}
 * in the workspace, and then selects experts greedily: starting from the empty
 * set, n_pick times add the expert outside S that minimises
 *     sum_t || O*_t - sum_{j in (S + i) and in T_k(h_t)} c_{t,j} ||^2
 * (the inner sum runs over the experts the token actually routes to: the
 * truncation output of Eq. 7 with the original weights; ties -> lower index).
 * The loop works on the per-token k x k Gram matrices of the c_{t,i} in fp64.
 *   order_host      [n_pick] experts in the order picked (host, written)
 *   objective_host  [n_pick] value of the objective after each pick (host, may be NULL)
 *   gold_energy_host sum_t ||O*_t||^2, the objective of the empty set (host, may be NULL)
 *   out_star        device [M, d] in out_dtype: receives O* (may be NULL)
 * The layer's routing state afterwards is that of the unpruned pass.  Allocates
 * its scratch on the first call of the handle; synchronises `stream`.
 * order_host can be passed to moespec_set_static_ranking of a MOESPEC_STATIC layer
 * over the same weights to run the layer with the oracle's shortlist.
 * Errors: BAD_HANDLE, NULL_POINTER, INVALID_ARG, UNSUPPORTED, OUT_OF_MEMORY, CUDA,
 * or the device status of the unpruned pass. */
int moespec_oracle_ranking(moespec_layer_t *layer, const void *hidden, int M, int k, int n_pick,
                           int *order_host, double *objective_host, double *gold_energy_host,
                           void *out_star, void *stream);

/* Gram matrices of the last moespec_oracle_ranking call: host [M, k, k] fp64,
 * G[t][a][b] = c_{t,a} . c_{t,b} with a, b the token's natural top-k slots in rank order. */
int moespec_get_gram(moespec_layer_t *layer, double *gram_host);

/* ||O_S - O*||_F^2 / ||O*||_F^2 over the M tokens (Section 4.5).  out_S, out_star:
 * device [M, d] in the layer's out_dtype.  *err_host receives the ratio (0 when both
 * are zero, +inf when only O* is); sums_host, if not NULL, the two sums
 * {numerator, denominator}.  Fixed summation order; synchronises `stream`. */
int moespec_reconstruction_error(moespec_layer_t *layer, const void *out_S, const void *out_star, int M,
                                 double *err_host, double *sums_host, void *stream);

const char *moespec_strerror(int status);
/* cudaError_t of the most recent failing CUDA call on this thread (0 if none). */
int moespec_last_cuda_error(void);
/* major*100 + minor; 110 added the stack, the analysis mode and the early-start FFN kernel;
 * 120 the expert-parallel shard (resident_first / resident_count at the end of moespec_layer_desc). */
int moespec_version(void);

#ifdef __cplusplus
}
#endif
#endif /* MOESPEC_H_ */
