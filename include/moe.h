/*
 * libmoe — top-2 Mixture-of-Experts layer forward with expert pruning and
 * dynamic expert skipping, and the layer-wise pruning search
 * (arXiv 2402.14800), as CUDA kernels for sm_100a.
 *
 * C ABI.  Conventions shared by every call:
 *   - "device" pointers are CUDA device memory of the current device, owned by
 *     the caller unless stated; "host" pointers are ordinary host memory.
 *   - bf16 tensors are row-major with the last index contiguous and a 16-byte
 *     aligned base address.
 *   - Calls return MOE_OK (0) or a negative moe_status; moe_layer_create returns
 *     NULL on failure.  moe_last_error() gives a thread-local message for the
 *     last failing call.  No C++ exception crosses this boundary.
 *   - Work is enqueued on the handle's stream (default: the legacy stream 0) and
 *     is asynchronous unless the call returns results to host memory.
 *   - A handle must not be used from two host threads at once: its scratch
 *     buffers are shared by all of its calls.
 *   - A call takes at most 2^24 tokens.
 */
#ifndef MOE_H_
#define MOE_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum moe_status {
  MOE_OK = 0,
  MOE_ERR_INVALID_ARG = -1,       /* null/misaligned pointer, bad mask, r out of range, ... */
  MOE_ERR_UNSUPPORTED_SHAPE = -2, /* h or f not a multiple of 64, E > 16, ... */
  MOE_ERR_CUDA = -3,              /* a CUDA runtime/driver call failed */
  MOE_ERR_OOM = -4,               /* device memory for weights or scratch not available */
  MOE_ERR_DEVICE_TIMEOUT = -5,    /* a bounded wait inside a kernel expired */
  MOE_ERR_ARCH = -6               /* the current device is not sm_100 */
} moe_status;

#define MOE_MAX_EXPERTS 16

typedef struct moe_layer moe_layer_t; /* opaque, owned by the library */

/*
 * Build one MoE layer (Sec. 3.1) restricted to the kept experts (Sec. 3.2:
 * pruned experts are discarded together with their router rows).
 *   W_gate [E][h]     bf16 device   router, one row per expert
 *   W1     [E][f][h]  bf16 device   gate projection of the SwiGLU expert
 *   W3     [E][f][h]  bf16 device   up projection
 *   W2     [E][h][f]  bf16 device   down projection
 *   kept_mask         bit e set <=> expert e is kept; at least 2 bits (top-2)
 * The kept router rows and kept experts are COPIED into library-owned buffers
 * in the layout the kernels want, so the handle occupies popcount(mask)/E of
 * the layer's bytes and the caller may free its tensors when this returns
 * (the call synchronises the device).  Requires h % 64 == 0, f % 64 == 0,
 * 2 <= E <= 16, and an sm_100 device.
 */
moe_layer_t* moe_layer_create(const void* W_gate, const void* W1, const void* W3, const void* W2,
                              int h, int f, int E, uint32_t kept_mask);

/* Free the handle with its weights and scratch (synchronises its stream). */
void moe_layer_destroy(moe_layer_t* layer);

/* Stream (a cudaStream_t) that later calls on this handle enqueue on. */
int moe_set_stream(moe_layer_t* layer, void* cuda_stream);

/*
 * Let `layer` run out of `owner`'s scratch buffers instead of its own (a stack of
 * layers then needs one set of scratch, not one per layer).  Both must have the
 * same h and f and must never run at the same time; `owner` must outlive the
 * sharing.  owner == NULL returns `layer` to its own scratch.
 */
int moe_layer_share_scratch(moe_layer_t* layer, moe_layer_t* owner);

/*
 * Grow the handle's scratch now to what moe_forward / moe_forward_residual need
 * for any batch of 1 .. T_max tokens (both the small-batch and the large-batch
 * kernel sequences), so that no later forward call with T <= T_max allocates,
 * frees or synchronises the device: a serving loop calls this once at start-up,
 * and a CUDA-graph capture needs no warm-up call.  Not part of the paper's
 * method.  Synchronises the handle's stream when a buffer is replaced.
 * Errors: MOE_ERR_INVALID_ARG (T_max outside 1 .. 2^24), MOE_ERR_OOM.
 */
int moe_reserve(moe_layer_t* layer, int T_max);

/* Bytes of device memory the handle holds for weights: the kept experts' three
 * matrices and the router rows (stored padded with zero rows to 16 rows). */
size_t moe_layer_weight_bytes(const moe_layer_t* layer);

/* Bytes of device memory the handle currently holds as scratch. */
size_t moe_layer_scratch_bytes(const moe_layer_t* layer);

/*
 * Layer forward for T tokens (Sec. 3.1 Eq. 1-2, Sec. 3.2, Sec. 3.3, App. A.2):
 *   l = W_gate x over the kept experts, w = Softmax(l), e0/e1 = top-2 (ties to
 *   the lower expert index), e1 is skipped when w_e1 < beta * w_e0 (strict),
 *   z = w~_e0 E_e0(x) + w~_e1 E_e1(x) with w~ renormalised over the experts
 *   that run (w~_e0 = 1 after a skip), E_e(x) = W2_e (silu(W1_e x) * W3_e x).
 *   The SwiGLU activation and y are rounded to bf16; everything else is fp32.
 *   x [T][h] bf16 device (read), y [T][h] bf16 device (written); beta >= 0,
 *   beta = 0 never skips.  x and y may not overlap.  T = 0 is a no-op.
 *   routing_stats: NULL, or device memory of moe_routing_stats_bytes(T, E)
 *   bytes that receives the per-token routing record (layout below).
 * Asynchronous; nothing is retained after the kernels finish.
 */
int moe_forward(moe_layer_t* layer, const void* x, int T, float beta, void* y,
                void* routing_stats);

/* As moe_forward, but y = bf16(residual + z) with one rounding.  residual
 * [T][h] bf16 device may be the same buffer as y; NULL means 0. */
int moe_forward_residual(moe_layer_t* layer, const void* x, int T, float beta,
                         const void* residual, void* y, void* routing_stats);

/*
 * Layer forward in the general top-k setting with the generalised skipping
 * rule of App. A.2: e_0..e_{k-1} are the kept experts with the k largest routing
 * weights; the top i* of them run, where
 *     i* = min i  such that  sum_{m=i+1..k} w_m <= beta * sum_{m=1..k} w_m,
 * and the output is renormalised over those i*:
 *     z = sum_{m<=i*} w_m E_m(x) / sum_{m<=i*} w_m.
 * beta = 0 keeps all k, beta >= 1 keeps only the first.  (For k = 2 this is the
 * rule of moe_forward with beta/(1-beta) in place of beta and "<=" for "<".)
 * 1 <= k <= min(kept experts, 8).  Optional device outputs: idx_out [T][k] int32
 * original expert ids in order of decreasing weight, wn_out [T][k] the weights
 * applied (0 for skipped experts), n_active_out [T] int32 = i*.  x, y as in
 * moe_forward.  Asynchronous.
 */
int moe_forward_topk(moe_layer_t* layer, const void* x, int T, int k, float beta, void* y,
                     int32_t* idx_out, float* wn_out, int32_t* n_active_out);

/*
 * Distance between a token's two selected expert outputs,
 *   dist[t] = || E_e0(x_t) - E_e1(x_t) ||_2      (no skipping, kept experts only),
 * the quantity whose concentration App. A.2 assumes (D ~ const) when it derives
 * the skipping rule; for k = 2 the error of skipping token t is exactly
 * w~_e1 * dist[t].  x [T][h] bf16 device, dist [T] fp32 device.  Asynchronous.
 */
int moe_top2_distance(moe_layer_t* layer, const void* x, int T, float* dist);

/*
 * moe_forward with HOST buffers: copies x_host to the device, runs the layer,
 * copies y back and waits for it.  x_host/y_host [T][h] bf16; pinned memory
 * makes the copies asynchronous to the host but is not required.
 */
int moe_forward_host(moe_layer_t* layer, const void* x_host, int T, float beta, void* y_host);

/*
 * Routing record written by moe_forward when routing_stats != NULL.  Sections
 * in this order, each starting at a multiple of 16 bytes:
 *   int32  idx[T][2]      original ids of e0, e1
 *   float  wn[T][2]       weights applied to E_e0, E_e1 (1, 0 after a skip)
 *   float  ratio[T]       w_e1 / w_e0
 *   uint8  skipped[T]
 *   int32  count[E][2]    token-expert pairs that ran, per expert and slot
 *   int32  n_skipped
 *   int32  n_experts_touched   experts with at least one pair
 * moe_routing_stats_layout fills offsets[7] (bytes from the start, same order)
 * and returns the total size; moe_routing_stats_bytes returns only the size.
 */
size_t moe_routing_stats_layout(int T, int E, size_t offsets[7]);
size_t moe_routing_stats_bytes(int T, int E);

/*
 * beta for dynamic skipping (Sec. 3.3): the median over the T calibration
 * tokens of w_e1 / w_e0 under this layer's router; for even T the mean of the
 * two middle values.  x [T][h] bf16 device, T >= 1; *beta_out is host memory.
 * Synchronises the handle's stream.
 */
int moe_calibrate_beta(moe_layer_t* layer, const void* x, int T, float* beta_out);

/*
 * Layer-wise expert pruning search (Sec. 3.2, Eq. 3).  For every subset C of r
 * experts, in lexicographic order of the ascending index tuples, the pruned
 * layer F'(x, C) (router rows of the other experts removed, no skipping) is
 * compared with the unpruned layer F(x) over the T calibration tokens:
 *   losses[i] = || F'(x, C_i) - F(x) ||_F        (host, C(E, r) floats)
 *   *best_subset = bitmask of the first subset with the smallest loss (host)
 * Every expert is evaluated once per token (outputs kept in bf16) and each
 * subset only re-routes among its kept logits and gathers.  The handle must
 * have been created with all E experts kept; 2 <= r <= E.  x_calib [T][h] bf16
 * device, T >= 1.  Synchronises the handle's stream.
 */
int moe_prune_search(moe_layer_t* layer, const void* x_calib, int T, int r, float* losses,
                     uint32_t* best_subset);

/*
 * moe_calibrate_beta for callers that must not allocate device memory while they
 * run (a server whose own pool owns the whole GPU, a loop that cannot take the
 * device-wide synchronisation of cudaMalloc).  The paper has no counterpart;
 * the result is the same median of w_e1 / w_e0 (Sec. 3.3).
 *   W_gate_kept [r][h] bf16 device: the router rows of the kept experts, in
 *   ascending expert order (the whole W_gate when nothing is pruned);
 *   x [T][h] bf16 device; stream is a cudaStream_t; *beta_out is host memory.
 * The scratch of the two kernels (per-token routing record, 21 bytes per token)
 * lives in a fixed array inside the library image, about 340 KB that every GPU
 * loading the library holds until the process exits; T is therefore limited to
 * MOE_NOALLOC_MAX_TOKENS and larger T is rejected with MOE_ERR_INVALID_ARG.
 * The call makes no cudaMalloc/cudaFree and calls no allocating library
 * routine.  Its first call on a device is a warm-up: it looks up the array's
 * device address (cudaGetSymbolAddress), and under CUDA's lazy module loading
 * that look-up or the first launch may load this part of the library onto the
 * device, which takes device memory once (the code and the array).  Make that
 * first call at start-up, before any stream capture and before the device is
 * handed to the caller's own memory pool; the calls after it take nothing.
 * All calls share the one array, which keeps the previous call's contents:
 * every element that is read is rewritten first, so nothing needs clearing,
 * but two calls that overlap on the GPU (different streams or threads) race.
 * Synchronises the stream.
 */
#define MOE_NOALLOC_MAX_TOKENS 16384
int moe_calibrate_beta_noalloc(const void* W_gate_kept, const void* x, int T, int h, int r,
                               void* cuda_stream, float* beta_out);

/*
 * The same search for several subset sizes r_list[0..n_r-1] at once (Sec. 3.2:
 * the cached layer inputs and the experts' outputs on them do not depend on r,
 * only the enumeration does): the experts are evaluated once, for the smallest
 * size, and every size is enumerated over those outputs.  losses (host) receives
 * the C(E, r_list[0]) values of the first size, then those of the second, and so
 * on, each block in the order moe_prune_search uses; best_subsets (host) one
 * bitmask per size.  Results equal those of one moe_prune_search call per size.
 * 1 <= n_r <= 16; everything else as moe_prune_search.
 */
int moe_prune_search_multi(moe_layer_t* layer, const void* x_calib, int T, const int* r_list,
                           int n_r, float* losses, uint32_t* best_subsets);

/*
 * Progressive variant of the search (the paper's ablation of layer-wise vs
 * progressive pruning, Sec. 4.4 "Ablation"): the pruned layer is evaluated on
 * x_pruned, calibration states that already went through the pruned earlier
 * layers, while the target stays the unpruned model's cached output of this
 * layer:   losses[i] = || F'(x_pruned, C_i) - F_ref ||_F.
 * x_pruned [T][h] bf16 device; F_ref [T][h] fp32 device (the cached layer
 * output, without the residual); everything else as moe_prune_search.
 */
int moe_prune_search_progressive(moe_layer_t* layer, const void* x_pruned, const float* F_ref,
                                 int T, int r, float* losses, uint32_t* best_subset);

/*
 * Expert co-selection counts (App. A.1): counts[a][b] (host, E x E int32, row a) is
 * the number of the T tokens whose largest routing weight is expert a and second
 * largest expert b under this layer's router, original expert ids, no skipping.
 * The activation frequency of expert e is the sum of row e and column e.
 * x [T][h] bf16 device.  Synchronises the handle's stream.
 */
int moe_coselection(moe_layer_t* layer, const void* x, int T, int32_t* counts);

/*
 * The activation-frequency pruning baseline (Sec. 4.1, "Comparison with Other
 * Expert Pruning Baselines"): bitmask of the r experts with the highest
 * activation frequency in `counts` (as written by moe_coselection; ties to the
 * lower index).  Host only.  Returns 0 for invalid arguments.
 */
uint32_t moe_frequency_subset(const int32_t* counts, int E, int r);

/* Number of subsets moe_prune_search scores: C(E, r), 0 if out of range. */
long moe_num_subsets(int E, int r);

/*
 * RMSNorm with unit gain, out = bf16(x / sqrt(mean(x^2) + eps)), the
 * normalisation placed before each MoE layer when layers are stacked.
 * x, out [T][h] bf16 device (may alias); stream is a cudaStream_t.
 */
int moe_rmsnorm(const void* x, int T, int h, float eps, void* out, void* cuda_stream);

/*
 * A stack of MoE layers with attention left out:
 *   x_{l+1} = x_l + MoE_l(RMSNorm(x_l)),  l = 0 .. n_layers-1,
 * each layer with its own kept experts and its own betas[l] (host array, NULL
 * for no skipping).  x [T][h] bf16 device is not modified; y [T][h] receives
 * x_{n_layers}.  All layers must share h and run on the first layer's stream.
 * eps is the RMSNorm epsilon.
 */
int moe_stack_forward(moe_layer_t* const* layers, int n_layers, const void* x, int T,
                      const float* betas, float eps, void* y);

/*
 * Per-stage device time of moe_forward, for benchmarks.  While enabled, every
 * forward call on the handle records CUDA events on its stream at the stage
 * boundaries (not part of the paper's method; a few microseconds per call):
 *   stage 0  router + permutation (Sec. 3.1-3.3 routing, gather of routed rows)
 *   stage 1  gate/up grouped GEMM with the SwiGLU epilogue
 *   stage 2  down-projection grouped GEMM
 *   stage 3  combine (Eq. 2)
 * The searches record too: per chunk of 8192 calibration tokens one set of marks
 * (stage 0 routing + permutation, 1 gate/up GEMM, 2 down GEMM, 3 empty) and one
 * more set for the enumerations (stages 0-2 empty, 3 enumeration + reduction),
 * so a search of n chunks counts as n + 1 calls.
 * moe_profile_read synchronises the stream, writes the milliseconds summed over
 * the calls recorded since the last enable/read into stage_ms[MOE_PROFILE_STAGES]
 * and their number into *calls (host memory), and starts a new window.  At most
 * 8192 calls are recorded per window.
 */
#define MOE_PROFILE_STAGES 4
int moe_profile_enable(moe_layer_t* layer, int on);
int moe_profile_read(moe_layer_t* layer, float* stage_ms, int* calls);

/* 0 when no kernel of this handle has reported a bounded wait expiring since
 * the last call of this function, else MOE_ERR_DEVICE_TIMEOUT.  Synchronises. */
int moe_device_status(moe_layer_t* layer);

/* Message of the last failing call on this host thread ("" if none). */
const char* moe_last_error(void);

#ifdef __cplusplus
}
#endif
#endif /* MOE_H_ */
