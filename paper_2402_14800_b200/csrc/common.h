// Internal declarations shared by the translation units of libmoe.
#pragma once

#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "moe.h"

namespace moe {

typedef __nv_bfloat16 bf16;

constexpr int kMaxE = MOE_MAX_EXPERTS;
constexpr int kTileRows = 128;            // token rows per row tile of the grouped GEMMs
constexpr int kRouteTokPerBlock = 16;     // tokens routed by one block (one warp per token)
constexpr int kHistCols = 2 * kMaxE + 1;  // per (expert, slot) pair counts + skipped count
constexpr int kInterleave = 16;           // W1/W3 rows are interleaved in groups of 16
constexpr int kDecodeMaxT = 256;          // up to here the small-batch path (weights read once) is used
constexpr int kTokensDPerExpert = 40;      // small batches with this many tokens per expert or more: token-major decode GEMM
constexpr int kTokensDMaxKept = 6;         // ... on layers with at most this many kept experts
constexpr int kDecodeKbPerItem = 112;      // k-blocks (of 64) per split-K item, decode down-proj

// Device-resident description of one permuted batch, written by the scan kernel
// (or by set_dense_meta for the search) and read by every later kernel.
struct Meta {
  int32_t count[kMaxE];            // token-expert pairs that run, per kept expert (compact index)
  int32_t count_slot[kMaxE][2];    // the same, split by top-2 slot
  int32_t off[kMaxE + 1];          // first permuted row of each expert's group (padded groups)
  int32_t tile_prefix[kMaxE + 1];  // cumulative number of 128-row tiles
  int32_t rows_total;              // off[r]
  int32_t n_skipped;
  int32_t n_touched;
  int32_t reserved;
};

struct KeptIds {
  int32_t id[kMaxE];  // compact index -> original expert id
};

// Programmatic dependent launch: a kernel launched this way may start while its predecessor
// in the stream is still draining; it must call pdl_wait() before touching anything the
// predecessor wrote (or still reads).  Every kernel on the forward path calls
// pdl_launch_dependents() and pdl_wait() first thing (the GEMMs after their set-up), so the
// stream order of all memory accesses is unchanged and only launch latency and prologues overlap.
//
// THE RULE for every kernel launched with launch_pdl: whatever an earlier kernel of the stream
// may have written (token rows, routing records, permutation tables, the batch description,
// activations, expert outputs, the residual) is read with ld_l2() below (ld.global.cg), never
// through a `const T* __restrict__` parameter with a plain dereference or __ldg.  Such a kernel
// is resident while its predecessors still write, no kernel boundary invalidates the SM's L1 in
// between, and the non-coherent path (ld.global.nc, which the compiler may pick for const
// __restrict__ data) is only defined for data that does not change during the kernel's lifetime:
// an L1 line cached on this SM before the writer finished would be stale.  Only data that is
// constant from the creation of the handle on (router rows, expert weights) keeps __ldg or the
// streaming loads.  Operands that reach the SM through TMA are read at L2 by construction.
#ifdef __CUDACC__
__device__ __forceinline__ uint4 ld_l2(const uint4* p) { return __ldcg(p); }
__device__ __forceinline__ float4 ld_l2(const float4* p) { return __ldcg(p); }
__device__ __forceinline__ int ld_l2(const int32_t* p) { return __ldcg(p); }
__device__ __forceinline__ float ld_l2(const float* p) { return __ldcg(p); }
__device__ __forceinline__ int ld_l2(const uint8_t* p) { return (int)__ldcg(p); }
__device__ __forceinline__ float ld_l2(const __nv_bfloat16* p) {
  return __uint_as_float((uint32_t)__ldcg(reinterpret_cast<const unsigned short*>(p)) << 16);
}
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_launch_dependents() {
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}

// MOE_NO_PDL=1 (read when a handle is created) launches everything with plain stream order.
inline bool g_pdl_enabled = true;

template <typename... KArgs, typename... Args>
cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                       Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = g_pdl_enabled ? 1 : 0;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}
#endif

#ifdef __CUDACC__
// The same launch in plain stream order (the kernel's griddepcontrol instructions are no-ops).
template <typename... KArgs, typename... Args>
cudaError_t launch_plain(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                         Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}
#endif

// Stores the message moe_last_error() returns on this thread and returns `code` (api.cu).
int set_error(int code, const char* fmt, ...);

// ---- routing / permutation / element-wise kernels (route_permute.cu) --------------------
struct RouteOut {
  int32_t* idx;       // [T][2] compact expert index
  float* wn;          // [T][2]
  float* ratio;       // [T]
  uint8_t* skipped;   // [T]
  float* logits;      // [T][r] or null
  int32_t* blk_hist;  // [nblk][kHistCols] or null
  // user-visible routing record (all null when not requested)
  int32_t* s_idx;
  float* s_wn;
  float* s_ratio;
  uint8_t* s_skipped;
};

cudaError_t launch_router(const bf16* x, const bf16* Wg, int T, int h, int r, float beta,
                          const KeptIds& kept, const RouteOut& out, cudaStream_t st);
// Large batches (T > kDecodeMaxT): the logits on the tensor cores (gemm_sm100.cu), the decision as
// in launch_router.  Wg16 = the kept router rows padded with zero rows to kMaxE rows.
cudaError_t launch_router_tc(const bf16* x, const bf16* Wg16, int T, int h, int r, float beta,
                             const KeptIds& kept, const RouteOut& out, int* status, cudaStream_t st);
// T <= kDecodeMaxT: router with one block per token; permutation + gather with one block per token
cudaError_t launch_router_small(const bf16* x, const bf16* Wg, int T, int h, int r, float beta,
                                const KeptIds& kept, const RouteOut& out, cudaStream_t st);
cudaError_t launch_route_single(const bf16* x, const bf16* Wg, int h, int r, float beta,
                                const KeptIds& kept, const RouteOut& out, int pad, Meta* meta,
                                int32_t* pair_pos, int32_t* row_token, bf16* xperm, int32_t* s_count,
                                int32_t* s_nskipped, int32_t* s_ntouched, int E, cudaStream_t st);
cudaError_t launch_permute_gather_small(const bf16* x, const int32_t* idx, const uint8_t* skipped, int T,
                                        int h, int r, int pad, Meta* meta, int32_t* pair_pos,
                                        int32_t* row_token, bf16* xperm, int32_t* s_count,
                                        int32_t* s_nskipped, int32_t* s_ntouched, const KeptIds& kept,
                                        int E, cudaStream_t st);
cudaError_t launch_scan(const int32_t* blk_hist, int nblk, int r, int pad, int32_t* blk_base,
                        Meta* meta, int32_t* s_count, int32_t* s_nskipped, int32_t* s_ntouched,
                        const KeptIds& kept, int E, cudaStream_t st);
cudaError_t launch_scatter(const int32_t* idx, const uint8_t* skipped, const int32_t* blk_base,
                           const Meta* meta, int T, int32_t* pair_pos, int32_t* row_token,
                           cudaStream_t st);
cudaError_t launch_gather(const bf16* x, const int32_t* row_token, const Meta* meta, int h,
                          int cap_rows, bf16* xperm, cudaStream_t st);
cudaError_t launch_combine(const float* O, int ksplit, size_t split_stride, const int32_t* pair_pos,
                           const float* wn, const bf16* residual, int T, int h, bf16* y,
                           cudaStream_t st);
// general top-k path (k slots per token instead of two)
cudaError_t launch_router_topk(const bf16* x, const bf16* Wg, int T, int h, int r, int k, float beta,
                               const KeptIds& kept, int32_t* idx, float* wn, int32_t* nact,
                               int32_t* u_idx, float* u_wn, int32_t* u_nact, float* logits,
                               cudaStream_t st);
cudaError_t launch_count_topk(const int32_t* idx, const int32_t* nact, int T, int k,
                              int32_t* blk_hist, cudaStream_t st);
cudaError_t launch_scatter_topk(const int32_t* idx, const int32_t* nact, const int32_t* blk_base,
                                const Meta* meta, int T, int k, int32_t* pair_pos,
                                int32_t* row_token, cudaStream_t st);
cudaError_t launch_combine_topk(const float* O, int ksplit, size_t split_stride,
                                const int32_t* pair_pos, const float* wn, int k, int T, int h,
                                bf16* y, cudaStream_t st);
cudaError_t launch_coselection(const int32_t* idx, int T, int E, const KeptIds& kept, int32_t* counts,
                               cudaStream_t st);
cudaError_t launch_top2_distance(const float* O, int ksplit, size_t split_stride,
                                 const int32_t* pair_pos, int T, int h, float* dist, cudaStream_t st);
cudaError_t launch_rmsnorm(const bf16* x, int T, int h, float eps, bf16* out, cudaStream_t st);
cudaError_t launch_set_dense_meta(Meta* meta, int E, int rows_per_expert, int off_stride,
                                  cudaStream_t st);
// k-th smallest (0-based) of ratio[T] for k = k0 and k1, written to out[0], out[1]
cudaError_t launch_select2(const float* ratio, int T, int k0, int k1, float* out, cudaStream_t st);
// W13[c][32q + s] = W1[id[c]][16q + s] (s < 16) | W3[id[c]][16q + s - 16] (s >= 16)
cudaError_t launch_interleave(const bf16* W1, const bf16* W3, const KeptIds& kept, int r, int f,
                              int h, bf16* W13, cudaStream_t st);

// ---- grouped GEMMs (gemm_sm100.cu) ----------------------------------------------------
enum GemmOut { kOutActBf16 = 0, kOutF32 = 1, kOutBf16 = 2 };

struct GemmArgs {
  const Meta* meta;
  int r;         // kept experts
  int K;         // contraction length (h for gate/up, f for down)
  int n_w_rows;  // weight rows per expert (2f interleaved for gate/up, h for down)
  // token-side operand rows: a_row = a_row_base + a_off_mul * off[c] + 128 * m
  int a_row_base, a_off_mul;
  // output rows: out_row = out_row_base + out_off_mul * off[c] + 128 * m; column offset c * out_col_mul
  int out_row_base, out_off_mul;
  long long out_col_mul;
  long long out_ld;        // elements between output rows
  void* out;               // bf16 activations / fp32 outputs / bf16 expert outputs
  long long split_stride;  // elements between split-K partial planes (decode down-proj)
  int* status;             // device error word
  // weight-major kernel: arrival counters (kTailHeaderBytes, zero between launches) followed by
  // the partial tiles of the K-sliced tail items; null = no slicing
  float* tail;
};

constexpr size_t kTailHeaderBytes = 4096;  // four arrival counters per tail item
constexpr size_t kTailBufferBytes = kTailHeaderBytes + (size_t)1024 * 128 * 128 * 4;  // 1024 slots of 128 tokens

int gemm_init_driver_api();  // resolves cuTensorMapEncodeTiled; 0 on success
int make_map_2d(CUtensorMap* m, const void* base, uint64_t inner, uint64_t rows, uint32_t box_rows);
int make_map_3d(CUtensorMap* m, const void* base, uint64_t inner, uint64_t rows, uint64_t planes,
                uint32_t box_rows);

struct GemmMaps {
  CUtensorMap w;     // weights [planes = r][rows][K], box 64 x (256 or 128) x 1
  CUtensorMap t[4];  // token-side operand [rows][K], boxes of 16 / 32 / 64 / 128 rows
};

// Token rows are the 128-row MMA operand, weights the 256-wide one (large T).
cudaError_t launch_gemm_tokens_m(bool gate_up, GemmOut out_kind, const GemmMaps& maps,
                                 const GemmArgs& a, cudaStream_t st);
// Weight rows are the 128-row MMA operand, tokens the narrow one (small T): weights stream once.
cudaError_t launch_gemm_tokens_d(bool gate_up, const GemmMaps& maps, const GemmArgs& a, int kb_per_item,
                                 cudaStream_t st);
cudaError_t launch_gemm_weights_m(bool gate_up, const GemmMaps& maps, const GemmArgs& a,
                                  int kb_per_item, int max_tokens_per_tile, cudaStream_t st);
// Single-token forward on the CUDA cores (T = 1 only): routing + gate/up matrix-vector kernel,
// then the down projection with the weighted sum of Eq. 2, which writes y.
cudaError_t gemv_single_setup();
bool gemv_single_fits(int h, int f);
cudaError_t launch_gemv_route_gate_up(const bf16* x, const bf16* Wg, const bf16* W13, int r, int h, int f,
                                      float beta, const KeptIds& kept, const RouteOut& ro, Meta* meta,
                                      int32_t* pair_pos, int32_t* row_token, int32_t* s_count,
                                      int32_t* s_nskipped, int32_t* s_ntouched, int E, bf16* act,
                                      cudaStream_t st);
cudaError_t launch_gemv_down_combine(const bf16* act, const bf16* W2, const int32_t* idx,
                                     const uint8_t* skipped, const float* wn, const bf16* residual,
                                     int h, int f, bf16* y, cudaStream_t st);
// Plain CUDA-core kernels of the same contractions, for bring-up and debugging only
// (MOE_DEBUG_SIMT=1); never selected otherwise.
cudaError_t launch_simt_gate_up(const bf16* A, const bf16* W13, const GemmArgs& a, int cap_rows,
                                cudaStream_t st);
cudaError_t launch_simt_down(const bf16* A, const bf16* W2, const GemmArgs& a, int cap_rows,
                             GemmOut out_kind, cudaStream_t st);
cudaError_t gemm_set_attributes();
// Test hook: one CTA runs the GEMMs' bounded wait on a barrier nobody arrives on, then their
// abort path (see moe_test_hooks.h).
cudaError_t launch_wait_expiry(int* status, unsigned long long limit_ns, cudaStream_t st);

// ---- search (search.cu) ---------------------------------------------------------------
// Where the enumeration finds the expert outputs.  Dense (topk_idx == null): Yall[T][E][h].
// Pruned work: only each token's K = E - r + 2 top-ranked experts were evaluated;
// topk_idx[T][K] lists them in rank order and their outputs are rows of a permuted buffer,
// row (t / chunk_tokens) * chunk_rows + pair_pos[t][rank].
struct EnumSource {
  const int32_t* topk_idx;
  const int32_t* pair_pos;
  int chunk_tokens;
  int chunk_rows;
  int k_stride;  // ranked experts recorded per token in topk_idx / pair_pos (>= E - r + 2)
};
int enumerate_num_blocks(int T, int nC);
cudaError_t launch_enumerate(const float* logits, const bf16* Yall, int T, int E, int r, int h,
                             const uint32_t* subsets, int nC, float* partial, double* loss_sq,
                             float* losses, const float* Fref, const EnumSource& src,
                             cudaStream_t st);

}  // namespace moe
