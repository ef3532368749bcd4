// C ABI of libmoe: handle, argument checks, scratch management and the kernel sequences.
#include <math.h>
#include <stdarg.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include <algorithm>
#include <vector>

#include "common.h"
#include "moe_test_hooks.h"

using namespace moe;

namespace {

thread_local char g_err[512] = "";

int fail(int code, const char* fmt, ...) {
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(g_err, sizeof(g_err), fmt, ap);
  va_end(ap);
  return code;
}

#define CUDA_TRY(expr)                                                                   \
  do {                                                                                   \
    cudaError_t e_ = (expr);                                                             \
    if (e_ != cudaSuccess)                                                               \
      return fail(e_ == cudaErrorMemoryAllocation ? MOE_ERR_OOM : MOE_ERR_CUDA, "%s: %s", \
                  #expr, cudaGetErrorString(e_));                                        \
  } while (0)

constexpr int kMaxTokens = 1 << 24;  // per call; keeps every row index and byte count in range
constexpr long kMaxSubsetsPerPass = 16384;  // subsets of several sizes share an enumeration pass up to here
inline int popc(uint32_t v) { return __builtin_popcount(v); }
inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }
inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// Binomial coefficients from Pascal's triangle (n <= 16 here).
long binom(int n, int k) {
  if (n < 0 || k < 0 || k > n || n > 2 * kMaxE) return 0;
  long row[2 * kMaxE + 2] = {1};
  for (int i = 1; i <= n; ++i)
    for (int j = i; j >= 1; --j) row[j] += row[j - 1];
  return row[k];
}

// Test hook (moe_test_set_free_bytes_limit): an upper bound on what cudaMemGetInfo may report.
long long g_free_bytes_limit = -1;

cudaError_t free_device_bytes(size_t* free_b) {
  size_t total_b = 0;
  cudaError_t e = cudaMemGetInfo(free_b, &total_b);
  if (e == cudaSuccess && g_free_bytes_limit >= 0 && *free_b > (size_t)g_free_bytes_limit)
    *free_b = (size_t)g_free_bytes_limit;
  return e;
}

// A device buffer that only grows.
struct Buf {
  void* p = nullptr;
  size_t bytes = 0;
};

}  // namespace

// Scratch of the kernel sequences.  Every handle owns one; a stack of layers runs all of
// its layers out of the first layer's workspace.
struct Workspace {
  size_t scratch_bytes = 0;
  // routing scratch (capacity in tokens)
  int cap_route_T = 0;
  Buf idx, wn, ratio, skipped, blk_hist, blk_base, pair_pos, meta, status, sel;
  // GEMM scratch (capacity in permuted rows)
  int cap_rows = 0;
  int map_h = 0, map_f = 0;
  Buf row_token, xperm, act, O, tail;
  CUtensorMap tok_x[4], tok_act[4];  // boxes of 16/32/64/128 rows over xperm and act
  // search scratch
  Buf s_logits, s_yall, s_act, s_subsets, s_partial, s_loss_sq, s_losses, s_xpad, s_meta, s_xperm, s_rowtok;
  // host staging and stack scratch
  Buf hx, hy, xn, cosel;
  // general top-k path
  Buf k_idx, k_wn, k_pos, k_nact;
};

int moe::set_error(int code, const char* fmt, ...) {
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(g_err, sizeof(g_err), fmt, ap);
  va_end(ap);
  return code;
}

struct moe_layer {
  int h = 0, f = 0, E = 0, r = 0;
  uint32_t kept_mask = 0;
  KeptIds kept;
  bf16* Wg = nullptr;   // [r][h]
  bf16* W13 = nullptr;  // [r][2f][h], gate/up rows interleaved by 16
  bf16* W2 = nullptr;   // [r][h][f]
  size_t weight_bytes = 0;
  cudaStream_t stream = 0;
  bool debug_simt = false;
  int decode_kernel = 0;  // small batches: 0 = by batch size, 1 = weight-major, 2 = token-major (MOE_DECODE_KERNEL=wm|td)
  bool single_gemv = true;    // T = 1 runs the matrix-vector kernels (MOE_SINGLE_KERNEL=gemm: the GEMM path)
  bool search_dense = false;  // MOE_SEARCH_DENSE=1: evaluate all E experts per token in the search
  CUtensorMap w13_256, w13_128, w2_256, w2_128;
  Workspace own;
  Workspace* ws = &own;
  // per-stage device timing (off unless moe_profile_enable)
  bool prof = false;
  std::vector<cudaEvent_t> prof_ev;  // MOE_PROFILE_STAGES + 1 marks per recorded call
  size_t prof_used = 0;
  int* h_status = nullptr;  // pinned host copy of the device status word
};

namespace {

int grow(moe_layer* L, Buf& b, size_t bytes) {
  if (bytes <= b.bytes) return MOE_OK;
  if (b.p) {
    cudaStreamSynchronize(L->stream);
    cudaFree(b.p);
    L->ws->scratch_bytes -= b.bytes;
    b.p = nullptr;
    b.bytes = 0;
  }
  size_t free_b = 0;
  if (free_device_bytes(&free_b) == cudaSuccess && bytes > free_b)
    return fail(MOE_ERR_OOM, "scratch of %zu bytes does not fit (%zu free)", bytes, free_b);
  cudaError_t e = cudaMalloc(&b.p, bytes);
  if (e != cudaSuccess) {
    b.p = nullptr;
    cudaGetLastError();
    return fail(MOE_ERR_OOM, "cudaMalloc(%zu): %s", bytes, cudaGetErrorString(e));
  }
  b.bytes = bytes;
  L->ws->scratch_bytes += bytes;
  return MOE_OK;
}

void release(moe_layer* L, Buf& b) {
  if (b.p) cudaFree(b.p);
  L->own.scratch_bytes -= b.bytes;
  b.p = nullptr;
  b.bytes = 0;
}

int ensure_route(moe_layer* L, int T) {
  int rc;
  if ((rc = grow(L, L->ws->meta, sizeof(Meta)))) return rc;
  if (!L->ws->status.p) {
    if ((rc = grow(L, L->ws->status, 16))) return rc;
    CUDA_TRY(cudaMemsetAsync(L->ws->status.p, 0, 16, L->stream));
  }
  if ((rc = grow(L, L->ws->sel, 16))) return rc;
  if (T <= L->ws->cap_route_T) return MOE_OK;
  const size_t nblk = (T + kRouteTokPerBlock - 1) / kRouteTokPerBlock;
  // a buffer that fails to grow is gone: the capacity is void until every buffer has grown
  L->ws->cap_route_T = 0;
  if ((rc = grow(L, L->ws->idx, (size_t)T * 8))) return rc;
  if ((rc = grow(L, L->ws->wn, (size_t)T * 8))) return rc;
  if ((rc = grow(L, L->ws->ratio, (size_t)T * 4))) return rc;
  if ((rc = grow(L, L->ws->skipped, align_up((size_t)T, 16)))) return rc;
  if ((rc = grow(L, L->ws->pair_pos, (size_t)T * 8))) return rc;
  if ((rc = grow(L, L->ws->blk_hist, nblk * kHistCols * 4))) return rc;
  if ((rc = grow(L, L->ws->blk_base, nblk * kMaxE * 4))) return rc;
  L->ws->cap_route_T = T;
  return MOE_OK;
}

inline bool decode_mode(int T) { return T <= kDecodeMaxT; }
// Small batches run the weight-major GEMM unless the experts hold many tokens each (about
// 2T/r): from kTokensDPerExpert on, the token-major decode GEMM is faster on layers of at most
// kTokensDMaxKept kept experts (measured crossover; with 8 experts the weight-major kernel won
// up to the largest small batch, 64 tokens per expert).
inline bool decode_weights_m(const moe_layer* L, int T) {
  return L->decode_kernel == 1 ||
         (L->decode_kernel == 0 && (2 * T < kTokensDPerExpert * L->r || L->r > kTokensDMaxKept));
}
inline int rows_for(const moe_layer* L, int T, int k = 2) {
  const int pad = decode_mode(T) ? 16 : kTileRows;
  return (int)align_up((size_t)k * T + (size_t)L->r * pad, 16);
}
// k-blocks per work item of the small-batch down projection: with one or two tokens at most four
// experts are touched, and finer items spread their few weight tiles over more SMs
inline int down_kb_per_item(int T) { return T <= 2 ? (kDecodeKbPerItem + 1) / 2 : kDecodeKbPerItem; }
inline int ksplit_for(const moe_layer* L, int T) {
  const int KB = (L->f + 63) / 64;
  return (KB + down_kb_per_item(T) - 1) / down_kb_per_item(T);
}

int build_token_maps(GemmMaps& m, const void* base, uint64_t inner, uint64_t rows) {
  for (int b = 0; b < 4; ++b)
    if (make_map_2d(&m.t[b], base, inner, rows, 16u << b))
      return fail(MOE_ERR_CUDA, "cuTensorMapEncodeTiled failed for a token-side operand");
  return MOE_OK;
}

int ensure_gemm(moe_layer* L, int T, int k = 2) {
  // capacity in rows: large enough for this T in its mode, at least 256 (TMA boxes)
  int need = (int)align_up((size_t)rows_for(L, T, k), kTileRows) + kTileRows;
  if (need < 256) need = 256;
  size_t need_O = (size_t)need * L->h * (decode_mode(T) ? ksplit_for(L, T) : 1);
  if (need <= L->ws->cap_rows && need_O * 4 <= L->ws->O.bytes && L->ws->map_h == L->h &&
      L->ws->map_f == L->f)
    return MOE_OK;
  if (need < L->ws->cap_rows) need = L->ws->cap_rows;
  int rc;
  L->ws->cap_rows = 0;  // void until every buffer has grown and the tensor maps are rebuilt
  if ((rc = grow(L, L->ws->row_token, (size_t)need * 4))) return rc;
  if ((rc = grow(L, L->ws->xperm, (size_t)need * L->h * 2))) return rc;
  if ((rc = grow(L, L->ws->act, (size_t)need * L->f * 2))) return rc;
  if ((rc = grow(L, L->ws->O, need_O * 4))) return rc;
  const void* tail_before = L->ws->tail.p;
  if ((rc = grow(L, L->ws->tail, kTailBufferBytes))) return rc;
  if (L->ws->tail.p != tail_before)  // the arrival counters start at zero and return to zero
    CUDA_TRY(cudaMemsetAsync(L->ws->tail.p, 0, kTailHeaderBytes, L->stream));
  L->ws->cap_rows = need;
  L->ws->map_h = L->h;
  L->ws->map_f = L->f;
  GemmMaps tmp;
  if ((rc = build_token_maps(tmp, L->ws->xperm.p, L->h, need))) return rc;
  memcpy(L->ws->tok_x, tmp.t, sizeof(tmp.t));
  if ((rc = build_token_maps(tmp, L->ws->act.p, L->f, need))) return rc;
  memcpy(L->ws->tok_act, tmp.t, sizeof(tmp.t));
  return MOE_OK;
}

// Records a stage boundary on the handle's stream while profiling is on.
void mark(moe_layer* L) {
  if (!L->prof) return;
  if (L->prof_used == L->prof_ev.size()) {
    if (L->prof_ev.size() >= 5 * 8192) return;  // enough samples; stop recording
    cudaEvent_t e;
    if (cudaEventCreate(&e) != cudaSuccess) return;
    L->prof_ev.push_back(e);
  }
  cudaEventRecord(L->prof_ev[L->prof_used++], L->stream);
}

int check_status(moe_layer* L) {
  // the status word is read into pinned memory: a copy to pageable memory is staged by the runtime
  if (!L->h_status && cudaHostAlloc((void**)&L->h_status, sizeof(int), cudaHostAllocDefault) != cudaSuccess) {
    cudaGetLastError();
    L->h_status = nullptr;
  }
  int st_pageable = 0;
  int* dst = L->h_status ? L->h_status : &st_pageable;
  CUDA_TRY(cudaMemcpyAsync(dst, L->ws->status.p, 4, cudaMemcpyDeviceToHost, L->stream));
  CUDA_TRY(cudaStreamSynchronize(L->stream));
  const int st = *dst;
  if (st != 0) {
    cudaMemsetAsync(L->ws->status.p, 0, 4, L->stream);
    // an aborted GEMM may have left arrival counters of its K-sliced tail items behind
    if (L->ws->tail.p) cudaMemsetAsync(L->ws->tail.p, 0, kTailHeaderBytes, L->stream);
    return fail(MOE_ERR_DEVICE_TIMEOUT, "a bounded wait inside a GEMM kernel expired");
  }
  return MOE_OK;
}

// The two grouped GEMMs of the experts over a batch described by `meta`.
int run_expert_gemms(moe_layer* L, const Meta* meta, bool weights_m, const GemmMaps& m_gu,
                     const GemmMaps& m_dn, GemmArgs gu, GemmArgs dn, GemmOut dn_kind,
                     const bf16* gu_A, const bf16* dn_A, int simt_rows, int T = 0) {
  gu.meta = meta; dn.meta = meta;
  gu.r = L->r; dn.r = L->r;
  gu.K = L->h; gu.n_w_rows = 2 * L->f;
  dn.K = L->f; dn.n_w_rows = L->h;
  gu.status = (int*)L->ws->status.p; dn.status = (int*)L->ws->status.p;
  if (L->debug_simt) {
    CUDA_TRY(launch_simt_gate_up(gu_A, L->W13, gu, simt_rows, L->stream));
    mark(L);
    CUDA_TRY(launch_simt_down(dn_A, L->W2, dn, simt_rows, dn_kind, L->stream));
  } else if (weights_m && decode_weights_m(L, T)) {
    CUDA_TRY(launch_gemm_weights_m(true, m_gu, gu, (L->h + 63) / 64, T, L->stream));
    mark(L);
    CUDA_TRY(launch_gemm_weights_m(false, m_dn, dn, down_kb_per_item(T), T, L->stream));
  } else if (weights_m) {
    CUDA_TRY(launch_gemm_tokens_d(true, m_gu, gu, (L->h + 63) / 64, L->stream));
    mark(L);
    CUDA_TRY(launch_gemm_tokens_d(false, m_dn, dn, down_kb_per_item(T), L->stream));
  } else {
    CUDA_TRY(launch_gemm_tokens_m(true, kOutActBf16, m_gu, gu, L->stream));
    mark(L);
    CUDA_TRY(launch_gemm_tokens_m(false, dn_kind, m_dn, dn, L->stream));
  }
  return MOE_OK;
}

// dist != nullptr: instead of combining, write || E_e0(x) - E_e1(x) ||_2 per token (y unused)
int forward_impl(moe_layer* L, const void* x, int T, float beta, const void* residual, void* y,
                 void* stats, float* dist = nullptr) {
  if (!L) return fail(MOE_ERR_INVALID_ARG, "layer is NULL");
  if (T < 0 || T > kMaxTokens) return fail(MOE_ERR_INVALID_ARG, "T = %d outside 0..%d", T, kMaxTokens);
  if (T == 0) return MOE_OK;
  if (!x || (!y && !dist)) return fail(MOE_ERR_INVALID_ARG, "x or the output is NULL");
  if (!aligned16(x) || !aligned16(y) || !aligned16(residual) || !aligned16(stats))
    return fail(MOE_ERR_INVALID_ARG, "x, y, residual and routing_stats must be 16-byte aligned");
  if (!(beta >= 0.f)) return fail(MOE_ERR_INVALID_ARG, "beta must be >= 0");
  if (x == y) return fail(MOE_ERR_INVALID_ARG, "x and y may not overlap");
  int rc;
  if ((rc = ensure_route(L, T))) return rc;
  if ((rc = ensure_gemm(L, T))) return rc;
  cudaStream_t st = L->stream;
  const bool dec = decode_mode(T);
  const int nblk = (T + kRouteTokPerBlock - 1) / kRouteTokPerBlock;
  const int rows_cap = rows_for(L, T);

  RouteOut ro;
  memset(&ro, 0, sizeof(ro));
  ro.idx = (int32_t*)L->ws->idx.p; ro.wn = (float*)L->ws->wn.p; ro.ratio = (float*)L->ws->ratio.p;
  ro.skipped = (uint8_t*)L->ws->skipped.p; ro.blk_hist = (int32_t*)L->ws->blk_hist.p;
  int32_t *s_count = nullptr, *s_nsk = nullptr, *s_nt = nullptr;
  if (stats) {
    size_t off[7];
    moe_routing_stats_layout(T, L->E, off);
    char* s = (char*)stats;
    ro.s_idx = (int32_t*)(s + off[0]); ro.s_wn = (float*)(s + off[1]);
    ro.s_ratio = (float*)(s + off[2]); ro.s_skipped = (uint8_t*)(s + off[3]);
    s_count = (int32_t*)(s + off[4]); s_nsk = (int32_t*)(s + off[5]); s_nt = (int32_t*)(s + off[6]);
  }
  Meta* meta = (Meta*)L->ws->meta.p;
  if (L->prof && (L->prof_used % (MOE_PROFILE_STAGES + 1)) != 0) L->prof_used = 0;
  mark(L);
  const bool single_gemv = T == 1 && L->single_gemv && !L->debug_simt && !dist;
  if (single_gemv) {
    mark(L);  // (no routing stage of its own)
    // one token: routing inside the gate/up matrix-vector kernel; the second kernel also forms
    // the weighted sum and writes y
    CUDA_TRY(launch_gemv_route_gate_up((const bf16*)x, L->Wg, L->W13, L->r, L->h, L->f, beta, L->kept, ro,
                                       meta, (int32_t*)L->ws->pair_pos.p, (int32_t*)L->ws->row_token.p,
                                       s_count, s_nsk, s_nt, L->E, (bf16*)L->ws->act.p, st));
    mark(L);
    CUDA_TRY(launch_gemv_down_combine((const bf16*)L->ws->act.p, L->W2, ro.idx, ro.skipped, ro.wn,
                                      (const bf16*)residual, L->h, L->f, (bf16*)y, st));
    mark(L);
    mark(L);
    return MOE_OK;
  }
  if (T == 1) {
    CUDA_TRY(launch_route_single((const bf16*)x, L->Wg, L->h, L->r, beta, L->kept, ro, 16, meta,
                                 (int32_t*)L->ws->pair_pos.p, (int32_t*)L->ws->row_token.p,
                                 (bf16*)L->ws->xperm.p, s_count, s_nsk, s_nt, L->E, st));
  } else if (dec) {
    CUDA_TRY(launch_router_small((const bf16*)x, L->Wg, T, L->h, L->r, beta, L->kept, ro, st));
    CUDA_TRY(launch_permute_gather_small((const bf16*)x, ro.idx, ro.skipped, T, L->h, L->r, 16, meta,
                                         (int32_t*)L->ws->pair_pos.p, (int32_t*)L->ws->row_token.p,
                                         (bf16*)L->ws->xperm.p, s_count, s_nsk, s_nt, L->kept, L->E, st));
  } else {
    // the tensor-core router wins from about 64 tiles of 128 tokens on (T = 8192: routing stage
    // 0.144 -> 0.115 ms, T = 32768: 0.52 -> 0.35 ms; T = 4096 equal, T = 2048 slower on its 16 CTAs)
    if (L->debug_simt || T < 64 * kTileRows)
      CUDA_TRY(launch_router((const bf16*)x, L->Wg, T, L->h, L->r, beta, L->kept, ro, st));
    else
      CUDA_TRY(launch_router_tc((const bf16*)x, L->Wg, T, L->h, L->r, beta, L->kept, ro,
                                (int*)L->ws->status.p, st));
    CUDA_TRY(launch_scan(ro.blk_hist, nblk, L->r, kTileRows, (int32_t*)L->ws->blk_base.p, meta,
                         s_count, s_nsk, s_nt, L->kept, L->E, st));
    CUDA_TRY(cudaMemsetAsync(L->ws->row_token.p, 0xff, (size_t)rows_cap * 4, st));
    CUDA_TRY(launch_scatter(ro.idx, ro.skipped, (int32_t*)L->ws->blk_base.p, meta, T,
                            (int32_t*)L->ws->pair_pos.p, (int32_t*)L->ws->row_token.p, st));
  }
  if (!dec)
    CUDA_TRY(launch_gather((const bf16*)x, (int32_t*)L->ws->row_token.p, meta, L->h, rows_cap,
                           (bf16*)L->ws->xperm.p, st));
  mark(L);

  GemmArgs gu, dn;
  memset(&gu, 0, sizeof(gu));
  memset(&dn, 0, sizeof(dn));
  gu.a_off_mul = 1; gu.out_off_mul = 1; gu.out_ld = L->f; gu.out = L->ws->act.p;
  dn.a_off_mul = 1; dn.out_off_mul = 1; dn.out_ld = L->h; dn.out = L->ws->O.p;
  const bool wm = dec && !L->debug_simt;
  if (wm) {
    gu.tail = (float*)L->ws->tail.p; dn.tail = (float*)L->ws->tail.p;
  }
  const int ksplit = wm ? ksplit_for(L, T) : 1;
  const size_t split_stride = (size_t)rows_cap * L->h;
  dn.split_stride = (long long)split_stride;
  GemmMaps m_gu, m_dn;
  m_gu.w = (wm && decode_weights_m(L, T)) ? L->w13_128 : L->w13_256;
  m_dn.w = (wm && decode_weights_m(L, T)) ? L->w2_128 : L->w2_256;
  memcpy(m_gu.t, L->ws->tok_x, sizeof(m_gu.t));
  memcpy(m_dn.t, L->ws->tok_act, sizeof(m_dn.t));
  rc = run_expert_gemms(L, meta, wm, m_gu, m_dn, gu, dn, kOutF32, (const bf16*)L->ws->xperm.p,
                        (const bf16*)L->ws->act.p, rows_cap, T);
  if (rc) return rc;
  mark(L);
  if (dist)
    CUDA_TRY(launch_top2_distance((const float*)L->ws->O.p, ksplit, split_stride,
                                  (int32_t*)L->ws->pair_pos.p, T, L->h, dist, st));
  else
    CUDA_TRY(launch_combine((const float*)L->ws->O.p, ksplit, split_stride, (int32_t*)L->ws->pair_pos.p,
                            (float*)L->ws->wn.p, (const bf16*)residual, T, L->h, (bf16*)y, st));
  mark(L);
  return MOE_OK;
}

}  // namespace

// ======================================================================================
extern "C" {

const char* moe_last_error(void) { return g_err; }

long moe_num_subsets(int E, int r) {
  if (E < 2 || E > kMaxE || r < 2 || r > E) return 0;
  return binom(E, r);
}

size_t moe_routing_stats_layout(int T, int E, size_t offsets[7]) {
  size_t o = 0;
  const size_t sizes[7] = {(size_t)T * 8, (size_t)T * 8, (size_t)T * 4, (size_t)T,
                           (size_t)E * 8, 4, 4};
  for (int i = 0; i < 7; ++i) {
    if (offsets) offsets[i] = o;
    o = align_up(o + sizes[i], 16);
  }
  return o;
}

size_t moe_routing_stats_bytes(int T, int E) { return moe_routing_stats_layout(T, E, nullptr); }

moe_layer_t* moe_layer_create(const void* W_gate, const void* W1, const void* W3, const void* W2,
                              int h, int f, int E, uint32_t kept_mask) {
  g_err[0] = 0;
  if (!W_gate || !W1 || !W3 || !W2) { fail(MOE_ERR_INVALID_ARG, "a weight pointer is NULL"); return nullptr; }
  if (!aligned16(W_gate) || !aligned16(W1) || !aligned16(W3) || !aligned16(W2)) {
    fail(MOE_ERR_INVALID_ARG, "weight pointers must be 16-byte aligned");
    return nullptr;
  }
  if (E < 2 || E > kMaxE) { fail(MOE_ERR_UNSUPPORTED_SHAPE, "E = %d outside 2..%d", E, kMaxE); return nullptr; }
  if (h < 64 || f < 64 || h % 64 || f % 64) {
    fail(MOE_ERR_UNSUPPORTED_SHAPE, "h = %d and f = %d must be positive multiples of 64", h, f);
    return nullptr;
  }
  if (kept_mask >> E) { fail(MOE_ERR_INVALID_ARG, "kept_mask has bits beyond expert %d", E - 1); return nullptr; }
  if (popc(kept_mask) < 2) { fail(MOE_ERR_INVALID_ARG, "kept_mask keeps fewer than 2 experts"); return nullptr; }

  int dev = 0, major = 0;
  if (cudaGetDevice(&dev) != cudaSuccess ||
      cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) {
    cudaGetLastError();
    fail(MOE_ERR_CUDA, "no usable CUDA device");
    return nullptr;
  }
  if (major != 10) { fail(MOE_ERR_ARCH, "device has compute capability %d.x, sm_100 is required", major); return nullptr; }
  if (gemm_init_driver_api()) { fail(MOE_ERR_CUDA, "cuTensorMapEncodeTiled is not available"); return nullptr; }
  cudaError_t e = gemm_set_attributes();
  if (e == cudaSuccess) e = gemv_single_setup();
  if (e != cudaSuccess) { fail(MOE_ERR_CUDA, "kernel attributes: %s", cudaGetErrorString(e)); return nullptr; }

  moe_layer* L = new (std::nothrow) moe_layer();
  if (!L) { fail(MOE_ERR_OOM, "host allocation failed"); return nullptr; }
  L->h = h; L->f = f; L->E = E; L->kept_mask = kept_mask; L->r = popc(kept_mask);
  for (int e_ = 0, c = 0; e_ < kMaxE; ++e_) {
    if (e_ < E && ((kept_mask >> e_) & 1u)) L->kept.id[c++] = e_;
  }
  for (int c = L->r; c < kMaxE; ++c) L->kept.id[c] = 0;
  const char* dbg = getenv("MOE_DEBUG_SIMT");
  L->debug_simt = dbg && dbg[0] == '1';
  const char* dk = getenv("MOE_DECODE_KERNEL");
  L->decode_kernel = (dk && !strcmp(dk, "wm")) ? 1 : ((dk && !strcmp(dk, "td")) ? 2 : 0);
  const char* sk = getenv("MOE_SINGLE_KERNEL");
  L->single_gemv = !(sk && !strcmp(sk, "gemm")) && L->decode_kernel == 0 && gemv_single_fits(h, f);
  const char* nopdl = getenv("MOE_NO_PDL");
  if (nopdl) g_pdl_enabled = nopdl[0] != '1';
  const char* dense = getenv("MOE_SEARCH_DENSE");
  L->search_dense = dense && dense[0] == '1';

  // the router rows are padded with zero rows to kMaxE rows (the tensor-core router's operand)
  const size_t n_gate = (size_t)kMaxE * h * 2, n_13 = (size_t)L->r * 2 * f * h * 2,
               n_2 = (size_t)L->r * h * f * 2;
  size_t free_b = 0;
  if (free_device_bytes(&free_b) != cudaSuccess) free_b = ~(size_t)0;
  if (n_gate + n_13 + n_2 > free_b) {
    fail(MOE_ERR_OOM, "weights of %zu bytes do not fit (%zu free)", n_gate + n_13 + n_2, free_b);
    delete L;
    return nullptr;
  }
  bool ok = cudaMalloc((void**)&L->Wg, n_gate) == cudaSuccess &&
            cudaMalloc((void**)&L->W13, n_13) == cudaSuccess &&
            cudaMalloc((void**)&L->W2, n_2) == cudaSuccess;
  if (!ok) {
    cudaGetLastError();
    fail(MOE_ERR_OOM, "cudaMalloc of the layer weights failed");
    moe_layer_destroy(L);
    return nullptr;
  }
  L->weight_bytes = n_gate + n_13 + n_2;
  ok = cudaMemsetAsync(L->Wg, 0, n_gate, 0) == cudaSuccess;
  for (int c = 0; c < L->r && ok; ++c) {
    const int id = L->kept.id[c];
    ok = ok && cudaMemcpyAsync(L->Wg + (size_t)c * h, (const bf16*)W_gate + (size_t)id * h,
                               (size_t)h * 2, cudaMemcpyDeviceToDevice, 0) == cudaSuccess;
    ok = ok && cudaMemcpyAsync(L->W2 + (size_t)c * h * f, (const bf16*)W2 + (size_t)id * h * f,
                               (size_t)h * f * 2, cudaMemcpyDeviceToDevice, 0) == cudaSuccess;
  }
  ok = ok && launch_interleave((const bf16*)W1, (const bf16*)W3, L->kept, L->r, f, h, L->W13, 0) ==
                 cudaSuccess;
  ok = ok && cudaDeviceSynchronize() == cudaSuccess;
  if (!ok) {
    fail(MOE_ERR_CUDA, "copying the weights failed: %s", cudaGetErrorString(cudaGetLastError()));
    moe_layer_destroy(L);
    return nullptr;
  }
  if (make_map_3d(&L->w13_256, L->W13, h, 2 * (uint64_t)f, L->r, 256) ||
      make_map_3d(&L->w13_128, L->W13, h, 2 * (uint64_t)f, L->r, 128) ||
      make_map_3d(&L->w2_256, L->W2, f, h, L->r, 256) ||
      make_map_3d(&L->w2_128, L->W2, f, h, L->r, 128)) {
    fail(MOE_ERR_CUDA, "cuTensorMapEncodeTiled failed for the weights");
    moe_layer_destroy(L);
    return nullptr;
  }
  return L;
}

void moe_layer_destroy(moe_layer_t* L) {
  if (!L) return;
  cudaStreamSynchronize(L->stream);
  Buf* bufs[] = {&L->own.idx, &L->own.wn, &L->own.ratio, &L->own.skipped, &L->own.blk_hist, &L->own.blk_base, &L->own.pair_pos,
                 &L->own.meta, &L->own.status, &L->own.sel, &L->own.row_token, &L->own.xperm, &L->own.act, &L->own.O, &L->own.tail,
                 &L->own.s_logits, &L->own.s_yall, &L->own.s_act, &L->own.s_subsets, &L->own.s_partial, &L->own.s_loss_sq,
                 &L->own.s_losses, &L->own.s_xpad, &L->own.s_meta, &L->own.s_xperm, &L->own.s_rowtok, &L->own.hx, &L->own.hy, &L->own.xn, &L->own.cosel, &L->own.k_idx, &L->own.k_wn, &L->own.k_pos, &L->own.k_nact};
  for (Buf* b : bufs) release(L, *b);
  for (cudaEvent_t e : L->prof_ev) cudaEventDestroy(e);
  if (L->h_status) cudaFreeHost(L->h_status);
  if (L->Wg) cudaFree(L->Wg);
  if (L->W13) cudaFree(L->W13);
  if (L->W2) cudaFree(L->W2);
  delete L;
}

int moe_set_stream(moe_layer_t* L, void* cuda_stream) {
  if (!L) return fail(MOE_ERR_INVALID_ARG, "layer is NULL");
  L->stream = (cudaStream_t)cuda_stream;
  return MOE_OK;
}

int moe_reserve(moe_layer_t* L, int T_max) {
  if (!L) return fail(MOE_ERR_INVALID_ARG, "layer is NULL");
  if (T_max < 1 || T_max > kMaxTokens) return fail(MOE_ERR_INVALID_ARG, "T_max = %d outside 1..%d", T_max, kMaxTokens);
  int rc;
  if ((rc = ensure_route(L, T_max))) return rc;
  // the small-batch sequences want split-K planes, the large-batch ones more rows: take both
  if ((rc = ensure_gemm(L, T_max < kDecodeMaxT ? T_max : kDecodeMaxT))) return rc;
  if ((rc = ensure_gemm(L, 1))) return rc;  // one or two tokens use finer split-K items
  if ((rc = ensure_gemm(L, T_max))) return rc;
  return MOE_OK;
}

void moe_test_set_free_bytes_limit(long long bytes) { g_free_bytes_limit = bytes; }

int moe_test_wait_expiry(moe_layer_t* L, unsigned limit_us, int poison_tail) {
  if (!L) return fail(MOE_ERR_INVALID_ARG, "layer is NULL");
  if (limit_us < 1 || limit_us > 100000) return fail(MOE_ERR_INVALID_ARG, "limit_us = %u outside 1..100000", limit_us);
  int rc;
  if ((rc = ensure_route(L, 1))) return rc;
  if (poison_tail) {
    if ((rc = ensure_gemm(L, 1))) return rc;
    CUDA_TRY(cudaMemsetAsync(L->ws->tail.p, 0x01, 64, L->stream));
  }
  CUDA_TRY(launch_wait_expiry((int*)L->ws->status.p, (unsigned long long)limit_us * 1000ull, L->stream));
  return MOE_OK;
}

size_t moe_layer_weight_bytes(const moe_layer_t* L) { return L ? L->weight_bytes : 0; }
size_t moe_layer_scratch_bytes(const moe_layer_t* L) { return L ? L->own.scratch_bytes : 0; }

int moe_forward(moe_layer_t* L, const void* x, int T, float beta, void* y, void* routing_stats) {
  return forward_impl(L, x, T, beta, nullptr, y, routing_stats);
}

int moe_forward_residual(moe_layer_t* L, const void* x, int T, float beta, const void* residual,
                         void* y, void* routing_stats) {
  return forward_impl(L, x, T, beta, residual, y, routing_stats);
}

int moe_top2_distance(moe_layer_t* L, const void* x, int T, float* dist) {
  if (!dist) return fail(MOE_ERR_INVALID_ARG, "dist is NULL");
  return forward_impl(L, x, T, 0.f, nullptr, nullptr, nullptr, dist);
}

int moe_forward_topk(moe_layer_t* L, const void* x, int T, int k, float beta, void* y,
                     int32_t* idx_out, float* wn_out, int32_t* n_active_out) {
  if (!L) return fail(MOE_ERR_INVALID_ARG, "layer is NULL");
  if (T < 0 || T > kMaxTokens) return fail(MOE_ERR_INVALID_ARG, "T = %d outside 0..%d", T, kMaxTokens);
  if (k < 1 || k > L->r || k > 8) return fail(MOE_ERR_INVALID_ARG, "k = %d outside 1..min(kept experts, 8)", k);
  if (T == 0) return MOE_OK;
  if (!x || !y || x == y) return fail(MOE_ERR_INVALID_ARG, "x and y must be distinct and non-NULL");
  if (!aligned16(x) || !aligned16(y)) return fail(MOE_ERR_INVALID_ARG, "x and y must be 16-byte aligned");
  if (!(beta >= 0.f)) return fail(MOE_ERR_INVALID_ARG, "beta must be >= 0");
  int rc;
  if ((rc = ensure_route(L, T))) return rc;
  if ((rc = ensure_gemm(L, T, k))) return rc;
  Workspace& W = *L->ws;
  if ((rc = grow(L, W.k_idx, (size_t)T * k * 4))) return rc;
  if ((rc = grow(L, W.k_wn, (size_t)T * k * 4))) return rc;
  if ((rc = grow(L, W.k_pos, (size_t)T * k * 4))) return rc;
  if ((rc = grow(L, W.k_nact, (size_t)T * 4))) return rc;
  cudaStream_t st = L->stream;
  const bool dec = decode_mode(T);
  const int nblk = (T + kRouteTokPerBlock - 1) / kRouteTokPerBlock;
  const int rows_cap = rows_for(L, T, k);
  Meta* meta = (Meta*)W.meta.p;
  int32_t* idx = (int32_t*)W.k_idx.p;
  int32_t* nact = (int32_t*)W.k_nact.p;
  CUDA_TRY(launch_router_topk((const bf16*)x, L->Wg, T, L->h, L->r, k, beta, L->kept, idx,
                              (float*)W.k_wn.p, nact, idx_out, wn_out, n_active_out, nullptr, st));
  CUDA_TRY(launch_count_topk(idx, nact, T, k, (int32_t*)W.blk_hist.p, st));
  CUDA_TRY(launch_scan((int32_t*)W.blk_hist.p, nblk, L->r, dec ? 16 : kTileRows, (int32_t*)W.blk_base.p,
                       meta, nullptr, nullptr, nullptr, L->kept, L->E, st));
  CUDA_TRY(cudaMemsetAsync(W.row_token.p, 0xff, (size_t)rows_cap * 4, st));
  CUDA_TRY(launch_scatter_topk(idx, nact, (int32_t*)W.blk_base.p, meta, T, k, (int32_t*)W.k_pos.p,
                               (int32_t*)W.row_token.p, st));
  CUDA_TRY(launch_gather((const bf16*)x, (int32_t*)W.row_token.p, meta, L->h, rows_cap,
                         (bf16*)W.xperm.p, st));
  GemmArgs gu, dn;
  memset(&gu, 0, sizeof(gu));
  memset(&dn, 0, sizeof(dn));
  gu.a_off_mul = 1; gu.out_off_mul = 1; gu.out_ld = L->f; gu.out = W.act.p;
  dn.a_off_mul = 1; dn.out_off_mul = 1; dn.out_ld = L->h; dn.out = W.O.p;
  const bool wm = dec && !L->debug_simt;
  if (wm) {
    gu.tail = (float*)W.tail.p; dn.tail = (float*)W.tail.p;
  }
  const int ksplit = wm ? ksplit_for(L, T) : 1;
  const size_t split_stride = (size_t)rows_cap * L->h;
  dn.split_stride = (long long)split_stride;
  GemmMaps m_gu, m_dn;
  m_gu.w = (wm && decode_weights_m(L, T)) ? L->w13_128 : L->w13_256;
  m_dn.w = (wm && decode_weights_m(L, T)) ? L->w2_128 : L->w2_256;
  memcpy(m_gu.t, W.tok_x, sizeof(m_gu.t));
  memcpy(m_dn.t, W.tok_act, sizeof(m_dn.t));
  const bool prof_saved = L->prof;
  L->prof = false;
  rc = run_expert_gemms(L, meta, wm, m_gu, m_dn, gu, dn, kOutF32, (const bf16*)W.xperm.p,
                        (const bf16*)W.act.p, rows_cap, T);
  L->prof = prof_saved;
  if (rc) return rc;
  CUDA_TRY(launch_combine_topk((const float*)W.O.p, ksplit, split_stride, (int32_t*)W.k_pos.p,
                               (float*)W.k_wn.p, k, T, L->h, (bf16*)y, st));
  return MOE_OK;
}

int moe_forward_host(moe_layer_t* L, const void* x_host, int T, float beta, void* y_host) {
  if (!L) return fail(MOE_ERR_INVALID_ARG, "layer is NULL");
  if (T < 0 || T > kMaxTokens) return fail(MOE_ERR_INVALID_ARG, "T = %d outside 0..%d", T, kMaxTokens);
  if (T == 0) return MOE_OK;
  if (!x_host || !y_host) return fail(MOE_ERR_INVALID_ARG, "x_host or y_host is NULL");
  const size_t bytes = (size_t)T * L->h * 2;
  int rc;
  if ((rc = grow(L, L->ws->hx, bytes))) return rc;
  if ((rc = grow(L, L->ws->hy, bytes))) return rc;
  CUDA_TRY(cudaMemcpyAsync(L->ws->hx.p, x_host, bytes, cudaMemcpyHostToDevice, L->stream));
  if ((rc = forward_impl(L, L->ws->hx.p, T, beta, nullptr, L->ws->hy.p, nullptr))) return rc;
  CUDA_TRY(cudaMemcpyAsync(y_host, L->ws->hy.p, bytes, cudaMemcpyDeviceToHost, L->stream));
  return check_status(L);
}

int moe_calibrate_beta(moe_layer_t* L, const void* x, int T, float* beta_out) {
  if (!L) return fail(MOE_ERR_INVALID_ARG, "layer is NULL");
  if (!x || !beta_out) return fail(MOE_ERR_INVALID_ARG, "x or beta_out is NULL");
  if (T < 1 || T > kMaxTokens)
    return fail(MOE_ERR_INVALID_ARG, "T = %d outside 1..%d calibration tokens", T, kMaxTokens);
  if (!aligned16(x)) return fail(MOE_ERR_INVALID_ARG, "x must be 16-byte aligned");
  int rc;
  if ((rc = ensure_route(L, T))) return rc;
  RouteOut ro;
  memset(&ro, 0, sizeof(ro));
  ro.idx = (int32_t*)L->ws->idx.p; ro.wn = (float*)L->ws->wn.p; ro.ratio = (float*)L->ws->ratio.p;
  ro.skipped = (uint8_t*)L->ws->skipped.p;
  CUDA_TRY(launch_router((const bf16*)x, L->Wg, T, L->h, L->r, 0.f, L->kept, ro, L->stream));
  CUDA_TRY(launch_select2(ro.ratio, T, (T - 1) / 2, T / 2, (float*)L->ws->sel.p, L->stream));
  float v[2];
  CUDA_TRY(cudaMemcpyAsync(v, L->ws->sel.p, 8, cudaMemcpyDeviceToHost, L->stream));
  CUDA_TRY(cudaStreamSynchronize(L->stream));
  *beta_out = (T & 1) ? v[0] : (float)(((double)v[0] + (double)v[1]) * 0.5);
  return MOE_OK;
}

int moe_coselection(moe_layer_t* L, const void* x, int T, int32_t* counts) {
  if (!L) return fail(MOE_ERR_INVALID_ARG, "layer is NULL");
  if (!x || !counts) return fail(MOE_ERR_INVALID_ARG, "x or counts is NULL");
  if (T < 0 || T > kMaxTokens) return fail(MOE_ERR_INVALID_ARG, "T = %d outside 0..%d", T, kMaxTokens);
  if (!aligned16(x)) return fail(MOE_ERR_INVALID_ARG, "x must be 16-byte aligned");
  const int E = L->E;
  memset(counts, 0, sizeof(int32_t) * E * E);
  if (T == 0) return MOE_OK;
  int rc;
  if ((rc = ensure_route(L, T))) return rc;
  if ((rc = grow(L, L->ws->cosel, (size_t)E * E * 4))) return rc;
  RouteOut ro;
  memset(&ro, 0, sizeof(ro));
  ro.idx = (int32_t*)L->ws->idx.p; ro.wn = (float*)L->ws->wn.p; ro.ratio = (float*)L->ws->ratio.p;
  ro.skipped = (uint8_t*)L->ws->skipped.p;
  CUDA_TRY(cudaMemsetAsync(L->ws->cosel.p, 0, (size_t)E * E * 4, L->stream));
  CUDA_TRY(launch_router((const bf16*)x, L->Wg, T, L->h, L->r, 0.f, L->kept, ro, L->stream));
  CUDA_TRY(launch_coselection(ro.idx, T, E, L->kept, (int32_t*)L->ws->cosel.p, L->stream));
  CUDA_TRY(cudaMemcpyAsync(counts, L->ws->cosel.p, (size_t)E * E * 4, cudaMemcpyDeviceToHost, L->stream));
  CUDA_TRY(cudaStreamSynchronize(L->stream));
  return MOE_OK;
}

uint32_t moe_frequency_subset(const int32_t* counts, int E, int r) {
  if (!counts || E < 2 || E > kMaxE || r < 1 || r > E) return 0;
  // activation frequency of an expert = tokens that have it in either slot of their top-2
  struct Entry { long long tokens; int expert; };
  std::vector<Entry> by_use(E);
  for (int e = 0; e < E; ++e) {
    long long row = 0, col = 0;
    for (int o = 0; o < E; ++o) { row += counts[e * E + o]; col += counts[o * E + e]; }
    by_use[e] = {row + col, e};
  }
  // most used first; equal use keeps the lower expert index first
  std::stable_sort(by_use.begin(), by_use.end(),
                   [](const Entry& a, const Entry& b) { return a.tokens > b.tokens; });
  uint32_t mask = 0;
  for (int i = 0; i < r; ++i) mask |= 1u << by_use[i].expert;
  return mask;
}

// Subsets of r of E experts in lexicographic order of their ascending index tuples.  With the
// bits of a mask read in reverse (expert 0 as the most significant bit) that order is numerically
// descending, so the masks are produced as E-bit words with r bits set in ascending numeric order
// (next word with the same number of bits: ripple the lowest run of ones), then reversed in
// order and in bit position.
static std::vector<uint32_t> subset_masks(int E, int r) {
  std::vector<uint32_t> words;
  words.reserve(binom(E, r));
  const uint32_t limit = E >= 32 ? 0xffffffffu : ((1u << E) - 1u);
  uint32_t w = (1u << r) - 1u;
  for (;;) {
    words.push_back(w);
    const uint32_t lowest = w & (0u - w);
    const uint32_t ripple = w + lowest;
    if (ripple > limit || ripple == 0) break;
    w = ripple | (((w ^ ripple) >> 2) / lowest);
    if (w > limit) break;
  }
  std::vector<uint32_t> masks(words.size());
  for (size_t i = 0; i < words.size(); ++i) {
    const uint32_t rev_word = words[words.size() - 1 - i];
    uint32_t m = 0;
    for (int b = 0; b < E; ++b)
      if ((rev_word >> b) & 1u) m |= 1u << (E - 1 - b);
    masks[i] = m;
  }
  return masks;
}

// The search for n_r subset sizes rs[] over one evaluation of the experts: losses holds the
// C(E, rs[0]) + C(E, rs[1]) + ... values one after the other, best_subset one mask per size.
static int search_impl(moe_layer_t* L, const void* x_calib, const float* F_ref, int T, const int* rs,
                       int n_r, float* losses, uint32_t* best_subset) {
  if (!L) return fail(MOE_ERR_INVALID_ARG, "layer is NULL");
  if (!x_calib || !losses || !best_subset)
    return fail(MOE_ERR_INVALID_ARG, "x_calib, losses or best_subset is NULL");
  if (!aligned16(x_calib)) return fail(MOE_ERR_INVALID_ARG, "x_calib must be 16-byte aligned");
  if (T < 1 || T > kMaxTokens)
    return fail(MOE_ERR_INVALID_ARG, "T = %d outside 1..%d calibration tokens", T, kMaxTokens);
  if (L->r != L->E)
    return fail(MOE_ERR_INVALID_ARG, "the search needs a layer created with all %d experts kept", L->E);
  if (!rs || n_r < 1 || n_r > kMaxE) return fail(MOE_ERR_INVALID_ARG, "no subset sizes given (or more than %d)", kMaxE);
  int r = L->E;  // the smallest size: it needs the most experts evaluated per token
  long nC = 0;   // subsets of all sizes together
  for (int i = 0; i < n_r; ++i) {
    if (rs[i] < 2 || rs[i] > L->E) return fail(MOE_ERR_INVALID_ARG, "r = %d outside 2..%d", rs[i], L->E);
    if (rs[i] < r) r = rs[i];
    nC += binom(L->E, rs[i]);
  }
  const int E = L->E, h = L->h, f = L->f;
  cudaStream_t st = L->stream;
  int rc;
  if ((rc = ensure_route(L, T))) return rc;

  const int Tc = T < 8192 ? T : 8192;  // tokens per chunk of expert evaluations
  const int Tc_pad = (int)align_up((size_t)Tc, kTileRows);
  const int nchunks = (T + Tc - 1) / Tc;
  // per-block partial losses of an enumeration pass (a pass takes at most kMaxSubsetsPerPass
  // subsets, or one whole size if that alone is more)
  size_t partial_floats = 0;
  {
    long pass = 0;
    for (int i = 0; i <= n_r; ++i) {
      const long n = i < n_r ? binom(E, rs[i]) : 0;
      if (i == n_r || (pass > 0 && pass + n > kMaxSubsetsPerPass)) {
        const size_t need = (size_t)enumerate_num_blocks(T, (int)pass) * (size_t)pass;
        if (need > partial_floats) partial_floats = need;
        pass = 0;
      }
      pass += n;
    }
  }
  // A subset of r experts always contains two of a token's K = E - r + 2 top-ranked experts,
  // so only those K need to be evaluated per token (all of them when K = E).
  const int K = E - r + 2;
  const bool pruned_work = K < E && !L->search_dense;
  Workspace& W = *L->ws;
  if ((rc = grow(L, W.s_logits, (size_t)T * E * 4))) return rc;
  if ((rc = grow(L, W.s_subsets, (size_t)nC * 4))) return rc;
  if ((rc = grow(L, W.s_partial, partial_floats * 4))) return rc;
  if ((rc = grow(L, W.s_loss_sq, (size_t)nC * 8))) return rc;
  if ((rc = grow(L, W.s_losses, (size_t)nC * 4))) return rc;
  if ((rc = grow(L, W.s_meta, sizeof(Meta)))) return rc;
  Meta* meta = (Meta*)W.s_meta.p;
  // While profiling, every chunk records one set of stage marks (permutation, gate/up, down, an
  // empty fourth stage) and the enumerations one more (three empty stages, then stage 3).
  const bool prof_saved = L->prof;
  if (L->prof && (L->prof_used % (MOE_PROFILE_STAGES + 1)) != 0) L->prof_used = 0;
  EnumSource src = {nullptr, nullptr, 0, 0, 0};
  GemmMaps m_gu, m_dn;
  m_gu.w = L->w13_256;
  m_dn.w = L->w2_256;

  if (pruned_work) {
    const int rows_chunk = (int)align_up((size_t)K * Tc + (size_t)E * kTileRows, kTileRows);
    if ((rc = grow(L, W.s_yall, (size_t)nchunks * rows_chunk * h * 2))) return rc;
    if ((rc = grow(L, W.s_act, ((size_t)rows_chunk + kTileRows) * f * 2))) return rc;
    if ((rc = grow(L, W.s_xperm, ((size_t)rows_chunk + kTileRows) * h * 2))) return rc;
    if ((rc = grow(L, W.s_rowtok, (size_t)rows_chunk * 4))) return rc;
    if ((rc = grow(L, W.k_idx, (size_t)T * K * 4))) return rc;
    if ((rc = grow(L, W.k_wn, (size_t)T * K * 4))) return rc;
    if ((rc = grow(L, W.k_pos, (size_t)T * K * 4))) return rc;
    if ((rc = grow(L, W.k_nact, (size_t)T * 4))) return rc;
    if ((rc = build_token_maps(m_gu, W.s_xperm.p, h, (uint64_t)rows_chunk + kTileRows))) return rc;
    if ((rc = build_token_maps(m_dn, W.s_act.p, f, (uint64_t)rows_chunk + kTileRows))) return rc;
    for (int c = 0; c < nchunks; ++c) {
      const int t0 = c * Tc;
      const int rows = (T - t0) < Tc ? (T - t0) : Tc;
      const int nblk = (rows + kRouteTokPerBlock - 1) / kRouteTokPerBlock;
      const bf16* xc = (const bf16*)x_calib + (size_t)t0 * h;
      int32_t* idx = (int32_t*)W.k_idx.p + (size_t)t0 * K;
      int32_t* nact = (int32_t*)W.k_nact.p + t0;
      int32_t* pos = (int32_t*)W.k_pos.p + (size_t)t0 * K;
      mark(L);
      // beta = -1: the skipping rule never fires, every token keeps its K top-ranked experts
      cudaError_t e = launch_router_topk(xc, L->Wg, rows, h, E, K, -1.0f, L->kept, idx,
                                         (float*)W.k_wn.p + (size_t)t0 * K, nact, nullptr, nullptr,
                                         nullptr, (float*)W.s_logits.p + (size_t)t0 * E, st);
      if (e == cudaSuccess) e = launch_count_topk(idx, nact, rows, K, (int32_t*)W.blk_hist.p, st);
      if (e == cudaSuccess)
        e = launch_scan((int32_t*)W.blk_hist.p, nblk, E, kTileRows, (int32_t*)W.blk_base.p, meta, nullptr,
                        nullptr, nullptr, L->kept, E, st);
      if (e == cudaSuccess) e = cudaMemsetAsync(W.s_rowtok.p, 0xff, (size_t)rows_chunk * 4, st);
      if (e == cudaSuccess)
        e = launch_scatter_topk(idx, nact, (int32_t*)W.blk_base.p, meta, rows, K, pos,
                                (int32_t*)W.s_rowtok.p, st);
      if (e == cudaSuccess)
        e = launch_gather(xc, (int32_t*)W.s_rowtok.p, meta, h, rows_chunk, (bf16*)W.s_xperm.p, st);
      if (e != cudaSuccess) {
        L->prof = prof_saved;
        return fail(MOE_ERR_CUDA, "search permutation: %s", cudaGetErrorString(e));
      }
      mark(L);
      GemmArgs gu, dn;
      memset(&gu, 0, sizeof(gu));
      memset(&dn, 0, sizeof(dn));
      gu.a_off_mul = 1; gu.out_off_mul = 1; gu.out_ld = f; gu.out = W.s_act.p;
      dn.a_off_mul = 1; dn.out_off_mul = 1; dn.out_row_base = c * rows_chunk; dn.out_ld = h;
      dn.out = W.s_yall.p;
      if ((rc = run_expert_gemms(L, meta, false, m_gu, m_dn, gu, dn, kOutBf16, (const bf16*)W.s_xperm.p,
                                 (const bf16*)W.s_act.p, rows_chunk))) {
        L->prof = prof_saved;
        return rc;
      }
      mark(L);
      mark(L);
    }
    src.topk_idx = (const int32_t*)W.k_idx.p;
    src.pair_pos = (const int32_t*)W.k_pos.p;
    src.chunk_tokens = Tc;
    src.chunk_rows = rows_chunk;
    src.k_stride = K;
  } else {
    if ((rc = grow(L, W.s_yall, (size_t)T * E * h * 2))) return rc;
    if ((rc = grow(L, W.s_act, ((size_t)E * Tc_pad + kTileRows) * f * 2))) return rc;
    // token-side operand of the gate/up GEMM: x itself (padded copy when shorter than one box)
    const bf16* xa = (const bf16*)x_calib;
    uint64_t xa_rows = (uint64_t)T;
    if (T < kTileRows) {
      if ((rc = grow(L, W.s_xpad, (size_t)kTileRows * h * 2))) return rc;
      CUDA_TRY(cudaMemsetAsync(W.s_xpad.p, 0, (size_t)kTileRows * h * 2, st));
      CUDA_TRY(cudaMemcpyAsync(W.s_xpad.p, x_calib, (size_t)T * h * 2, cudaMemcpyDeviceToDevice, st));
      xa = (const bf16*)W.s_xpad.p;
      xa_rows = kTileRows;
    }
    if ((rc = build_token_maps(m_gu, xa, h, xa_rows))) return rc;
    if ((rc = build_token_maps(m_dn, W.s_act.p, f, (uint64_t)E * Tc_pad + kTileRows))) return rc;
    // all logits (Sec. 3.2: the unpruned layer's routing), then every expert on every token
    RouteOut ro;
    memset(&ro, 0, sizeof(ro));
    ro.idx = (int32_t*)W.idx.p; ro.wn = (float*)W.wn.p; ro.ratio = (float*)W.ratio.p;
    ro.skipped = (uint8_t*)W.skipped.p; ro.logits = (float*)W.s_logits.p;
    mark(L);
    CUDA_TRY(launch_router((const bf16*)x_calib, L->Wg, T, h, E, 0.f, L->kept, ro, st));
    for (int t0 = 0; t0 < T; t0 += Tc) {
      const int rows = (T - t0) < Tc ? (T - t0) : Tc;
      if (t0 > 0) mark(L);
      CUDA_TRY(launch_set_dense_meta(meta, E, rows, Tc_pad, st));
      mark(L);
      GemmArgs gu, dn;
      memset(&gu, 0, sizeof(gu));
      memset(&dn, 0, sizeof(dn));
      gu.a_row_base = t0; gu.a_off_mul = 0; gu.out_off_mul = 1; gu.out_ld = f; gu.out = W.s_act.p;
      dn.a_off_mul = 1; dn.out_row_base = t0; dn.out_off_mul = 0; dn.out_col_mul = h;
      dn.out_ld = (long long)E * h; dn.out = W.s_yall.p;
      if ((rc = run_expert_gemms(L, meta, false, m_gu, m_dn, gu, dn, kOutBf16, xa,
                                 (const bf16*)W.s_act.p, rows))) {
        L->prof = prof_saved;
        return rc;
      }
      mark(L);
      mark(L);
    }
  }
  L->prof = prof_saved;
  for (int i = 0; i < MOE_PROFILE_STAGES; ++i) mark(L);
  // One enumeration for all subset sizes over the same expert outputs.  Which pair of experts a
  // subset routes a token to depends on the subset alone (its two highest-ranked kept experts,
  // which lie within the token's E - r + 2 <= K top-ranked ones), so the subsets of every size go
  // through one pass that reads each token's K expert outputs once; every loss is computed by
  // the same operations in the same order as in a pass of its own size.
  std::vector<std::vector<uint32_t>> masks(n_r);
  for (int i = 0; i < n_r; ++i) masks[i] = subset_masks(E, rs[i]);
  size_t o = 0;
  for (int i0 = 0; i0 < n_r;) {
    // sizes i0 .. i1 - 1 go through one pass (as many as the per-warp loss table has room for)
    std::vector<uint32_t> batch = masks[i0];
    int i1 = i0 + 1;
    while (i1 < n_r && batch.size() + masks[i1].size() <= (size_t)kMaxSubsetsPerPass) {
      batch.insert(batch.end(), masks[i1].begin(), masks[i1].end());
      ++i1;
    }
    const size_t n = batch.size();
    CUDA_TRY(cudaMemcpyAsync(W.s_subsets.p, batch.data(), n * 4, cudaMemcpyHostToDevice, st));
    CUDA_TRY(launch_enumerate((const float*)W.s_logits.p, (const bf16*)W.s_yall.p, T, E, r, h,
                              (const uint32_t*)W.s_subsets.p, (int)n, (float*)W.s_partial.p,
                              (double*)W.s_loss_sq.p, (float*)W.s_losses.p, F_ref, src, st));
    CUDA_TRY(cudaMemcpyAsync(losses + o, L->ws->s_losses.p, n * 4, cudaMemcpyDeviceToHost, st));
    // the host list is reused for the next pass: the copy above must have left it
    if (i1 < n_r) CUDA_TRY(cudaStreamSynchronize(st));
    o += n;
    i0 = i1;
  }
  mark(L);
  if ((rc = check_status(L))) return rc;
  o = 0;
  for (int i = 0; i < n_r; ++i) {
    const size_t n = masks[i].size();
    size_t best = 0;
    for (size_t c = 1; c < n; ++c)
      if (losses[o + c] < losses[o + best]) best = c;
    best_subset[i] = masks[i][best];
    o += n;
  }
  return MOE_OK;
}

int moe_prune_search(moe_layer_t* L, const void* x_calib, int T, int r, float* losses,
                     uint32_t* best_subset) {
  return search_impl(L, x_calib, nullptr, T, &r, 1, losses, best_subset);
}

int moe_prune_search_multi(moe_layer_t* L, const void* x_calib, int T, const int* r_list, int n_r,
                           float* losses, uint32_t* best_subsets) {
  return search_impl(L, x_calib, nullptr, T, r_list, n_r, losses, best_subsets);
}

int moe_prune_search_progressive(moe_layer_t* L, const void* x_pruned, const float* F_ref, int T,
                                 int r, float* losses, uint32_t* best_subset) {
  if (!F_ref) return fail(MOE_ERR_INVALID_ARG, "F_ref is NULL");
  if (!aligned16(F_ref)) return fail(MOE_ERR_INVALID_ARG, "F_ref must be 16-byte aligned");
  return search_impl(L, x_pruned, F_ref, T, &r, 1, losses, best_subset);
}

int moe_rmsnorm(const void* x, int T, int h, float eps, void* out, void* cuda_stream) {
  if (T < 0 || h < 8 || h % 8) return fail(MOE_ERR_INVALID_ARG, "bad T = %d or h = %d", T, h);
  if (T == 0) return MOE_OK;
  if (!x || !out || !aligned16(x) || !aligned16(out))
    return fail(MOE_ERR_INVALID_ARG, "x and out must be non-NULL and 16-byte aligned");
  CUDA_TRY(launch_rmsnorm((const bf16*)x, T, h, eps, (bf16*)out, (cudaStream_t)cuda_stream));
  return MOE_OK;
}

int moe_stack_forward(moe_layer_t* const* layers, int n_layers, const void* x, int T,
                      const float* betas, float eps, void* y) {
  if (!layers || n_layers < 1) return fail(MOE_ERR_INVALID_ARG, "no layers");
  if (T < 0 || T > kMaxTokens) return fail(MOE_ERR_INVALID_ARG, "T = %d outside 0..%d", T, kMaxTokens);
  if (T == 0) return MOE_OK;
  if (!x || !y || x == y) return fail(MOE_ERR_INVALID_ARG, "x and y must be distinct and non-NULL");
  moe_layer* L0 = layers[0];
  if (!L0) return fail(MOE_ERR_INVALID_ARG, "layer 0 is NULL");
  for (int l = 0; l < n_layers; ++l)
    if (!layers[l] || layers[l]->h != L0->h)
      return fail(MOE_ERR_INVALID_ARG, "layer %d is NULL or has a different h", l);
  int rc;
  if ((rc = grow(L0, L0->ws->xn, (size_t)T * L0->h * 2))) return rc;
  const void* cur = x;
  for (int l = 0; l < n_layers; ++l) {
    moe_layer* L = layers[l];
    cudaStream_t saved = L->stream;
    Workspace* saved_ws = L->ws;
    L->stream = L0->stream;
    if (L->f == L0->f) L->ws = L0->ws;
    rc = MOE_OK;
    cudaError_t e = launch_rmsnorm((const bf16*)cur, T, L->h, eps, (bf16*)L0->ws->xn.p, L0->stream);
    if (e != cudaSuccess) rc = fail(MOE_ERR_CUDA, "rmsnorm: %s", cudaGetErrorString(e));
    if (!rc) rc = forward_impl(L, L0->ws->xn.p, T, betas ? betas[l] : 0.f, cur, y, nullptr);
    L->stream = saved;
    L->ws = saved_ws;
    if (rc) return rc;
    cur = y;
  }
  return MOE_OK;
}

int moe_layer_share_scratch(moe_layer_t* L, moe_layer_t* owner) {
  if (!L) return fail(MOE_ERR_INVALID_ARG, "layer is NULL");
  if (!owner || owner == L) {
    L->ws = &L->own;
    return MOE_OK;
  }
  if (owner->h != L->h || owner->f != L->f)
    return fail(MOE_ERR_INVALID_ARG, "scratch can only be shared between layers of the same h and f");
  if (owner->ws != &owner->own)
    return fail(MOE_ERR_INVALID_ARG, "the owner itself borrows its scratch");
  L->ws = &owner->own;
  return MOE_OK;
}

int moe_profile_enable(moe_layer_t* L, int on) {
  if (!L) return fail(MOE_ERR_INVALID_ARG, "layer is NULL");
  L->prof = on != 0;
  L->prof_used = 0;
  return MOE_OK;
}

int moe_profile_read(moe_layer_t* L, float* stage_ms, int* calls) {
  if (!L || !stage_ms || !calls) return fail(MOE_ERR_INVALID_ARG, "NULL argument");
  CUDA_TRY(cudaStreamSynchronize(L->stream));
  const size_t per = MOE_PROFILE_STAGES + 1;
  const size_t n = L->prof_used / per;
  for (int s = 0; s < MOE_PROFILE_STAGES; ++s) stage_ms[s] = 0.f;
  for (size_t c = 0; c < n; ++c)
    for (int s = 0; s < MOE_PROFILE_STAGES; ++s) {
      float ms = 0.f;
      CUDA_TRY(cudaEventElapsedTime(&ms, L->prof_ev[c * per + s], L->prof_ev[c * per + s + 1]));
      stage_ms[s] += ms;
    }
  *calls = (int)n;
  L->prof_used = 0;
  return MOE_OK;
}

int moe_device_status(moe_layer_t* L) {
  if (!L) return fail(MOE_ERR_INVALID_ARG, "layer is NULL");
  if (!L->ws->status.p) {
    CUDA_TRY(cudaStreamSynchronize(L->stream));
    return MOE_OK;
  }
  return check_status(L);
}

}  // extern "C"
