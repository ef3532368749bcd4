// Device helpers shared by the routing kernels and the single-token kernels.
#pragma once
#include "common.h"

namespace moe {

__device__ __forceinline__ float bf16_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }

__device__ __forceinline__ void unpack8(const uint4& v, float* f) {
  f[0] = bf16_lo(v.x); f[1] = bf16_hi(v.x);
  f[2] = bf16_lo(v.y); f[3] = bf16_hi(v.y);
  f[4] = bf16_lo(v.z); f[5] = bf16_hi(v.z);
  f[6] = bf16_lo(v.w); f[7] = bf16_hi(v.w);
}

__device__ __forceinline__ uint32_t pack2(float a, float b) {
  __nv_bfloat162 p = __floats2bfloat162_rn(a, b);
  return *reinterpret_cast<uint32_t*>(&p);
}

// Routing decision of one token from its r logits (Sec. 3.1, Eq. 1; skip test of Sec. 3.3;
// weight 1 for the first expert after a skip, App. A.2).  p1 = w_e1 / w_e0.
template <int R>
__device__ __forceinline__ void route_choose(const float (&acc)[R], int r, float beta, int& e0,
                                             int& e1, bool& skip, float& w0, float& w1, float& p1) {
  // top-2 on the logits (softmax is increasing) in one sweep over the kept experts in index
  // order: a logit displaces the leader or the runner-up only when strictly larger, so of equal
  // logits the lower index ranks first
  float l0 = acc[0], l1 = 0.f;
  e0 = 0;
  e1 = -1;
#pragma unroll
  for (int c = 1; c < R; ++c) {
    if (c < r) {
      const float v = acc[c];
      if (v > l0) { l1 = l0; e1 = e0; l0 = v; e0 = c; }
      else if (e1 < 0 || v > l1) { l1 = v; e1 = c; }
    }
  }
  // softmax numerators relative to the maximum: p_e0 = 1, p_e1 = exp(l1 - l0); the
  // denominator cancels in the ratio, the skip test and the normalised weights
  p1 = expf(l1 - l0);
  skip = p1 < beta * 1.0f;
  if (skip) { w0 = 1.f; w1 = 0.f; }
  else { const float d = 1.0f + p1; w0 = 1.0f / d; w1 = p1 / d; }
}

// The same decision by one thread, which also writes the per-token record.
template <int R>
__device__ __forceinline__ void route_decide(const float (&acc)[R], int r, float beta, int t,
                                             const KeptIds& kept, const RouteOut& o, int& e0,
                                             int& e1, bool& skip) {
  float w0, w1, p1;
  route_choose<R>(acc, r, beta, e0, e1, skip, w0, w1, p1);
  o.idx[2 * t] = e0; o.idx[2 * t + 1] = e1;
  o.wn[2 * t] = w0; o.wn[2 * t + 1] = w1;
  o.ratio[t] = p1;
  o.skipped[t] = skip ? 1 : 0;
  if (o.s_idx) {
    o.s_idx[2 * t] = kept.id[e0]; o.s_idx[2 * t + 1] = kept.id[e1];
    o.s_wn[2 * t] = w0; o.s_wn[2 * t + 1] = w1;
    o.s_ratio[t] = p1;
    o.s_skipped[t] = skip ? 1 : 0;
  }
  if (o.logits) {
#pragma unroll
    for (int c = 0; c < R; ++c)
      if (c < r) o.logits[(size_t)t * r + c] = acc[c];
  }
}

// Batch description of a single token (one thread): one permuted row for e0, one for e1 unless
// it was skipped (e1 < 0); p0 / p1 return those rows (p1 = -1 after a skip).
__device__ __forceinline__ void publish_single(int e0, int e1, int pad, const KeptIds& kept, Meta* meta,
                                               int32_t* pair_pos, int32_t* row_token, int32_t* s_count,
                                               int32_t* s_nskipped, int32_t* s_ntouched, int E, int& p0,
                                               int& p1) {
  const bool skip = e1 < 0;
  int off = 0, tiles = 0;
  p0 = 0;
  p1 = -1;
  meta->off[0] = 0;
  meta->tile_prefix[0] = 0;
  for (int c = 0; c < kMaxE; ++c) {
    const int n0 = (c == e0), n1 = (c == e1);
    const int n = n0 + n1;
    if (c == e0) p0 = off;
    if (c == e1) p1 = off;
    off += (n + pad - 1) / pad * pad;
    tiles += (n + kTileRows - 1) / kTileRows;
    meta->count[c] = n;
    meta->count_slot[c][0] = n0;
    meta->count_slot[c][1] = n1;
    meta->off[c + 1] = off;
    meta->tile_prefix[c + 1] = tiles;
  }
  meta->rows_total = off;
  meta->n_skipped = skip ? 1 : 0;
  meta->n_touched = skip ? 1 : 2;
  meta->reserved = 0;
  pair_pos[0] = p0;
  pair_pos[1] = p1;
  row_token[p0] = 0;
  if (!skip) row_token[p1] = 0;
  if (s_count) {
    for (int e = 0; e < E; ++e) { s_count[2 * e] = 0; s_count[2 * e + 1] = 0; }
    s_count[2 * kept.id[e0]] = 1;
    if (!skip) s_count[2 * kept.id[e1] + 1] = 1;
    *s_nskipped = skip ? 1 : 0;
    *s_ntouched = skip ? 1 : 2;
  }
}

}  // namespace moe
