// Router, token permutation, combine and the small element-wise kernels.
//
//   router_kernel   Sec. 3.1 (logits, softmax, top-2, Eq. 1), Sec. 3.2 (kept experts only),
//                   Sec. 3.3 (skip test), App. A.2 (weight 1 after a skip); warp per token.
//   scan / scatter  stable counting sort of the token-expert pairs that run, by expert;
//                   no atomics, the order is a function of the routing alone.
//   gather          copies the routed rows of x into expert-contiguous order.
//   combine         Eq. 2: y = bf16(residual + w~_e0 o_e0 + w~_e1 o_e1), slot 0 first.
//
// Every kernel here that is launched as a programmatic dependent reads what earlier kernels of
// the stream wrote with ld_l2 (the rule beside launch_pdl): token rows, routing records,
// histograms, the batch description, expert outputs, the residual.  The router rows never
// change and keep ld.global.nc.
#include "common.h"
#include "route_device.cuh"

namespace moe {

namespace {

// Small batches: one block per token, all loads of a thread independent of each other, so the
// kernel costs a couple of memory round trips instead of a serial walk over the row.
template <int R>
__global__ void __launch_bounds__(256)
router_small_kernel(const bf16* x, const bf16* __restrict__ Wg, int T, int h, int r,
                    float beta, KeptIds kept, RouteOut o) {
  pdl_launch_dependents();
  pdl_wait();
  __shared__ float s_part[8][R];
  const int t = blockIdx.x;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int nvec = h >> 3;
  float acc[R];
#pragma unroll
  for (int c = 0; c < R; ++c) acc[c] = 0.f;
  const uint4* xr = reinterpret_cast<const uint4*>(x + (size_t)t * h);
  for (int v = threadIdx.x; v < nvec; v += 256) {
    float xf[8];
    unpack8(ld_l2(xr + v), xf);
#pragma unroll
    for (int c = 0; c < R; ++c) {
      if (c < r) {
        float wf[8];
        unpack8(__ldg(reinterpret_cast<const uint4*>(Wg + (size_t)c * h) + v), wf);
#pragma unroll
        for (int k = 0; k < 8; ++k) acc[c] = fmaf(xf[k], wf[k], acc[c]);
      }
    }
  }
#pragma unroll
  for (int c = 0; c < R; ++c) {
#pragma unroll
    for (int s = 16; s > 0; s >>= 1) acc[c] += __shfl_xor_sync(0xffffffffu, acc[c], s);
    if (lane == 0) s_part[warp][c] = acc[c];
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    float l[R];
#pragma unroll
    for (int c = 0; c < R; ++c) {
      float v = 0.f;
#pragma unroll
      for (int w = 0; w < 8; ++w) v += s_part[w][c];
      l[c] = v;
    }
    int e0, e1;
    bool skip;
    route_decide<R>(l, r, beta, t, kept, o, e0, e1, skip);
  }
}

// A single token (batch-1 decoding): routing, the (trivial) permutation, the batch description
// and the copy of the token's row in one block, in place of the two launches above.  The
// records it writes are those of router_small_kernel + permute_gather_small_kernel for T = 1.
template <int R>
__global__ void __launch_bounds__(256)
route_single_kernel(const bf16* x, const bf16* __restrict__ Wg, int h, int r, float beta,
                    KeptIds kept, RouteOut o, int pad, Meta* meta, int32_t* __restrict__ pair_pos,
                    int32_t* __restrict__ row_token, bf16* __restrict__ xperm, int32_t* s_count,
                    int32_t* s_nskipped, int32_t* s_ntouched, int E) {
  pdl_launch_dependents();
  pdl_wait();
  __shared__ float s_part[8][R];
  __shared__ int s_p[2];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int nvec = h >> 3;
  float acc[R];
#pragma unroll
  for (int c = 0; c < R; ++c) acc[c] = 0.f;
  const uint4* xr = reinterpret_cast<const uint4*>(x);
  for (int v = threadIdx.x; v < nvec; v += 256) {
    float xf[8];
    unpack8(ld_l2(xr + v), xf);
#pragma unroll
    for (int c = 0; c < R; ++c) {
      if (c < r) {
        float wf[8];
        unpack8(__ldg(reinterpret_cast<const uint4*>(Wg + (size_t)c * h) + v), wf);
#pragma unroll
        for (int k = 0; k < 8; ++k) acc[c] = fmaf(xf[k], wf[k], acc[c]);
      }
    }
  }
#pragma unroll
  for (int c = 0; c < R; ++c) {
#pragma unroll
    for (int s = 16; s > 0; s >>= 1) acc[c] += __shfl_xor_sync(0xffffffffu, acc[c], s);
    if (lane == 0) s_part[warp][c] = acc[c];
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    float l[R];
#pragma unroll
    for (int c = 0; c < R; ++c) {
      float v = 0.f;
#pragma unroll
      for (int w = 0; w < 8; ++w) v += s_part[w][c];
      l[c] = v;
    }
    int e0, e1;
    bool skip;
    route_decide<R>(l, r, beta, 0, kept, o, e0, e1, skip);
    if (skip) e1 = -1;
    publish_single(e0, e1, pad, kept, meta, pair_pos, row_token, s_count, s_nskipped, s_ntouched, E,
                   s_p[0], s_p[1]);
  }
  __syncthreads();
  const int p0 = s_p[0], p1 = s_p[1];
  uint4* d0 = reinterpret_cast<uint4*>(xperm + (size_t)p0 * h);
  uint4* d1 = reinterpret_cast<uint4*>(xperm + (size_t)(p1 < 0 ? p0 : p1) * h);
  for (int v = threadIdx.x; v < nvec; v += 256) {
    const uint4 val = ld_l2(xr + v);
    d0[v] = val;
    if (p1 >= 0) d1[v] = val;
  }
}

// Small batches: permutation and gather in one launch, one block per token.  Every block
// recomputes the (tiny) histogram and offsets from the routing record, places its own token's
// pairs and copies the token's row to them; block 0 also publishes the batch description.
// Padding rows of the groups are left as they are: in the weight-major GEMM a token row only
// feeds its own accumulator column, and the columns of padding rows are never stored.
__global__ void __launch_bounds__(kDecodeMaxT)
permute_gather_small_kernel(const bf16* x, const int32_t* idx, const uint8_t* skipped, int T, int h, int r, int pad,
                            Meta* meta, int32_t* __restrict__ pair_pos,
                            int32_t* __restrict__ row_token, bf16* __restrict__ xperm,
                            int32_t* s_count, int32_t* s_nskipped, int32_t* s_ntouched, KeptIds kept,
                            int E) {
  pdl_launch_dependents();
  pdl_wait();
  __shared__ int s_e[kDecodeMaxT][2];
  __shared__ int s_cnt[kMaxE][2];
  __shared__ int s_off[kMaxE + 1];
  __shared__ int s_nsk;
  __shared__ int s_p[2];
  const int i = threadIdx.x;
  const int t = blockIdx.x;
  {
    int e0 = -1, e1 = -1;
    if (i < T) {
      e0 = ld_l2(idx + 2 * i);
      e1 = ld_l2(skipped + i) ? -1 : ld_l2(idx + 2 * i + 1);
    }
    s_e[i][0] = e0;
    s_e[i][1] = e1;
  }
  __syncthreads();
  if (i < 2 * r) {
    const int c = i >> 1, slot = i & 1;
    int n = 0;
    for (int q = 0; q < T; ++q) n += (s_e[q][slot] == c);
    s_cnt[c][slot] = n;
  } else if (i == 2 * kMaxE) {
    int n = 0;
    for (int q = 0; q < T; ++q) n += (s_e[q][1] < 0);
    s_nsk = n;
  }
  __syncthreads();
  if (i == 0) {
    int off = 0, tiles = 0, touched = 0;
    s_off[0] = 0;
    for (int c = 0; c < kMaxE; ++c) {
      const int n = c < r ? s_cnt[c][0] + s_cnt[c][1] : 0;
      off += (n + pad - 1) / pad * pad;
      tiles += (n + kTileRows - 1) / kTileRows;
      touched += (n > 0);
      s_off[c + 1] = off;
      if (t == 0) {
        meta->count[c] = n;
        meta->count_slot[c][0] = c < r ? s_cnt[c][0] : 0;
        meta->count_slot[c][1] = c < r ? s_cnt[c][1] : 0;
        meta->off[c + 1] = off;
        meta->tile_prefix[c + 1] = tiles;
      }
    }
    if (t == 0) {
      meta->off[0] = 0;
      meta->tile_prefix[0] = 0;
      meta->rows_total = off;
      meta->n_skipped = s_nsk;
      meta->n_touched = touched;
      meta->reserved = 0;
      if (s_count) {
        for (int e = 0; e < E; ++e) { s_count[2 * e] = 0; s_count[2 * e + 1] = 0; }
        for (int c = 0; c < r; ++c) {
          s_count[2 * kept.id[c]] = s_cnt[c][0];
          s_count[2 * kept.id[c] + 1] = s_cnt[c][1];
        }
        *s_nskipped = s_nsk;
        *s_ntouched = touched;
      }
    }
  }
  __syncthreads();
  if (i < 2) {
    const int c = s_e[t][i];
    int pos = -1;
    if (c >= 0) {
      int rank = 0;
      for (int q = 0; q < t; ++q) rank += (s_e[q][0] == c) + (s_e[q][1] == c);
      pos = s_off[c] + rank;
      row_token[pos] = t;
    }
    pair_pos[2 * t + i] = pos;
    s_p[i] = pos;
  }
  __syncthreads();
  const int nvec = h >> 3;
  const uint4* src = reinterpret_cast<const uint4*>(x + (size_t)t * h);
  const int p0 = s_p[0], p1 = s_p[1];
  uint4* d0 = reinterpret_cast<uint4*>(xperm + (size_t)p0 * h);
  uint4* d1 = reinterpret_cast<uint4*>(xperm + (size_t)(p1 < 0 ? p0 : p1) * h);
  for (int v = i; v < nvec; v += blockDim.x) {
    const uint4 val = ld_l2(src + v);
    d0[v] = val;
    if (p1 >= 0) d1[v] = val;
  }
}

// Large batches: one warp per token, kRouteTokPerBlock tokens per block (whose pair counts go
// to the block's histogram row).  A lane first fetches its whole share of the token's row (the
// loads that come from DRAM, all independent), then walks it against the router rows, which
// sit in L1 after the block's first pass.

template <int R>
__global__ void __launch_bounds__(32 * kRouteTokPerBlock)
router_kernel(const bf16* x, const bf16* __restrict__ Wg, int T, int h, int r,
              float beta, KeptIds kept, RouteOut o) {
  pdl_launch_dependents();
  pdl_wait();
  __shared__ int s_e[kRouteTokPerBlock][2];
  __shared__ int s_skip[kRouteTokPerBlock];
  constexpr int kRouteXVec = R > 8 ? 8 : 16;  // 16-byte vectors of the row a lane holds at a time
  const int tl = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int t = blockIdx.x * kRouteTokPerBlock + tl;
  const int nvec = h >> 3;

  float acc[R];
#pragma unroll
  for (int c = 0; c < R; ++c) acc[c] = 0.f;
  // a token past the end reads the last token's row; its result is dropped below
  const uint4* xr = reinterpret_cast<const uint4*>(x + (size_t)min(t, T - 1) * h);
  for (int v0 = lane; v0 < nvec; v0 += 32 * kRouteXVec) {
    uint4 xv[kRouteXVec];
#pragma unroll
    for (int i = 0; i < kRouteXVec; ++i)
      xv[i] = (v0 + 32 * i < nvec) ? ld_l2(xr + v0 + 32 * i) : make_uint4(0u, 0u, 0u, 0u);
#pragma unroll
    for (int i = 0; i < kRouteXVec; ++i) {
      const int v = v0 + 32 * i;
      if (v < nvec) {
        uint4 wv[R];
#pragma unroll
        for (int c = 0; c < R; ++c)
          if (c < r) wv[c] = __ldg(reinterpret_cast<const uint4*>(Wg + (size_t)c * h) + v);
        float xf[8];
        unpack8(xv[i], xf);
#pragma unroll
        for (int c = 0; c < R; ++c) {
          if (c < r) {
            float wf[8];
            unpack8(wv[c], wf);
#pragma unroll
            for (int k = 0; k < 8; ++k) acc[c] = fmaf(xf[k], wf[k], acc[c]);
          }
        }
      }
    }
  }
#pragma unroll
  for (int c = 0; c < R; ++c) {
#pragma unroll
    for (int s = 16; s > 0; s >>= 1) acc[c] += __shfl_xor_sync(0xffffffffu, acc[c], s);
  }
  if (lane == 0) {
    if (t >= T) {
      s_e[tl][0] = -1; s_e[tl][1] = -1; s_skip[tl] = 0;
    } else {
      int e0, e1;
      bool skip;
      route_decide<R>(acc, r, beta, t, kept, o, e0, e1, skip);
      s_e[tl][0] = e0;
      s_e[tl][1] = skip ? -1 : e1;
      s_skip[tl] = skip ? 1 : 0;
    }
  }
  __syncthreads();
  if (o.blk_hist && threadIdx.x < kHistCols) {
    int n = 0;
    if (threadIdx.x == 2 * kMaxE) {
      for (int i = 0; i < kRouteTokPerBlock; ++i) n += s_skip[i];
    } else {
      const int c = threadIdx.x >> 1, slot = threadIdx.x & 1;
      for (int i = 0; i < kRouteTokPerBlock; ++i) n += (s_e[i][slot] == c);
    }
    o.blk_hist[(size_t)blockIdx.x * kHistCols + threadIdx.x] = n;
  }
}

// ---------------------------------------------------------------------------------- scan

// One block.  Warp c scans the per-block counts of expert c over the blocks in order, which
// gives every block its first position inside the expert's group; thread 0 then lays the
// groups out (each padded to `pad` rows) and counts the 128-row tiles.
__global__ void __launch_bounds__(1024)
scan_kernel(const int32_t* blk_hist, int nblk, int r, int pad,
            int32_t* __restrict__ blk_base, Meta* meta, int32_t* s_count, int32_t* s_nskipped,
            int32_t* s_ntouched, KeptIds kept, int E) {
  pdl_launch_dependents();
  pdl_wait();
  __shared__ int s_tot[kMaxE][2];
  __shared__ int s_skipped;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (warp < r) {
    int run = 0, run0 = 0;
    // the loads of a step do not depend on the running sums: let several steps be in flight
#pragma unroll 4
    for (int b0 = 0; b0 < nblk; b0 += 32) {
      const int b = b0 + lane;
      int v0 = 0, v1 = 0;
      if (b < nblk) {
        v0 = ld_l2(blk_hist + (size_t)b * kHistCols + 2 * warp);
        v1 = ld_l2(blk_hist + (size_t)b * kHistCols + 2 * warp + 1);
      }
      const int v = v0 + v1;
      int inc = v;
#pragma unroll
      for (int s = 1; s < 32; s <<= 1) {
        const int n = __shfl_up_sync(0xffffffffu, inc, s);
        if (lane >= s) inc += n;
      }
      if (b < nblk) blk_base[(size_t)b * kMaxE + warp] = run + inc - v;
      run += __shfl_sync(0xffffffffu, inc, 31);
      int t0 = v0;
#pragma unroll
      for (int s = 16; s > 0; s >>= 1) t0 += __shfl_xor_sync(0xffffffffu, t0, s);
      run0 += t0;
    }
    if (lane == 0) { s_tot[warp][0] = run0; s_tot[warp][1] = run - run0; }
  } else if (warp == kMaxE) {
    int n = 0;
    for (int b = lane; b < nblk; b += 32) n += ld_l2(blk_hist + (size_t)b * kHistCols + 2 * kMaxE);
#pragma unroll
    for (int s = 16; s > 0; s >>= 1) n += __shfl_xor_sync(0xffffffffu, n, s);
    if (lane == 0) s_skipped = n;
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    int off = 0, tiles = 0, touched = 0;
    meta->off[0] = 0;
    meta->tile_prefix[0] = 0;
    for (int c = 0; c < kMaxE; ++c) {
      const int n0 = c < r ? s_tot[c][0] : 0, n1 = c < r ? s_tot[c][1] : 0;
      const int n = n0 + n1;
      meta->count[c] = n;
      meta->count_slot[c][0] = n0;
      meta->count_slot[c][1] = n1;
      off += (n + pad - 1) / pad * pad;
      tiles += (n + kTileRows - 1) / kTileRows;
      touched += (n > 0);
      meta->off[c + 1] = off;
      meta->tile_prefix[c + 1] = tiles;
    }
    meta->rows_total = off;
    meta->n_skipped = s_skipped;
    meta->n_touched = touched;
    meta->reserved = 0;
    if (s_count) {
      for (int e = 0; e < E; ++e) { s_count[2 * e] = 0; s_count[2 * e + 1] = 0; }
      for (int c = 0; c < r; ++c) {
        s_count[2 * kept.id[c]] = s_tot[c][0];
        s_count[2 * kept.id[c] + 1] = s_tot[c][1];
      }
      *s_nskipped = s_skipped;
      *s_ntouched = touched;
    }
  }
}

// ------------------------------------------------------------------------------- scatter

// Position of pair (t, slot) = start of its expert's group + pairs of that expert in earlier
// blocks + pairs of that expert among the earlier tokens of this block.
__global__ void __launch_bounds__(2 * kRouteTokPerBlock)
scatter_kernel(const int32_t* idx, const uint8_t* skipped, const int32_t* blk_base, const Meta* meta, int T,
               int32_t* __restrict__ pair_pos, int32_t* __restrict__ row_token) {
  pdl_launch_dependents();
  pdl_wait();
  __shared__ int s_e[kRouteTokPerBlock][2];
  const int tl = threadIdx.x >> 1, slot = threadIdx.x & 1;
  const int t = blockIdx.x * kRouteTokPerBlock + tl;
  int c = -1;
  if (t < T) {
    c = ld_l2(idx + 2 * t + slot);
    if (slot == 1 && ld_l2(skipped + t)) c = -1;
  }
  s_e[tl][slot] = c;
  __syncthreads();
  if (t >= T) return;
  int pos = -1;
  if (c >= 0) {
    int rank = 0;
    for (int i = 0; i < tl; ++i) rank += (s_e[i][0] == c) + (s_e[i][1] == c);
    pos = ld_l2(&meta->off[c]) + ld_l2(blk_base + (size_t)blockIdx.x * kMaxE + c) + rank;
    row_token[pos] = t;
  }
  pair_pos[2 * t + slot] = pos;
}

// -------------------------------------------------------------------------------- gather

__global__ void __launch_bounds__(256)
gather_kernel(const bf16* x, const int32_t* row_token, const Meta* meta, int h,
              bf16* __restrict__ xperm) {
  pdl_launch_dependents();
  pdl_wait();
  const int rows = ld_l2(&meta->rows_total);
  const int lane = threadIdx.x & 31;
  const int nvec = h >> 3;
  for (int row = blockIdx.x * 8 + (threadIdx.x >> 5); row < rows; row += gridDim.x * 8) {
    const int t = ld_l2(row_token + row);
    uint4* dst = reinterpret_cast<uint4*>(xperm + (size_t)row * h);
    if (t >= 0) {
      const uint4* src = reinterpret_cast<const uint4*>(x + (size_t)t * h);
      for (int v = lane; v < nvec; v += 32) dst[v] = ld_l2(src + v);
    } else {
      for (int v = lane; v < nvec; v += 32) dst[v] = make_uint4(0, 0, 0, 0);
    }
  }
}

// ------------------------------------------------------------------------------- combine

__global__ void __launch_bounds__(128)
combine_kernel(const float* O, int ksplit, size_t split_stride, const int32_t* pair_pos,
               const float* wn, const bf16* residual, int T, int h, bf16* y) {
  pdl_launch_dependents();
  pdl_wait();
  const int t = blockIdx.x;
  const int p0 = ld_l2(pair_pos + 2 * t), p1 = ld_l2(pair_pos + 2 * t + 1);
  const float w0 = ld_l2(wn + 2 * t), w1 = ld_l2(wn + 2 * t + 1);
  const int nvec = h >> 3;
  for (int v = blockIdx.y * blockDim.x + threadIdx.x; v < nvec; v += gridDim.y * blockDim.x) {
    float a[8], b[8];
#pragma unroll
    for (int k = 0; k < 8; ++k) { a[k] = 0.f; b[k] = 0.f; }
#pragma unroll 4
    for (int s = 0; s < ksplit; ++s) {
      const float4* o0 = reinterpret_cast<const float4*>(O + s * split_stride + (size_t)p0 * h) + 2 * v;
      const float4 q0 = ld_l2(o0), q1 = ld_l2(o0 + 1);
      a[0] += q0.x; a[1] += q0.y; a[2] += q0.z; a[3] += q0.w;
      a[4] += q1.x; a[5] += q1.y; a[6] += q1.z; a[7] += q1.w;
      if (p1 >= 0) {
        const float4* o1 = reinterpret_cast<const float4*>(O + s * split_stride + (size_t)p1 * h) + 2 * v;
        const float4 r0 = ld_l2(o1), r1 = ld_l2(o1 + 1);
        b[0] += r0.x; b[1] += r0.y; b[2] += r0.z; b[3] += r0.w;
        b[4] += r1.x; b[5] += r1.y; b[6] += r1.z; b[7] += r1.w;
      }
    }
    float z[8];
#pragma unroll
    for (int k = 0; k < 8; ++k) z[k] = (p1 >= 0) ? fmaf(w1, b[k], w0 * a[k]) : w0 * a[k];
    if (residual) {
      float rf[8];
      unpack8(ld_l2(reinterpret_cast<const uint4*>(residual + (size_t)t * h) + v), rf);
#pragma unroll
      for (int k = 0; k < 8; ++k) z[k] += rf[k];
    }
    uint4 outv;
    outv.x = pack2(z[0], z[1]); outv.y = pack2(z[2], z[3]);
    outv.z = pack2(z[4], z[5]); outv.w = pack2(z[6], z[7]);
    reinterpret_cast<uint4*>(y + (size_t)t * h)[v] = outv;
  }
}


// ------------------------------------------------------------------ general top-k path

// Top-k routing with the generalised skipping rule of App. A.2, one block per token:
//   e_0..e_{k-1} = kept experts with the k largest logits (ties to the lower index),
//   p_m = exp(l_em - l_e0);  keep the top i* = min i : sum_{m>i} p_m <= beta * sum_{m<=k} p_m;
//   weights p_m / sum_{m<=i*} p_m.  The fp32 summation orders are fixed: total ascending in m,
//   tails from the smallest upwards, kept mass ascending in m.
__global__ void __launch_bounds__(256)
router_topk_kernel(const bf16* __restrict__ x, const bf16* __restrict__ Wg, int T, int h, int r,
                   int k, float beta, KeptIds kept, int32_t* __restrict__ idx,
                   float* __restrict__ wn, int32_t* __restrict__ nact, int32_t* u_idx, float* u_wn,
                   int32_t* u_nact, float* logits) {
  __shared__ float s_part[8][kMaxE];
  const int t = blockIdx.x;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int nvec = h >> 3;
  float acc[kMaxE];
#pragma unroll
  for (int c = 0; c < kMaxE; ++c) acc[c] = 0.f;
  const uint4* xr = reinterpret_cast<const uint4*>(x + (size_t)t * h);
  for (int v = threadIdx.x; v < nvec; v += 256) {
    float xf[8];
    unpack8(ld_l2(xr + v), xf);
#pragma unroll
    for (int c = 0; c < kMaxE; ++c) {
      if (c < r) {
        float wf[8];
        unpack8(__ldg(reinterpret_cast<const uint4*>(Wg + (size_t)c * h) + v), wf);
#pragma unroll
        for (int q = 0; q < 8; ++q) acc[c] = fmaf(xf[q], wf[q], acc[c]);
      }
    }
  }
#pragma unroll
  for (int c = 0; c < kMaxE; ++c) {
#pragma unroll
    for (int s = 16; s > 0; s >>= 1) acc[c] += __shfl_xor_sync(0xffffffffu, acc[c], s);
    if (lane == 0) s_part[warp][c] = acc[c];
  }
  __syncthreads();
  // Ranking by counting, one thread per kept expert: the rank of expert c is the number of kept
  // experts that beat it (larger logit, or equal logit and lower index), so the expert of rank m
  // is the m-th choice.  The k chosen experts' softmax numerators relative to the largest,
  // p_m = exp(l_m - l_0), then go through the three fixed-order sums of the rule, which one
  // thread evaluates (k <= 8 values).
  __shared__ float s_l[kMaxE];
  __shared__ float s_p[kMaxE];
  __shared__ int s_sel[kMaxE];
  const int c = threadIdx.x;
  if (c < r) {
    float v = 0.f;
    for (int w = 0; w < 8; ++w) v += s_part[w][c];
    s_l[c] = v;
    if (logits) logits[(size_t)t * r + c] = v;
  }
  __syncthreads();
  if (c < r) {
    const float mine = s_l[c];
    int rank = 0;
    for (int d = 0; d < r; ++d) {
      const float o = s_l[d];
      rank += (o > mine) || (o == mine && d < c);
    }
    if (rank < k) s_sel[rank] = c;
  }
  __syncthreads();
  if (c < k) s_p[c] = expf(s_l[s_sel[c]] - s_l[s_sel[0]]);
  __syncthreads();
  if (c != 0) return;
  // i* = the smallest i in 1..k whose dropped mass p_i + .. + p_{k-1} (added from the smallest
  // value upwards) is at most beta times the whole mass p_0 + .. + p_{k-1} (added in rank order)
  float whole = 0.f;
  for (int m = 0; m < k; ++m) whole += s_p[m];
  const float bound = beta * whole;
  int istar = 1;
  {
    float dropped = 0.f;   // mass beyond rank i - 1, for i = k, k - 1, ..: walk down while it fits
    int i = k;
    while (i > 1 && dropped + s_p[i - 1] <= bound) { dropped += s_p[i - 1]; --i; }
    // dropped = p_i + .. + p_{k-1} fits; p_{i-1} + dropped does not (or i = 1)
    istar = i;
  }
  float kept_mass = 0.f;
  for (int m = 0; m < istar; ++m) kept_mass += s_p[m];
  for (int m = 0; m < k; ++m) {
    const float w = m < istar ? s_p[m] / kept_mass : 0.f;
    const int e = s_sel[m];
    idx[(size_t)t * k + m] = e;
    wn[(size_t)t * k + m] = w;
    if (u_idx) u_idx[(size_t)t * k + m] = kept.id[e];
    if (u_wn) u_wn[(size_t)t * k + m] = w;
  }
  nact[t] = istar;
  if (u_nact) u_nact[t] = istar;
}

// Per block of kRouteTokPerBlock tokens: active pairs per expert, in the column layout scan_kernel reads
// (the pairs go to the slot-0 column, the skipped pairs to the last column).
__global__ void __launch_bounds__(kHistCols < 64 ? 64 : kHistCols)
count_topk_kernel(const int32_t* __restrict__ idx, const int32_t* __restrict__ nact, int T, int k,
                  int32_t* __restrict__ blk_hist) {
  const int t0 = blockIdx.x * kRouteTokPerBlock;
  const int col = threadIdx.x;
  if (col >= kHistCols) return;
  int n = 0;
  const int t1 = min(T, t0 + kRouteTokPerBlock);
  if (col == 2 * kMaxE) {
    for (int t = t0; t < t1; ++t) n += k - nact[t];
  } else if ((col & 1) == 0) {
    const int c = col >> 1;
    for (int t = t0; t < t1; ++t)
      for (int m = 0; m < nact[t]; ++m) n += (idx[(size_t)t * k + m] == c);
  }
  blk_hist[(size_t)blockIdx.x * kHistCols + col] = n;
}

// Position of pair (t, m): start of the expert's group + pairs of that expert in earlier
// blocks + pairs of that expert among the earlier tokens of this block.
__global__ void __launch_bounds__(kRouteTokPerBlock)
scatter_topk_kernel(const int32_t* __restrict__ idx, const int32_t* __restrict__ nact,
                    const int32_t* __restrict__ blk_base, const Meta* __restrict__ meta, int T,
                    int k, int32_t* __restrict__ pair_pos, int32_t* __restrict__ row_token) {
  __shared__ int s_e[kRouteTokPerBlock][kMaxE];
  const int tl = threadIdx.x;
  const int t = blockIdx.x * kRouteTokPerBlock + tl;
  for (int m = 0; m < k; ++m) s_e[tl][m] = (t < T && m < nact[t]) ? idx[(size_t)t * k + m] : -1;
  __syncthreads();
  if (t >= T) return;
  for (int m = 0; m < k; ++m) {
    const int c = s_e[tl][m];
    int pos = -1;
    if (c >= 0) {
      int rank = 0;
      for (int i = 0; i < tl; ++i)
        for (int q = 0; q < k; ++q) rank += (s_e[i][q] == c);
      pos = meta->off[c] + blk_base[(size_t)blockIdx.x * kMaxE + c] + rank;
      row_token[pos] = t;
    }
    pair_pos[(size_t)t * k + m] = pos;
  }
}

__global__ void __launch_bounds__(128)
combine_topk_kernel(const float* __restrict__ O, int ksplit, size_t split_stride,
                    const int32_t* __restrict__ pair_pos, const float* __restrict__ wn, int k,
                    int T, int h, bf16* y) {
  const int t = blockIdx.x;
  const int nvec = h >> 3;
  for (int v = blockIdx.y * blockDim.x + threadIdx.x; v < nvec; v += gridDim.y * blockDim.x) {
    float z[8];
#pragma unroll
    for (int q = 0; q < 8; ++q) z[q] = 0.f;
    for (int m = 0; m < k; ++m) {
      const int p = pair_pos[(size_t)t * k + m];
      if (p < 0) continue;
      const float w = wn[(size_t)t * k + m];
      float a[8];
#pragma unroll
      for (int q = 0; q < 8; ++q) a[q] = 0.f;
      for (int s = 0; s < ksplit; ++s) {
        const float4* o = reinterpret_cast<const float4*>(O + s * split_stride + (size_t)p * h) + 2 * v;
        const float4 q0 = o[0], q1 = o[1];
        a[0] += q0.x; a[1] += q0.y; a[2] += q0.z; a[3] += q0.w;
        a[4] += q1.x; a[5] += q1.y; a[6] += q1.z; a[7] += q1.w;
      }
#pragma unroll
      for (int q = 0; q < 8; ++q) z[q] = fmaf(w, a[q], z[q]);
    }
    uint4 outv;
    outv.x = pack2(z[0], z[1]); outv.y = pack2(z[2], z[3]);
    outv.z = pack2(z[4], z[5]); outv.w = pack2(z[6], z[7]);
    reinterpret_cast<uint4*>(y + (size_t)t * h)[v] = outv;
  }
}

// --------------------------------------------------------------------------- co-selection

// counts[a][b] += 1 for every token whose top-2 is (a, b) (App. A.1).  Integer counts: block
// histograms in shared memory, then integer atomics, so the result is exact and order-free.
__global__ void __launch_bounds__(256)
coselection_kernel(const int32_t* __restrict__ idx, int T, int E, KeptIds kept,
                   int32_t* __restrict__ counts) {
  __shared__ int s_c[kMaxE * kMaxE];
  for (int i = threadIdx.x; i < kMaxE * kMaxE; i += blockDim.x) s_c[i] = 0;
  __syncthreads();
  for (int t = blockIdx.x * blockDim.x + threadIdx.x; t < T; t += gridDim.x * blockDim.x)
    atomicAdd(&s_c[kept.id[idx[2 * t]] * kMaxE + kept.id[idx[2 * t + 1]]], 1);
  __syncthreads();
  for (int i = threadIdx.x; i < kMaxE * kMaxE; i += blockDim.x) {
    const int a = i / kMaxE, b = i % kMaxE;
    if (a < E && b < E && s_c[i]) atomicAdd(&counts[a * E + b], s_c[i]);
  }
}

// ------------------------------------------------------------------------- top-2 distance

// D_t = || E_e0(x_t) - E_e1(x_t) ||_2, the quantity App. A.2 observes to be concentrated.
__global__ void __launch_bounds__(256)
top2_distance_kernel(const float* O, int ksplit, size_t split_stride, const int32_t* pair_pos, int T,
                     int h, float* __restrict__ dist) {
  __shared__ float s_part[8];
  pdl_launch_dependents();
  pdl_wait();
  const int t = blockIdx.x;
  const int p0 = ld_l2(pair_pos + 2 * t), p1 = ld_l2(pair_pos + 2 * t + 1);
  float acc = 0.f;
  if (p1 >= 0) {
    for (int i = threadIdx.x; i < h; i += blockDim.x) {
      float a = 0.f, b = 0.f;
      for (int s = 0; s < ksplit; ++s) {
        a += ld_l2(O + s * split_stride + (size_t)p0 * h + i);
        b += ld_l2(O + s * split_stride + (size_t)p1 * h + i);
      }
      const float d = a - b;
      acc = fmaf(d, d, acc);
    }
  }
#pragma unroll
  for (int s = 16; s > 0; s >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, s);
  if ((threadIdx.x & 31) == 0) s_part[threadIdx.x >> 5] = acc;
  __syncthreads();
  if (threadIdx.x == 0) {
    float tot = 0.f;
    for (int w = 0; w < 8; ++w) tot += s_part[w];
    dist[t] = sqrtf(tot);
  }
}

// ------------------------------------------------------------------------------- rmsnorm

__global__ void __launch_bounds__(256)
rmsnorm_kernel(const bf16* x, int T, int h, float eps, bf16* out) {
  pdl_launch_dependents();
  pdl_wait();
  __shared__ float s_part[8];
  const int t = blockIdx.x;
  const int nvec = h >> 3;
  const uint4* xr = reinterpret_cast<const uint4*>(x + (size_t)t * h);
  float ss = 0.f;
  for (int v = threadIdx.x; v < nvec; v += blockDim.x) {
    float f[8];
    unpack8(ld_l2(xr + v), f);
#pragma unroll
    for (int k = 0; k < 8; ++k) ss = fmaf(f[k], f[k], ss);
  }
#pragma unroll
  for (int s = 16; s > 0; s >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, s);
  if ((threadIdx.x & 31) == 0) s_part[threadIdx.x >> 5] = ss;
  __syncthreads();
  float tot = 0.f;
#pragma unroll
  for (int w = 0; w < 8; ++w) tot += s_part[w];
  const float inv = 1.0f / sqrtf(tot / (float)h + eps);
  for (int v = threadIdx.x; v < nvec; v += blockDim.x) {
    float f[8];
    unpack8(ld_l2(xr + v), f);
    uint4 o;
    o.x = pack2(f[0] * inv, f[1] * inv); o.y = pack2(f[2] * inv, f[3] * inv);
    o.z = pack2(f[4] * inv, f[5] * inv); o.w = pack2(f[6] * inv, f[7] * inv);
    reinterpret_cast<uint4*>(out + (size_t)t * h)[v] = o;
  }
}

// ---------------------------------------------------------------------------- dense meta

__global__ void set_dense_meta_kernel(Meta* meta, int E, int rows, int off_stride) {
  if (threadIdx.x != 0) return;
  const int tiles = (rows + kTileRows - 1) / kTileRows;
  for (int c = 0; c <= kMaxE; ++c) {
    const int cc = c < E ? c : E;
    meta->off[c] = cc * off_stride;
    meta->tile_prefix[c] = cc * tiles;
    if (c < kMaxE) {
      meta->count[c] = c < E ? rows : 0;
      meta->count_slot[c][0] = meta->count[c];
      meta->count_slot[c][1] = 0;
    }
  }
  meta->rows_total = E * off_stride;
  meta->n_skipped = 0;
  meta->n_touched = E;
  meta->reserved = 0;
}

// -------------------------------------------------------------------------------- select

__device__ __forceinline__ uint32_t float_key(float f) {
  const uint32_t u = __float_as_uint(f);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
__device__ __forceinline__ float key_float(uint32_t k) {
  return __uint_as_float((k & 0x80000000u) ? (k & 0x7fffffffu) : ~k);
}

// Exact k-th smallest by radix selection on the ordered bit patterns, 8 bits per pass.
__global__ void __launch_bounds__(1024)
select2_kernel(const float* __restrict__ v, int n, int k0, int k1, float* out) {
  __shared__ unsigned hist[256];
  __shared__ unsigned s_prefix;
  __shared__ int s_k;
  for (int which = 0; which < 2; ++which) {
    if (threadIdx.x == 0) { s_prefix = 0; s_k = which ? k1 : k0; }
    unsigned mask = 0;
    for (int pass = 3; pass >= 0; --pass) {
      const int shift = pass * 8;
      if (threadIdx.x < 256) hist[threadIdx.x] = 0;
      __syncthreads();
      const unsigned prefix = s_prefix;
      for (int i = threadIdx.x; i < n; i += blockDim.x) {
        const unsigned key = float_key(v[i]);
        if ((key & mask) == prefix) atomicAdd(&hist[(key >> shift) & 255u], 1u);
      }
      __syncthreads();
      if (threadIdx.x == 0) {
        int k = s_k;
        unsigned bin = 0;
        for (; bin < 255; ++bin) {
          if (k < (int)hist[bin]) break;
          k -= (int)hist[bin];
        }
        s_k = k;
        s_prefix = prefix | (bin << shift);
      }
      mask |= 0xffu << shift;
      __syncthreads();
    }
    if (threadIdx.x == 0) out[which] = key_float(s_prefix);
    __syncthreads();
  }
}

// ---------------------------------------------------------------------------- interleave

__global__ void __launch_bounds__(256)
interleave_kernel(const bf16* __restrict__ W1, const bf16* __restrict__ W3, KeptIds kept, int r,
                  int f, int h, bf16* __restrict__ W13) {
  const long long rows = (long long)r * 2 * f;
  const int lane = threadIdx.x & 31;
  const int nvec = h >> 3;
  for (long long row = (long long)blockIdx.x * 8 + (threadIdx.x >> 5); row < rows;
       row += (long long)gridDim.x * 8) {
    const int c = (int)(row / (2 * f));
    const int R = (int)(row % (2 * f));
    const int q = R / (2 * kInterleave), s = R % (2 * kInterleave);
    const bf16* src = (s < kInterleave)
        ? W1 + ((size_t)kept.id[c] * f + (size_t)q * kInterleave + s) * h
        : W3 + ((size_t)kept.id[c] * f + (size_t)q * kInterleave + s - kInterleave) * h;
    const uint4* sv = reinterpret_cast<const uint4*>(src);
    uint4* dv = reinterpret_cast<uint4*>(W13 + (size_t)row * h);
    for (int v = lane; v < nvec; v += 32) dv[v] = __ldg(sv + v);
  }
}

}  // namespace

// ------------------------------------------------------------------------------ launchers

cudaError_t launch_router(const bf16* x, const bf16* Wg, int T, int h, int r, float beta,
                          const KeptIds& kept, const RouteOut& out, cudaStream_t st) {
  const int nblk = (T + kRouteTokPerBlock - 1) / kRouteTokPerBlock;
  switch (r) {
    case 2: return launch_pdl(router_kernel<2>, dim3(nblk), dim3(32 * kRouteTokPerBlock), 0, st, x, Wg, T, h, r, beta, kept, out);
    case 3: case 4: return launch_pdl(router_kernel<4>, dim3(nblk), dim3(32 * kRouteTokPerBlock), 0, st, x, Wg, T, h, r, beta, kept, out);
    case 5: case 6: return launch_pdl(router_kernel<6>, dim3(nblk), dim3(32 * kRouteTokPerBlock), 0, st, x, Wg, T, h, r, beta, kept, out);
    case 7: case 8: return launch_pdl(router_kernel<8>, dim3(nblk), dim3(32 * kRouteTokPerBlock), 0, st, x, Wg, T, h, r, beta, kept, out);
    default: return launch_pdl(router_kernel<kMaxE>, dim3(nblk), dim3(32 * kRouteTokPerBlock), 0, st, x, Wg, T, h, r, beta, kept, out);
  }
  return cudaGetLastError();
}

cudaError_t launch_router_small(const bf16* x, const bf16* Wg, int T, int h, int r, float beta,
                                const KeptIds& kept, const RouteOut& out, cudaStream_t st) {
  switch (r) {
    case 2: return launch_pdl(router_small_kernel<2>, dim3(T), dim3(256), 0, st, x, Wg, T, h, r, beta, kept, out);
    case 3: case 4: return launch_pdl(router_small_kernel<4>, dim3(T), dim3(256), 0, st, x, Wg, T, h, r, beta, kept, out);
    case 5: case 6: return launch_pdl(router_small_kernel<6>, dim3(T), dim3(256), 0, st, x, Wg, T, h, r, beta, kept, out);
    case 7: case 8: return launch_pdl(router_small_kernel<8>, dim3(T), dim3(256), 0, st, x, Wg, T, h, r, beta, kept, out);
    default: return launch_pdl(router_small_kernel<kMaxE>, dim3(T), dim3(256), 0, st, x, Wg, T, h, r, beta, kept, out);
  }
  return cudaGetLastError();
}

cudaError_t launch_route_single(const bf16* x, const bf16* Wg, int h, int r, float beta,
                                const KeptIds& kept, const RouteOut& out, int pad, Meta* meta,
                                int32_t* pair_pos, int32_t* row_token, bf16* xperm, int32_t* s_count,
                                int32_t* s_nskipped, int32_t* s_ntouched, int E, cudaStream_t st) {
#define MOE_ROUTE_SINGLE(R)                                                                        \
  return launch_pdl(route_single_kernel<R>, dim3(1), dim3(256), 0, st, x, Wg, h, r, beta, kept, out, \
                    pad, meta, pair_pos, row_token, xperm, s_count, s_nskipped, s_ntouched, E)
  switch (r) {
    case 2: MOE_ROUTE_SINGLE(2);
    case 3: case 4: MOE_ROUTE_SINGLE(4);
    case 5: case 6: MOE_ROUTE_SINGLE(6);
    case 7: case 8: MOE_ROUTE_SINGLE(8);
    default: MOE_ROUTE_SINGLE(kMaxE);
  }
#undef MOE_ROUTE_SINGLE
}

cudaError_t launch_permute_gather_small(const bf16* x, const int32_t* idx, const uint8_t* skipped, int T,
                                        int h, int r, int pad, Meta* meta, int32_t* pair_pos,
                                        int32_t* row_token, bf16* xperm, int32_t* s_count,
                                        int32_t* s_nskipped, int32_t* s_ntouched, const KeptIds& kept,
                                        int E, cudaStream_t st) {
  return launch_pdl(permute_gather_small_kernel, dim3(T), dim3(kDecodeMaxT), 0, st, x, idx, skipped, T, h,
                    r, pad, meta, pair_pos, row_token, xperm, s_count, s_nskipped, s_ntouched, kept, E);
}

cudaError_t launch_scan(const int32_t* blk_hist, int nblk, int r, int pad, int32_t* blk_base,
                        Meta* meta, int32_t* s_count, int32_t* s_nskipped, int32_t* s_ntouched,
                        const KeptIds& kept, int E, cudaStream_t st) {
  return launch_pdl(scan_kernel, dim3(1), dim3(1024), 0, st, blk_hist, nblk, r, pad, blk_base, meta,
                    s_count, s_nskipped, s_ntouched, kept, E);
}

cudaError_t launch_scatter(const int32_t* idx, const uint8_t* skipped, const int32_t* blk_base,
                           const Meta* meta, int T, int32_t* pair_pos, int32_t* row_token,
                           cudaStream_t st) {
  const int nblk = (T + kRouteTokPerBlock - 1) / kRouteTokPerBlock;
  return launch_pdl(scatter_kernel, dim3(nblk), dim3(2 * kRouteTokPerBlock), 0, st, idx, skipped,
                    blk_base, meta, T, pair_pos, row_token);
}

cudaError_t launch_gather(const bf16* x, const int32_t* row_token, const Meta* meta, int h,
                          int cap_rows, bf16* xperm, cudaStream_t st) {
  int blocks = (cap_rows + 7) / 8;
  if (blocks > 148 * 16) blocks = 148 * 16;
  if (blocks < 1) blocks = 1;
  return launch_pdl(gather_kernel, dim3(blocks), dim3(256), 0, st, x, row_token, meta, h, xperm);
}

cudaError_t launch_combine(const float* O, int ksplit, size_t split_stride, const int32_t* pair_pos,
                           const float* wn, const bf16* residual, int T, int h, bf16* y,
                           cudaStream_t st) {
  int ychunks = ((h >> 3) + 127) / 128;
  if (T > 4096) ychunks = 1;  // plenty of blocks already
  return launch_pdl(combine_kernel, dim3(T, ychunks), dim3(128), 0, st, O, ksplit, split_stride,
                    pair_pos, wn, residual, T, h, y);
}

cudaError_t launch_router_topk(const bf16* x, const bf16* Wg, int T, int h, int r, int k, float beta,
                               const KeptIds& kept, int32_t* idx, float* wn, int32_t* nact,
                               int32_t* u_idx, float* u_wn, int32_t* u_nact, float* logits,
                               cudaStream_t st) {
  router_topk_kernel<<<T, 256, 0, st>>>(x, Wg, T, h, r, k, beta, kept, idx, wn, nact, u_idx, u_wn, u_nact,
                                        logits);
  return cudaGetLastError();
}

cudaError_t launch_count_topk(const int32_t* idx, const int32_t* nact, int T, int k,
                              int32_t* blk_hist, cudaStream_t st) {
  const int nblk = (T + kRouteTokPerBlock - 1) / kRouteTokPerBlock;
  count_topk_kernel<<<nblk, kHistCols < 64 ? 64 : kHistCols, 0, st>>>(idx, nact, T, k, blk_hist);
  return cudaGetLastError();
}

cudaError_t launch_scatter_topk(const int32_t* idx, const int32_t* nact, const int32_t* blk_base,
                                const Meta* meta, int T, int k, int32_t* pair_pos,
                                int32_t* row_token, cudaStream_t st) {
  const int nblk = (T + kRouteTokPerBlock - 1) / kRouteTokPerBlock;
  scatter_topk_kernel<<<nblk, kRouteTokPerBlock, 0, st>>>(idx, nact, blk_base, meta, T, k, pair_pos,
                                                          row_token);
  return cudaGetLastError();
}

cudaError_t launch_combine_topk(const float* O, int ksplit, size_t split_stride,
                                const int32_t* pair_pos, const float* wn, int k, int T, int h,
                                bf16* y, cudaStream_t st) {
  int ychunks = ((h >> 3) + 127) / 128;
  if (T > 4096) ychunks = 1;
  combine_topk_kernel<<<dim3(T, ychunks), 128, 0, st>>>(O, ksplit, split_stride, pair_pos, wn, k, T, h, y);
  return cudaGetLastError();
}

cudaError_t launch_coselection(const int32_t* idx, int T, int E, const KeptIds& kept, int32_t* counts,
                               cudaStream_t st) {
  int blocks = (T + 255) / 256;
  if (blocks > 148 * 4) blocks = 148 * 4;
  coselection_kernel<<<blocks, 256, 0, st>>>(idx, T, E, kept, counts);
  return cudaGetLastError();
}

cudaError_t launch_top2_distance(const float* O, int ksplit, size_t split_stride,
                                 const int32_t* pair_pos, int T, int h, float* dist, cudaStream_t st) {
  return launch_pdl(top2_distance_kernel, dim3(T), dim3(256), 0, st, O, ksplit, split_stride, pair_pos,
                    T, h, dist);
}

cudaError_t launch_rmsnorm(const bf16* x, int T, int h, float eps, bf16* out, cudaStream_t st) {
  return launch_pdl(rmsnorm_kernel, dim3(T), dim3(256), 0, st, x, T, h, eps, out);
}

cudaError_t launch_set_dense_meta(Meta* meta, int E, int rows_per_expert, int off_stride,
                                  cudaStream_t st) {
  set_dense_meta_kernel<<<1, 32, 0, st>>>(meta, E, rows_per_expert, off_stride);
  return cudaGetLastError();
}

cudaError_t launch_select2(const float* ratio, int T, int k0, int k1, float* out, cudaStream_t st) {
  select2_kernel<<<1, 1024, 0, st>>>(ratio, T, k0, k1, out);
  return cudaGetLastError();
}

cudaError_t launch_interleave(const bf16* W1, const bf16* W3, const KeptIds& kept, int r, int f,
                              int h, bf16* W13, cudaStream_t st) {
  interleave_kernel<<<148 * 8, 256, 0, st>>>(W1, W3, kept, r, f, h, W13);
  return cudaGetLastError();
}

}  // namespace moe
