// Subset enumeration of the layer-wise pruning search (Sec. 3.2, Eq. 3).
//
// Input: router logits l[T][E] and Yall[t][e] = bf16(E_e(x_t)) for every token and expert.
// For a kept subset C the pruned layer routes token t to the two highest-ranked experts
// (by logit) that are in C, so per token only pairs of its top (E - r + 2) ranked experts can
// occur.  One warp per token computes the squared error of each such pair against the
// unpruned output once (from the Gram matrix of the expert outputs' differences, see
// pair_errors_fast), then adds it to every subset that selects the pair.
//   loss(C) = sqrt( sum_t || F'(x_t, C) - F(x_t) ||^2 )
// Reduction order is fixed: tokens of a warp in order (fp32), warps of a block in order,
// blocks in order (fp64); no atomics.
#include "common.h"

namespace moe {

namespace {

constexpr int kTokPerWarp = 2;
constexpr int kMaxBlocks = 148 * 16;

__device__ __forceinline__ void unpack8f(const uint4& v, float* f) {
  f[0] = __uint_as_float(v.x << 16); f[1] = __uint_as_float(v.x & 0xffff0000u);
  f[2] = __uint_as_float(v.y << 16); f[3] = __uint_as_float(v.y & 0xffff0000u);
  f[4] = __uint_as_float(v.z << 16); f[5] = __uint_as_float(v.z & 0xffff0000u);
  f[6] = __uint_as_float(v.w << 16); f[7] = __uint_as_float(v.w & 0xffff0000u);
}

// Normalised top-2 weights of the pair (first, second) from their logits: the softmax
// denominator cancels (Eq. 1), p = exp(l_second - l_first).
__device__ __forceinline__ void pair_weights(float l_first, float l_second, float& wa, float& wb) {
  const float p = expf(l_second - l_first);
  const float d = 1.0f + p;
  wa = 1.0f / d;
  wb = p / d;
}

// Squared errors of all pairs among the K top-ranked experts of one token.
//
// With y_0 .. y_{K-1} the token's expert outputs in rank order and w~_a + w~_b = 1 (Eq. 1), the
// pruned layer's output for the pair (i, j) is  y_0 + w~_i u_i + w~_j u_j  with the differences
// u_a = y_a - y_0 (u_0 = 0), and the target is  y_0 + w~'_1 u_1  (the unpruned output: the two
// top-ranked experts) or, for the progressive search, a given row f:  y_0 - g  with g = y_0 - f.
// Every error vector is therefore a combination of the NV = K - 1 (+ 1) vectors u_1 .. u_{K-1}
// (, g), and its squared norm follows from their Gram matrix: NV (NV + 1) / 2 dot products per
// element instead of four operations for each of the K (K - 1) / 2 pairs, a third of the
// arithmetic at K = 6.  Forming the differences first (exactly, from bf16 values) keeps the
// cancellation between similar expert outputs out of the accumulated sums; the pair (0, 1) has
// all coefficients zero and an error of exactly 0.  `ref` (optional) is the target row f in fp32.
// The rows of the next 8-element slice are fetched before the current one is used.
template <int K, bool REF>
__device__ __forceinline__ void pair_errors_fast(const bf16* __restrict__ Yt, int h,
                                                 const int* order, const int* rowoff,
                                                 const float* l, int lane,
                                                 float* s_err /* [16*16] */,
                                                 const float* __restrict__ ref) {
  constexpr int NV = K - 1 + (REF ? 1 : 0);
  constexpr int NG = NV * (NV + 1) / 2;
  float G[NG > 0 ? NG : 1];
#pragma unroll
  for (int q = 0; q < NG; ++q) G[q] = 0.f;
  const uint4* rows[K];
#pragma unroll
  for (int i = 0; i < K; ++i) rows[i] = reinterpret_cast<const uint4*>(Yt + (size_t)rowoff[i] * h);
  const int nvec = h >> 3;
  uint4 cur[K], nxt[K];
  float4 cref0 = make_float4(0.f, 0.f, 0.f, 0.f), cref1 = cref0, nref0 = cref0, nref1 = cref0;
  if (lane < nvec) {
#pragma unroll
    for (int i = 0; i < K; ++i) cur[i] = __ldg(rows[i] + lane);
    if (REF) {
      cref0 = __ldg(reinterpret_cast<const float4*>(ref) + 2 * lane);
      cref1 = __ldg(reinterpret_cast<const float4*>(ref) + 2 * lane + 1);
    }
  }
  for (int v = lane; v < nvec; v += 32) {
    if (v + 32 < nvec) {
#pragma unroll
      for (int i = 0; i < K; ++i) nxt[i] = __ldg(rows[i] + v + 32);
      if (REF) {
        nref0 = __ldg(reinterpret_cast<const float4*>(ref) + 2 * (v + 32));
        nref1 = __ldg(reinterpret_cast<const float4*>(ref) + 2 * (v + 32) + 1);
      }
    }
    const float fr[8] = {cref0.x, cref0.y, cref0.z, cref0.w, cref1.x, cref1.y, cref1.z, cref1.w};
#pragma unroll
    for (int k = 0; k < 8; ++k) {
      // element k of each row, straight from the packed registers
      float yk[K];
#pragma unroll
      for (int i = 0; i < K; ++i) {
        const uint32_t w = (k >> 1) == 0 ? cur[i].x : ((k >> 1) == 1 ? cur[i].y : ((k >> 1) == 2 ? cur[i].z : cur[i].w));
        yk[i] = (k & 1) ? __uint_as_float(w & 0xffff0000u) : __uint_as_float(w << 16);
      }
      float u[NV > 0 ? NV : 1];
#pragma unroll
      for (int a = 0; a < K - 1; ++a) u[a] = yk[a + 1] - yk[0];
      if (REF) u[K - 1] = yk[0] - fr[k];
      int q = 0;
#pragma unroll
      for (int a = 0; a < NV; ++a)
#pragma unroll
        for (int b = a; b < NV; ++b, ++q) G[q] = fmaf(u[a], u[b], G[q]);
    }
#pragma unroll
    for (int i = 0; i < K; ++i) cur[i] = nxt[i];
    if (REF) { cref0 = nref0; cref1 = nref1; }
  }
#pragma unroll
  for (int q = 0; q < NG; ++q) {
#pragma unroll
    for (int s = 16; s > 0; s >>= 1) G[q] += __shfl_xor_sync(0xffffffffu, G[q], s);
  }
  // lane p evaluates pair p = (i, j), all pairs at once: err = sum_ab c_a c_b G_ab with
  // c = w~_i e_{i-1} + w~_j e_{j-1} - (target), every lane holding the reduced G
  constexpr int NP = K * (K - 1) / 2;
  if (lane < NP) {
    int i = 0, rem = lane;
    while (rem >= K - 1 - i) { rem -= K - 1 - i; ++i; }
    const int j = i + 1 + rem;
    float wt0, wt1, wa, wb;
    pair_weights(l[order[0]], l[order[1]], wt0, wt1);  // the unpruned output: the two top-ranked experts
    pair_weights(l[order[i]], l[order[j]], wa, wb);
    float c[NV > 0 ? NV : 1];
#pragma unroll
    for (int a = 0; a < NV; ++a) {
      c[a] = 0.f;
      if (a == i - 1) c[a] += wa;   // u_i (nothing for i = 0: u_0 = 0)
      if (a == j - 1) c[a] += wb;   // u_j
    }
    if (REF) c[NV - 1] += 1.0f;     // + g
    else c[0] -= wt1;               // - w~'_1 u_1
    double e = 0.0;
    int q = 0;
#pragma unroll
    for (int a = 0; a < NV; ++a)
#pragma unroll
      for (int b = a; b < NV; ++b, ++q)
        e += (double)(a == b ? c[a] * c[a] : 2.0f * c[a] * c[b]) * (double)G[q];
    s_err[i * kMaxE + j] = e > 0.0 ? (float)e : 0.f;
  }
}

// The same for any K, one pair at a time (rows are re-read from cache).
__device__ __forceinline__ void pair_errors_generic(const bf16* __restrict__ Yt, int h, int K,
                                                    const int* order, const int* rowoff,
                                                    const float* l, int lane, float* s_err,
                                                    const float* __restrict__ ref) {
  float w0, w1;
  pair_weights(l[order[0]], l[order[1]], w0, w1);
  const uint4* r0 = reinterpret_cast<const uint4*>(Yt + (size_t)rowoff[0] * h);
  const uint4* r1 = reinterpret_cast<const uint4*>(Yt + (size_t)rowoff[1] * h);
  for (int i = 0; i < K; ++i)
    for (int j = i + 1; j < K; ++j) {
      float wa, wb;
      pair_weights(l[order[i]], l[order[j]], wa, wb);
      const uint4* ri = reinterpret_cast<const uint4*>(Yt + (size_t)rowoff[i] * h);
      const uint4* rj = reinterpret_cast<const uint4*>(Yt + (size_t)rowoff[j] * h);
      float e = 0.f;
      for (int v = lane; v < (h >> 3); v += 32) {
        float y0[8], y1[8], yi[8], yj[8];
        unpack8f(__ldg(r0 + v), y0);
        unpack8f(__ldg(r1 + v), y1);
        unpack8f(__ldg(ri + v), yi);
        unpack8f(__ldg(rj + v), yj);
#pragma unroll
        for (int k = 0; k < 8; ++k) {
          const float F = ref ? ref[8 * v + k] : fmaf(w1, y1[k], w0 * y0[k]);
          const float d = fmaf(wb, yj[k], wa * yi[k]) - F;
          e = fmaf(d, d, e);
        }
      }
#pragma unroll
      for (int s = 16; s > 0; s >>= 1) e += __shfl_xor_sync(0xffffffffu, e, s);
      if (lane == 0) s_err[i * kMaxE + j] = e;
    }
}

// KT = K for the Gram form (K = 2 .. 6), 0 for any K through the generic form; REF = a target row
// per token is given (progressive search).
template <int KT, bool REF>
__global__ void __launch_bounds__(128)
enumerate_kernel(const float* __restrict__ logits, const bf16* __restrict__ Yall, int T, int E,
                 int r, int h, const uint32_t* __restrict__ subsets, int nC,
                 float* __restrict__ partial, const float* __restrict__ Fref, EnumSource src) {
  extern __shared__ float s_dyn[];
  const int nwarps = blockDim.x >> 5;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  float* acc = s_dyn + (size_t)warp * nC;  // [nC] per warp
  float* base_err = s_dyn + (size_t)nwarps * nC;
  float* s_err = base_err + warp * (kMaxE * kMaxE);
  int* base_order = reinterpret_cast<int*>(base_err + nwarps * (kMaxE * kMaxE));
  int* s_order = base_order + warp * kMaxE;
  float* s_l = reinterpret_cast<float*>(base_order + nwarps * kMaxE) + warp * kMaxE;
  int* s_row = reinterpret_cast<int*>(base_order + 2 * nwarps * kMaxE) + warp * kMaxE;

  for (int s = lane; s < nC; s += 32) acc[s] = 0.f;
  const int K = E - r + 2;
  const int gw = blockIdx.x * nwarps + warp;
  const int stride = gridDim.x * nwarps;
  for (int t = gw; t < T; t += stride) {
    __syncwarp();
    // rank of every expert by (logit descending, index ascending)
    float mine = 0.f;
    if (lane < E) {
      mine = logits[(size_t)t * E + lane];
      s_l[lane] = mine;
    }
    __syncwarp();
    if (src.topk_idx) {
      // only the K top-ranked experts were evaluated; they are listed in rank order, and their
      // outputs sit in the permuted row pair_pos[t][rank] of the token's chunk
      if (lane < K) {
        s_order[lane] = src.topk_idx[(size_t)t * src.k_stride + lane];
        s_row[lane] = (t / src.chunk_tokens) * src.chunk_rows + src.pair_pos[(size_t)t * src.k_stride + lane];
      }
    } else if (lane < E) {
      int rank = 0;
      for (int e = 0; e < E; ++e) {
        const float o = s_l[e];
        rank += (o > mine) || (o == mine && e < lane);
      }
      s_order[rank] = lane;
      s_row[rank] = lane;
    }
    __syncwarp();
    const bf16* Yt = src.topk_idx ? Yall : Yall + (size_t)t * E * h;
    const float* ref = Fref ? Fref + (size_t)t * h : nullptr;
if (KT > 0) pair_errors_fast<(KT > 0 ? KT : 2), REF>(Yt, h, s_order, s_row, s_l, lane, s_err, ref);
    else pair_errors_generic(Yt, h, K, s_order, s_row, s_l, lane, s_err, ref);
    __syncwarp();
    for (int s = lane; s < nC; s += 32) {
      const uint32_t mask = subsets[s];
      int i = -1, j = -1;
      for (int q = 0; q < K; ++q) {  // the two best kept experts are always among the top K
        if ((mask >> s_order[q]) & 1u) {
          if (i < 0) i = q;
          else { j = q; break; }
        }
      }
      acc[s] += s_err[i * kMaxE + j];
    }
  }
  __syncthreads();
  for (int s = threadIdx.x; s < nC; s += blockDim.x) {
    float v = 0.f;
    for (int w = 0; w < nwarps; ++w) v += s_dyn[(size_t)w * nC + s];
    partial[(size_t)blockIdx.x * nC + s] = v;
  }
}

// One warp per subset: lane i adds blocks i, i+32, ... in order, then a fixed shuffle tree;
// the order depends only on the number of blocks, so the result is reproducible.
__global__ void __launch_bounds__(32)
reduce_partials_kernel(const float* __restrict__ partial, int nblk, int nC,
                       double* __restrict__ loss_sq, float* __restrict__ losses) {
  const int s = blockIdx.x;
  const int lane = threadIdx.x;
  double v = 0.0;
  for (int b = lane; b < nblk; b += 32) v += (double)partial[(size_t)b * nC + s];
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  if (lane == 0) {
    loss_sq[s] = v;
    losses[s] = (float)sqrt(v);
  }
}

int warps_for(int nC) { return nC <= 2048 ? 4 : 1; }

}  // namespace

int enumerate_num_blocks(int T, int nC) {
  const int per_block = warps_for(nC) * kTokPerWarp;
  int n = (T + per_block - 1) / per_block;
  if (n > kMaxBlocks) n = kMaxBlocks;
  if (n < 1) n = 1;
  return n;
}

cudaError_t launch_enumerate(const float* logits, const bf16* Yall, int T, int E, int r, int h,
                             const uint32_t* subsets, int nC, float* partial, double* loss_sq,
                             float* losses, const float* Fref, const EnumSource& src,
                             cudaStream_t st) {
  const int nw = warps_for(nC);
  const int nblk = enumerate_num_blocks(T, nC);
  const size_t smem = ((size_t)nw * nC + (size_t)nw * kMaxE * kMaxE + 3 * (size_t)nw * kMaxE) * 4;
  if (smem > 96 * 1024) return cudaErrorInvalidValue;
  const int K = E - r + 2;
  void (*kernel)(const float*, const bf16*, int, int, int, int, const uint32_t*, int, float*, const float*,
                 EnumSource) = nullptr;
#define MOE_ENUM_PICK(KK)                                                                   \
  case KK: kernel = Fref ? enumerate_kernel<KK, true> : enumerate_kernel<KK, false>; break
  switch (K) {
    MOE_ENUM_PICK(2);
    MOE_ENUM_PICK(3);
    MOE_ENUM_PICK(4);
    MOE_ENUM_PICK(5);
    MOE_ENUM_PICK(6);
    default: kernel = Fref ? enumerate_kernel<0, true> : enumerate_kernel<0, false>; break;
  }
#undef MOE_ENUM_PICK
  if (smem > 48 * 1024) {
    cudaError_t ea = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 96 * 1024);
    if (ea != cudaSuccess) return ea;
  }
  kernel<<<nblk, nw * 32, smem, st>>>(logits, Yall, T, E, r, h, subsets, nC, partial, Fref, src);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  reduce_partials_kernel<<<nC, 32, 0, st>>>(partial, nblk, nC, loss_sq, losses);
  return cudaGetLastError();
}

}  // namespace moe
