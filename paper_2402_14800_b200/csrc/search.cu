// Subset enumeration of the layer-wise pruning search (Sec. 3.2, Eq. 3).
//
// Input: router logits l[T][E] and Yall[t][e] = bf16(E_e(x_t)) for every token and expert.
// For a kept subset C the pruned layer routes token t to the two highest-ranked experts
// (by logit) that are in C, so per token only pairs of its top (E - r + 2) ranked experts can
// occur.  One warp per token computes the squared error of each such pair against the
// unpruned output once, then adds it to every subset that selects the pair.
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

// Squared errors of all pairs among the K top-ranked experts, pair accumulators in registers.
// `ref` (optional) is the token's target row F_ref[h] in fp32; without it the target is the
// unpruned output built from the two top-ranked experts.
template <int K>
__device__ __forceinline__ void pair_errors_fast(const bf16* __restrict__ Yt, int h,
                                                 const int* order, const int* rowoff,
                                                 const float* l, int lane,
                                                 float* s_err /* [16*16] */,
                                                 const float* __restrict__ ref) {
  constexpr int NP = K * (K - 1) / 2;
  float wa[NP], wb[NP], err[NP];
  {
    int p = 0;
#pragma unroll
    for (int i = 0; i < K; ++i)
#pragma unroll
      for (int j = i + 1; j < K; ++j, ++p) {
        pair_weights(l[order[i]], l[order[j]], wa[p], wb[p]);
        err[p] = 0.f;
      }
  }
  const uint4* rows[K];
#pragma unroll
  for (int i = 0; i < K; ++i) rows[i] = reinterpret_cast<const uint4*>(Yt + (size_t)rowoff[i] * h);
  for (int v = lane; v < (h >> 3); v += 32) {
    float y[K][8];
#pragma unroll
    for (int i = 0; i < K; ++i) unpack8f(__ldg(rows[i] + v), y[i]);
    float fr[8];
    if (ref) {
      const float4 r0 = __ldg(reinterpret_cast<const float4*>(ref) + 2 * v);
      const float4 r1 = __ldg(reinterpret_cast<const float4*>(ref) + 2 * v + 1);
      fr[0] = r0.x; fr[1] = r0.y; fr[2] = r0.z; fr[3] = r0.w;
      fr[4] = r1.x; fr[5] = r1.y; fr[6] = r1.z; fr[7] = r1.w;
    }
#pragma unroll
    for (int k = 0; k < 8; ++k) {
      const float F = ref ? fr[k] : fmaf(wb[0], y[1][k], wa[0] * y[0][k]);
      int p = 0;
#pragma unroll
      for (int i = 0; i < K; ++i)
#pragma unroll
        for (int j = i + 1; j < K; ++j, ++p) {
          const float d = fmaf(wb[p], y[j][k], wa[p] * y[i][k]) - F;
          err[p] = fmaf(d, d, err[p]);
        }
    }
  }
  int p = 0;
#pragma unroll
  for (int i = 0; i < K; ++i)
#pragma unroll
    for (int j = i + 1; j < K; ++j, ++p) {
      float e = err[p];
#pragma unroll
      for (int s = 16; s > 0; s >>= 1) e += __shfl_xor_sync(0xffffffffu, e, s);
      if (lane == 0) s_err[i * kMaxE + j] = e;
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
    switch (K) {
      case 2: pair_errors_fast<2>(Yt, h, s_order, s_row, s_l, lane, s_err, ref); break;
      case 3: pair_errors_fast<3>(Yt, h, s_order, s_row, s_l, lane, s_err, ref); break;
      case 4: pair_errors_fast<4>(Yt, h, s_order, s_row, s_l, lane, s_err, ref); break;
      case 5: pair_errors_fast<5>(Yt, h, s_order, s_row, s_l, lane, s_err, ref); break;
      case 6: pair_errors_fast<6>(Yt, h, s_order, s_row, s_l, lane, s_err, ref); break;
      default: pair_errors_generic(Yt, h, K, s_order, s_row, s_l, lane, s_err, ref); break;
    }
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
  static bool attr_set = false;
  if (!attr_set) {
    cudaError_t e = cudaFuncSetAttribute(enumerate_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         96 * 1024);
    if (e != cudaSuccess) return e;
    attr_set = true;
  }
  if (smem > 96 * 1024) return cudaErrorInvalidValue;
  enumerate_kernel<<<nblk, nw * 32, smem, st>>>(logits, Yall, T, E, r, h, subsets, nC, partial, Fref, src);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  reduce_partials_kernel<<<nC, 32, 0, st>>>(partial, nblk, nC, loss_sq, losses);
  return cudaGetLastError();
}

}  // namespace moe
