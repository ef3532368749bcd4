// Single-token forward (T = 1, batch-1 decoding): the whole layer as two kernels on the CUDA
// cores.  One token against one or two experts is no contraction worth a tensor core: every
// weight byte is used once, so the kernels only have to keep enough plain 16-byte loads in
// flight to saturate HBM.  They need no tensor-memory allocation, no pipeline set-up, no
// K-slices and no partial planes.
//
//   gemv_route_gate_up_kernel  every block routes the token itself (Sec. 3.1 logits over the kept
//                              experts, top-2, skip test of Sec. 3.3: the same few thousand
//                              multiply-adds in every block, in the same order, so all blocks
//                              agree), block 0 writes the routing record, then the blocks stream
//                              the gate and up rows of the token's experts.
//   gemv_down_combine_kernel   down projection of both experts and the weighted sum of Eq. 2
//                              (plus the optional residual), written to y.
//
// Rounding points are those of the GEMM path: fp32 accumulation, silu(g)*u rounded to bf16,
// expert outputs kept in fp32, the weighted sum rounded to bf16 once.
#include "common.h"
#include "route_device.cuh"

namespace moe {
namespace {

// acc += <8 bf16 of a, 8 bf16 of w>, ascending element order
__device__ __forceinline__ float dot8(const uint4& a, const uint4& w, float acc) {
  acc = fmaf(bf16_lo(a.x), bf16_lo(w.x), acc); acc = fmaf(bf16_hi(a.x), bf16_hi(w.x), acc);
  acc = fmaf(bf16_lo(a.y), bf16_lo(w.y), acc); acc = fmaf(bf16_hi(a.y), bf16_hi(w.y), acc);
  acc = fmaf(bf16_lo(a.z), bf16_lo(w.z), acc); acc = fmaf(bf16_hi(a.z), bf16_hi(w.z), acc);
  acc = fmaf(bf16_lo(a.w), bf16_lo(w.w), acc); acc = fmaf(bf16_hi(a.w), bf16_hi(w.w), acc);
  return acc;
}

// Weights are read once: streaming loads (evict-first) leave L2 to the token row, the
// activations and the routing record.
__device__ __forceinline__ uint4 ld_stream(const uint4* p) { return __ldcs(p); }

// Whatever an earlier kernel of the stream wrote (the token row, the activations, the routing
// record, the residual) is read with ld_l2 (see the rule beside launch_pdl).

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int s = 16; s > 0; s >>= 1) v += __shfl_xor_sync(0xffffffffu, v, s);
  return v;
}

constexpr int kGuThreads = 512;  // two blocks per SM
constexpr int kDnThreads = 896;  // one block per SM (148 x 28 warps cover 4096 output rows in one go)

// Routing of the token by every block, then act[slot][j] = bf16( silu(W1_e[j] . x) * (W3_e[j] . x) )
// for the experts e of slot 0 and, unless it was skipped, slot 1.
// Routing: thread v multiplies chunk v of the token row (8 values) with the same chunk of each
// kept router row; warp sums, then the warps' partial sums in ascending order.
// Streaming: a warp takes one feature j at a time, the gate row and the up row of the
// interleaved weight matrix (4h bytes), eight 16-byte loads per lane in flight; features are
// dealt round-robin to all warps of the grid.
struct SingleOut {
  RouteOut ro;
  Meta* meta;
  int32_t *pair_pos, *row_token, *s_count, *s_nskipped, *s_ntouched;
  int E;
};

template <int R>
__global__ void __launch_bounds__(kGuThreads, 2)
gemv_route_gate_up_kernel(const bf16* __restrict__ x, const bf16* __restrict__ Wg,
                          const bf16* __restrict__ W13, int r, int h, int f, float beta, KeptIds kept,
                          SingleOut out, bf16* __restrict__ act) {
  extern __shared__ uint4 s_x[];  // the token row, h / 8 chunks of 8 bf16
  __shared__ float s_part[kGuThreads / 32][R];
  pdl_launch_dependents();
  pdl_wait();
  const int nvec = h >> 3;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  float acc[R];
#pragma unroll
  for (int c = 0; c < R; ++c) acc[c] = 0.f;
  for (int v = threadIdx.x; v < nvec; v += kGuThreads) {
    const uint4 xv = ld_l2(reinterpret_cast<const uint4*>(x) + v);
    s_x[v] = xv;
    constexpr int G = R < 8 ? R : 8;  // router rows fetched together
#pragma unroll
    for (int cb = 0; cb < R; cb += G) {
      uint4 wv[G];
#pragma unroll
      for (int c = 0; c < G; ++c)
        if (cb + c < r) wv[c] = ld_l2(reinterpret_cast<const uint4*>(Wg + (size_t)(cb + c) * h) + v);
#pragma unroll
      for (int c = 0; c < G; ++c)
        if (cb + c < r) acc[cb + c] = dot8(xv, wv[c], acc[cb + c]);
    }
  }
#pragma unroll
  for (int c = 0; c < R; ++c) {
    acc[c] = warp_sum(acc[c]);
    if (lane == 0) s_part[warp][c] = acc[c];
  }
  __syncthreads();
  float l[R];
#pragma unroll
  for (int c = 0; c < R; ++c) {
    float v = 0.f;
#pragma unroll
    for (int w = 0; w < kGuThreads / 32; ++w) v += s_part[w][c];
    l[c] = v;
  }
  int e0, e1;
  bool skip;
  if (blockIdx.x == 0 && threadIdx.x == 0) {
    route_decide<R>(l, r, beta, 0, kept, out.ro, e0, e1, skip);
    int p0, p1;
    publish_single(e0, skip ? -1 : e1, 16, kept, out.meta, out.pair_pos, out.row_token, out.s_count,
                   out.s_nskipped, out.s_ntouched, out.E, p0, p1);
  } else {
    float w0, w1, p1;
    route_choose<R>(l, r, beta, e0, e1, skip, w0, w1, p1);
  }
  const int nwarps = gridDim.x * (kGuThreads / 32);
  const int total = (skip ? 1 : 2) * f;
  // a block takes 16 consecutive features at a time: contiguous gate rows and up rows
  for (int task = blockIdx.x * (kGuThreads / 32) + warp; task < total; task += nwarps) {
    const int s = task >= f ? 1 : 0;
    const int j = task - s * f;
    const int q = j / kInterleave, i = j % kInterleave;
    const uint4* g = reinterpret_cast<const uint4*>(
        W13 + ((size_t)(s ? e1 : e0) * 2 * f + (size_t)2 * kInterleave * q + i) * h);
    const uint4* u = g + (size_t)kInterleave * nvec;
    float ag = 0.f, au = 0.f;
    int v = lane;
    for (; v + 96 < nvec; v += 128) {
      uint4 wg[4], wu[4];
#pragma unroll
      for (int k = 0; k < 4; ++k) { wg[k] = ld_stream(g + v + 32 * k); wu[k] = ld_stream(u + v + 32 * k); }
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        const uint4 xv = s_x[v + 32 * k];
        ag = dot8(xv, wg[k], ag);
        au = dot8(xv, wu[k], au);
      }
    }
    for (; v < nvec; v += 32) {
      const uint4 xv = s_x[v];
      ag = dot8(xv, ld_stream(g + v), ag);
      au = dot8(xv, ld_stream(u + v), au);
    }
    ag = warp_sum(ag);
    au = warp_sum(au);
    if (lane == 0) act[(size_t)s * f + j] = __float2bfloat16_rn(ag / (1.0f + expf(-ag)) * au);
  }
}

// y[n] = bf16( w0 * (W2_e0[n] . act_e0) + w1 * (W2_e1[n] . act_e1) [+ residual[n]] ), slot 1
// left out when the second expert was skipped (Eq. 2 and the skipping rule of Sec. 3.3).
// A warp takes one output row n: 2f bytes of each expert's down matrix, eight loads per lane
// in flight; rows are dealt round-robin over the blocks so that every SM gets its share.
__global__ void __launch_bounds__(kDnThreads, 1)
gemv_down_combine_kernel(const bf16* __restrict__ act, const bf16* __restrict__ W2,
                         const int32_t* __restrict__ idx, const uint8_t* __restrict__ skipped,
                         const float* __restrict__ wn, const bf16* residual, int h, int f,
                         bf16* __restrict__ y) {
  extern __shared__ uint4 s_act[];  // slot 0 then slot 1, f / 8 chunks each
  pdl_launch_dependents();
  pdl_wait();
  const int nvec = f >> 3;
  const int c0 = ld_l2(idx), c1 = ld_l2(idx + 1);  // compact expert indices of the two slots
  const float w0 = ld_l2(wn), w1 = ld_l2(wn + 1);
  const int nslot = ld_l2(skipped) ? 1 : 2;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int n_first = blockIdx.x + gridDim.x * warp;
  for (int v = threadIdx.x; v < nslot * nvec; v += kDnThreads)
    s_act[v] = ld_l2(reinterpret_cast<const uint4*>(act) + v);
  __syncthreads();
  for (int n = n_first; n < h; n += gridDim.x * (kDnThreads / 32)) {
    float o0 = 0.f, o1 = 0.f;
    for (int s = 0; s < nslot; ++s) {
      const uint4* w = reinterpret_cast<const uint4*>(W2 + ((size_t)(s ? c1 : c0) * h + n) * f);
      const uint4* av = s_act + s * nvec;
      float acc = 0.f;
      int v = lane;
      for (; v + 224 < nvec; v += 256) {
        uint4 wv[8];
#pragma unroll
        for (int k = 0; k < 8; ++k) wv[k] = ld_stream(w + v + 32 * k);
#pragma unroll
        for (int k = 0; k < 8; ++k) acc = dot8(av[v + 32 * k], wv[k], acc);
      }
      for (; v < nvec; v += 32) acc = dot8(av[v], ld_stream(w + v), acc);
      acc = warp_sum(acc);
      if (s) o1 = acc; else o0 = acc;
    }
    if (lane == 0) {
      float z = (nslot == 2) ? fmaf(w1, o1, w0 * o0) : w0 * o0;
      if (residual) z += ld_l2(residual + n);
      y[n] = __float2bfloat16_rn(z);
    }
  }
}

int g_sms = 0;                             // SMs of the device the kernels were set up on
constexpr size_t kDnMaxSmem = 200 * 1024;  // two activation rows: f <= 51200

}  // namespace

// Once per process, with the device current, before the first launch (moe_layer_create).
cudaError_t gemv_single_setup() {
  if (g_sms > 0) return cudaSuccess;
  cudaError_t e = cudaFuncSetAttribute(gemv_down_combine_kernel,
                                       cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kDnMaxSmem);
  if (e != cudaSuccess) return e;
  int dev = 0;
  if ((e = cudaGetDevice(&dev)) != cudaSuccess) return e;
  return cudaDeviceGetAttribute(&g_sms, cudaDevAttrMultiProcessorCount, dev);
}

// Shapes whose token row and two activation rows fit the kernels' shared memory.
bool gemv_single_fits(int h, int f) { return (size_t)h * 2 <= 48 * 1024 && (size_t)4 * f <= kDnMaxSmem; }

cudaError_t launch_gemv_route_gate_up(const bf16* x, const bf16* Wg, const bf16* W13, int r, int h, int f,
                                      float beta, const KeptIds& kept, const RouteOut& ro, Meta* meta,
                                      int32_t* pair_pos, int32_t* row_token, int32_t* s_count,
                                      int32_t* s_nskipped, int32_t* s_ntouched, int E, bf16* act,
                                      cudaStream_t st) {
  const int sms = g_sms > 0 ? g_sms : 148;
  SingleOut out;
  out.ro = ro; out.meta = meta; out.pair_pos = pair_pos; out.row_token = row_token;
  out.s_count = s_count; out.s_nskipped = s_nskipped; out.s_ntouched = s_ntouched; out.E = E;
#define MOE_GEMV_ROUTE(R)                                                                            \
  return launch_pdl(gemv_route_gate_up_kernel<R>, dim3(2 * sms), dim3(kGuThreads), (size_t)h * 2, st, x, \
                    Wg, W13, r, h, f, beta, kept, out, act)
  switch (r) {
    case 2: MOE_GEMV_ROUTE(2);
    case 3: case 4: MOE_GEMV_ROUTE(4);
    case 5: case 6: MOE_GEMV_ROUTE(6);
    case 7: case 8: MOE_GEMV_ROUTE(8);
    default: MOE_GEMV_ROUTE(kMaxE);
  }
#undef MOE_GEMV_ROUTE
}

cudaError_t launch_gemv_down_combine(const bf16* act, const bf16* W2, const int32_t* idx,
                                     const uint8_t* skipped, const float* wn, const bf16* residual,
                                     int h, int f, bf16* y, cudaStream_t st) {
  const int sms = g_sms > 0 ? g_sms : 148;
  return launch_pdl(gemv_down_combine_kernel, dim3(sms), dim3(kDnThreads), (size_t)4 * f, st, act, W2,
                    idx, skipped, wn, residual, h, f, y);
}

}  // namespace moe
