// Single-token forward (T = 1, batch-1 decoding): the expert FFNs as two matrix-vector kernels
// on the CUDA cores.  One token against one or two experts is no contraction worth a tensor
// core: every weight byte is used once, so the kernels only have to keep enough plain 16-byte
// loads in flight to saturate HBM.  They need no tensor-memory allocation, no pipeline set-up,
// no K-slices and no partial planes, and the second one finishes the layer (Eq. 2: the
// weighted sum over the token's experts, plus the optional residual), so a step is three
// launches: route_single_kernel, gemv_gate_up_kernel, gemv_down_combine_kernel.
//
// Rounding points are those of the GEMM path: fp32 accumulation, silu(g)*u rounded to bf16,
// expert outputs kept in fp32, the weighted sum rounded to bf16 once.
#include "common.h"

namespace moe {
namespace {

__device__ __forceinline__ float lo_f(uint32_t v) { return __uint_as_float(v << 16); }
__device__ __forceinline__ float hi_f(uint32_t v) { return __uint_as_float(v & 0xffff0000u); }

// acc += <8 bf16 of a, 8 bf16 of w>, ascending element order
__device__ __forceinline__ float dot8(const uint4& a, const uint4& w, float acc) {
  acc = fmaf(lo_f(a.x), lo_f(w.x), acc); acc = fmaf(hi_f(a.x), hi_f(w.x), acc);
  acc = fmaf(lo_f(a.y), lo_f(w.y), acc); acc = fmaf(hi_f(a.y), hi_f(w.y), acc);
  acc = fmaf(lo_f(a.z), lo_f(w.z), acc); acc = fmaf(hi_f(a.z), hi_f(w.z), acc);
  acc = fmaf(lo_f(a.w), lo_f(w.w), acc); acc = fmaf(hi_f(a.w), hi_f(w.w), acc);
  return acc;
}

// Weights are read once: streaming loads (evict-first) leave L2 to the token row, the
// activations and the routing record.
__device__ __forceinline__ uint4 ld_stream(const uint4* p) { return __ldcs(p); }

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int s = 16; s > 0; s >>= 1) v += __shfl_xor_sync(0xffffffffu, v, s);
  return v;
}

constexpr int kGuThreads = 512;  // two blocks per SM
constexpr int kDnThreads = 896;  // one block per SM (148 x 28 warps cover 4096 output rows in one go)

// The (at most two) experts of the token, as compact indices in ascending order, with the
// permuted row each of them reads and writes.
struct Active {
  int n, c0, c1, row0, row1;
};
__device__ __forceinline__ Active active_experts(const Meta* meta, int r) {
  Active a;
  a.n = 0;
  a.c0 = a.c1 = a.row0 = a.row1 = 0;
  for (int c = 0; c < r; ++c) {
    if (meta->count[c] > 0) {
      if (a.n == 0) { a.c0 = c; a.row0 = meta->off[c]; }
      if (a.n == 1) { a.c1 = c; a.row1 = meta->off[c]; }
      ++a.n;
    }
  }
  if (a.n > 2) a.n = 2;
  return a;
}

// act[row(c)][j] = bf16( silu(W1_c[j] . x) * (W3_c[j] . x) ) for the token's experts c.
// A warp takes one feature j at a time: the gate row and the up row of the interleaved
// weight matrix (16 KB), eight 16-byte loads per lane in flight.  Features are dealt
// round-robin to all warps of the grid.
__global__ void __launch_bounds__(kGuThreads, 2)
gemv_gate_up_kernel(const bf16* __restrict__ x, const bf16* __restrict__ W13,
                    const Meta* __restrict__ meta, int r, int h, int f, bf16* __restrict__ act) {
  extern __shared__ uint4 s_x[];  // the token row, h / 8 chunks of 8 bf16
  pdl_launch_dependents();
  pdl_wait();
  const int nvec = h >> 3;
  for (int v = threadIdx.x; v < nvec; v += kGuThreads) s_x[v] = __ldg(reinterpret_cast<const uint4*>(x) + v);
  const Active a = active_experts(meta, r);
  __syncthreads();
  const int lane = threadIdx.x & 31;
  const int nwarps = gridDim.x * (kGuThreads / 32);
  const int total = a.n * f;
  for (int task = blockIdx.x * (kGuThreads / 32) + (threadIdx.x >> 5); task < total; task += nwarps) {
    const int s = task >= f ? 1 : 0;
    const int j = task - s * f;
    const int q = j / kInterleave, i = j % kInterleave;
    const uint4* g = reinterpret_cast<const uint4*>(
        W13 + ((size_t)(s ? a.c1 : a.c0) * 2 * f + (size_t)2 * kInterleave * q + i) * h);
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
    if (lane == 0)
      act[(size_t)(s ? a.row1 : a.row0) * f + j] = __float2bfloat16_rn(ag / (1.0f + expf(-ag)) * au);
  }
}

// y[n] = bf16( w0 * (W2_e0[n] . act_e0) + w1 * (W2_e1[n] . act_e1) [+ residual[n]] ), slot 1
// left out when the second expert was skipped (Eq. 2 and the skipping rule of Sec. 3.3).
// A warp takes one output row n: 2f bytes of each expert's down matrix, eight loads per lane
// in flight; rows are dealt round-robin over the blocks so that every SM gets its share.
__global__ void __launch_bounds__(kDnThreads, 1)
gemv_down_combine_kernel(const bf16* __restrict__ act, const bf16* __restrict__ W2,
                         const Meta* __restrict__ meta, const int32_t* __restrict__ pair_pos,
                         const float* __restrict__ wn, const bf16* residual, int r, int h, int f,
                         bf16* __restrict__ y) {
  extern __shared__ uint4 s_act[];  // slot 0 then slot 1, f / 8 chunks each
  pdl_launch_dependents();
  pdl_wait();
  const int nvec = f >> 3;
  const int p0 = pair_pos[0], p1 = pair_pos[1];
  const float w0 = wn[0], w1 = wn[1];
  // the expert behind each slot: the group that starts at the slot's permuted row
  int c0 = 0, c1 = 0;
  for (int c = 0; c < r; ++c) {
    if (meta->count[c] > 0) {
      if (meta->off[c] == p0) c0 = c;
      if (meta->off[c] == p1) c1 = c;
    }
  }
  const int nslot = p1 >= 0 ? 2 : 1;
  for (int v = threadIdx.x; v < nslot * nvec; v += kDnThreads) {
    const int s = v >= nvec ? 1 : 0;
    s_act[v] = __ldg(reinterpret_cast<const uint4*>(act + (size_t)(s ? p1 : p0) * f) + (v - s * nvec));
  }
  __syncthreads();
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  for (int n = blockIdx.x + gridDim.x * warp; n < h; n += gridDim.x * (kDnThreads / 32)) {
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
      if (residual) z += __bfloat162float(residual[n]);
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

cudaError_t launch_gemv_gate_up(const bf16* x, const bf16* W13, const Meta* meta, int r, int h, int f,
                                bf16* act, cudaStream_t st) {
  const int sms = g_sms > 0 ? g_sms : 148;
  return launch_pdl(gemv_gate_up_kernel, dim3(2 * sms), dim3(kGuThreads), (size_t)h * 2, st, x, W13, meta,
                    r, h, f, act);
}

cudaError_t launch_gemv_down_combine(const bf16* act, const bf16* W2, const Meta* meta,
                                     const int32_t* pair_pos, const float* wn, const bf16* residual,
                                     int r, int h, int f, bf16* y, cudaStream_t st) {
  const int sms = g_sms > 0 ? g_sms : 148;
  return launch_pdl(gemv_down_combine_kernel, dim3(sms), dim3(kDnThreads), (size_t)4 * f, st, act, W2,
                    meta, pair_pos, wn, residual, r, h, f, y);
}

}  // namespace moe
