// Grouped GEMMs of the SwiGLU experts on the 5th-generation tensor cores (tcgen05),
// operands staged in shared memory by TMA, accumulators in tensor memory.
//
//   E_e(x) = W2_e ( silu(W1_e x) * (W3_e x) )      (Sec. 3.1; Mixtral's SwiGLU form)
//
// Three persistent, warp-specialised kernels share one pipeline skeleton:
//   gemm_tokens_m   256 token rows x 256 weight rows per item on two accumulators; for large
//                   batches, where the work is a dense contraction bound by the tensor pipe.
//   gemm_weights_m  128 weight rows x (16..128) tokens per item; for small batches, where
//                   every weight byte is streamed from HBM exactly once.
//   gemm_tokens_d   up to 128 token rows x 256 weight rows per item; small batches with many
//                   tokens per expert (twice the weight bytes per trip round the MMA loop).
// Warp 0 issues TMA loads, warp 1 issues the MMAs (one lane) and owns the tensor memory, the
// other warps run the epilogue out of tensor memory (in the small-batch kernels while the next
// item accumulates in the other half of it).
//
// W1/W3 are stored interleaved (16 gate rows, 16 up rows, ...) so that one accumulator tile
// holds both halves of a SwiGLU feature and the epilogue can fuse silu(g) * u.
//
// Every wait on an mbarrier is bounded: when it expires the CTA raises its abort flag, all
// roles leave their loops, outstanding copies and MMAs are drained (again bounded), tensor
// memory is released and the device status word is set.
#include <stdio.h>

#include "common.h"
#include "route_device.cuh"

namespace moe {

namespace {

constexpr int BK = 64;            // k elements per pipeline stage = one 128-byte swizzle span
constexpr int UMMA_K = 16;        // k elements per tcgen05.mma (bf16)
constexpr int kBand = 16;         // row tiles that sweep the weight tiles together (L2 reuse)
constexpr unsigned long long kWaitLimitNs = 4000000000ull;
constexpr unsigned long long kDrainLimitNs = 2000000ull;

constexpr int kThreads = 192;

// ------------------------------------------------------------------------------ PTX glue

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ unsigned long long gtimer() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes)
               : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n"
      " .reg .pred p;\n"
      " mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n"
      " selp.u32 %0, 1, 0, p;\n"
      "}\n"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded wait.  Returns false when the CTA is aborting (this wait or another one expired).
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag,
                                          unsigned long long limit_ns = kWaitLimitNs) {
  if (mbar_try_wait(bar, parity)) return true;
  const unsigned long long t0 = gtimer();
  unsigned spins = 0;
  while (!mbar_try_wait(bar, parity)) {
    if ((++spins & 0xffu) == 0) {
      if (*abort_flag) return false;
      if (gtimer() - t0 > limit_ns) {
        *abort_flag = 1;
        return false;
      }
    }
  }
  return true;
}
__device__ __forceinline__ void fence_barrier_init() {
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void fence_proxy_async() {
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int c0, int c1,
                                            uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes"
      " [%0], [%1, {%2, %3}], [%4];"
      ::"r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(bar)
      : "memory");
}
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* map, int c0, int c1,
                                            int c2, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes"
      " [%0], [%1, {%2, %3, %4}], [%5];"
      ::"r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(c2), "r"(bar)
      : "memory");
}
// the same with an L2 eviction policy (weights that are read exactly once)
__device__ __forceinline__ uint64_t l2_policy_evict_first() {
  uint64_t p;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(p));
  return p;
}
__device__ __forceinline__ void tma_load_3d_hint(uint32_t dst, const CUtensorMap* map, int c0, int c1,
                                                 int c2, uint32_t bar, uint64_t policy) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint"
      " [%0], [%1, {%2, %3, %4}], [%5], %6;"
      ::"r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(c2), "r"(bar), "l"(policy)
      : "memory");
}
__device__ __forceinline__ void tmem_alloc(uint32_t smem_dst, uint32_t ncols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_dst),
               "r"(ncols)
               : "memory");
}
__device__ __forceinline__ void tmem_relinquish() {
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols)
               : "memory");
}
__device__ __forceinline__ void tc_fence_before() {
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
}
__device__ __forceinline__ void tc_fence_after() {
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar)
               : "memory");
}
// D[tmem] (+)= A[smem] * B[smem]^T, bf16 inputs, fp32 accumulation
__device__ __forceinline__ void umma_bf16(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc,
                                          uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n"
      " .reg .pred p;\n"
      " setp.ne.b32 p, %4, 0;\n"
      " tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n"
      "}\n"
      ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
      : "memory");
}
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t* v) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]),
        "=r"(v[7]), "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]),
        "=r"(v[14]), "=r"(v[15]), "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]),
        "=r"(v[21]), "=r"(v[22]), "=r"(v[23]), "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]),
        "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t* v) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
      : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]),
        "=r"(v[7]), "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]),
        "=r"(v[14]), "=r"(v[15])
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() {
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

// Shared-memory matrix descriptor of a K-major bf16 tile whose rows are 128 bytes (64
// elements), written by TMA with the 128-byte swizzle: 8-row groups are 1024 bytes apart.
__device__ __forceinline__ uint64_t smem_desc_k128(uint32_t saddr) {
  uint64_t d = 0;
  d |= (uint64_t)((saddr & 0x3ffffu) >> 4);  // start address / 16
  d |= (uint64_t)1 << 16;                    // leading byte offset / 16 (unused with swizzle)
  d |= (uint64_t)(1024 >> 4) << 32;          // stride byte offset / 16
  d |= (uint64_t)1 << 46;                    // descriptor version of sm_100
  d |= (uint64_t)2 << 61;                    // 128-byte swizzle
  return d;
}
// Instruction descriptor: bf16 x bf16 -> fp32, both operands K-major, M x N tile.
__device__ __forceinline__ uint32_t idesc_bf16(int M, int N) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(N >> 3) << 17) |
         ((uint32_t)(M >> 4) << 24);
}

__device__ __forceinline__ float silu_mul(float g, float u) {
  return g / (1.0f + __expf(-g)) * u;
}
__device__ __forceinline__ uint32_t pack_bf16(float a, float b) {
  __nv_bfloat162 p = __floats2bfloat162_rn(a, b);
  return *reinterpret_cast<uint32_t*>(&p);
}

struct Bars {
  unsigned long long full[8];
  unsigned long long empty[8];
  unsigned long long tmem_full[2];
  unsigned long long tmem_empty[2];
  unsigned long long drain;
  uint32_t tmem_base;
  int abort_flag;
};

template <int NS>
__device__ __forceinline__ void setup_barriers(Bars& b, uint32_t tmem_empty_arrivals = 4) {
  if (threadIdx.x == 0) {
    for (int s = 0; s < NS; ++s) {
      mbar_init(smem_u32(&b.full[s]), 1);
      mbar_init(smem_u32(&b.empty[s]), 1);
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(smem_u32(&b.tmem_full[i]), 1);
      mbar_init(smem_u32(&b.tmem_empty[i]), tmem_empty_arrivals);
    }
    mbar_init(smem_u32(&b.drain), 1);
    b.abort_flag = 0;
    fence_barrier_init();
    fence_proxy_async();
  }
}

// Common tail: after an abort, wait (bounded) for loads and MMAs that are still in flight,
// report, and release tensor memory.
template <int TMEM_COLS>
__device__ __forceinline__ void teardown(Bars& b, uint32_t tmem_base, uint32_t issued, uint32_t NS,
                                         int* status) {
  tc_fence_before();
  __syncthreads();
  const int aborted = *(volatile int*)&b.abort_flag;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (aborted) {
    if (warp == 0 && lane == 0) {
      // the last min(issued, NS) stages may still have a load in flight
      int dummy = 0;
      const uint32_t n = issued < NS ? issued : NS;
      for (uint32_t i = 0; i < n; ++i) {
        const uint32_t it = issued - 1 - i;
        mbar_wait(smem_u32(&b.full[it % NS]), (it / NS) & 1u, &dummy, kDrainLimitNs);
      }
      if (status) atomicExch(status, 1);
    }
    if (warp == 1 && lane == 0) {
      int dummy = 0;
      umma_commit(smem_u32(&b.drain));
      mbar_wait(smem_u32(&b.drain), 0, &dummy, kDrainLimitNs);
    }
    __syncthreads();
  }
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, TMEM_COLS);
  }
}

// ------------------------------------------------------------------------ gemm_tokens_m
//
// Large batches.  One CTA computes 256 token rows x 256 weight rows per item: per k-block of 64
// it stages two 128-row token tiles and one 256-row weight tile (64 KB) and issues eight MMAs,
// four into each of two accumulators that together fill all 512 tensor-memory columns.  What
// bounds this kernel is the traffic from L2 to shared memory and its latency (measured: with 2 /
// 3 / 4 stages of a 128 x 256 tile the tensor pipe was busy in proportion to the stages, and an
// L2 prefetch stream made it slower), so the tile is as large as tensor memory allows: a
// 256 x 256 tile moves 2/3 of the bytes of a 128 x 256 tile per FLOP, and three stages of it
// cover 3 x 1024 pipe cycles of latency instead of 4 x 512.  The price is that the accumulators
// are not double-buffered: the MMAs of the next item wait until the epilogue warps have read the
// previous item out of tensor memory, which is why there are many epilogue warps (each reads
// 32 lanes x 128 or 64 columns) and why accumulator 0 is released before accumulator 1.
// An item whose second 128 rows are all padding (an expert group's odd last row tile) runs as
// a half item: no second token tile, no MMAs into accumulator 1.

struct TileM {
  int c, nt, a_row, out_row, rows_valid;  // rows_valid in 1 .. 256
};

constexpr int TM_NS = 3;
constexpr int TM_A_HALF = 128 * 128;        // 128 token rows x 64 bf16
constexpr int TM_A_BYTES = 2 * TM_A_HALF;   // two token tiles
constexpr int TM_B_BYTES = 256 * 128;       // 256 weight rows x 64 bf16
constexpr int TM_STAGE = TM_A_BYTES + TM_B_BYTES;
constexpr int TM_SMEM = TM_NS * TM_STAGE + 1024;
constexpr int TM_BN = 256;
// Epilogue warps per CTA: 2 accumulators x 4 tensor-memory lane quarters x 1 or 2 column halves.
// The SwiGLU epilogue (an exponential and a division per output) is the long one and, with the
// accumulators single-buffered, sits on the critical path between two items: 16 warps (gate/up
// launch 11.3 vs 12.2 ms at 32768 tokens).  The plain copies of the down projection were
// 4 % faster with 8 (5.48 vs 5.72 ms): its items are 3.5 times as long, and fewer warps wait.
template <bool GATE_UP> struct TmCfg {
  static constexpr int kEpiWarps = GATE_UP ? 16 : 8;
  static constexpr int kThreads = 64 + 32 * kEpiWarps;
};

// An item covers `unit` row tiles of 128 (2 normally; 1 for launches with too few items to fill
// the machine with double row tiles: the kernel decides, see below).  Items of expert c:
// ceil(row tiles / unit) x Nt weight tiles, ordered band of kBand / unit row items -> weight
// tile -> row item, so that the items in flight share few token tiles and weight tiles in L2.
__device__ __forceinline__ void decode_tile_m(const Meta& m, const GemmArgs& a, int item, int Nt,
                                              int unit, TileM& t) {
  int c = 0, first = 0;
  for (;;) {
    const int mtu = (m.tile_prefix[c + 1] - m.tile_prefix[c] + unit - 1) / unit;
    if (c + 1 >= a.r || item < first + mtu * Nt) break;
    first += mtu * Nt;
    ++c;
  }
  const int local = item - first;
  const int Mtu = (m.tile_prefix[c + 1] - m.tile_prefix[c] + unit - 1) / unit;
  const int band_items = kBand / unit;
  const int band = local / (band_items * Nt);
  const int rem = local - band * band_items * Nt;
  const int band_rows = min(band_items, Mtu - band * band_items);
  t.nt = rem / band_rows;
  const int mt = band * band_items + rem - t.nt * band_rows;
  const int rows = unit * kTileRows;
  t.c = c;
  t.a_row = a.a_row_base + a.a_off_mul * m.off[c] + rows * mt;
  t.out_row = a.out_row_base + a.out_off_mul * m.off[c] + rows * mt;
  t.rows_valid = min(rows, m.count[c] - rows * mt);
}

__device__ __forceinline__ int num_items_m(const Meta& m, const GemmArgs& a, int Nt, int unit) {
  int n = 0;
  for (int c = 0; c < a.r; ++c) n += ((m.tile_prefix[c + 1] - m.tile_prefix[c] + unit - 1) / unit) * Nt;
  return n;
}

// Epilogue of 128 accumulator rows x columns [32 j0, 32 j1) of one accumulator: this thread owns
// tensor-memory lane `row` (one token row) and walks the columns in chunks of 32.
template <bool GATE_UP, int OUT>
__device__ __forceinline__ void store_tile_tokens_m(uint32_t taddr, const GemmArgs& args, int nt, int c,
                                                    int out_row, int rows_valid, int row, int j0, int j1) {
  const bool row_ok = row < rows_valid;
  const long long orow = (long long)(out_row + row) * args.out_ld + (long long)c * args.out_col_mul;
#pragma unroll 1
  for (int j = j0; j < j1; ++j) {
    const int col0 = nt * TM_BN + 32 * j;  // first weight row of this chunk
    if (col0 >= args.n_w_rows) break;        // warp-uniform
    uint32_t v[32];
    tmem_ld32(taddr + 32 * j, v);
    tmem_ld_wait();
    if (GATE_UP) {
      // chunk = 16 gate rows then 16 up rows of the features col0/2 .. col0/2 + 15
      uint32_t o[8];
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        const float a0 = silu_mul(__uint_as_float(v[2 * i]), __uint_as_float(v[16 + 2 * i]));
        const float a1 = silu_mul(__uint_as_float(v[2 * i + 1]), __uint_as_float(v[17 + 2 * i]));
        o[i] = pack_bf16(a0, a1);
      }
      if (row_ok) {
        uint4* dst = reinterpret_cast<uint4*>(reinterpret_cast<bf16*>(args.out) + orow + (col0 >> 1));
        dst[0] = make_uint4(o[0], o[1], o[2], o[3]);
        dst[1] = make_uint4(o[4], o[5], o[6], o[7]);
      }
    } else if (OUT == kOutF32) {
      if (row_ok) {
        float4* dst = reinterpret_cast<float4*>(reinterpret_cast<float*>(args.out) + orow + col0);
#pragma unroll
        for (int i = 0; i < 8; ++i)
          dst[i] = make_float4(__uint_as_float(v[4 * i]), __uint_as_float(v[4 * i + 1]),
                               __uint_as_float(v[4 * i + 2]), __uint_as_float(v[4 * i + 3]));
      }
    } else {
      if (row_ok) {
        uint4* dst = reinterpret_cast<uint4*>(reinterpret_cast<bf16*>(args.out) + orow + col0);
#pragma unroll
        for (int i = 0; i < 4; ++i)
          dst[i] = make_uint4(
              pack_bf16(__uint_as_float(v[8 * i]), __uint_as_float(v[8 * i + 1])),
              pack_bf16(__uint_as_float(v[8 * i + 2]), __uint_as_float(v[8 * i + 3])),
              pack_bf16(__uint_as_float(v[8 * i + 4]), __uint_as_float(v[8 * i + 5])),
              pack_bf16(__uint_as_float(v[8 * i + 6]), __uint_as_float(v[8 * i + 7])));
      }
    }
  }
}

template <bool GATE_UP, int OUT>
__global__ void __launch_bounds__(TmCfg<GATE_UP>::kThreads, 1)
gemm_tokens_m_kernel(const __grid_constant__ GemmMaps maps, const GemmArgs args) {
  extern __shared__ uint8_t smem_raw[];
  __shared__ Bars bars;
  __shared__ Meta s_meta;
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  // tmem_empty[a]: one arrival per epilogue warp of accumulator a
  constexpr int TM_EPI_WARPS = TmCfg<GATE_UP>::kEpiWarps;
  setup_barriers<4>(bars, TM_EPI_WARPS / 2);
  if (warp == 1) {
    tmem_alloc(smem_u32(&bars.tmem_base), 512);
    tmem_relinquish();
  }
  // everything above is independent of the preceding kernels; their results are read from here on
  pdl_wait();
  for (int i = threadIdx.x; i < (int)(sizeof(Meta) / 4); i += blockDim.x)
    reinterpret_cast<int32_t*>(&s_meta)[i] = ld_l2(reinterpret_cast<const int32_t*>(args.meta) + i);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *(volatile uint32_t*)&bars.tmem_base;
  volatile int* abort_flag = &bars.abort_flag;

  const int KB = (args.K + BK - 1) / BK;
  const int Nt = (args.n_w_rows + TM_BN - 1) / TM_BN;
  // Items of 256 token rows move a third fewer bytes per FLOP, but a launch needs enough of them:
  // an item of one row tile (4 stages of 48 KB: one token tile + the weight tile; every item a
  // half item, the accumulators alternate, which double-buffers them) takes about 0.58 of a
  // double-row item's time, and the last, partly filled round of a launch costs a whole item.
  // Every CTA compares the rounds of both forms from the real group sizes (2048 tokens, down
  // projection: 3 rounds of double-row items 0.55 ms, 4 rounds of single-row items 0.50 ms;
  // 3072 tokens: 3 rounds 0.60 ms against 6 rounds 0.72 ms).
  const int grid = (int)gridDim.x;
  const int rounds1 = (num_items_m(s_meta, args, Nt, 1) + grid - 1) / grid;
  const int rounds2 = (num_items_m(s_meta, args, Nt, 2) + grid - 1) / grid;
  const bool single = 58 * rounds1 < 100 * rounds2;
  const int unit = single ? 1 : 2;
  const uint32_t ns = single ? 4u : (uint32_t)TM_NS;
  const uint32_t stage_bytes = single ? (uint32_t)(TM_A_HALF + TM_B_BYTES) : (uint32_t)TM_STAGE;
  const uint32_t b_off = single ? (uint32_t)TM_A_HALF : (uint32_t)TM_A_BYTES;
  const int n_items = num_items_m(s_meta, args, Nt, unit);
  uint32_t issued = 0;

  if (warp == 0) {
    // ---- TMA producer
    uint32_t it = 0, s = 0, ph = 0;
    bool ok = true;
    for (int item = blockIdx.x; item < n_items && ok; item += gridDim.x) {
      TileM t;
      decode_tile_m(s_meta, args, item, Nt, unit, t);
      const bool full_item = t.rows_valid > kTileRows;
      const uint32_t bytes = TM_B_BYTES + (full_item ? TM_A_BYTES : TM_A_HALF);
      for (int kb = 0; kb < KB; ++kb, ++it) {
        ok = __all_sync(0xffffffffu, mbar_wait(smem_u32(&bars.empty[s]), ph ^ 1u, abort_flag));
        if (!ok) break;
        if (lane == 0) {
          const uint32_t full = smem_u32(&bars.full[s]);
          const uint32_t sa = smem_base + s * stage_bytes;
          mbar_expect_tx(full, bytes);
          tma_load_2d(sa, &maps.t[3], kb * BK, t.a_row, full);
          tma_load_3d(sa + b_off, &maps.w, kb * BK, t.nt * TM_BN, t.c, full);
          if (full_item) tma_load_2d(sa + TM_A_HALF, &maps.t[3], kb * BK, t.a_row + kTileRows, full);
        }
        if (++s == ns) { s = 0; ph ^= 1u; }
        __syncwarp();
      }
    }
    issued = it;
  } else if (warp == 1) {
    // ---- MMA issuer.  A full item uses both accumulators (rows 0-127 in accumulator 0, rows
    // 128-255 in accumulator 1); half items take the accumulators in turn.  n0 / n1 count the
    // uses of each accumulator, nh the half items; the epilogue warps count the same way.
    // The loop of this warp, not the tensor pipe, sets the pace whenever it spends more than about
    // one MMA's time between two MMAs (the pipe queues little beyond the MMA it executes), so the
    // body of a k-block is kept short, and the commit that releases a stage is issued after the
    // first MMA of the NEXT k-block instead of between two k-blocks, where it would sit next to
    // the wait for the next stage's data.  A commit covers every MMA issued before it, so the
    // stage is released slightly later than it could be, never earlier.  (Measured side by side:
    // the deferred commit 5 % faster; the loop run by one lane with the others parked, or the wait
    // for the next stage moved between the MMAs as well, each 4-7 % slower.)
    const uint32_t idesc = idesc_bf16(128, TM_BN);
    uint32_t s = 0, ph = 0, n0 = 0, n1 = 0, nh = 0;
    uint32_t owed_bar = 0;  // empty barrier of the stage whose release is still to be committed
    bool ok = true;
    for (int item = blockIdx.x; item < n_items && ok; item += gridDim.x) {
      TileM t;
      decode_tile_m(s_meta, args, item, Nt, unit, t);
      const bool full_item = t.rows_valid > kTileRows;
      const uint32_t a0 = full_item ? 0u : (nh & 1u);  // accumulator of the first (or only) 128 rows
      const uint32_t d0 = tmem_base + a0 * TM_BN;
      for (int kb = 0; kb < KB; ++kb) {
        bool ready = mbar_wait(smem_u32(&bars.full[s]), ph, abort_flag);
        // the accumulators must have been read out of tensor memory before they are overwritten
        if (kb == 0) {
          ready = ready && mbar_wait(smem_u32(&bars.tmem_empty[a0]), ((a0 ? n1 : n0) & 1u) ^ 1u, abort_flag);
          if (full_item) ready = ready && mbar_wait(smem_u32(&bars.tmem_empty[1]), (n1 & 1u) ^ 1u, abort_flag);
        }
        ok = __all_sync(0xffffffffu, ready);
        if (!ok) break;
        tc_fence_after();
        if (lane == 0) {
          const uint32_t sa = smem_base + s * stage_bytes;
          const uint64_t bdesc = smem_desc_k128(sa + b_off);
          const uint64_t adesc0 = smem_desc_k128(sa);
          const uint32_t acc_flag = kb > 0 ? 1u : 0u;
          umma_bf16(d0, adesc0, bdesc, idesc, acc_flag);
          if (owed_bar) umma_commit(owed_bar);
          umma_bf16(d0, adesc0 + 2, bdesc + 2, idesc, 1u);
          umma_bf16(d0, adesc0 + 4, bdesc + 4, idesc, 1u);
          umma_bf16(d0, adesc0 + 6, bdesc + 6, idesc, 1u);
          if (kb == KB - 1) umma_commit(smem_u32(&bars.tmem_full[a0]));  // these rows can be read already
          if (full_item) {
            const uint64_t adesc1 = smem_desc_k128(sa + TM_A_HALF);
            umma_bf16(tmem_base + TM_BN, adesc1, bdesc, idesc, acc_flag);
            umma_bf16(tmem_base + TM_BN, adesc1 + 2, bdesc + 2, idesc, 1u);
            umma_bf16(tmem_base + TM_BN, adesc1 + 4, bdesc + 4, idesc, 1u);
            umma_bf16(tmem_base + TM_BN, adesc1 + 6, bdesc + 6, idesc, 1u);
            if (kb == KB - 1) umma_commit(smem_u32(&bars.tmem_full[1]));
          }
        }
        owed_bar = smem_u32(&bars.empty[s]);
        if (++s == ns) { s = 0; ph ^= 1u; }
        __syncwarp();
      }
      if (full_item) { ++n0; ++n1; }
      else { if (a0) ++n1; else ++n0; ++nh; }
    }
    if (ok && owed_bar && lane == 0) umma_commit(owed_bar);
    __syncwarp();
  } else {
    // ---- epilogue: warp w may touch tensor-memory lanes 32 (w % 4) .. + 31.  The first half of
    // the epilogue warps reads accumulator 0, the second half accumulator 1; where an accumulator
    // has eight warps, the first four take the first 128 columns and the other four the rest.
    const int e = warp - 2;
    const uint32_t acc = (uint32_t)(e / (TM_EPI_WARPS / 2));
    const int half = (e / 4) % (TM_EPI_WARPS / 8);   // which share of the 8 column chunks
    constexpr int kChunks = 64 / TM_EPI_WARPS;        // 32-column chunks per warp (4 or 8)
    const int wq = warp & 3;
    const int row = 32 * wq + lane;
    uint32_t n = 0, nh = 0;  // uses of this warp's accumulator so far; half items so far
    bool ok = true;
    for (int item = blockIdx.x; item < n_items && ok; item += gridDim.x) {
      TileM t;
      decode_tile_m(s_meta, args, item, Nt, unit, t);
      const bool full_item = t.rows_valid > kTileRows;
      int row_half = (int)acc;  // a full item: accumulator a holds rows 128 a ..
      if (!full_item) {
        const uint32_t a0 = nh & 1u;
        ++nh;
        if (a0 != acc) continue;  // the other accumulator's item
        row_half = 0;
      }
      ok = __all_sync(0xffffffffu, mbar_wait(smem_u32(&bars.tmem_full[acc]), n & 1u, abort_flag));
      if (!ok) break;
      ++n;
      tc_fence_after();
      const uint32_t taddr = tmem_base + ((uint32_t)(32 * wq) << 16) + acc * TM_BN;
      store_tile_tokens_m<GATE_UP, OUT>(taddr, args, t.nt, t.c, t.out_row + row_half * kTileRows,
                                        t.rows_valid - row_half * kTileRows, row, kChunks * half,
                                        kChunks * (half + 1));
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&bars.tmem_empty[acc]));
    }
  }
  // the dependents may be scheduled once every CTA is this far: a grid that waits on an SM for the
  // whole run of this kernel costs issue slots and power
  pdl_launch_dependents();
  teardown<512>(bars, tmem_base, issued, ns, args.status);
}

// ----------------------------------------------------------------------- gemm_weights_m

// A pipeline stage holds two k-blocks (one barrier wait and one commit per 32 KB of weights: the
// loop of the MMA-issuing warp, not memory, bounds this kernel):
//   [weights kb][weights kb+1][tokens kb][tokens kb+1], token slots of TOK rows.
// TOK = 64 (batches of at most 64 tokens): 4 stages of 48 KB; TOK = 128: 3 stages of 64 KB.
// (Smaller slots with more stages were measured: 5 x 40 KB equal, 6 x 36 KB 4-5 % slower.)
constexpr int WM_A_BYTES = 128 * 128;  // 128 weight rows x 64 bf16
template <int TOK> struct WmCfg {
  static constexpr int kTokBytes = TOK * 128;
  static constexpr int kStage = 2 * (WM_A_BYTES + kTokBytes);
  static constexpr int kNS = TOK <= 64 ? 4 : 3;
  static constexpr int kSmem = kNS * kStage + 1024;
};
constexpr int WM_BN = 128;

struct ItemW {
  int c, mt, ks, tok_row, out_row, cnt, bucket, kb0, kb1;
  int tail_slot;  // >= 0: this is one K-slice of a tail item and goes to the tail buffer
  int tail_item;  // which tail item the slice belongs to
  int nslice;     // non-empty K-slices of that tail item
};

// Work list of the weight-major kernel.  The base items (expert row tile x weight tile x
// k-chunk) are dealt round-robin to the `grid` CTAs.  The `rem` items left over after the full
// rounds would keep part of the machine busy for a whole item's time, so they are cut into
// `KSt` K-slices each.  The slices come FIRST in the work list and are dealt like items; each
// leaves an fp32 partial tile in the tail buffer, and the slice of an item that finishes last
// adds the partial tiles up in slice order and writes the regular output (the order of arrival
// does not change the result).  That happens while the CTAs are busy with their regular items,
// off the critical path, and the last round of the launch is a full one.
// KSt minimises the modelled time of the slices, rounds x (k-blocks per slice + kSliceFixedKb),
// among the values whose slices fit the tail buffer and whose fold stays below kFoldLoads loads
// per thread; KSt = 1 (no slicing) competes too.
struct SchedW {
  int Mt, KS, KB, kb_per_item;
  int n_base, full, rem, KSt, kbs, n_slices, n_total;
  int slot_floats;  // floats between the partial tiles of two slices
};

constexpr int kMinSliceKb = 4;                     // a slice covers at least this many k-blocks
constexpr int kSliceFixedKb = 6;                   // modelled fixed cost of a slice, in k-blocks
constexpr int kFoldLoads = 512;                    // tokens x slices one thread adds up at most
constexpr int kTailHeaderFloats = (int)(kTailHeaderBytes / 4);  // arrival counters come first

// Warp-collective: all 32 lanes of a converged warp call it and get the same result.
// tile_w = weight rows of an item (128 weight-major, 256 token-major); a partial tile holds
// tile_w floats per token; kst_cap bounds the slices by what the fold may load per thread.
__device__ __forceinline__ SchedW make_sched_w(const Meta& m, const GemmArgs& a, int kb_per_item,
                                               int grid, int tile_w = 128, int kst_cap = 0) {
  SchedW s;
  s.KB = (a.K + BK - 1) / BK;
  s.kb_per_item = kb_per_item;
  s.KS = (s.KB + kb_per_item - 1) / kb_per_item;
  s.Mt = (a.n_w_rows + tile_w - 1) / tile_w;
  s.n_base = m.tile_prefix[a.r] * s.Mt * s.KS;
  s.full = (s.n_base / grid) * grid;
  s.rem = s.n_base - s.full;
  s.KSt = 1;
  s.kbs = kb_per_item;
  int maxcnt = 1;
  for (int c = 0; c < a.r; ++c) maxcnt = max(maxcnt, min(m.count[c], WM_BN));
  const int slot_tokens = (maxcnt + 15) & ~15;
  s.slot_floats = tile_w * slot_tokens;
  if (a.tail != nullptr && s.rem > 0) {
    const int n_slots = (int)((kTailBufferBytes - kTailHeaderBytes) / ((size_t)s.slot_floats * 4));
    const int kst_fold = kst_cap > 0 ? kst_cap : kFoldLoads / slot_tokens;
    const int want = (int)(threadIdx.x & 31) + 1;  // this lane tries `want` slices per item
    const int kbs = (kb_per_item + want - 1) / want;
    const int kst = (kb_per_item + kbs - 1) / kbs;
    const int slices = s.rem * kst;
    const bool valid = want == 1 || (kbs >= kMinSliceKb && slices <= n_slots && kst <= kst_fold);
    const int rounds = (slices + grid - 1) / grid;
    const unsigned cost = valid ? (unsigned)(rounds * (kbs + kSliceFixedKb)) : 0xffffffu;
    const unsigned best = __reduce_min_sync(0xffffffffu, (cost << 6) | (unsigned)kst);
    s.KSt = (int)(best & 63u);
    s.kbs = (kb_per_item + s.KSt - 1) / s.KSt;
  }
  if (s.KSt <= 1) {
    s.KSt = 1;
    s.kbs = kb_per_item;
    s.full = s.n_base;
    s.rem = 0;
  }
  s.n_slices = s.rem * s.KSt;
  s.n_total = s.n_slices + s.full;
  return s;
}

__device__ __forceinline__ void decode_item_w(const Meta& m, const GemmArgs& a, const SchedW& s,
                                              int item, ItemW& w) {
  int base = item - s.n_slices, sub = 0;
  w.tail_slot = -1;
  if (item < s.n_slices) {  // the slices come first
    base = s.full + item / s.KSt;
    sub = item - (item / s.KSt) * s.KSt;
    w.tail_slot = item;
  }
  const int ks = base % s.KS;
  const int rest = base / s.KS;
  const int mt = rest % s.Mt;
  const int rt = rest / s.Mt;
  int c = 0;
  while (c + 1 < a.r && m.tile_prefix[c + 1] <= rt) ++c;
  const int n0 = (rt - m.tile_prefix[c]) * WM_BN;
  w.c = c;
  w.mt = mt;
  w.ks = ks;
  w.cnt = min(WM_BN, m.count[c] - n0);
  w.bucket = w.cnt <= 16 ? 0 : (w.cnt <= 32 ? 1 : (w.cnt <= 64 ? 2 : 3));
  w.tok_row = a.a_row_base + a.a_off_mul * m.off[c] + n0;
  w.out_row = a.out_row_base + a.out_off_mul * m.off[c] + n0;
  w.kb0 = ks * s.kb_per_item;
  w.kb1 = min(s.KB, w.kb0 + s.kb_per_item);
  if (w.tail_slot >= 0) {
    w.tail_item = w.tail_slot / s.KSt;
    w.nslice = (w.kb1 - w.kb0 + s.kbs - 1) / s.kbs;  // a short last k-chunk has fewer slices
    w.kb0 += sub * s.kbs;
    w.kb1 = min(w.kb1, w.kb0 + s.kbs);  // empty beyond nslice
  }
}

// Adds up the K-slices of one tail item for the 32 weight rows of epilogue warp `wq` (this
// lane: one weight row) and tokens n0 .. n0 + nt - 1 (nt <= NT) in slice order and writes the
// regular output.  SUB slices are loaded before they are added: NT x SUB loads are in flight.
template <bool GATE_UP, int NT, int SUB>
__device__ __forceinline__ void fold_slices(const GemmArgs& args, const ItemW& w, const float* src,
                                            int slot_floats, int n0, int nt, int wq, int lane) {
  float acc[NT];
#pragma unroll
  for (int i = 0; i < NT; ++i) acc[i] = 0.f;
  src += n0 * 128;
  for (int sub0 = 0; sub0 < w.nslice; sub0 += SUB) {
    float v[SUB][NT];
#pragma unroll
    for (int u = 0; u < SUB; ++u)
#pragma unroll
      for (int i = 0; i < NT; ++i)
        v[u][i] = (sub0 + u < w.nslice && i < nt)
                      ? __ldcg(src + (size_t)(sub0 + u) * slot_floats + i * 128) : 0.f;
#pragma unroll
    for (int u = 0; u < SUB; ++u)
#pragma unroll
      for (int i = 0; i < NT; ++i) acc[i] += v[u][i];
  }
  const int wrow = w.mt * 128 + 32 * wq + lane;
  const int feat = (wrow >> 5) * kInterleave + (lane & 15);
  const bool rows_ok = w.mt * 128 + 32 * wq < args.n_w_rows;
#pragma unroll
  for (int i = 0; i < NT; ++i) {
    if (i < nt) {
      if (GATE_UP) {
        const float other = __shfl_xor_sync(0xffffffffu, acc[i], 16);
        if (rows_ok && lane < 16)
          reinterpret_cast<bf16*>(args.out)[(long long)(w.out_row + n0 + i) * args.out_ld + feat] =
              __float2bfloat16_rn(silu_mul(acc[i], other));
      } else if (wrow < args.n_w_rows) {
        reinterpret_cast<float*>(args.out)[(long long)w.ks * args.split_stride +
                                           (long long)(w.out_row + n0 + i) * args.out_ld + wrow] = acc[i];
      }
    }
  }
}

template <bool GATE_UP, int TOK>
__global__ void __launch_bounds__(kThreads, 1)
gemm_weights_m_kernel(const __grid_constant__ GemmMaps maps, const GemmArgs args, int kb_per_item) {
  extern __shared__ uint8_t smem_raw[];
  __shared__ Bars bars;
  __shared__ Meta s_meta;
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  using Cfg = WmCfg<TOK>;
  constexpr int WM_NS = Cfg::kNS;
  constexpr int WM_STAGE = Cfg::kStage;
  constexpr int WM_TOK_BYTES = Cfg::kTokBytes;
  setup_barriers<WM_NS>(bars);
  if (warp == 1) {
    tmem_alloc(smem_u32(&bars.tmem_base), 256);
    tmem_relinquish();
  }
  // everything above is independent of the preceding kernels; their results are read from here on
  pdl_wait();
  for (int i = threadIdx.x; i < (int)(sizeof(Meta) / 4); i += blockDim.x)
    reinterpret_cast<int32_t*>(&s_meta)[i] = ld_l2(reinterpret_cast<const int32_t*>(args.meta) + i);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *(volatile uint32_t*)&bars.tmem_base;
  volatile int* abort_flag = &bars.abort_flag;

  const SchedW sched = make_sched_w(s_meta, args, kb_per_item, (int)gridDim.x);
  const int n_items = sched.n_total;
  uint32_t issued = 0;

  if (warp == 0) {
    uint32_t it = 0;
    bool ok = true;
    const uint64_t evict_first = l2_policy_evict_first();
    for (int item = blockIdx.x; item < n_items && ok; item += gridDim.x) {
      ItemW w;
      decode_item_w(s_meta, args, sched, item, w);
      if (w.kb0 >= w.kb1) continue;
      const uint32_t bytes = WM_A_BYTES + (16u << w.bucket) * 128u;  // of one k-block
      for (int kb = w.kb0; kb < w.kb1; kb += 2, ++it) {
        const uint32_t s = it % WM_NS, ph = (it / WM_NS) & 1u;
        const int nk = min(2, w.kb1 - kb);
        ok = __all_sync(0xffffffffu, mbar_wait(smem_u32(&bars.empty[s]), ph ^ 1u, abort_flag));
        if (!ok) break;
        if (lane == 0) {
          const uint32_t full = smem_u32(&bars.full[s]);
          const uint32_t sa = smem_base + s * WM_STAGE;
          mbar_expect_tx(full, bytes * nk);
          for (int j = 0; j < nk; ++j) {
            // every weight byte is read exactly once: do not let it push the token rows, the
            // activations and the partial sums out of L2
            tma_load_3d_hint(sa + j * WM_A_BYTES, &maps.w, (kb + j) * BK, w.mt * 128, w.c, full, evict_first);
            tma_load_2d(sa + 2 * WM_A_BYTES + j * WM_TOK_BYTES, &maps.t[w.bucket], (kb + j) * BK, w.tok_row, full);
          }
        }
        __syncwarp();
      }
    }
    issued = it;
  } else if (warp == 1) {
    uint32_t it = 0, tile_it = 0;
    bool ok = true;
    for (int item = blockIdx.x; item < n_items && ok; item += gridDim.x) {
      ItemW w;
      decode_item_w(s_meta, args, sched, item, w);
      if (w.kb0 >= w.kb1) continue;
      const uint32_t idesc = idesc_bf16(128, 16 << w.bucket);
      const uint32_t buf = tile_it & 1u, bph = (tile_it >> 1) & 1u;
      ok = __all_sync(0xffffffffu, mbar_wait(smem_u32(&bars.tmem_empty[buf]), bph ^ 1u, abort_flag));
      if (!ok) break;
      tc_fence_after();
      const uint32_t d_tmem = tmem_base + buf * WM_BN;
      for (int kb = w.kb0; kb < w.kb1; kb += 2, ++it) {
        const uint32_t s = it % WM_NS, ph = (it / WM_NS) & 1u;
        const int nk = min(2, w.kb1 - kb);
        ok = __all_sync(0xffffffffu, mbar_wait(smem_u32(&bars.full[s]), ph, abort_flag));
        if (!ok) break;
        tc_fence_after();
        if (lane == 0) {
          const uint32_t sa = smem_base + s * WM_STAGE;
          for (int j = 0; j < nk; ++j) {
            const uint64_t adesc = smem_desc_k128(sa + j * WM_A_BYTES);
            const uint64_t bdesc = smem_desc_k128(sa + 2 * WM_A_BYTES + j * WM_TOK_BYTES);
#pragma unroll
            for (int k = 0; k < BK / UMMA_K; ++k)
              umma_bf16(d_tmem, adesc + 2 * k, bdesc + 2 * k, idesc, (kb + j > w.kb0 || k > 0) ? 1u : 0u);
          }
          umma_commit(smem_u32(&bars.empty[s]));
          if (kb + nk >= w.kb1) umma_commit(smem_u32(&bars.tmem_full[buf]));
        }
        __syncwarp();
      }
      ++tile_it;
    }
  } else {
    const int wq = warp & 3;
    uint32_t tile_it = 0;
    bool ok = true;
    for (int item = blockIdx.x; item < n_items && ok; item += gridDim.x) {
      ItemW w;
      decode_item_w(s_meta, args, sched, item, w);
      if (w.kb0 >= w.kb1) continue;
      const uint32_t buf = tile_it & 1u, bph = (tile_it >> 1) & 1u;
      ok = __all_sync(0xffffffffu, mbar_wait(smem_u32(&bars.tmem_full[buf]), bph, abort_flag));
      if (!ok) break;
      tc_fence_after();
      const uint32_t taddr = tmem_base + ((uint32_t)(32 * wq) << 16) + buf * WM_BN;
      const int wrow = w.mt * 128 + 32 * wq + lane;  // weight row held by this lane
      const int nchunk = (w.cnt + 15) >> 4;
      if (w.tail_slot >= 0) {
        // K-slice of a tail item: raw fp32 partial tile [token][weight row of the tile]
        float* slots = args.tail + kTailHeaderFloats;
        float* outp = slots + (size_t)w.tail_slot * sched.slot_floats + 32 * wq + lane;
#pragma unroll 1
        for (int j = 0; j < nchunk; ++j) {
          uint32_t v[16];
          tmem_ld16(taddr + 16 * j, v);
          tmem_ld_wait();
#pragma unroll
          for (int i = 0; i < 16; ++i) {
            const int n = 16 * j + i;
            if (n < w.cnt) outp[n * 128] = __uint_as_float(v[i]);
          }
        }
        // The accumulator has been read: hand the buffer back before the slower part.  Each
        // epilogue warp owns 32 weight rows of the tile in every slice; it counts its arrival,
        // and the warp that arrives last folds those rows of the item.
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&bars.tmem_empty[buf]));
        ++tile_it;
        __threadfence();
        __syncwarp();
        int* counter = reinterpret_cast<int*>(args.tail) + w.tail_item * 4 + wq;
        int last = 0;
        if (lane == 0) last = atomicAdd(counter, 1) == w.nslice - 1;
        last = __shfl_sync(0xffffffffu, last, 0);
        if (!last) continue;
        __threadfence();
        const float* src = slots + (size_t)(w.tail_item * sched.KSt) * sched.slot_floats + 32 * wq + lane;
        const int sf = sched.slot_floats;
        // few tokens: many slices in flight per token; many tokens: many tokens in flight
        if (w.cnt <= 2) fold_slices<GATE_UP, 2, 16>(args, w, src, sf, 0, w.cnt, wq, lane);
        else if (w.cnt <= 4) fold_slices<GATE_UP, 4, 8>(args, w, src, sf, 0, w.cnt, wq, lane);
        else if (w.cnt <= 8) fold_slices<GATE_UP, 8, 4>(args, w, src, sf, 0, w.cnt, wq, lane);
        else
          for (int n0 = 0; n0 < w.cnt; n0 += 16)
            fold_slices<GATE_UP, 16, 2>(args, w, src, sf, n0, min(16, w.cnt - n0), wq, lane);
        if (lane == 0) *counter = 0;  // ready for the next launch
        continue;
      } else if (GATE_UP) {
        // lanes 0-15 hold gate rows, lanes 16-31 the up rows of the same 16 features
        const int feat = (wrow >> 5) * kInterleave + (lane & 15);
        const bool lane_ok = (lane < 16) && (w.mt * 128 + 32 * wq < args.n_w_rows);
        bf16* outp = reinterpret_cast<bf16*>(args.out) + (long long)w.out_row * args.out_ld + feat;
#pragma unroll 1
        for (int j = 0; j < nchunk; ++j) {
          uint32_t v[16];
          tmem_ld16(taddr + 16 * j, v);
          tmem_ld_wait();
#pragma unroll
          for (int i = 0; i < 16; ++i) {
            const float mine = __uint_as_float(v[i]);
            const float other = __shfl_xor_sync(0xffffffffu, mine, 16);
            const int n = 16 * j + i;
            if (lane_ok && n < w.cnt)
              outp[(long long)n * args.out_ld] = __float2bfloat16_rn(silu_mul(mine, other));
          }
        }
      } else {
        const bool lane_ok = wrow < args.n_w_rows;
        float* outp = reinterpret_cast<float*>(args.out) + (long long)w.ks * args.split_stride +
                      (long long)w.out_row * args.out_ld + wrow;
#pragma unroll 1
        for (int j = 0; j < nchunk; ++j) {
          uint32_t v[16];
          tmem_ld16(taddr + 16 * j, v);
          tmem_ld_wait();
#pragma unroll
          for (int i = 0; i < 16; ++i) {
            const int n = 16 * j + i;
            if (lane_ok && n < w.cnt) outp[(long long)n * args.out_ld] = __uint_as_float(v[i]);
          }
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&bars.tmem_empty[buf]));
      ++tile_it;
    }
  }
  pdl_launch_dependents();
  teardown<256>(bars, tmem_base, issued, WM_NS, args.status);
}

// ----------------------------------------------------------------------- gemm_tokens_d
//
// Small batches (T <= 256), token-major.  The warp that issues the MMAs spends about 550 cycles
// per k-block whatever the tile (four instructions of ~57 cycles each when N <= 64, a commit of
// ~120, the barrier wait and fences), which bounds an SM of the weight-major kernel at 16 KB of
// weights per k-block.  With the weights as the N operand a k-block carries 256 rows = 32 KB
// (four instructions of 128 cycles), twice the bytes per trip round the loop.  The token tile is
// the M operand: only the rows the expert really has are loaded (boxes of 16 to 128 rows), the
// rest of its 128-row slot is zero and its accumulator rows are never stored.  Work items, the
// K-slices of the remainder that run first and their fold are those of the weight-major kernel,
// with 256-row weight tiles.

constexpr int TD_NS = 4;
constexpr int TD_A_BYTES = 128 * 128;  // slot of the token tile (16 .. 128 rows loaded)
constexpr int TD_B_BYTES = 256 * 128;  // 256 weight rows x 64 bf16
constexpr int TD_STAGE = TD_A_BYTES + TD_B_BYTES;
constexpr int TD_SMEM = TD_NS * TD_STAGE + 1024;
constexpr int TD_BN = 256;
constexpr int kFoldSlicesD = 8;  // the fold of this kernel reads 256 floats per slice and token

// 32 accumulator columns of one token row -> output (SwiGLU + bf16, or fp32), as in
// store_tile_tokens_m.  col0 = first weight row of the chunk, orow = element offset of the row.
template <bool GATE_UP>
__device__ __forceinline__ void store_chunk_d(const float* v, const GemmArgs& args, long long orow, int col0) {
  if (GATE_UP) {
    uint32_t o[8];
#pragma unroll
    for (int i = 0; i < 8; ++i)
      o[i] = pack_bf16(silu_mul(v[2 * i], v[16 + 2 * i]), silu_mul(v[2 * i + 1], v[17 + 2 * i]));
    uint4* dst = reinterpret_cast<uint4*>(reinterpret_cast<bf16*>(args.out) + orow + (col0 >> 1));
    dst[0] = make_uint4(o[0], o[1], o[2], o[3]);
    dst[1] = make_uint4(o[4], o[5], o[6], o[7]);
  } else {
    float4* dst = reinterpret_cast<float4*>(reinterpret_cast<float*>(args.out) + orow + col0);
#pragma unroll
    for (int i = 0; i < 8; ++i) dst[i] = make_float4(v[4 * i], v[4 * i + 1], v[4 * i + 2], v[4 * i + 3]);
  }
}

template <bool GATE_UP>
__global__ void __launch_bounds__(kThreads, 1)
gemm_tokens_d_kernel(const __grid_constant__ GemmMaps maps, const GemmArgs args, int kb_per_item) {
  extern __shared__ uint8_t smem_raw[];
  __shared__ Bars bars;
  __shared__ Meta s_meta;
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  setup_barriers<TD_NS>(bars);
  if (warp == 1) {
    tmem_alloc(smem_u32(&bars.tmem_base), 512);
    tmem_relinquish();
  }
  // Rows of the token slots that no load ever writes feed the tensor core all the same: start
  // them at zero (multiplying zeros costs far less power than multiplying stale data).
  {
    uint8_t* gen = smem_raw + (smem_base - smem_u32(smem_raw));
    for (int s = 0; s < TD_NS; ++s)
      for (int i = threadIdx.x; i < TD_A_BYTES / 16; i += blockDim.x)
        reinterpret_cast<uint4*>(gen + s * TD_STAGE)[i] = make_uint4(0u, 0u, 0u, 0u);
    fence_proxy_async();
  }
  pdl_wait();
  for (int i = threadIdx.x; i < (int)(sizeof(Meta) / 4); i += blockDim.x)
    reinterpret_cast<int32_t*>(&s_meta)[i] = ld_l2(reinterpret_cast<const int32_t*>(args.meta) + i);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *(volatile uint32_t*)&bars.tmem_base;
  volatile int* abort_flag = &bars.abort_flag;

  const SchedW sched = make_sched_w(s_meta, args, kb_per_item, (int)gridDim.x, TD_BN, kFoldSlicesD);
  const int n_items = sched.n_total;
  uint32_t issued = 0;

  if (warp == 0) {
    uint32_t it = 0;
    bool ok = true;
    const uint64_t evict_first = l2_policy_evict_first();
    for (int item = blockIdx.x; item < n_items && ok; item += gridDim.x) {
      ItemW w;
      decode_item_w(s_meta, args, sched, item, w);
      if (w.kb0 >= w.kb1) continue;
      const uint32_t bytes = TD_B_BYTES + (16u << w.bucket) * 128u;
      for (int kb = w.kb0; kb < w.kb1; ++kb, ++it) {
        const uint32_t s = it % TD_NS, ph = (it / TD_NS) & 1u;
        ok = __all_sync(0xffffffffu, mbar_wait(smem_u32(&bars.empty[s]), ph ^ 1u, abort_flag));
        if (!ok) break;
        if (lane == 0) {
          const uint32_t full = smem_u32(&bars.full[s]);
          const uint32_t sa = smem_base + s * TD_STAGE;
          mbar_expect_tx(full, bytes);
          tma_load_3d_hint(sa + TD_A_BYTES, &maps.w, kb * BK, w.mt * TD_BN, w.c, full, evict_first);
          tma_load_2d(sa, &maps.t[w.bucket], kb * BK, w.tok_row, full);
        }
        __syncwarp();
      }
    }
    issued = it;
  } else if (warp == 1) {
    uint32_t it = 0, tile_it = 0;
    bool ok = true;
    for (int item = blockIdx.x; item < n_items && ok; item += gridDim.x) {
      ItemW w;
      decode_item_w(s_meta, args, sched, item, w);
      if (w.kb0 >= w.kb1) continue;
      // up to 64 token rows: the M = 64 form (half the multiplications, hence less board power)
      const uint32_t idesc = idesc_bf16(w.cnt <= 64 ? 64 : 128, TD_BN);
      const uint32_t buf = tile_it & 1u, bph = (tile_it >> 1) & 1u;
      ok = __all_sync(0xffffffffu, mbar_wait(smem_u32(&bars.tmem_empty[buf]), bph ^ 1u, abort_flag));
      if (!ok) break;
      tc_fence_after();
      const uint32_t d_tmem = tmem_base + buf * TD_BN;
      for (int kb = w.kb0; kb < w.kb1; ++kb, ++it) {
        const uint32_t s = it % TD_NS, ph = (it / TD_NS) & 1u;
        ok = __all_sync(0xffffffffu, mbar_wait(smem_u32(&bars.full[s]), ph, abort_flag));
        if (!ok) break;
        tc_fence_after();
        if (lane == 0) {
          const uint32_t sa = smem_base + s * TD_STAGE;
          const uint64_t adesc = smem_desc_k128(sa);
          const uint64_t bdesc = smem_desc_k128(sa + TD_A_BYTES);
#pragma unroll
          for (int k = 0; k < BK / UMMA_K; ++k)
            umma_bf16(d_tmem, adesc + 2 * k, bdesc + 2 * k, idesc, (kb > w.kb0 || k > 0) ? 1u : 0u);
          umma_commit(smem_u32(&bars.empty[s]));
          if (kb == w.kb1 - 1) umma_commit(smem_u32(&bars.tmem_full[buf]));
        }
        __syncwarp();
      }
      ++tile_it;
    }
  } else {
    // epilogue warp wq reads tensor-memory lanes 32 wq .. 32 wq + 31.  M = 128: lane l of the
    // tile is token row l.  M = 64: rows 16 q .. 16 q + 15 sit in lanes 32 q .. 32 q + 15.
    const int wq = warp & 3;
    uint32_t tile_it = 0;
    bool ok = true;
    for (int item = blockIdx.x; item < n_items && ok; item += gridDim.x) {
      ItemW w;
      decode_item_w(s_meta, args, sched, item, w);
      if (w.kb0 >= w.kb1) continue;
      const uint32_t buf = tile_it & 1u, bph = (tile_it >> 1) & 1u;
      ok = __all_sync(0xffffffffu, mbar_wait(smem_u32(&bars.tmem_full[buf]), bph, abort_flag));
      if (!ok) break;
      tc_fence_after();
      ++tile_it;
      const uint32_t taddr = tmem_base + ((uint32_t)(32 * wq) << 16) + buf * TD_BN;
      const bool m64 = w.cnt <= 64;
      const int row = m64 ? 16 * wq + lane : 32 * wq + lane;
      const bool warp_has_rows = (m64 ? 16 * wq : 32 * wq) < w.cnt;  // warp-uniform
      const bool row_ok = row < w.cnt && (!m64 || lane < 16);
      const long long orow = (long long)(w.out_row + row) * args.out_ld +
                             (GATE_UP ? 0ll : (long long)w.ks * args.split_stride);
      const int nchunk = min(TD_BN, args.n_w_rows - w.mt * TD_BN) / 32;  // 32-column chunks in range
      if (w.tail_slot < 0) {
        if (warp_has_rows) {
#pragma unroll 1
          for (int j = 0; j < nchunk; ++j) {
            uint32_t v[32];
            tmem_ld32(taddr + 32 * j, v);
            tmem_ld_wait();
            if (row_ok) store_chunk_d<GATE_UP>(reinterpret_cast<const float*>(v), args, orow, w.mt * TD_BN + 32 * j);
          }
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&bars.tmem_empty[buf]));
        continue;
      }
      // K-slice of a tail item: fp32 partial tile [token][256 weight rows]
      float* slots = args.tail + kTailHeaderFloats;
      if (warp_has_rows) {
        float4* outp = reinterpret_cast<float4*>(slots + (size_t)w.tail_slot * sched.slot_floats + row * TD_BN);
#pragma unroll 1
        for (int j = 0; j < nchunk; ++j) {
          uint32_t v[32];
          tmem_ld32(taddr + 32 * j, v);
          tmem_ld_wait();
          if (row_ok) {
#pragma unroll
            for (int i = 0; i < 8; ++i)
              outp[8 * j + i] = make_float4(__uint_as_float(v[4 * i]), __uint_as_float(v[4 * i + 1]),
                                            __uint_as_float(v[4 * i + 2]), __uint_as_float(v[4 * i + 3]));
          }
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&bars.tmem_empty[buf]));
      if (!warp_has_rows) continue;
      // the warp that arrives last for these 32 token rows of the item folds them
      __threadfence();
      __syncwarp();
      int* counter = reinterpret_cast<int*>(args.tail) + w.tail_item * 4 + wq;
      int last = 0;
      if (lane == 0) last = atomicAdd(counter, 1) == w.nslice - 1;
      last = __shfl_sync(0xffffffffu, last, 0);
      if (!last) continue;
      __threadfence();
      if (row_ok) {
        const float* src = slots + (size_t)(w.tail_item * sched.KSt) * sched.slot_floats + row * TD_BN;
#pragma unroll 1
        for (int j = 0; j < nchunk; ++j) {
          float v[32];
#pragma unroll
          for (int i = 0; i < 32; ++i) v[i] = 0.f;
#pragma unroll 2
          for (int sub = 0; sub < w.nslice; ++sub) {
            const float4* p = reinterpret_cast<const float4*>(src + (size_t)sub * sched.slot_floats + 32 * j);
            float4 q[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) q[i] = __ldcg(p + i);
#pragma unroll
            for (int i = 0; i < 8; ++i) {
              v[4 * i] += q[i].x; v[4 * i + 1] += q[i].y; v[4 * i + 2] += q[i].z; v[4 * i + 3] += q[i].w;
            }
          }
          store_chunk_d<GATE_UP>(v, args, orow, w.mt * TD_BN + 32 * j);
        }
      }
      __syncwarp();
      if (lane == 0) *counter = 0;  // ready for the next launch
    }
  }
  pdl_launch_dependents();
  teardown<512>(bars, tmem_base, issued, TD_NS, args.status);
}

// -------------------------------------------------------------------- router_tc (large T)
//
// Router logits of a large batch on the tensor cores (Sec. 3.1: l = W_gate x over the kept
// experts): a [T x h] x [h x 16] contraction that has to read every token row once and nothing
// else, so it runs at the rate the rows arrive.  One CTA takes tiles of 128 tokens in turn: the
// producer warp streams the tile's k-blocks (128 rows x 64 values, 16 KB) and the matching
// k-blocks of the 16 padded router rows (2 KB) through an 8-stage ring, one lane issues four
// M128 N16 K16 MMAs per k-block.
// The tensor core does not round its fp32 accumulation the IEEE way, and over a whole row of
// 4096 products with outlier channels that left the logits accurate to 5e-5 only.  So the
// accumulator holds no more than kRouterChunkKb k-blocks (128 products) at a time: the MMA lane
// alternates between two 16-column accumulators, one chunk each, and the four epilogue warps, one
// thread per token, read every chunk out of tensor memory and add it to the token's logits with
// IEEE fp32 additions in chunk order.  The routing decision (top-2, skip test, weights:
// route_decide) is then taken exactly as the CUDA-core routers take it.  Each epilogue warp also
// writes the pair counts of its two blocks of 16 tokens, the histogram rows the permutation's
// scan reads.

constexpr int RT_NS = 8;
constexpr int RT_X_BYTES = 128 * 128;   // 128 token rows x 64 bf16
constexpr int RT_W_BYTES = 16 * 128;    // 16 router rows x 64 bf16
constexpr int RT_STAGE = RT_X_BYTES + RT_W_BYTES;
constexpr int RT_SMEM = RT_NS * RT_STAGE + 1024;
constexpr int RT_N = 16;                // accumulator columns = padded router rows
constexpr int kRouterChunkKb = 2;       // k-blocks accumulated inside the tensor core at a time

struct RouterMaps {
  CUtensorMap x;   // token rows [T][h], box 64 x 128
  CUtensorMap wg;  // router rows [16][h] (rows beyond the kept experts are zero), box 64 x 16
};

template <int R>
__global__ void __launch_bounds__(kThreads, 1)
router_tc_kernel(const __grid_constant__ RouterMaps maps, int T, int h, int r, float beta, KeptIds kept,
                 RouteOut o, int* status) {
  extern __shared__ uint8_t smem_raw[];
  __shared__ Bars bars;
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  setup_barriers<RT_NS>(bars);
  if (warp == 1) {
    tmem_alloc(smem_u32(&bars.tmem_base), 32);
    tmem_relinquish();
  }
  pdl_launch_dependents();
  pdl_wait();  // the token rows may have been written by the stream's previous kernel
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *(volatile uint32_t*)&bars.tmem_base;
  volatile int* abort_flag = &bars.abort_flag;
  const int KB = (h + BK - 1) / BK;
  const int n_chunks = (KB + kRouterChunkKb - 1) / kRouterChunkKb;
  const int n_tiles = (T + 127) / 128;
  uint32_t issued = 0;

  if (warp == 0) {
    uint32_t it = 0, s = 0, ph = 0;
    bool ok = true;
    for (int tile = blockIdx.x; tile < n_tiles && ok; tile += gridDim.x) {
      for (int kb = 0; kb < KB; ++kb, ++it) {
        ok = __all_sync(0xffffffffu, mbar_wait(smem_u32(&bars.empty[s]), ph ^ 1u, abort_flag));
        if (!ok) break;
        if (lane == 0) {
          const uint32_t full = smem_u32(&bars.full[s]);
          const uint32_t sa = smem_base + s * RT_STAGE;
          mbar_expect_tx(full, RT_STAGE);
          tma_load_2d(sa, &maps.x, kb * BK, tile * 128, full);
          tma_load_2d(sa + RT_X_BYTES, &maps.wg, kb * BK, 0, full);
        }
        if (++s == RT_NS) { s = 0; ph ^= 1u; }
        __syncwarp();
      }
    }
    issued = it;
  } else if (warp == 1) {
    const uint32_t idesc = idesc_bf16(128, RT_N);
    uint32_t s = 0, ph = 0, chunk_it = 0;
    bool ok = true;
    for (int tile = blockIdx.x; tile < n_tiles && ok; tile += gridDim.x) {
      for (int kb = 0; kb < KB; ++kb) {
        const bool first = kb % kRouterChunkKb == 0;
        const bool last = kb % kRouterChunkKb == kRouterChunkKb - 1 || kb == KB - 1;
        const uint32_t buf = chunk_it & 1u, bph = (chunk_it >> 1) & 1u;
        bool ready = mbar_wait(smem_u32(&bars.full[s]), ph, abort_flag);
        if (first) ready = ready && mbar_wait(smem_u32(&bars.tmem_empty[buf]), bph ^ 1u, abort_flag);
        ok = __all_sync(0xffffffffu, ready);
        if (!ok) break;
        tc_fence_after();
        if (lane == 0) {
          const uint32_t sa = smem_base + s * RT_STAGE;
          const uint64_t adesc = smem_desc_k128(sa);
          const uint64_t bdesc = smem_desc_k128(sa + RT_X_BYTES);
          const uint32_t d_tmem = tmem_base + buf * RT_N;
#pragma unroll
          for (int k = 0; k < BK / UMMA_K; ++k)
            umma_bf16(d_tmem, adesc + 2 * k, bdesc + 2 * k, idesc, (!first || k > 0) ? 1u : 0u);
          umma_commit(smem_u32(&bars.empty[s]));
          if (last) umma_commit(smem_u32(&bars.tmem_full[buf]));
        }
        if (last) ++chunk_it;
        if (++s == RT_NS) { s = 0; ph ^= 1u; }
        __syncwarp();
      }
    }
  } else {
    // epilogue warp wq owns tensor-memory lanes 32 wq .. 32 wq + 31 = tokens 32 wq .. of the tile
    const int wq = warp & 3;
    uint32_t chunk_it = 0;
    bool ok = true;
    for (int tile = blockIdx.x; tile < n_tiles && ok; tile += gridDim.x) {
      float acc[R], lost[R];  // compensated (Kahan) sums of the chunks: `lost` carries what an addition dropped
#pragma unroll
      for (int c = 0; c < R; ++c) { acc[c] = 0.f; lost[c] = 0.f; }
      for (int ch = 0; ch < n_chunks; ++ch, ++chunk_it) {
        const uint32_t buf = chunk_it & 1u, bph = (chunk_it >> 1) & 1u;
        ok = __all_sync(0xffffffffu, mbar_wait(smem_u32(&bars.tmem_full[buf]), bph, abort_flag));
        if (!ok) break;
        tc_fence_after();
        uint32_t v[16];
        tmem_ld16(tmem_base + ((uint32_t)(32 * wq) << 16) + buf * RT_N, v);
        tmem_ld_wait();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&bars.tmem_empty[buf]));
#pragma unroll
        for (int c = 0; c < R; ++c) {
          const float term = __fsub_rn(__uint_as_float(v[c]), lost[c]);
          const float sum = __fadd_rn(acc[c], term);
          lost[c] = __fsub_rn(__fsub_rn(sum, acc[c]), term);
          acc[c] = sum;
        }
      }
      if (!ok) break;
      const int t = tile * 128 + 32 * wq + lane;
      int e0 = -1, e1 = -1;
      bool skip = false;
      if (t < T) {
        route_decide<R>(acc, r, beta, t, kept, o, e0, e1, skip);
        if (skip) e1 = -1;
      }
      if (o.blk_hist) {
        // pair counts of the two blocks of kRouteTokPerBlock = 16 tokens this warp holds
        const int blk = (tile * 128 + 32 * wq) / kRouteTokPerBlock;
        const int nblk = (T + kRouteTokPerBlock - 1) / kRouteTokPerBlock;
#pragma unroll 1
        for (int col = 0; col < kHistCols; ++col) {
          bool hit;
          if (col == 2 * kMaxE) hit = skip;
          else hit = ((col & 1) ? e1 : e0) == (col >> 1);
          const unsigned m = __ballot_sync(0xffffffffu, hit);
          if (lane == 0) {
            if (blk < nblk) o.blk_hist[(size_t)blk * kHistCols + col] = __popc(m & 0xffffu);
            if (blk + 1 < nblk) o.blk_hist[(size_t)(blk + 1) * kHistCols + col] = __popc(m >> 16);
          }
        }
      }
    }
  }
  teardown<32>(bars, tmem_base, issued, RT_NS, status);
}

// ------------------------------------------------------------------ wait-expiry test hook

// One CTA with the GEMMs' barrier block and a tensor-memory allocation.  Warp 0 waits, with the
// GEMMs' own bounded wait, for phase 0 of a barrier on which nothing ever arrives; the wait runs
// out after limit_ns, raises the abort flag, and the common teardown drains, reports and releases
// tensor memory exactly as it does for a GEMM whose pipeline stalled.  Nothing is in flight, so
// nothing can fault or spin beyond the limit.
__global__ void __launch_bounds__(kThreads, 1)
wait_expiry_kernel(int* status, unsigned long long limit_ns) {
  __shared__ Bars bars;
  const int warp = threadIdx.x >> 5;
  setup_barriers<1>(bars);
  if (warp == 1) {
    tmem_alloc(smem_u32(&bars.tmem_base), 32);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *(volatile uint32_t*)&bars.tmem_base;
  volatile int* abort_flag = &bars.abort_flag;
  if (warp == 0) {
    // the producer's wait of the GEMMs, on the phase that only an arrival could complete
    (void)__all_sync(0xffffffffu, mbar_wait(smem_u32(&bars.full[0]), 0u, abort_flag, limit_ns));
  } else if (warp == 1) {
    // the other roles poll their own barriers and leave when the flag is up
    (void)__all_sync(0xffffffffu, mbar_wait(smem_u32(&bars.tmem_empty[0]), 0u, abort_flag, 2 * limit_ns));
  } else {
    (void)__all_sync(0xffffffffu, mbar_wait(smem_u32(&bars.tmem_full[0]), 0u, abort_flag, 2 * limit_ns));
  }
  teardown<32>(bars, tmem_base, 0u, 1u, status);
}

// ------------------------------------------------------------ CUDA-core debug kernels

__device__ __forceinline__ float dot8(const uint4& a, const uint4& b, float acc) {
  const uint32_t aw[4] = {a.x, a.y, a.z, a.w}, bw[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    acc = fmaf(__uint_as_float(aw[i] << 16), __uint_as_float(bw[i] << 16), acc);
    acc = fmaf(__uint_as_float(aw[i] & 0xffff0000u), __uint_as_float(bw[i] & 0xffff0000u), acc);
  }
  return acc;
}

__global__ void __launch_bounds__(128)
simt_gate_up_kernel(const bf16* __restrict__ A, const bf16* __restrict__ W13, GemmArgs a) {
  const int c = blockIdx.z, i = blockIdx.x;
  const Meta* m = a.meta;
  if (i >= m->count[c]) return;
  const int f = a.n_w_rows / 2, h = a.K;
  const int j = blockIdx.y * 128 + threadIdx.x;
  if (j >= f) return;
  const int q = j / kInterleave, s = j % kInterleave;
  const long long a_row = a.a_row_base + (long long)a.a_off_mul * m->off[c] + i;
  const long long o_row = a.out_row_base + (long long)a.out_off_mul * m->off[c] + i;
  const uint4* xr = reinterpret_cast<const uint4*>(A + a_row * h);
  const uint4* g = reinterpret_cast<const uint4*>(W13 + ((size_t)c * a.n_w_rows + 32 * q + s) * h);
  const uint4* u = reinterpret_cast<const uint4*>(W13 + ((size_t)c * a.n_w_rows + 32 * q + 16 + s) * h);
  float ag = 0.f, au = 0.f;
  for (int v = 0; v < h / 8; ++v) {
    const uint4 xv = xr[v];
    ag = dot8(xv, g[v], ag);
    au = dot8(xv, u[v], au);
  }
  reinterpret_cast<bf16*>(a.out)[o_row * a.out_ld + c * a.out_col_mul + j] =
      __float2bfloat16_rn(ag / (1.0f + expf(-ag)) * au);
}

template <int OUT>
__global__ void __launch_bounds__(128)
simt_down_kernel(const bf16* __restrict__ A, const bf16* __restrict__ W2, GemmArgs a) {
  const int c = blockIdx.z, i = blockIdx.x;
  const Meta* m = a.meta;
  if (i >= m->count[c]) return;
  const int h = a.n_w_rows, f = a.K;
  const int n = blockIdx.y * 128 + threadIdx.x;
  if (n >= h) return;
  const long long a_row = a.a_row_base + (long long)a.a_off_mul * m->off[c] + i;
  const long long o_row = a.out_row_base + (long long)a.out_off_mul * m->off[c] + i;
  const uint4* ar = reinterpret_cast<const uint4*>(A + a_row * f);
  const uint4* w = reinterpret_cast<const uint4*>(W2 + ((size_t)c * h + n) * f);
  float acc = 0.f;
  for (int v = 0; v < f / 8; ++v) acc = dot8(ar[v], w[v], acc);
  const long long o = o_row * a.out_ld + c * a.out_col_mul + n;
  if (OUT == kOutF32) reinterpret_cast<float*>(a.out)[o] = acc;
  else reinterpret_cast<bf16*>(a.out)[o] = __float2bfloat16_rn(acc);
}

// ------------------------------------------------------------------------- tensor maps

// Every tensor map asks for 256-byte L2 promotion (128 bytes or none measured 1.0-1.5 % slower
// for the small-batch kernels and equal for the large-batch one).
constexpr CUtensorMapL2promotion kL2Promotion = CU_TENSOR_MAP_L2_PROMOTION_L2_256B;

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*,
                                  const cuuint64_t*, const cuuint64_t*, const cuuint32_t*,
                                  const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeTiledFn g_encode = nullptr;
int g_num_sms = 0;

}  // namespace

int gemm_init_driver_api() {
  if (g_encode) return 0;
  void* fn = nullptr;
  cudaDriverEntryPointQueryResult q;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q) != cudaSuccess ||
      q != cudaDriverEntryPointSuccess || !fn)
    return -1;
  g_encode = reinterpret_cast<EncodeTiledFn>(fn);
  return 0;
}

int make_map_2d(CUtensorMap* m, const void* base, uint64_t inner, uint64_t rows, uint32_t box_rows) {
  if (!g_encode) return -1;
  cuuint64_t dims[2] = {inner, rows};
  cuuint64_t strides[1] = {inner * 2};
  cuuint32_t box[2] = {BK, box_rows};
  cuuint32_t es[2] = {1, 1};
  CUresult rc = g_encode(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims,
                         strides, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE,
                         CU_TENSOR_MAP_SWIZZLE_128B, kL2Promotion,
                         CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return rc == CUDA_SUCCESS ? 0 : -(int)rc;
}

int make_map_3d(CUtensorMap* m, const void* base, uint64_t inner, uint64_t rows, uint64_t planes,
                uint32_t box_rows) {
  if (!g_encode) return -1;
  cuuint64_t dims[3] = {inner, rows, planes};
  cuuint64_t strides[2] = {inner * 2, inner * rows * 2};
  cuuint32_t box[3] = {BK, box_rows, 1};
  cuuint32_t es[3] = {1, 1, 1};
  CUresult rc = g_encode(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims,
                         strides, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE,
                         CU_TENSOR_MAP_SWIZZLE_128B, kL2Promotion,
                         CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return rc == CUDA_SUCCESS ? 0 : -(int)rc;
}

cudaError_t gemm_set_attributes() {
  cudaError_t e;
#define SET_ATTR(k, bytes)                                                                 \
  e = cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);         \
  if (e != cudaSuccess) return e;
  SET_ATTR((gemm_tokens_m_kernel<true, kOutActBf16>), TM_SMEM)
  SET_ATTR((gemm_tokens_m_kernel<false, kOutF32>), TM_SMEM)
  SET_ATTR((gemm_tokens_m_kernel<false, kOutBf16>), TM_SMEM)
  SET_ATTR((gemm_weights_m_kernel<true, 64>), WmCfg<64>::kSmem)
  SET_ATTR((gemm_weights_m_kernel<false, 64>), WmCfg<64>::kSmem)
  SET_ATTR((gemm_weights_m_kernel<true, 128>), WmCfg<128>::kSmem)
  SET_ATTR((gemm_weights_m_kernel<false, 128>), WmCfg<128>::kSmem)
  SET_ATTR((router_tc_kernel<2>), RT_SMEM)
  SET_ATTR((router_tc_kernel<4>), RT_SMEM)
  SET_ATTR((router_tc_kernel<6>), RT_SMEM)
  SET_ATTR((router_tc_kernel<8>), RT_SMEM)
  SET_ATTR((router_tc_kernel<kMaxE>), RT_SMEM)
  SET_ATTR((gemm_tokens_d_kernel<true>), TD_SMEM)
  SET_ATTR((gemm_tokens_d_kernel<false>), TD_SMEM)
#undef SET_ATTR
  int dev = 0;
  e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  return cudaDeviceGetAttribute(&g_num_sms, cudaDevAttrMultiProcessorCount, dev);
}

cudaError_t launch_router_tc(const bf16* x, const bf16* Wg16, int T, int h, int r, float beta,
                             const KeptIds& kept, const RouteOut& out, int* status, cudaStream_t st) {
  RouterMaps maps;
  if (make_map_2d(&maps.x, x, (uint64_t)h, (uint64_t)T, 128) || make_map_2d(&maps.wg, Wg16, (uint64_t)h, kMaxE, RT_N))
    return cudaErrorInvalidValue;
  const int n_tiles = (T + 127) / 128;
  int grid = g_num_sms > 0 ? g_num_sms : 148;
  if (grid > n_tiles) grid = n_tiles;
#define MOE_ROUTER_TC(R)                                                                          \
  return launch_pdl(router_tc_kernel<R>, dim3(grid), dim3(kThreads), RT_SMEM, st, maps, T, h, r, beta, kept, \
                    out, status)
  switch (r) {
    case 2: MOE_ROUTER_TC(2);
    case 3: case 4: MOE_ROUTER_TC(4);
    case 5: case 6: MOE_ROUTER_TC(6);
    case 7: case 8: MOE_ROUTER_TC(8);
    default: MOE_ROUTER_TC(kMaxE);
  }
#undef MOE_ROUTER_TC
}

cudaError_t launch_wait_expiry(int* status, unsigned long long limit_ns, cudaStream_t st) {
  wait_expiry_kernel<<<1, kThreads, 0, st>>>(status, limit_ns);
  return cudaGetLastError();
}

cudaError_t launch_gemm_tokens_m(bool gate_up, GemmOut out_kind, const GemmMaps& maps,
                                 const GemmArgs& args, cudaStream_t st) {
  const int grid = g_num_sms > 0 ? g_num_sms : 148;
  const GemmArgs& a = args;
  // Plain stream order for these long kernels: launched as programmatic dependents they measured
  // 3-5 % slower at T = 8192 (5.35 vs 5.0-5.1 ms per step), while the short kernels around them and
  // the weight-major kernels gain from the overlap.
  if (gate_up)
    return launch_plain(gemm_tokens_m_kernel<true, kOutActBf16>, dim3(grid), dim3(TmCfg<true>::kThreads), TM_SMEM, st, maps, a);
  if (out_kind == kOutF32)
    return launch_plain(gemm_tokens_m_kernel<false, kOutF32>, dim3(grid), dim3(TmCfg<false>::kThreads), TM_SMEM, st, maps, a);
  return launch_plain(gemm_tokens_m_kernel<false, kOutBf16>, dim3(grid), dim3(TmCfg<false>::kThreads), TM_SMEM, st, maps, a);
}

cudaError_t launch_gemm_tokens_d(bool gate_up, const GemmMaps& maps, const GemmArgs& a, int kb_per_item,
                                 cudaStream_t st) {
  const int grid = g_num_sms > 0 ? g_num_sms : 148;
  if (gate_up)
    return launch_pdl(gemm_tokens_d_kernel<true>, dim3(grid), dim3(kThreads), TD_SMEM, st, maps, a,
                      kb_per_item);
  return launch_pdl(gemm_tokens_d_kernel<false>, dim3(grid), dim3(kThreads), TD_SMEM, st, maps, a,
                    kb_per_item);
}

template <int TOK>
static cudaError_t launch_wm(bool gate_up, const GemmMaps& maps, const GemmArgs& a, int kb_per_item, int grid,
                             cudaStream_t st) {
  if (gate_up)
    return launch_pdl(gemm_weights_m_kernel<true, TOK>, dim3(grid), dim3(kThreads), WmCfg<TOK>::kSmem, st, maps,
                      a, kb_per_item);
  return launch_pdl(gemm_weights_m_kernel<false, TOK>, dim3(grid), dim3(kThreads), WmCfg<TOK>::kSmem, st, maps,
                    a, kb_per_item);
}

cudaError_t launch_gemm_weights_m(bool gate_up, const GemmMaps& maps, const GemmArgs& a,
                                  int kb_per_item, int max_tokens_per_tile, cudaStream_t st) {
  const int grid = g_num_sms > 0 ? g_num_sms : 148;
  // no expert group can exceed the batch: small batches take the layout with 64-row token slots
  if (max_tokens_per_tile <= 64) return launch_wm<64>(gate_up, maps, a, kb_per_item, grid, st);
  return launch_wm<128>(gate_up, maps, a, kb_per_item, grid, st);
}

cudaError_t launch_simt_gate_up(const bf16* A, const bf16* W13, const GemmArgs& a, int cap_rows,
                                cudaStream_t st) {
  const int f = a.n_w_rows / 2;
  dim3 grid(cap_rows, (f + 127) / 128, a.r);
  simt_gate_up_kernel<<<grid, 128, 0, st>>>(A, W13, a);
  return cudaGetLastError();
}

cudaError_t launch_simt_down(const bf16* A, const bf16* W2, const GemmArgs& a, int cap_rows,
                             GemmOut out_kind, cudaStream_t st) {
  dim3 grid(cap_rows, (a.n_w_rows + 127) / 128, a.r);
  if (out_kind == kOutF32) simt_down_kernel<kOutF32><<<grid, 128, 0, st>>>(A, W2, a);
  else simt_down_kernel<kOutBf16><<<grid, 128, 0, st>>>(A, W2, a);
  return cudaGetLastError();
}

}  // namespace moe
