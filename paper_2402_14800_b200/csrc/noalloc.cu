// Beta calibration that allocates nothing.
//
// Some callers of this library must not allocate device memory once they are running: a
// serving process that hands the whole device to its own memory pool at start-up (a later
// cudaMalloc then fails or fragments the pool), or a latency-critical loop that cannot
// afford the device-wide synchronisation cudaMalloc implies.  moe_calibrate_beta grows
// scratch buffers with cudaMalloc on first use, so it is closed to them.  The entry point
// here runs the same two kernels (router, exact median selection) with their scratch in a
// fixed array that is part of the library image: every GPU that loads the library holds
// those bytes until the process exits, which is why the size limit is modest.
#include <mutex>

#include "common.h"

namespace moe {

namespace {

constexpr int kMaxT = MOE_NOALLOC_MAX_TOKENS;

// Layout of the static scratch: what the router writes per token, and the two selected values.
struct StaticScratch {
  int32_t idx[2 * kMaxT];
  float wn[2 * kMaxT];
  float ratio[kMaxT];
  uint8_t skipped[kMaxT];
  float sel[4];
};

// In host code this name is only a handle for cudaGetSymbolAddress, never a device address.
static __device__ __align__(256) unsigned char g_noalloc_scratch[sizeof(StaticScratch)];

constexpr int kMaxDevices = 64;
std::mutex g_mu;
void* g_scratch_ptr[kMaxDevices] = {};

// Device address of the scratch array on the current device, resolved once per device.
int scratch_address(StaticScratch** out) {
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return set_error(MOE_ERR_CUDA, "cudaGetDevice: %s", cudaGetErrorString(e));
  if (dev < 0 || dev >= kMaxDevices) return set_error(MOE_ERR_CUDA, "device index %d not supported", dev);
  std::lock_guard<std::mutex> lock(g_mu);
  if (!g_scratch_ptr[dev]) {
    void* p = nullptr;
    e = cudaGetSymbolAddress(&p, g_noalloc_scratch);
    if (e != cudaSuccess || !p)
      return set_error(MOE_ERR_CUDA, "cudaGetSymbolAddress(static scratch): %s", cudaGetErrorString(e));
    g_scratch_ptr[dev] = p;
  }
  *out = static_cast<StaticScratch*>(g_scratch_ptr[dev]);
  return MOE_OK;
}

}  // namespace

}  // namespace moe

using namespace moe;

extern "C" int moe_calibrate_beta_noalloc(const void* W_gate_kept, const void* x, int T, int h,
                                          int r, void* cuda_stream, float* beta_out) {
  if (!W_gate_kept || !x || !beta_out)
    return set_error(MOE_ERR_INVALID_ARG, "W_gate_kept, x or beta_out is NULL");
  if ((reinterpret_cast<uintptr_t>(W_gate_kept) & 15u) || (reinterpret_cast<uintptr_t>(x) & 15u))
    return set_error(MOE_ERR_INVALID_ARG, "W_gate_kept and x must be 16-byte aligned");
  if (r < 2 || r > kMaxE) return set_error(MOE_ERR_INVALID_ARG, "r = %d outside 2..%d", r, kMaxE);
  if (h < 8 || h % 8) return set_error(MOE_ERR_UNSUPPORTED_SHAPE, "h = %d must be a positive multiple of 8", h);
  if (T < 1) return set_error(MOE_ERR_INVALID_ARG, "T = %d: at least one calibration token is needed", T);
  if (T > kMaxT)
    return set_error(MOE_ERR_INVALID_ARG,
                     "T = %d exceeds the %d tokens the static scratch holds; use moe_calibrate_beta", T,
                     kMaxT);
  StaticScratch* s = nullptr;
  int rc = scratch_address(&s);
  if (rc) return rc;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  KeptIds ids;
  for (int c = 0; c < kMaxE; ++c) ids.id[c] = c;
  RouteOut ro = {};
  ro.idx = s->idx;
  ro.wn = s->wn;
  ro.ratio = s->ratio;
  ro.skipped = s->skipped;
  // Every element the selection reads (ratio[0..T)) is written by the router first, so stale
  // contents of an earlier call are never seen and nothing needs clearing.
  cudaError_t e = launch_router(static_cast<const bf16*>(x), static_cast<const bf16*>(W_gate_kept),
                                T, h, r, 0.f, ids, ro, st);
  if (e != cudaSuccess) return set_error(MOE_ERR_CUDA, "router launch: %s", cudaGetErrorString(e));
  e = launch_select2(s->ratio, T, (T - 1) / 2, T / 2, s->sel, st);
  if (e != cudaSuccess) return set_error(MOE_ERR_CUDA, "select launch: %s", cudaGetErrorString(e));
  float v[2] = {0.f, 0.f};
  e = cudaMemcpyAsync(v, s->sel, sizeof(v), cudaMemcpyDeviceToHost, st);
  if (e == cudaSuccess) e = cudaStreamSynchronize(st);
  if (e != cudaSuccess) return set_error(MOE_ERR_CUDA, "reading the result: %s", cudaGetErrorString(e));
  *beta_out = (T & 1) ? v[0] : (float)(((double)v[0] + (double)v[1]) * 0.5);
  return MOE_OK;
}
