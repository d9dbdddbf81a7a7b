// moe_vqlr_route_noalloc: router scores + top-k + affinities for callers that cannot allocate.
//
// Some callers of this library may not call cudaMalloc at all: code that runs while a memory
// pool owns the whole device, plug-ins loaded into a serving process whose allocator must see
// every byte, or hosts that forbid driver allocations after start-up.  moe_vqlr_create()
// allocates a workspace, so such callers cannot use it.  This entry point is the routing step
// of the layer on its own, with the one piece of scratch it needs -- the [T][E] fp32 logits
// that the scoring kernel writes and the top-k kernel reads -- placed in a fixed array in the
// library's device data segment.  Nothing is allocated or freed here, by the CUDA runtime or
// by any other library.
//
// Consequences of the fixed array, all part of the contract:
//   * sizes are bounded: T <= 16 tokens, E <= 1024 experts (64 KiB); larger requests are
//     rejected with MOE_VQLR_ERR_UNSUPPORTED before anything is launched;
//   * every GPU that loads the library holds the 64 KiB until the process exits;
//   * the array is shared by every call on a device and keeps the previous call's contents.
//     A call overwrites all T*E entries it later reads, so nothing needs clearing, but two
//     calls that overlap on the GPU (different streams, or different host threads) race on
//     it: serialise them;
//   * the first call on each device looks up the array's device address (a runtime query, no
//     allocation).  Make that first call outside any stream capture.
#include "moe_vqlr.h"

#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <mutex>

namespace {

constexpr int kNaMaxT = 16;
constexpr int kNaMaxE = 1024;
constexpr int kNaMaxK = 32;
constexpr int kNaMaxDevices = 64;

// Scratch for the logits.  In host code this name is only a handle for the runtime's symbol
// queries, never a device address: the kernels get the pointer that cudaGetSymbolAddress returns.
static __device__ __align__(256) float g_na_logits[kNaMaxT * kNaMaxE];

std::mutex g_na_mutex;
float* g_na_ptr[kNaMaxDevices];   // device address of g_na_logits per device, filled on first use

typedef __nv_bfloat16 bf16;

__device__ __forceinline__ float na_lo(uint32_t u) { return __uint_as_float(u << 16); }
__device__ __forceinline__ float na_hi(uint32_t u) { return __uint_as_float(u & 0xffff0000u); }

__device__ __forceinline__ float na_dot8(const uint4& a, const uint4& b, float acc) {
  acc = fmaf(na_lo(a.x), na_lo(b.x), acc); acc = fmaf(na_hi(a.x), na_hi(b.x), acc);
  acc = fmaf(na_lo(a.y), na_lo(b.y), acc); acc = fmaf(na_hi(a.y), na_hi(b.y), acc);
  acc = fmaf(na_lo(a.z), na_lo(b.z), acc); acc = fmaf(na_hi(a.z), na_hi(b.z), acc);
  acc = fmaf(na_lo(a.w), na_lo(b.w), acc); acc = fmaf(na_hi(a.w), na_hi(b.w), acc);
  return acc;
}

// One warp per expert row, all tokens; writes logits[t][e] into the scratch.
__global__ void __launch_bounds__(256)
k_na_logits(const bf16* __restrict__ x, const bf16* __restrict__ router_w,
            const float* __restrict__ bias, int T, int E, int H, float* __restrict__ logits) {
  const int lane = threadIdx.x & 31;
  const int e = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  if (e >= E) return;
  const uint4* w4 = reinterpret_cast<const uint4*>(router_w + (size_t)e * H);
  const float b = bias ? bias[e] : 0.f;
  for (int t = 0; t < T; ++t) {
    const uint4* x4 = reinterpret_cast<const uint4*>(x + (size_t)t * H);
    float acc = 0.f;
    for (int c = lane; c < H / 8; c += 32) acc = na_dot8(__ldg(w4 + c), __ldg(x4 + c), acc);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
    if (lane == 0) logits[(size_t)t * E + e] = acc + b;
  }
}

// One warp per token: k rounds of arg-max over the scratch row, order (logit descending, id
// ascending); affinities = softmax over the selected logits (renorm) or over all E.
__global__ void __launch_bounds__(32 * kNaMaxT)
k_na_topk(const float* __restrict__ logits, int T, int E, int k, int renorm,
          int32_t* __restrict__ topk_id, float* __restrict__ topk_w) {
  const int lane = threadIdx.x & 31, t = threadIdx.x >> 5;
  if (t >= T) return;
  const float* row = logits + (size_t)t * E;
  unsigned int taken = 0;          // bit j: expert lane + 32*j already selected (E <= 1024)
  float sel_l = -INFINITY;
  int sel_id = 0;
  for (int s = 0; s < k; ++s) {
    float bv = -INFINITY;
    int bi = 0x7fffffff;
    for (int e = lane, j = 0; e < E; e += 32, ++j) {
      const float v = row[e];
      if (!((taken >> j) & 1u) && v > bv) { bv = v; bi = e; }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      const float ov = __shfl_xor_sync(0xffffffffu, bv, o);
      const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
      if (ov > bv || (ov == bv && oi < bi)) { bv = ov; bi = oi; }
    }
    if (bi >= E) bi = s;           // only NaN / -inf left: stay in bounds
    if (lane == (bi & 31)) taken |= 1u << (bi >> 5);
    if (lane == s) { sel_l = bv; sel_id = bi; }
  }
  const float lmax = __shfl_sync(0xffffffffu, sel_l, 0);
  const float ev = lane < k ? expf(sel_l - lmax) : 0.f;
  float denom = ev;
  if (!renorm)
    for (int e = lane, j = 0; e < E; e += 32, ++j)
      if (!((taken >> j) & 1u) && row[e] != -INFINITY) denom += expf(row[e] - lmax);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) denom += __shfl_xor_sync(0xffffffffu, denom, o);
  if (lane < k) {
    topk_id[(size_t)t * k + lane] = sel_id;
    topk_w[(size_t)t * k + lane] = ev / denom;
  }
}

}  // namespace

extern "C" int moe_vqlr_route_noalloc(const void* x, const void* router_w, const float* router_bias,
                                      int32_t T, int32_t E, int32_t H, int32_t k, int32_t renorm_topk,
                                      int32_t* topk_id, float* topk_w, void* cuda_stream) {
  if (!x || !router_w || !topk_id || !topk_w) return MOE_VQLR_ERR_INVALID_ARG;
  if (T < 1 || E < 1 || H < 8 || (H % 8) || k < 1 || k > E) return MOE_VQLR_ERR_INVALID_ARG;
  if (((reinterpret_cast<uintptr_t>(x) | reinterpret_cast<uintptr_t>(router_w)) & 15u) != 0)
    return MOE_VQLR_ERR_INVALID_ARG;
  if (T > kNaMaxT || E > kNaMaxE || k > kNaMaxK) return MOE_VQLR_ERR_UNSUPPORTED;   // beyond the fixed scratch

  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kNaMaxDevices) return MOE_VQLR_ERR_CUDA;
  float* scratch;
  {
    std::lock_guard<std::mutex> lock(g_na_mutex);
    if (!g_na_ptr[dev]) {   // first call on this device, with it current: resolve the symbol
      void* p = nullptr;
      if (cudaGetSymbolAddress(&p, g_na_logits) != cudaSuccess || !p) {
        cudaGetLastError();
        return MOE_VQLR_ERR_CUDA;
      }
      g_na_ptr[dev] = static_cast<float*>(p);
    }
    scratch = g_na_ptr[dev];
  }
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  k_na_logits<<<(E + 7) / 8, 256, 0, st>>>(static_cast<const bf16*>(x), static_cast<const bf16*>(router_w),
                                            router_bias, T, E, H, scratch);
  k_na_topk<<<1, 32 * T, 0, st>>>(scratch, T, E, k, renorm_topk ? 1 : 0, topk_id, topk_w);
  return cudaGetLastError() == cudaSuccess ? MOE_VQLR_OK : MOE_VQLR_ERR_CUDA;
}
