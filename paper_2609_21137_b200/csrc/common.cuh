// Shared definitions of the CUDA kernels: parameter block, bf16 helpers, warp reductions.
#pragma once
#include "moe_vqlr.h"
#ifndef __CUDACC_RTC__       // the run-time compiler has the device built-ins and takes no host headers
#include "moe_vqlr_bench.h"
#include <cuda_runtime.h>
#include <stdint.h>
#endif
#include <cuda_bf16.h>
#include <math_constants.h>

namespace {

constexpr int kMaxT = 16;      // tokens per call
constexpr int kMaxK = 32;      // experts per token
constexpr int kD = 8;          // VQ block length (one code word = 16 bytes of bf16)
constexpr int kTokGroup = 4;   // tokens of one expert handled per pass over its row
constexpr int kStages = 6;     // router_z, route, gateup, zdown, down, combine
const char* const kStageNames[kStages] = {"router_z", "route", "gateup", "zdown", "down", "combine"};

typedef __nv_bfloat16 bf16;

struct ProjDev {
  int kind;
  int out_dim, in_dim;
  int zslot;               // which z slot feeds the low-rank term (gate/up), -1 if none
  const uint4* codebook;   // [K] code words of 8 bf16 (d = 4: [K] words of 4 bf16, read as uint2)
  const void* idx;
  const bf16* basis;
  const bf16* factor;
  const bf16* dense;
};

struct Params {
  int H, I, E, k, S, K, r, renorm;
  int act;                 // expert activation: 0 = SiLU, 1 = GELU (tanh form), 2 = up-only experts, p = relu(u)^2
                           // (the gate projection then aliases up: kernels that know skip its work, the rest repeat it)
  int d;                   // VQ block length: 8 (one code word = 16 bytes) or 4 (8 bytes)
  int idx12;               // index maps hold 12-bit indices, two to three bytes (256 < K <= 4096); the uint16 kernels run
  int z_repeat;            // 1; ablation: every basis projection is computed this many times (once per selected expert)
  int n_zrows;             // rows of the stacked basis projection: (distinct gate/up bases) * r
  const bf16* router_w;
  const float* router_bias;
  ProjDev gate, up, down;
  // workspace
  float* logits;           // [maxT][E]
  float* z;                // [maxT][2][r]
  int* topk_id;            // [maxT][k]
  float* topk_w;           // [maxT][k]
  int* counts;             // [E]
  int* offsets;            // [E+1]
  int* pair_token;         // [maxT*(k+S)]  routed pairs sorted by expert, then shared experts' pairs
  int* pair_slot;          // [maxT*(k+S)]
  float* pair_w;           // [maxT*(k+S)]
  int* act_n;              // [1] number of active experts (routed with >=1 pair, then shared)
  int* act_e;              // [E+S] expert id
  int* act_off;            // [E+S] first pair position
  int* act_cnt;            // [E+S] pairs
  int* grp_n;              // [1] work groups of the tensor-core chain: (expert, first pair, <= 8 pairs)
  int* grp_e;              // [maxT*(k+S)]
  int* grp_off;            // [maxT*(k+S)]
  int* grp_cnt;            // [maxT*(k+S)]
  float* p;                // [maxT*(k+S)][I]   SwiGLU intermediate per pair position
  bf16* p_hi;              // [maxT*(k+S)][I]   p rounded to bf16 ...
  bf16* p_lo;              // [maxT*(k+S)][I]   ... and the bf16 remainder (p = hi + lo to 2^-17)
  float* zd;               // [maxT*(k+S)][r]   basis_down * p per pair position
  float* gpart;            // [parts][maxT*(k+S)][I]  partial gate tiles of the tensor-core chain
  float* upart;            // [parts][maxT*(k+S)][I]  partial up tiles
  float* ypart;            // [parts][maxT*(k+S)][H]  partial down tiles, by pair position
  float* zd_part;          // [maxT*(k+S)][slices][r] partial z_d of the fused kernel's slices
  int* inv_pos;            // [maxT][k+S]       pair position of (token, slot)
  int* status;             // [1] in pinned host memory mapped into the device: 0, or the code a kernel recorded
  int spin_limit;          // polls after which a device-side wait gives up (MOE_VQLR_ERR_TIMEOUT)
  int bar_fault;           // test switch: the persistent kernel's barriers wait for one arrival too many
  unsigned int* grid_bar;  // [2] arrivals and generation of the cooperative kernel's grid barrier
  long long* clk;          // optional phase stamps [kernel 4][block][warp 16][stamp 16], or NULL
  int clk_blocks;
};

#ifdef MOE_VQLR_JIT
// Run-time-compiled copies of the kernels know the layer: every integer of the parameter block is
// a constant of the compilation (the pointers stay arguments, so one copy serves all layers of a
// shape).
#define MOE_VQLR_JIT_PARAMS(P)                                                                          \
  do {                                                                                                  \
    (P).H = J_H; (P).I = J_I; (P).E = J_E; (P).k = J_TOPK; (P).S = J_S; (P).K = J_K; (P).r = J_R;       \
    (P).renorm = J_RENORM; (P).act = J_ACT; (P).d = J_D; (P).idx12 = J_IDX12; (P).z_repeat = J_ZREPEAT; \
    (P).n_zrows = J_NZROWS; (P).gate.zslot = J_ZSLOT_G; (P).up.zslot = J_ZSLOT_U;                       \
  } while (0)
#endif

// The model-specific expert activation phi applied to the gate output (Section 2.1):
// p = phi(g) * u.  act is uniform over the launch.
__device__ __forceinline__ float gated_act(float g, float u, int act) {
  if (act == 2) {                       // up-only experts (Section 5.7): the gate value is not used
    const float v = fmaxf(u, 0.f);
    return v * v;
  }
  if (act == 1) {
    const float t = tanhf(0.7978845608028654f * (g + 0.044715f * g * g * g));
    return 0.5f * g * (1.f + t) * u;
  }
  return g / (1.f + expf(-g)) * u;      // silu(g) * u
}

// Records a device-detected condition for the host (moe_vqlr_last_status).  The word lives in
// host memory, so it is a plain store: whichever block writes last wins, and every writer of a call
// reports a failure of that call.
__device__ __forceinline__ void set_status(const Params& P, int code) { *reinterpret_cast<volatile int*>(P.status) = code; }

// Optional tracing: lane 0 of a warp stores clock64() at phase `k` of kernel `kern`.
__device__ __forceinline__ void stamp(const long long* base_c, int clk_blocks, int kern, int k) {
  long long* base = const_cast<long long*>(base_c);
  if (base && (threadIdx.x & 31) == 0 && k < 16 && (int)blockIdx.x < clk_blocks && (threadIdx.x >> 5) < 16)
  {
#ifdef MOE_VQLR_TRACE_GLOBAL      // nanoseconds of the device-wide timer: comparable across SMs and kernels
    long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
#else
    const long long t = clock64();
#endif
    base[(((size_t)kern * clk_blocks + blockIdx.x) * 16 + (threadIdx.x >> 5)) * 16 + k] = t;
  }
}

__device__ __forceinline__ float bf_lo(uint32_t u) { return __uint_as_float(u << 16); }
__device__ __forceinline__ float bf_hi(uint32_t u) { return __uint_as_float(u & 0xffff0000u); }

__device__ __forceinline__ void unpack8(const uint4& v, float (&f)[8]) {
  f[0] = bf_lo(v.x); f[1] = bf_hi(v.x); f[2] = bf_lo(v.y); f[3] = bf_hi(v.y);
  f[4] = bf_lo(v.z); f[5] = bf_hi(v.z); f[6] = bf_lo(v.w); f[7] = bf_hi(v.w);
}

__device__ __forceinline__ float dot8(const float (&a)[8], const float (&b)[8], float acc) {
#pragma unroll
  for (int j = 0; j < 8; ++j) acc = fmaf(a[j], b[j], acc);
  return acc;
}

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// Twelve-bit packed index maps (the index width between one and two bytes: the deployed width
// changes only at an encoding boundary of K).  Indices 2q and 2q+1 of a map occupy bytes 3q..3q+2,
// little end first, i.e. a run of eight indices is a 96-bit little-endian number of 12-bit fields.
// Element `elem` (even) of a map that the kernels otherwise address as IdxT:
template <typename IdxT>
__device__ __forceinline__ const IdxT* idx_at(const IdxT* base, size_t elem, int idx12) {
  return idx12 ? reinterpret_cast<const IdxT*>(reinterpret_cast<const unsigned char*>(base) + (elem >> 1) * 3) : base + elem;
}
__device__ __forceinline__ void unpack_idx12x8(uint32_t w0, uint32_t w1, uint32_t w2, uint32_t (&id)[8]) {
  id[0] = w0 & 0xfffu;          id[1] = (w0 >> 12) & 0xfffu;
  id[2] = (w0 >> 24) | ((w1 & 0xfu) << 8);
  id[3] = (w1 >> 4) & 0xfffu;   id[4] = (w1 >> 16) & 0xfffu;
  id[5] = (w1 >> 28) | ((w2 & 0xffu) << 4);
  id[6] = (w2 >> 8) & 0xfffu;   id[7] = w2 >> 20;
}
// One index of a packed map (element `elem` counted from `base`).
__device__ __forceinline__ uint32_t read_idx12(const void* base, size_t elem) {
  const unsigned char* b = static_cast<const unsigned char*>(base) + (elem >> 1) * 3;
  return (elem & 1) ? ((uint32_t)b[1] >> 4) | ((uint32_t)b[2] << 4) : (uint32_t)b[0] | (((uint32_t)b[1] & 0xfu) << 8);
}

// Position of 16-byte block b of an activation row in shared memory.  Lane l of a warp walks
// blocks 8l..8l+7; XOR-ing the low three bits with l keeps the eight lanes of a quarter warp on
// distinct bank groups.
__device__ __forceinline__ int swz(int b) { return b ^ ((b >> 3) & 7); }

}  // namespace
