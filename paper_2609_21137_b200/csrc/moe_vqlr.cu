// One routed MoE decode layer on VQ + shared-basis low-rank expert weights (sm_100a).
// Host side of the C ABI declared in include/moe_vqlr.h plus the kernels it launches.
//
// Kernel chain of one call (all on the caller's stream):
//   k_router_z   router logits and the shared rank-r projections z = basis * x   (Section 4.1:
//                the work that does not depend on the routing decision)
//   k_route      top-k, affinities, grouping of (token, slot) pairs by expert
//   k_gateup     gate/up rows of every activated expert straight from indices + code book,
//                low-rank term joined in the same accumulator, SwiGLU               (Eq. 1)
//   k_zdown      z_d = basis_down * p per pair (only when the down projection is VQ+LR)
//   k_down       down rows over all activated experts with the affinity-weighted sum fused in
#include "moe_vqlr.h"

#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <cstdarg>
#include <cstdio>
#include <cstring>
#include <new>
#include <string>

namespace {

constexpr int kMaxT = 16;      // tokens per call
constexpr int kMaxK = 32;      // experts per token
constexpr int kD = 8;          // VQ block length (one code word = 16 bytes of bf16)
constexpr int kTokGroup = 4;   // tokens of one expert handled per pass over its row
constexpr int kStages = 5;     // router_z, route, gateup, zdown, down
const char* const kStageNames[kStages] = {"router_z", "route", "gateup", "zdown", "down"};

typedef __nv_bfloat16 bf16;

struct ProjDev {
  int kind;
  int out_dim, in_dim;
  int zslot;               // which z slot feeds the low-rank term (gate/up), -1 if none
  const uint4* codebook;   // [K] code words of 8 bf16
  const void* idx;
  const bf16* basis;
  const bf16* factor;
  const bf16* dense;
};

struct Params {
  int H, I, E, k, S, K, r, renorm;
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
  float* p;                // [maxT*(k+S)][I]   SwiGLU intermediate per pair position
  float* zd;               // [maxT*(k+S)][r]   basis_down * p per pair position
  int* status;             // [1]
};

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

// Position of 16-byte block b of an activation row in shared memory.  Lane l of a warp walks
// blocks 8l..8l+7; XOR-ing the low three bits with l keeps the eight lanes of a quarter warp on
// distinct bank groups.
__device__ __forceinline__ int swz(int b) { return b ^ ((b >> 3) & 7); }

// ---------------------------------------------------------------------------------------------
// k_router_z: one warp per row of [router_w ; basis_gate ; basis_up], all T tokens.
// The summation order of a row is fixed (lane-strided chunks, then an xor butterfly), so two
// identical router rows give bitwise identical logits.
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) k_router_z(const Params P, const bf16* __restrict__ x, int T) {
  const int lane = threadIdx.x & 31;
  const int row = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  if (row >= P.E + P.n_zrows) return;
  const bf16* wrow;
  float* dst;
  int dst_stride;
  float bias = 0.f;
  if (row < P.E) {
    wrow = P.router_w + (size_t)row * P.H;
    dst = P.logits + row;
    dst_stride = P.E;
    if (P.router_bias) bias = P.router_bias[row];
  } else {
    const int q = row - P.E;
    const int slot = q / P.r, rho = q - slot * P.r;
    const bf16* basis = (slot == P.gate.zslot && P.gate.basis) ? P.gate.basis : P.up.basis;
    wrow = basis + (size_t)rho * P.H;
    dst = P.z + slot * P.r + rho;
    dst_stride = 2 * P.r;
  }
  const int nchunk = P.H / 8;
  const uint4* w4 = reinterpret_cast<const uint4*>(wrow);
  for (int t0 = 0; t0 < T; t0 += kTokGroup) {
    float acc[kTokGroup] = {0.f, 0.f, 0.f, 0.f};
    for (int c = lane; c < nchunk; c += 32) {
      float wf[8];
      unpack8(__ldg(w4 + c), wf);
#pragma unroll
      for (int tt = 0; tt < kTokGroup; ++tt) {
        if (t0 + tt < T) {
          float xf[8];
          unpack8(__ldg(reinterpret_cast<const uint4*>(x + (size_t)(t0 + tt) * P.H) + c), xf);
          acc[tt] = dot8(wf, xf, acc[tt]);
        }
      }
    }
#pragma unroll
    for (int tt = 0; tt < kTokGroup; ++tt) {
      const float s = warp_sum(acc[tt]);
      if (lane == 0 && t0 + tt < T) dst[(size_t)(t0 + tt) * dst_stride] = s + bias;
    }
  }
}

// ---------------------------------------------------------------------------------------------
// k_route: one block, one warp per token.  Top-k by k rounds of warp arg-max with the order
// (logit descending, id ascending); softmax over the selected logits; counting sort of the
// pairs by expert; compact list of active experts with the shared experts appended.
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(32 * kMaxT) k_route(const Params P, int T) {
  extern __shared__ float s_dyn[];
  float* s_logit = s_dyn;                                  // [T][E]
  int* s_cnt = reinterpret_cast<int*>(s_dyn + T * P.E);    // [E]
  int* s_off = s_cnt + P.E;                                // [E+1]
  __shared__ int s_id[kMaxT * kMaxK];
  __shared__ float s_w[kMaxT * kMaxK];
  const int lane = threadIdx.x & 31, t = threadIdx.x >> 5;
  const int E = P.E, k = P.k;

  if (t < T) {
    for (int e = lane; e < E; e += 32) s_logit[t * E + e] = P.logits[(size_t)t * E + e];
    __syncwarp();
    float sel_l = -INFINITY;
    float rest = 0.f;
    for (int s = 0; s < k; ++s) {
      float bv = -INFINITY;
      int bi = 0x7fffffff;
      for (int e = lane; e < E; e += 32) {
        const float v = s_logit[t * E + e];
        if (v > bv) { bv = v; bi = e; }   // ascending e per lane: strict '>' keeps the lower id
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        const float ov = __shfl_xor_sync(0xffffffffu, bv, o);
        const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
        if (ov > bv || (ov == bv && oi < bi)) { bv = ov; bi = oi; }
      }
      if (bi >= E) {   // only NaN / -inf logits left: keep memory safe and report it
        bi = s;
        if (lane == 0) atomicExch(P.status, MOE_VQLR_ERR_INVALID_ARG);
      }
      if (lane == s) sel_l = bv;
      if (lane == 0) s_id[t * k + s] = bi;
      if (lane == (bi & 31)) s_logit[t * E + bi] = -INFINITY;   // taken
      __syncwarp();
    }
    const float lmax = __shfl_sync(0xffffffffu, sel_l, 0);
    const float ev = lane < k ? expf(sel_l - lmax) : 0.f;
    float denom = warp_sum(ev);
    if (!P.renorm) {
      for (int e = lane; e < E; e += 32) {
        const float v = s_logit[t * E + e];
        if (v != -INFINITY) rest += expf(v - lmax);
      }
      denom += warp_sum(rest);
    }
    if (lane < k) {
      const float w = ev / denom;
      s_w[t * k + lane] = w;
      P.topk_w[t * k + lane] = w;
    }
    __syncwarp();
    if (lane < k) P.topk_id[t * k + lane] = s_id[t * k + lane];
  }
  __syncthreads();

  const int n_pairs = T * k;
  for (int e = threadIdx.x; e < E; e += blockDim.x) {
    int c = 0;
    for (int q = 0; q < n_pairs; ++q) c += (s_id[q] == e);
    s_cnt[e] = c;
  }
  __syncthreads();
  if (threadIdx.x < 32) {
    // exclusive scan of counts and compaction of active experts, `chunk` experts per lane
    const int chunk = (E + 31) / 32;
    const int e0 = lane * chunk, e1 = min(E, e0 + chunk);
    int sum = 0, nact = 0;
    for (int e = e0; e < e1; ++e) { sum += s_cnt[e]; nact += (s_cnt[e] > 0); }
    int psum = sum, pact = nact;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int a = __shfl_up_sync(0xffffffffu, psum, o);
      const int b = __shfl_up_sync(0xffffffffu, pact, o);
      if (lane >= o) { psum += a; pact += b; }
    }
    int run = psum - sum, arun = pact - nact;
    for (int e = e0; e < e1; ++e) {
      s_off[e] = run;
      P.offsets[e] = run;
      P.counts[e] = s_cnt[e];
      if (s_cnt[e] > 0) {
        P.act_e[arun] = e;
        P.act_off[arun] = run;
        P.act_cnt[arun] = s_cnt[e];
        ++arun;
      }
      run += s_cnt[e];
    }
    const int total_act = __shfl_sync(0xffffffffu, pact, 31);
    if (lane == 31) { s_off[E] = psum; P.offsets[E] = psum; }
    // shared experts: every token, weight 1, pair positions after the routed ones
    for (int s = lane; s < P.S; s += 32) {
      P.act_e[total_act + s] = E + s;
      P.act_off[total_act + s] = n_pairs + s * T;
      P.act_cnt[total_act + s] = T;
    }
    if (lane == 0) *P.act_n = total_act + P.S;
  }
  __syncthreads();
  for (int e = threadIdx.x; e < E; e += blockDim.x) {
    int pos = s_off[e];
    if (s_cnt[e] == 0) continue;
    for (int q = 0; q < n_pairs; ++q)
      if (s_id[q] == e) {
        P.pair_token[pos] = q / k;
        P.pair_slot[pos] = q - (q / k) * k;
        P.pair_w[pos] = s_w[q];
        ++pos;
      }
  }
  for (int q = threadIdx.x; q < P.S * T; q += blockDim.x) {
    P.pair_token[n_pairs + q] = q % T;
    P.pair_slot[n_pairs + q] = k + q / T;
    P.pair_w[n_pairs + q] = 1.f;
  }
}

// ---------------------------------------------------------------------------------------------
// Row kernels.  A warp owns one output row of one expert; lane l walks chunks of eight blocks
// (one 16-byte / 8-byte load of uint16 / uint8 indices), looks every code word up in the
// shared-memory code book and multiplies it with the matching activation block.
// ---------------------------------------------------------------------------------------------
template <typename IdxT>
__device__ __forceinline__ void load_idx8(const IdxT* p, uint32_t (&id)[8]);

template <>
__device__ __forceinline__ void load_idx8<uint16_t>(const uint16_t* p, uint32_t (&id)[8]) {
  const uint4 v = __ldg(reinterpret_cast<const uint4*>(p));
  id[0] = v.x & 0xffffu; id[1] = v.x >> 16; id[2] = v.y & 0xffffu; id[3] = v.y >> 16;
  id[4] = v.z & 0xffffu; id[5] = v.z >> 16; id[6] = v.w & 0xffffu; id[7] = v.w >> 16;
}

template <>
__device__ __forceinline__ void load_idx8<uint8_t>(const uint8_t* p, uint32_t (&id)[8]) {
  const uint2 v = __ldg(reinterpret_cast<const uint2*>(p));
  id[0] = v.x & 0xffu; id[1] = (v.x >> 8) & 0xffu; id[2] = (v.x >> 16) & 0xffu; id[3] = v.x >> 24;
  id[4] = v.y & 0xffu; id[5] = (v.y >> 8) & 0xffu; id[6] = (v.y >> 16) & 0xffu; id[7] = v.y >> 24;
}

// VQ part of one row against up to kTokGroup bf16 activation rows held (swizzled) in shared
// memory.  nb = blocks per row.
template <typename IdxT>
__device__ __forceinline__ void vq_row_bf16x(const IdxT* __restrict__ idx_row, int nb,
                                             const uint4* __restrict__ s_cb,
                                             const uint4* __restrict__ s_x, int x_stride,
                                             const int (&tok)[kTokGroup], int nt,
                                             float (&acc)[kTokGroup], int lane) {
  if ((nb & 7) == 0) {
    for (int c = lane; c < (nb >> 3); c += 32) {
      uint32_t id[8];
      load_idx8<IdxT>(idx_row + c * 8, id);
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        float wf[8];
        unpack8(s_cb[id[j]], wf);
        const int b = swz(c * 8 + j);
#pragma unroll
        for (int tt = 0; tt < kTokGroup; ++tt)
          if (tt < nt) {
            float xf[8];
            unpack8(s_x[tok[tt] * x_stride + b], xf);
            acc[tt] = dot8(wf, xf, acc[tt]);
          }
      }
    }
  } else {   // rows whose index run is not a multiple of eight blocks: one index at a time
    for (int b0 = lane; b0 < nb; b0 += 32) {
      float wf[8];
      unpack8(s_cb[idx_row[b0]], wf);
      const int b = swz(b0);
#pragma unroll
      for (int tt = 0; tt < kTokGroup; ++tt)
        if (tt < nt) {
          float xf[8];
          unpack8(s_x[tok[tt] * x_stride + b], xf);
          acc[tt] = dot8(wf, xf, acc[tt]);
        }
    }
  }
}

// Dense bf16 row against bf16 activations in shared memory.
__device__ __forceinline__ void dense_row_bf16x(const bf16* __restrict__ wrow, int nb,
                                                const uint4* __restrict__ s_x, int x_stride,
                                                const int (&tok)[kTokGroup], int nt,
                                                float (&acc)[kTokGroup], int lane) {
  const uint4* w4 = reinterpret_cast<const uint4*>(wrow);
  for (int c = lane; c < nb; c += 32) {
    float wf[8];
    unpack8(__ldg(w4 + c), wf);
    const int b = swz(c);
#pragma unroll
    for (int tt = 0; tt < kTokGroup; ++tt)
      if (tt < nt) {
        float xf[8];
        unpack8(s_x[tok[tt] * x_stride + b], xf);
        acc[tt] = dot8(wf, xf, acc[tt]);
      }
  }
}

// Low-rank part of one row: sum_rho factor[rho] * z[token][rho], z in global memory (fp32).
__device__ __forceinline__ void lr_row(const bf16* __restrict__ frow, int r,
                                       const float* __restrict__ z, int z_stride,
                                       const int (&zrow)[kTokGroup], int nt,
                                       float (&acc)[kTokGroup], int lane) {
  for (int rho = lane; rho < r; rho += 32) {
    const float a = __bfloat162float(frow[rho]);
#pragma unroll
    for (int tt = 0; tt < kTokGroup; ++tt)
      if (tt < nt) acc[tt] = fmaf(a, z[(size_t)zrow[tt] * z_stride + rho], acc[tt]);
  }
}

template <typename IdxT>
__global__ void __launch_bounds__(512, 1)
k_gateup(const Params P, const bf16* __restrict__ x, int T, int two_books) {
  extern __shared__ uint4 s_u4[];
  const int nbH = P.H / kD;
  uint4* s_cb_g = s_u4;
  uint4* s_cb_u = two_books ? s_u4 + P.K : s_u4;
  const int n_cb = (P.gate.kind == MOE_VQLR_PROJ_VQLR || P.up.kind == MOE_VQLR_PROJ_VQLR)
                       ? (two_books ? 2 : 1) : 0;
  uint4* s_x = s_u4 + (size_t)n_cb * P.K;

  if (n_cb) {
    const uint4* src_g = P.gate.kind == MOE_VQLR_PROJ_VQLR ? P.gate.codebook : P.up.codebook;
    for (int i = threadIdx.x; i < P.K; i += blockDim.x) s_cb_g[i] = __ldg(src_g + i);
    if (two_books)
      for (int i = threadIdx.x; i < P.K; i += blockDim.x) s_cb_u[i] = __ldg(P.up.codebook + i);
  }
  const int xs = (nbH + 7) & ~7;   // row stride in blocks: the swizzle permutes within groups of 8
  const uint4* x4 = reinterpret_cast<const uint4*>(x);
  for (int i = threadIdx.x; i < T * nbH; i += blockDim.x) {
    const int t = i / nbH, b = i - t * nbH;
    s_x[t * xs + swz(b)] = __ldg(x4 + i);
  }
  __syncthreads();

  const int lane = threadIdx.x & 31;
  const int warps_per_block = blockDim.x >> 5;
  const int gwarp = blockIdx.x * warps_per_block + (threadIdx.x >> 5);
  const int nwarps = gridDim.x * warps_per_block;
  const int n_act = *P.act_n;
  const long long total = (long long)n_act * P.I;
  for (long long w = gwarp; w < total; w += nwarps) {
    const int a = (int)(w / P.I), i = (int)(w - (long long)a * P.I);
    const int e = P.act_e[a], off = P.act_off[a], cnt = P.act_cnt[a];
    const size_t row = (size_t)e * P.I + i;
    for (int q0 = 0; q0 < cnt; q0 += kTokGroup) {
      const int nt = min(kTokGroup, cnt - q0);
      int tok[kTokGroup];
#pragma unroll
      for (int tt = 0; tt < kTokGroup; ++tt) tok[tt] = tt < nt ? P.pair_token[off + q0 + tt] : 0;
      float g[kTokGroup] = {0.f, 0.f, 0.f, 0.f}, u[kTokGroup] = {0.f, 0.f, 0.f, 0.f};
      if (P.gate.kind == MOE_VQLR_PROJ_VQLR) {
        vq_row_bf16x<IdxT>(static_cast<const IdxT*>(P.gate.idx) + row * nbH, nbH, s_cb_g, s_x, xs,
                           tok, nt, g, lane);
        if (P.gate.zslot >= 0)
          lr_row(P.gate.factor + row * P.r, P.r, P.z + P.gate.zslot * P.r, 2 * P.r, tok, nt, g, lane);
      } else {
        dense_row_bf16x(P.gate.dense + row * P.H, nbH, s_x, xs, tok, nt, g, lane);
      }
      if (P.up.kind == MOE_VQLR_PROJ_VQLR) {
        vq_row_bf16x<IdxT>(static_cast<const IdxT*>(P.up.idx) + row * nbH, nbH, s_cb_u, s_x, xs,
                           tok, nt, u, lane);
        if (P.up.zslot >= 0)
          lr_row(P.up.factor + row * P.r, P.r, P.z + P.up.zslot * P.r, 2 * P.r, tok, nt, u, lane);
      } else {
        dense_row_bf16x(P.up.dense + row * P.H, nbH, s_x, xs, tok, nt, u, lane);
      }
#pragma unroll
      for (int tt = 0; tt < kTokGroup; ++tt) {
        const float gs = warp_sum(g[tt]), us = warp_sum(u[tt]);
        if (lane == 0 && tt < nt)
          P.p[(size_t)(off + q0 + tt) * P.I + i] = gs / (1.f + expf(-gs)) * us;   // silu(g) * u
      }
    }
  }
}

// z_d[pos][rho] = <basis_down[rho], p[pos]>: the low-rank input of a compressed down
// projection depends on the expert's own intermediate, so it is computed per pair.
__global__ void __launch_bounds__(256) k_zdown(const Params P, int n_pos) {
  const int lane = threadIdx.x & 31;
  const int w = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  if (w >= n_pos * P.r) return;
  const int pos = w / P.r, rho = w - pos * P.r;
  const bf16* brow = P.down.basis + (size_t)rho * P.I;
  const float* prow = P.p + (size_t)pos * P.I;
  float acc = 0.f;
  for (int i = lane; i < P.I; i += 32) acc = fmaf(__bfloat162float(brow[i]), prow[i], acc);
  acc = warp_sum(acc);
  if (lane == 0) P.zd[(size_t)pos * P.r + rho] = acc;
}

// k_down: a warp owns output row h for ALL activated experts and tokens, so the weighted sum
// over experts (Section 2.1) happens in its own accumulators in a fixed order (experts
// ascending, tokens ascending): no atomics, bitwise repeatable.
template <typename IdxT>
__global__ void __launch_bounds__(512, 1)
k_down(const Params P, bf16* __restrict__ out, int T) {
  extern __shared__ uint4 s_u4[];
  uint4* s_cb = s_u4;
  const bool vq = P.down.kind == MOE_VQLR_PROJ_VQLR;
  float* s_acc = reinterpret_cast<float*>(s_u4 + (vq ? P.K : 0));   // [warps][kMaxT]
  if (vq)
    for (int i = threadIdx.x; i < P.K; i += blockDim.x) s_cb[i] = __ldg(P.down.codebook + i);
  for (int i = threadIdx.x; i < (blockDim.x >> 5) * kMaxT; i += blockDim.x) s_acc[i] = 0.f;
  __syncthreads();

  const int lane = threadIdx.x & 31, wib = threadIdx.x >> 5;
  const int warps_per_block = blockDim.x >> 5;
  const int nwarps = gridDim.x * warps_per_block;
  const int n_act = *P.act_n;
  const int nbI = P.I / kD;
  float* my_acc = s_acc + wib * kMaxT;
  for (int h = blockIdx.x * warps_per_block + wib; h < P.H; h += nwarps) {
    for (int a = 0; a < n_act; ++a) {
      const int e = P.act_e[a], off = P.act_off[a], cnt = P.act_cnt[a];
      const size_t row = (size_t)e * P.H + h;
      for (int q = 0; q < cnt; ++q) {
        const int pos = off + q;
        const float* prow = P.p + (size_t)pos * P.I;
        float acc = 0.f;
        if (vq) {
          const IdxT* idx_row = static_cast<const IdxT*>(P.down.idx) + row * nbI;
          if ((nbI & 7) == 0) {
            for (int c = lane; c < (nbI >> 3); c += 32) {
              uint32_t id[8];
              load_idx8<IdxT>(idx_row + c * 8, id);
#pragma unroll
              for (int j = 0; j < 8; ++j) {
                float wf[8];
                unpack8(s_cb[id[j]], wf);
                const float4 p0 = *reinterpret_cast<const float4*>(prow + (c * 8 + j) * 8);
                const float4 p1 = *reinterpret_cast<const float4*>(prow + (c * 8 + j) * 8 + 4);
                const float pf[8] = {p0.x, p0.y, p0.z, p0.w, p1.x, p1.y, p1.z, p1.w};
                acc = dot8(wf, pf, acc);
              }
            }
          } else {
            for (int b = lane; b < nbI; b += 32) {
              float wf[8];
              unpack8(s_cb[idx_row[b]], wf);
              const float4 p0 = *reinterpret_cast<const float4*>(prow + b * 8);
              const float4 p1 = *reinterpret_cast<const float4*>(prow + b * 8 + 4);
              const float pf[8] = {p0.x, p0.y, p0.z, p0.w, p1.x, p1.y, p1.z, p1.w};
              acc = dot8(wf, pf, acc);
            }
          }
          if (P.r > 0 && P.down.factor) {
            const bf16* frow = P.down.factor + row * P.r;
            const float* zrow = P.zd + (size_t)pos * P.r;
            for (int rho = lane; rho < P.r; rho += 32)
              acc = fmaf(__bfloat162float(frow[rho]), zrow[rho], acc);
          }
        } else {
          const uint4* w4 = reinterpret_cast<const uint4*>(P.down.dense + row * P.I);
          for (int c = lane; c < nbI; c += 32) {
            float wf[8];
            unpack8(__ldg(w4 + c), wf);
            const float4 p0 = *reinterpret_cast<const float4*>(prow + c * 8);
            const float4 p1 = *reinterpret_cast<const float4*>(prow + c * 8 + 4);
            const float pf[8] = {p0.x, p0.y, p0.z, p0.w, p1.x, p1.y, p1.z, p1.w};
            acc = dot8(wf, pf, acc);
          }
        }
        acc = warp_sum(acc);
        if (lane == 0) my_acc[P.pair_token[pos]] += P.pair_w[pos] * acc;
      }
    }
    __syncwarp();
    if (lane < T) {
      out[(size_t)lane * P.H + h] = __float2bfloat16_rn(my_acc[lane]);
      my_acc[lane] = 0.f;
    }
    __syncwarp();
  }
}

// Largest index of an index map (create-time validation only).
template <typename IdxT>
__global__ void k_max_index(const IdxT* __restrict__ idx, size_t n, unsigned int* out) {
  unsigned int m = 0;
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n;
       i += (size_t)gridDim.x * blockDim.x)
    m = max(m, (unsigned int)idx[i]);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) m = max(m, __shfl_xor_sync(0xffffffffu, m, o));
  if ((threadIdx.x & 31) == 0) atomicMax(out, m);
}

thread_local std::string g_create_error;

}  // namespace

struct moe_vqlr_handle {
  moe_vqlr_config cfg;
  Params P;
  int device;
  int sm_count;
  int idx_bytes;
  int two_books;
  size_t smem_gateup_per_token, smem_gateup_fixed, smem_down;
  void* workspace;
  size_t workspace_bytes;
  bf16* x_stage;     // [maxT][H] device staging for the host-buffer entry point
  bf16* out_stage;   // [maxT][H]
  int64_t launches;
  int profiling;             // record an event after every stage of a call
  cudaEvent_t ev[kStages + 1];
  bool ev_valid;
  bool stage_ran[kStages];
  std::string error;
};

namespace {

int fail(moe_vqlr_handle* h, int code, const char* fmt, ...) {
  char buf[512];
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(buf, sizeof buf, fmt, ap);
  va_end(ap);
  if (h) h->error = buf; else g_create_error = buf;
  return code;
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

int check_proj(const moe_vqlr_proj& p, const char* name, int rank) {
  if (p.kind == MOE_VQLR_PROJ_VQLR) {
    if (!p.codebook || !p.idx) return fail(nullptr, MOE_VQLR_ERR_INVALID_ARG, "%s: codebook/idx is null", name);
    if (rank > 0 && (!p.basis || !p.factor))
      return fail(nullptr, MOE_VQLR_ERR_INVALID_ARG, "%s: rank > 0 but basis/factor is null", name);
    if (!aligned16(p.codebook) || !aligned16(p.idx) || !aligned16(p.basis) || !aligned16(p.factor))
      return fail(nullptr, MOE_VQLR_ERR_INVALID_ARG, "%s: pointers must be 16-byte aligned", name);
  } else if (p.kind == MOE_VQLR_PROJ_DENSE_BF16) {
    if (!p.dense) return fail(nullptr, MOE_VQLR_ERR_INVALID_ARG, "%s: dense is null", name);
    if (!aligned16(p.dense)) return fail(nullptr, MOE_VQLR_ERR_INVALID_ARG, "%s: dense must be 16-byte aligned", name);
  } else {
    return fail(nullptr, MOE_VQLR_ERR_INVALID_ARG, "%s: unknown kind %d", name, p.kind);
  }
  return MOE_VQLR_OK;
}

ProjDev make_proj(const moe_vqlr_proj& p, int out_dim, int in_dim) {
  ProjDev d;
  d.kind = p.kind;
  d.out_dim = out_dim;
  d.in_dim = in_dim;
  d.zslot = -1;
  d.codebook = static_cast<const uint4*>(p.codebook);
  d.idx = p.idx;
  d.basis = static_cast<const bf16*>(p.basis);
  d.factor = static_cast<const bf16*>(p.factor);
  d.dense = static_cast<const bf16*>(p.dense);
  return d;
}

template <typename T>
T* carve(char*& cur, size_t n) {
  T* p = reinterpret_cast<T*>(cur);
  cur += (n * sizeof(T) + 255) / 256 * 256;
  return p;
}

}  // namespace

extern "C" {

int moe_vqlr_create(const moe_vqlr_config* cfg, moe_vqlr_handle** out) {
  if (out) *out = nullptr;
  if (!cfg || !out) return fail(nullptr, MOE_VQLR_ERR_INVALID_ARG, "cfg/out is null");
  const int H = cfg->hidden, I = cfg->inter, E = cfg->n_experts, k = cfg->top_k, S = cfg->n_shared;
  const int K = cfg->codebook_size, r = cfg->rank, maxT = cfg->max_tokens;
  if (H <= 0 || I <= 0 || E <= 0 || k <= 0 || S < 0 || r < 0 || maxT <= 0)
    return fail(nullptr, MOE_VQLR_ERR_INVALID_ARG, "non-positive size");
  if (k > E) return fail(nullptr, MOE_VQLR_ERR_INVALID_ARG, "top_k %d > n_experts %d", k, E);
  if (!cfg->router_w || !aligned16(cfg->router_w))
    return fail(nullptr, MOE_VQLR_ERR_INVALID_ARG, "router_w null or not 16-byte aligned");
  if (cfg->vq_dim != kD) return fail(nullptr, MOE_VQLR_ERR_UNSUPPORTED, "vq_dim must be 8");
  if (H % kD || I % kD) return fail(nullptr, MOE_VQLR_ERR_UNSUPPORTED, "hidden and inter must be multiples of 8");
  if (k > kMaxK) return fail(nullptr, MOE_VQLR_ERR_UNSUPPORTED, "top_k > %d", kMaxK);
  if (maxT > kMaxT) return fail(nullptr, MOE_VQLR_ERR_UNSUPPORTED, "max_tokens > %d", kMaxT);
  const bool any_vq = cfg->gate.kind == MOE_VQLR_PROJ_VQLR || cfg->up.kind == MOE_VQLR_PROJ_VQLR ||
                      cfg->down.kind == MOE_VQLR_PROJ_VQLR;
  if (any_vq && (K <= 0 || K > 65536)) return fail(nullptr, MOE_VQLR_ERR_UNSUPPORTED, "codebook_size out of 1..65536");
  int rc;
  if ((rc = check_proj(cfg->gate, "gate", r)) || (rc = check_proj(cfg->up, "up", r)) ||
      (rc = check_proj(cfg->down, "down", r)))
    return rc;

  moe_vqlr_handle* h = new (std::nothrow) moe_vqlr_handle();
  if (!h) return fail(nullptr, MOE_VQLR_ERR_OOM, "host allocation failed");
  h->cfg = *cfg;
  h->launches = 0;
  h->workspace = nullptr;
  h->profiling = 0;
  h->ev_valid = false;
  for (auto& e : h->ev) e = nullptr;
  h->idx_bytes = K <= 256 ? 1 : 2;
  cudaError_t ce = cudaGetDevice(&h->device);
  cudaDeviceProp prop;
  if (ce == cudaSuccess) ce = cudaGetDeviceProperties(&prop, h->device);
  if (ce != cudaSuccess) {
    rc = fail(nullptr, MOE_VQLR_ERR_CUDA, "cudaGetDeviceProperties: %s", cudaGetErrorString(ce));
    delete h;
    return rc;
  }
  h->sm_count = prop.multiProcessorCount;

  Params& P = h->P;
  memset(&P, 0, sizeof P);
  P.H = H; P.I = I; P.E = E; P.k = k; P.S = S; P.K = any_vq ? K : 0; P.r = r;
  P.renorm = cfg->renorm_topk ? 1 : 0;
  P.router_w = static_cast<const bf16*>(cfg->router_w);
  P.router_bias = cfg->router_bias;
  P.gate = make_proj(cfg->gate, I, H);
  P.up = make_proj(cfg->up, I, H);
  P.down = make_proj(cfg->down, H, I);
  // z slots: gate -> 0, up -> 0 when it shares gate's basis, else 1
  int n_slots = 0;
  if (r > 0 && P.gate.kind == MOE_VQLR_PROJ_VQLR) P.gate.zslot = n_slots++;
  if (r > 0 && P.up.kind == MOE_VQLR_PROJ_VQLR) {
    if (P.gate.zslot >= 0 && P.up.basis == P.gate.basis) P.up.zslot = P.gate.zslot;
    else P.up.zslot = n_slots++;
  }
  // k_router_z maps stacked row q to slot q / r; with gate dense and up VQLR the single slot is up's
  P.n_zrows = n_slots * r;
  h->two_books = (P.gate.kind == MOE_VQLR_PROJ_VQLR && P.up.kind == MOE_VQLR_PROJ_VQLR &&
                  P.gate.codebook != P.up.codebook) ? 1 : 0;

  // shared memory budgets
  const bool gu_vq = P.gate.kind == MOE_VQLR_PROJ_VQLR || P.up.kind == MOE_VQLR_PROJ_VQLR;
  h->smem_gateup_fixed = gu_vq ? (size_t)(h->two_books ? 2 : 1) * K * 16 : 0;
  h->smem_gateup_per_token = (size_t)((H / kD + 7) / 8 * 8) * 16;
  h->smem_down = (P.down.kind == MOE_VQLR_PROJ_VQLR ? (size_t)K * 16 : 0) + 16 * kMaxT * sizeof(float);
  const size_t smem_gu_max = h->smem_gateup_fixed + h->smem_gateup_per_token * maxT;
  if (smem_gu_max > (size_t)prop.sharedMemPerBlockOptin || h->smem_down > (size_t)prop.sharedMemPerBlockOptin) {
    rc = fail(nullptr, MOE_VQLR_ERR_UNSUPPORTED, "shared memory need (%zu / %zu bytes) exceeds the device limit %zu",
              smem_gu_max, h->smem_down, (size_t)prop.sharedMemPerBlockOptin);
    delete h;
    return rc;
  }
  if (h->idx_bytes == 1) {
    cudaFuncSetAttribute(k_gateup<uint8_t>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_gu_max);
    cudaFuncSetAttribute(k_down<uint8_t>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)h->smem_down);
  } else {
    cudaFuncSetAttribute(k_gateup<uint16_t>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_gu_max);
    cudaFuncSetAttribute(k_down<uint16_t>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)h->smem_down);
  }
  cudaFuncSetAttribute(k_route, cudaFuncAttributeMaxDynamicSharedMemorySize,
                       (int)((size_t)maxT * E * 4 + (2 * (size_t)E + 1) * 4));

  // workspace
  const size_t n_pos = (size_t)maxT * (k + S);
  auto plan = [&](char* base) {
    char* cur = base;
    P.logits = carve<float>(cur, (size_t)maxT * E);
    P.z = carve<float>(cur, (size_t)maxT * 2 * (r > 0 ? r : 1));
    P.topk_id = carve<int>(cur, (size_t)maxT * k);
    P.topk_w = carve<float>(cur, (size_t)maxT * k);
    P.counts = carve<int>(cur, E);
    P.offsets = carve<int>(cur, E + 1);
    P.pair_token = carve<int>(cur, n_pos);
    P.pair_slot = carve<int>(cur, n_pos);
    P.pair_w = carve<float>(cur, n_pos);
    P.act_n = carve<int>(cur, 1);
    P.act_e = carve<int>(cur, E + S);
    P.act_off = carve<int>(cur, E + S);
    P.act_cnt = carve<int>(cur, E + S);
    P.p = carve<float>(cur, n_pos * I);
    P.zd = carve<float>(cur, n_pos * (r > 0 ? r : 1));
    P.status = carve<int>(cur, 1);
    h->x_stage = carve<bf16>(cur, (size_t)maxT * H);
    h->out_stage = carve<bf16>(cur, (size_t)maxT * H);
    return (size_t)(cur - base);
  };
  h->workspace_bytes = plan(nullptr);
  ce = cudaMalloc(&h->workspace, h->workspace_bytes);
  if (ce != cudaSuccess) {
    rc = fail(nullptr, MOE_VQLR_ERR_OOM, "cudaMalloc(%zu): %s", h->workspace_bytes, cudaGetErrorString(ce));
    cudaGetLastError();
    delete h;
    return rc;
  }
  plan(static_cast<char*>(h->workspace));
  cudaMemset(h->workspace, 0, h->workspace_bytes);

  if (cfg->flags & MOE_VQLR_FLAG_VALIDATE_INDICES) {
    unsigned int* d_max = reinterpret_cast<unsigned int*>(P.status);
    const moe_vqlr_proj* projs[3] = {&cfg->gate, &cfg->up, &cfg->down};
    for (int i = 0; i < 3; ++i) {
      if (projs[i]->kind != MOE_VQLR_PROJ_VQLR) continue;
      const size_t n = (size_t)(E + S) * H * I / kD;
      if (h->idx_bytes == 1) k_max_index<uint8_t><<<h->sm_count * 4, 256>>>(static_cast<const uint8_t*>(projs[i]->idx), n, d_max);
      else k_max_index<uint16_t><<<h->sm_count * 4, 256>>>(static_cast<const uint16_t*>(projs[i]->idx), n, d_max);
    }
    unsigned int mx = 0;
    ce = cudaMemcpy(&mx, d_max, sizeof mx, cudaMemcpyDeviceToHost);
    cudaMemset(P.status, 0, sizeof(int));
    if (ce != cudaSuccess || mx >= (unsigned int)K) {
      rc = ce != cudaSuccess ? fail(nullptr, MOE_VQLR_ERR_CUDA, "index validation: %s", cudaGetErrorString(ce))
                             : fail(nullptr, MOE_VQLR_ERR_BAD_INDEX, "index %u >= codebook_size %d", mx, K);
      cudaFree(h->workspace);
      delete h;
      return rc;
    }
  }
  ce = cudaDeviceSynchronize();
  if (ce != cudaSuccess) {
    rc = fail(nullptr, MOE_VQLR_ERR_CUDA, "create: %s", cudaGetErrorString(ce));
    cudaFree(h->workspace);
    delete h;
    return rc;
  }
  *out = h;
  return MOE_VQLR_OK;
}

int moe_vqlr_decode_layer(moe_vqlr_handle* h, const void* x, int32_t T, void* out,
                          const moe_vqlr_debug* dbg, void* cuda_stream) {
  if (!h) return MOE_VQLR_ERR_INVALID_ARG;
  if (!x || !out) return fail(h, MOE_VQLR_ERR_INVALID_ARG, "x/out is null");
  if (T < 1 || T > h->cfg.max_tokens) return fail(h, MOE_VQLR_ERR_INVALID_ARG, "T=%d outside 1..%d", T, h->cfg.max_tokens);
  if (!aligned16(x) || !aligned16(out)) return fail(h, MOE_VQLR_ERR_INVALID_ARG, "x/out must be 16-byte aligned");
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  const Params& P = h->P;
  const bf16* xb = static_cast<const bf16*>(x);
  bf16* ob = static_cast<bf16*>(out);

  const bool prof = h->profiling != 0;
  auto mark = [&](int i) { if (prof) cudaEventRecord(h->ev[i], st); };
  for (int i = 0; i < kStages; ++i) h->stage_ran[i] = false;
  mark(0);
  {
    const int rows = P.E + P.n_zrows;
    k_router_z<<<(rows + 7) / 8, 256, 0, st>>>(P, xb, T);
    h->stage_ran[0] = true;
  }
  mark(1);
  {
    const size_t smem = (size_t)T * P.E * 4 + (2 * (size_t)P.E + 1) * 4;
    k_route<<<1, 32 * T, smem, st>>>(P, T);
    h->stage_ran[1] = true;
  }
  mark(2);
  {
    const size_t smem = h->smem_gateup_fixed + h->smem_gateup_per_token * T;
    const int grid = h->sm_count;
    if (h->idx_bytes == 1) k_gateup<uint8_t><<<grid, 512, smem, st>>>(P, xb, T, h->two_books);
    else k_gateup<uint16_t><<<grid, 512, smem, st>>>(P, xb, T, h->two_books);
    h->stage_ran[2] = true;
  }
  mark(3);
  h->launches += 3;
  if (P.down.kind == MOE_VQLR_PROJ_VQLR && P.r > 0) {
    const int n_pos = T * (P.k + P.S);
    k_zdown<<<(n_pos * P.r + 7) / 8, 256, 0, st>>>(P, n_pos);
    h->launches += 1;
    h->stage_ran[3] = true;
  }
  mark(4);
  {
    const int grid = min(h->sm_count, (P.H + 15) / 16);
    if (h->idx_bytes == 1) k_down<uint8_t><<<grid, 512, h->smem_down, st>>>(P, ob, T);
    else k_down<uint16_t><<<grid, 512, h->smem_down, st>>>(P, ob, T);
    h->launches += 1;
    h->stage_ran[4] = true;
  }
  mark(5);
  h->ev_valid = prof;
  cudaError_t ce = cudaGetLastError();
  if (ce != cudaSuccess) return fail(h, MOE_VQLR_ERR_CUDA, "launch: %s", cudaGetErrorString(ce));

  if (dbg) {
    const size_t Tk = (size_t)T * P.k;
    struct { void* dst; const void* src; size_t n; } cp[] = {
        {dbg->logits, P.logits, (size_t)T * P.E * 4}, {dbg->topk_id, P.topk_id, Tk * 4},
        {dbg->topk_w, P.topk_w, Tk * 4},              {dbg->counts, P.counts, (size_t)P.E * 4},
        {dbg->offsets, P.offsets, (size_t)(P.E + 1) * 4},
        {dbg->pair_token, P.pair_token, Tk * 4},      {dbg->pair_slot, P.pair_slot, Tk * 4}};
    for (auto& c : cp)
      if (c.dst) {
        ce = cudaMemcpyAsync(c.dst, c.src, c.n, cudaMemcpyDeviceToDevice, st);
        if (ce != cudaSuccess) return fail(h, MOE_VQLR_ERR_CUDA, "debug copy: %s", cudaGetErrorString(ce));
      }
  }
  return MOE_VQLR_OK;
}

int moe_vqlr_decode_layer_host(moe_vqlr_handle* h, const void* x_host, int32_t T, void* out_host,
                               void* cuda_stream) {
  if (!h) return MOE_VQLR_ERR_INVALID_ARG;
  if (!x_host || !out_host) return fail(h, MOE_VQLR_ERR_INVALID_ARG, "x_host/out_host is null");
  if (T < 1 || T > h->cfg.max_tokens) return fail(h, MOE_VQLR_ERR_INVALID_ARG, "T=%d outside 1..%d", T, h->cfg.max_tokens);
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  const size_t bytes = (size_t)T * h->P.H * sizeof(bf16);
  cudaError_t ce = cudaMemcpyAsync(h->x_stage, x_host, bytes, cudaMemcpyHostToDevice, st);
  if (ce != cudaSuccess) return fail(h, MOE_VQLR_ERR_CUDA, "copy in: %s", cudaGetErrorString(ce));
  const int rc = moe_vqlr_decode_layer(h, h->x_stage, T, h->out_stage, nullptr, cuda_stream);
  if (rc != MOE_VQLR_OK) return rc;
  ce = cudaMemcpyAsync(out_host, h->out_stage, bytes, cudaMemcpyDeviceToHost, st);
  if (ce == cudaSuccess) ce = cudaStreamSynchronize(st);
  if (ce != cudaSuccess) return fail(h, MOE_VQLR_ERR_CUDA, "copy out: %s", cudaGetErrorString(ce));
  return MOE_VQLR_OK;
}

int moe_vqlr_destroy(moe_vqlr_handle* h) {
  if (!h) return MOE_VQLR_OK;
  for (auto& e : h->ev)
    if (e) cudaEventDestroy(e);
  cudaError_t ce = cudaFree(h->workspace);
  delete h;
  return ce == cudaSuccess ? MOE_VQLR_OK : MOE_VQLR_ERR_CUDA;
}

const char* moe_vqlr_last_error(const moe_vqlr_handle* h) {
  return h ? h->error.c_str() : g_create_error.c_str();
}

int moe_vqlr_set_profiling(moe_vqlr_handle* h, int32_t on) {
  if (!h) return MOE_VQLR_ERR_INVALID_ARG;
  if (on && !h->ev[0]) {
    for (auto& e : h->ev) {
      cudaError_t ce = cudaEventCreate(&e);
      if (ce != cudaSuccess) return fail(h, MOE_VQLR_ERR_CUDA, "cudaEventCreate: %s", cudaGetErrorString(ce));
    }
  }
  h->profiling = on ? 1 : 0;
  h->ev_valid = false;
  return MOE_VQLR_OK;
}

int moe_vqlr_stage_count(void) { return kStages; }

const char* moe_vqlr_stage_name(int32_t i) { return (i >= 0 && i < kStages) ? kStageNames[i] : ""; }

int moe_vqlr_last_stage_times(moe_vqlr_handle* h, float* ms_out, int32_t cap) {
  if (!h || !ms_out || cap < kStages) return h ? fail(h, MOE_VQLR_ERR_INVALID_ARG, "ms_out null or cap < %d", kStages) : MOE_VQLR_ERR_INVALID_ARG;
  if (!h->ev_valid) return fail(h, MOE_VQLR_ERR_INVALID_ARG, "no profiled call to report");
  cudaError_t ce = cudaEventSynchronize(h->ev[kStages]);
  if (ce != cudaSuccess) return fail(h, MOE_VQLR_ERR_CUDA, "event sync: %s", cudaGetErrorString(ce));
  for (int i = 0; i < kStages; ++i) {
    ms_out[i] = 0.f;
    if (h->stage_ran[i]) {
      ce = cudaEventElapsedTime(&ms_out[i], h->ev[i], h->ev[i + 1]);
      if (ce != cudaSuccess) return fail(h, MOE_VQLR_ERR_CUDA, "elapsed: %s", cudaGetErrorString(ce));
    }
  }
  return MOE_VQLR_OK;
}

int64_t moe_vqlr_launch_count(const moe_vqlr_handle* h) { return h ? h->launches : 0; }

int64_t moe_vqlr_workspace_bytes(const moe_vqlr_handle* h) { return h ? (int64_t)h->workspace_bytes : 0; }

}  // extern "C"
