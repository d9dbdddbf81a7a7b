// Generic kernels: one warp per output row, CUDA cores, any shape the interface accepts
// (ragged block counts, ranks that are not multiples of eight).  They are the path for shapes
// the tensor-core kernels do not cover.
#pragma once
#include "common.cuh"

namespace {

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
        if (lane == 0) set_status(P, MOE_VQLR_ERR_INVALID_ARG);
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

// The eight weights of 8-value block b of a row: one code word (d = 8) or two consecutive
// 4-value code words (d = 4, Section 5.5's shorter vectors: the row then has two indices per block).
// Eight indices of a packed twelve-bit row starting at element 8 c (a 4-byte boundary).
__device__ __forceinline__ void load_idx12x8(const void* row, int c, uint32_t (&id)[8]) {
  const uint32_t* w = reinterpret_cast<const uint32_t*>(static_cast<const unsigned char*>(row) + (size_t)c * 12);
  unpack_idx12x8(__ldg(w), __ldg(w + 1), __ldg(w + 2), id);
}

template <typename IdxT>
__device__ __forceinline__ uint4 row_block8(const IdxT* __restrict__ idx_row, int b, const uint4* __restrict__ s_cb, int d, int idx12 = 0) {
  if (d == 8) return s_cb[idx12 ? read_idx12(idx_row, b) : idx_row[b]];
  const uint2* cb2 = reinterpret_cast<const uint2*>(s_cb);
  const uint2 lo = cb2[idx_row[2 * b]], hi = cb2[idx_row[2 * b + 1]];
  return make_uint4(lo.x, lo.y, hi.x, hi.y);
}

// Code book of a projection into shared memory (K words of 2 d bytes).
__device__ __forceinline__ void stage_codebook(uint4* dst, const uint4* __restrict__ src, int K, int d) {
  if (d == 8) {
    for (int i = threadIdx.x; i < K; i += blockDim.x) dst[i] = __ldg(src + i);
  } else {
    uint2* d2 = reinterpret_cast<uint2*>(dst);
    const uint2* s2 = reinterpret_cast<const uint2*>(src);
    for (int i = threadIdx.x; i < K; i += blockDim.x) d2[i] = __ldg(s2 + i);
  }
}

// VQ part of one row against up to kTokGroup bf16 activation rows held (swizzled) in shared
// memory.  nb = 8-value blocks per row.
template <typename IdxT>
__device__ __forceinline__ void vq_row_bf16x(const IdxT* __restrict__ idx_row, int nb, int d,
                                             const uint4* __restrict__ s_cb,
                                             const uint4* __restrict__ s_x, int x_stride,
                                             const int (&tok)[kTokGroup], int nt,
                                             float (&acc)[kTokGroup], int lane, int idx12 = 0) {
  if (d == 8 && (nb & 7) == 0) {
    for (int c = lane; c < (nb >> 3); c += 32) {
      uint32_t id[8];
      if (idx12) load_idx12x8(idx_row, c, id); else load_idx8<IdxT>(idx_row + c * 8, id);
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
      unpack8(row_block8<IdxT>(idx_row, b0, s_cb, d, idx12), wf);
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
    stage_codebook(s_cb_g, src_g, P.K, P.d);
    if (two_books) stage_codebook(s_cb_u, P.up.codebook, P.K, P.d);
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
        vq_row_bf16x<IdxT>(idx_at(static_cast<const IdxT*>(P.gate.idx), row * (P.H / P.d), P.idx12), nbH, P.d, s_cb_g, s_x, xs,
                           tok, nt, g, lane, P.idx12);
        if (P.gate.zslot >= 0)
          lr_row(P.gate.factor + row * P.r, P.r, P.z + P.gate.zslot * P.r, 2 * P.r, tok, nt, g, lane);
      } else {
        dense_row_bf16x(P.gate.dense + row * P.H, nbH, s_x, xs, tok, nt, g, lane);
      }
      if (P.up.kind == MOE_VQLR_PROJ_VQLR) {
        vq_row_bf16x<IdxT>(idx_at(static_cast<const IdxT*>(P.up.idx), row * (P.H / P.d), P.idx12), nbH, P.d, s_cb_u, s_x, xs,
                           tok, nt, u, lane, P.idx12);
        if (P.up.zslot >= 0)
          lr_row(P.up.factor + row * P.r, P.r, P.z + P.up.zslot * P.r, 2 * P.r, tok, nt, u, lane);
      } else {
        dense_row_bf16x(P.up.dense + row * P.H, nbH, s_x, xs, tok, nt, u, lane);
      }
#pragma unroll
      for (int tt = 0; tt < kTokGroup; ++tt) {
        const float gs = warp_sum(g[tt]), us = warp_sum(u[tt]);
        if (lane == 0 && tt < nt)
          P.p[(size_t)(off + q0 + tt) * P.I + i] = gated_act(gs, us, P.act);   // phi(g) * u
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
  if (vq) stage_codebook(s_cb, P.down.codebook, P.K, P.d);
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
          const IdxT* idx_row = idx_at(static_cast<const IdxT*>(P.down.idx), row * (P.I / P.d), P.idx12);
          if (P.d == 8 && (nbI & 7) == 0) {
            for (int c = lane; c < (nbI >> 3); c += 32) {
              uint32_t id[8];
              if (P.idx12) load_idx12x8(idx_row, c, id); else load_idx8<IdxT>(idx_row + c * 8, id);
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
              unpack8(row_block8<IdxT>(idx_row, b, s_cb, P.d, P.idx12), wf);
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
__global__ void k_max_index(const IdxT* __restrict__ idx, size_t n, unsigned int* out, int idx12) {
  unsigned int m = 0;
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n;
       i += (size_t)gridDim.x * blockDim.x)
    m = max(m, idx12 ? read_idx12(idx, i) : (unsigned int)idx[i]);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) m = max(m, __shfl_xor_sync(0xffffffffu, m, o));
  if ((threadIdx.x & 31) == 0) atomicMax(out, m);
}

}  // namespace
