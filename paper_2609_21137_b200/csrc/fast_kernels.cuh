// Tensor-core kernels of the decode layer.
//
// Design.  Every projection here is "eight output rows of one expert times up to eight token
// vectors", with the contraction cut into slices of 32 blocks (256 values).  One warp owns one
// slice: it keeps the slice of the activations as mma A fragments in registers for as long as
// the expert does not change, and for each row tile it
//     loads 16 bytes of indices (8 code-word ids of row g),
//     fetches the 8 code words from the shared-memory code book (one 16-byte read each),
//     and feeds each code word straight into two mma.sync.m16n8k16 as the B fragment.
// The k order inside an mma is free as long as A and B agree, so the fragment layout is chosen
// such that a thread's B registers of two consecutive mma's are exactly one 16-byte code word
// and its A registers are exactly the matching 16-byte activation block: no unpacking, no
// shuffles, no FMAs on the CUDA cores.  Token rows 8..15 of the m16 tile are zero; experts
// with more than eight tokens take a second pass that reuses the same index registers.
// The low-rank term (Eq. 1) joins the same accumulator as more k: B = a row of the private
// factor, A = z split into bf16 hi + lo so that nothing is lost against fp32.
// The warps of a team (one per slice) add their partial tiles through shared memory in a fixed
// order; nothing uses floating-point atomics, so results repeat bit for bit.
//
// Kernel chain of a call, linked by programmatic dependent launch (each kernel starts its
// routing-independent prologue while its predecessor drains):
//   k_router_z  ->  k_gateup_mma (routing redone in every block from the logits)
//               ->  [k_zdown]  ->  k_down_mma  ->  k_combine
#pragma once
#include "common.cuh"

namespace {

constexpr int kFastThreads = 512;
constexpr int kDenseThreads = 384;   // dense gate/up: weight tiles in flight need more registers per thread
constexpr int kDownThreads = 384;    // down: hi + lo activation fragments need 64 registers per thread

__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_launch() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

__device__ __forceinline__ void team_sync(int id, int nthreads) {
  asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(nthreads) : "memory");
}

// D += A * B with A rows 8..15 zero.  a0 = A[g][2c..2c+1], a2 = A[g][2c+8..2c+9],
// b0 = B[2c..2c+1][g], b1 = B[2c+8..2c+9][g]; d0 = D[g][2c], d1 = D[g][2c+1] (g = lane/4, c = lane%4).
__device__ __forceinline__ void mma_tok8(float (&d)[4], uint32_t a0, uint32_t a2, uint32_t b0, uint32_t b1) {
  const uint32_t zero = 0u;
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
      : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
      : "r"(a0), "r"(zero), "r"(a2), "r"(zero), "r"(b0), "r"(b1));
}

// One 16-byte weight block w (8 bf16 along k) against the matching activation block a.
__device__ __forceinline__ void mma_block(float (&d)[4], const uint4& a, const uint4& w) {
  mma_tok8(d, a.x, a.y, w.x, w.y);
  mma_tok8(d, a.z, a.w, w.z, w.w);
}

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  const __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<const uint32_t*>(&v);
}

// Split eight fp32 values into bf16 hi and lo blocks: v = hi + lo up to 2^-17 relative.
__device__ __forceinline__ void split_hi_lo(const float4& p0, const float4& p1, uint4& hi, uint4& lo) {
  const float v[8] = {p0.x, p0.y, p0.z, p0.w, p1.x, p1.y, p1.z, p1.w};
  uint32_t h[4], l[4];
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    h[q] = pack_bf16(v[2 * q], v[2 * q + 1]);
    const float r0 = v[2 * q] - bf_lo(h[q]), r1 = v[2 * q + 1] - bf_hi(h[q]);
    l[q] = pack_bf16(r0, r1);
  }
  hi = make_uint4(h[0], h[1], h[2], h[3]);
  lo = make_uint4(l[0], l[1], l[2], l[3]);
}

template <typename IdxT>
__device__ __forceinline__ void unpack_idx8(const uint4& raw, uint32_t (&id)[8]);
template <>
__device__ __forceinline__ void unpack_idx8<uint16_t>(const uint4& v, uint32_t (&id)[8]) {
  id[0] = v.x & 0xffffu; id[1] = v.x >> 16; id[2] = v.y & 0xffffu; id[3] = v.y >> 16;
  id[4] = v.z & 0xffffu; id[5] = v.z >> 16; id[6] = v.w & 0xffffu; id[7] = v.w >> 16;
}
template <>
__device__ __forceinline__ void unpack_idx8<uint8_t>(const uint4& v, uint32_t (&id)[8]) {
  id[0] = v.x & 0xffu; id[1] = (v.x >> 8) & 0xffu; id[2] = (v.x >> 16) & 0xffu; id[3] = v.x >> 24;
  id[4] = v.y & 0xffu; id[5] = (v.y >> 8) & 0xffu; id[6] = (v.y >> 16) & 0xffu; id[7] = v.y >> 24;
}

// Eight indices of one row starting at block b0 (a multiple of 8): 16 bytes of uint16 or 8 of uint8.
template <typename IdxT>
__device__ __forceinline__ uint4 load_idx_raw(const IdxT* p) {
  if (sizeof(IdxT) == 2) return __ldg(reinterpret_cast<const uint4*>(p));
  const uint2 v = __ldg(reinterpret_cast<const uint2*>(p));
  return make_uint4(v.x, v.y, 0u, 0u);
}

// How one projection stage is cut up (computed on the host, see plan_stage()).
struct StagePlan {
  int nb;          // blocks per weight row = in_dim / 8
  int n_slices;    // ceil(nb / 32)
  int team_warps;  // warps that share one row tile (power of two <= 16)
  int n_teams;     // teams per block
  int tiles;       // row tiles per expert = out_dim / 8
  int n_lr;        // groups of 32 ranks = ceil(r / 32), 0 without a low-rank term
  int depth;       // tiles each warp keeps in flight in its shared-memory ring (2..4)
};

// ---------------------------------------------------------------------------------------------
// Routing inside a block: top-k by rank counting (rank = number of experts that beat this one
// in the order logit descending, id ascending), affinities, grouping.  All threads take part.
// ---------------------------------------------------------------------------------------------
struct RouteSmem {
  float* logit;     // [T][E]
  signed char* slot;// [T][E]  slot of expert e for token t, -1 if not selected
  int* sel_id;      // [T][k]
  float* sel_l;     // [T][k]
  float* w;         // [T][k]
  int* cnt;         // [E]
  int* off;         // [E+1]
  int* act_e;       // [E+S]
  int* act_off;     // [E+S]
  int* act_cnt;     // [E+S]
  int* pair_token;  // [T*(k+S)]
  int* n_act;       // [1]
};

__host__ __device__ inline size_t route_smem_bytes(int T, int E, int k, int S) {
  size_t b = (size_t)T * E * 4 + ((size_t)T * E + 15) / 16 * 16 + (size_t)T * k * 12 +
             (size_t)(2 * E + 1) * 4 + (size_t)(E + S) * 12 + (size_t)T * (k + S) * 4 + 16;
  return (b + 15) / 16 * 16;
}

__device__ inline RouteSmem carve_route(char* base, int T, int E, int k, int S) {
  RouteSmem r;
  r.logit = reinterpret_cast<float*>(base); base += (size_t)T * E * 4;
  r.slot = reinterpret_cast<signed char*>(base); base += ((size_t)T * E + 15) / 16 * 16;
  r.sel_id = reinterpret_cast<int*>(base); base += (size_t)T * k * 4;
  r.sel_l = reinterpret_cast<float*>(base); base += (size_t)T * k * 4;
  r.w = reinterpret_cast<float*>(base); base += (size_t)T * k * 4;
  r.cnt = reinterpret_cast<int*>(base); base += (size_t)E * 4;
  r.off = reinterpret_cast<int*>(base); base += (size_t)(E + 1) * 4;
  r.act_e = reinterpret_cast<int*>(base); base += (size_t)(E + S) * 4;
  r.act_off = reinterpret_cast<int*>(base); base += (size_t)(E + S) * 4;
  r.act_cnt = reinterpret_cast<int*>(base); base += (size_t)(E + S) * 4;
  r.pair_token = reinterpret_cast<int*>(base); base += (size_t)T * (k + S) * 4;
  r.n_act = reinterpret_cast<int*>(base);
  return r;
}

__device__ void route_in_block(const Params& P, int T, const RouteSmem& R, bool write_global) {
  const int E = P.E, k = P.k, S = P.S;
  const int tid = threadIdx.x, nthr = blockDim.x, lane = tid & 31, warp = tid >> 5;
  for (int i = tid; i < T * E; i += nthr) R.logit[i] = P.logits[i];
  __syncthreads();
  // rank of every (token, expert): four lanes share one pair and scan a quarter of the row each
  for (int q0 = 0; q0 < T * E; q0 += nthr >> 2) {     // uniform trip count: all lanes reach the shuffles
    const int q = q0 + (tid >> 2);
    const bool live = q < T * E;
    const int t = live ? q / E : 0, e = live ? q - t * E : 0;
    const float l = live ? R.logit[q] : 0.f;
    const float* row = R.logit + t * E;
    int rank = 0;
    if (live)
      for (int e2 = tid & 3; e2 < E; e2 += 4) {
        const float v = row[e2];
        rank += (v > l) || (v == l && e2 < e);
      }
    rank += __shfl_xor_sync(0xffffffffu, rank, 1);
    rank += __shfl_xor_sync(0xffffffffu, rank, 2);
    if (live && (tid & 3) == 0) {
      R.slot[q] = rank < k ? (signed char)rank : (signed char)-1;
      if (rank < k) { R.sel_id[t * k + rank] = e; R.sel_l[t * k + rank] = l; }
    }
  }
  __syncthreads();
  // affinities: one warp per token (blockDim >= 32 * T)
  for (int t = warp; t < T; t += nthr >> 5) {
    const float lmax = R.sel_l[t * k];
    const float ev = lane < k ? expf(R.sel_l[t * k + lane] - lmax) : 0.f;
    float denom = ev;
    if (!P.renorm)
      for (int e = lane; e < E; e += 32)
        if (R.slot[t * E + e] < 0) denom += expf(R.logit[t * E + e] - lmax);
    denom = warp_sum(denom);
    if (lane < k) R.w[t * k + lane] = ev / denom;
  }
  for (int e = tid; e < E; e += nthr) {
    int c = 0;
    for (int t = 0; t < T; ++t) c += R.slot[t * E + e] >= 0;
    R.cnt[e] = c;
  }
  __syncthreads();
  const int n_pairs = T * k;
  if (warp == 0) {
    const int chunk = (E + 31) / 32;
    const int e0 = lane * chunk, e1 = min(E, e0 + chunk);
    int sum = 0, nact = 0;
    for (int e = e0; e < e1; ++e) { sum += R.cnt[e]; nact += R.cnt[e] > 0; }
    int psum = sum, pact = nact;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int a = __shfl_up_sync(0xffffffffu, psum, o);
      const int b = __shfl_up_sync(0xffffffffu, pact, o);
      if (lane >= o) { psum += a; pact += b; }
    }
    int run = psum - sum, arun = pact - nact;
    for (int e = e0; e < e1; ++e) {
      R.off[e] = run;
      if (R.cnt[e] > 0) { R.act_e[arun] = e; R.act_off[arun] = run; R.act_cnt[arun] = R.cnt[e]; ++arun; }
      run += R.cnt[e];
    }
    const int total_act = __shfl_sync(0xffffffffu, pact, 31);
    if (lane == 31) R.off[E] = psum;
    for (int s = lane; s < S; s += 32) {
      R.act_e[total_act + s] = E + s;
      R.act_off[total_act + s] = n_pairs + s * T;
      R.act_cnt[total_act + s] = T;
    }
    if (lane == 0) *R.n_act = total_act + S;
  }
  __syncthreads();
  for (int e = tid; e < E; e += nthr) {
    if (R.cnt[e] == 0) continue;
    int pos = R.off[e];
    for (int t = 0; t < T; ++t) {
      const int s = R.slot[t * E + e];
      if (s >= 0) {
        R.pair_token[pos] = t;
        if (write_global) { P.pair_token[pos] = t; P.pair_slot[pos] = s; P.pair_w[pos] = R.w[t * k + s]; }
        ++pos;
      }
    }
  }
  for (int q = tid; q < S * T; q += nthr) {
    R.pair_token[n_pairs + q] = q % T;
    if (write_global) { P.pair_token[n_pairs + q] = q % T; P.pair_slot[n_pairs + q] = k + q / T; P.pair_w[n_pairs + q] = 1.f; }
  }
  __syncthreads();
  if (write_global) {
    for (int i = tid; i < T * k; i += nthr) { P.topk_id[i] = R.sel_id[i]; P.topk_w[i] = R.w[i]; }
    for (int e = tid; e <= E; e += nthr) { P.offsets[e] = R.off[e]; if (e < E) P.counts[e] = R.cnt[e]; }
    const int n_act = *R.n_act;
    for (int a = tid; a < n_act; a += nthr) { P.act_e[a] = R.act_e[a]; P.act_off[a] = R.act_off[a]; P.act_cnt[a] = R.act_cnt[a]; }
    if (tid == 0) *P.act_n = n_act;
  }
}

// ---------------------------------------------------------------------------------------------
// k_router_z_pdl: head of the chain.  One warp per (row of [router_w ; basis_gate ; basis_up],
// group of four tokens).  Per (row, token) the summation order is the one of k_router_z
// (lane-strided 16-byte chunks, sequential FMAs inside a chunk, xor butterfly), so identical
// router rows give bitwise identical logits.
// ---------------------------------------------------------------------------------------------
constexpr int kRouterWarps = 2;

__global__ void __launch_bounds__(32 * kRouterWarps) k_router_z_pdl(const Params P, const bf16* __restrict__ x, int T) {
  pdl_wait();      // the previous call's kernels may still read logits / z
  pdl_launch();
  const int lane = threadIdx.x & 31;
  const int unit = blockIdx.x * kRouterWarps + (threadIdx.x >> 5);
  const int n_rows = P.E + P.n_zrows;
  const int n_groups = (T + kTokGroup - 1) / kTokGroup;
  if (unit >= n_rows * n_groups) return;
  const int row = unit / n_groups, t0 = (unit - row * n_groups) * kTokGroup;
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
  const int nt = min(kTokGroup, T - t0);
  float acc[kTokGroup] = {0.f, 0.f, 0.f, 0.f};
  for (int c0 = 0; c0 < nchunk; c0 += 32 * 4) {          // four chunks per lane in flight
    uint4 wv[4], xv[4][kTokGroup];
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      const int c = c0 + q * 32 + lane;
      wv[q] = c < nchunk ? __ldg(w4 + c) : make_uint4(0, 0, 0, 0);
#pragma unroll
      for (int tt = 0; tt < kTokGroup; ++tt)
        xv[q][tt] = (c < nchunk && tt < nt) ? __ldg(reinterpret_cast<const uint4*>(x + (size_t)(t0 + tt) * P.H) + c)
                                            : make_uint4(0, 0, 0, 0);
    }
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      if (c0 + q * 32 + lane < nchunk) {
        float wf[8];
        unpack8(wv[q], wf);
#pragma unroll
        for (int tt = 0; tt < kTokGroup; ++tt) {
          float xf[8];
          unpack8(xv[q][tt], xf);
          acc[tt] = dot8(wf, xf, acc[tt]);
        }
      }
    }
  }
#pragma unroll
  for (int tt = 0; tt < kTokGroup; ++tt) {
    const float sum = warp_sum(acc[tt]);
    if (lane == 0 && tt < nt) dst[(size_t)(t0 + tt) * dst_stride] = sum + bias;
  }
}

// ---------------------------------------------------------------------------------------------
// Asynchronous copies: every warp streams the bytes it will need (indices, factor rows, dense
// weight rows) into a private shared-memory ring several tiles ahead, so that HBM latency is
// hidden without holding the data in registers.
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ void cp_async16(void* smem, const void* gptr) {
  const uint32_t sa = (uint32_t)__cvta_generic_to_shared(smem);
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(sa), "l"(gptr) : "memory");
}
__device__ __forceinline__ void cp_async8(void* smem, const void* gptr) {
  const uint32_t sa = (uint32_t)__cvta_generic_to_shared(smem);
  asm volatile("cp.async.ca.shared.global [%0], [%1], 8;" ::"r"(sa), "l"(gptr) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
// waits until at most `pending` of this thread's copy groups are still in flight
__device__ __forceinline__ void cp_async_wait_pending(int pending) {
  switch (pending) {
    case 0: asm volatile("cp.async.wait_group 0;" ::: "memory"); break;
    case 1: asm volatile("cp.async.wait_group 1;" ::: "memory"); break;
    case 2: asm volatile("cp.async.wait_group 2;" ::: "memory"); break;
    default: asm volatile("cp.async.wait_group 3;" ::: "memory"); break;
  }
}
template <typename IdxT>
__device__ __forceinline__ void cp_async_idx8(uint4* smem, const IdxT* gptr) {
  if (sizeof(IdxT) == 2) cp_async16(smem, gptr); else cp_async8(smem, gptr);
}
template <typename IdxT>
__device__ __forceinline__ uint4 ring_idx8(const uint4* smem) {
  if (sizeof(IdxT) == 2) return *smem;
  const uint2 v = *reinterpret_cast<const uint2*>(smem);
  return make_uint4(v.x, v.y, 0u, 0u);
}

constexpr int kMaxDepth = 4;

// ---------------------------------------------------------------------------------------------
// k_gateup_mma
// ---------------------------------------------------------------------------------------------
struct GuLayout {         // byte offsets into dynamic shared memory
  size_t cb_u, x, ring, fring, z, part, route, total;
};

__host__ __device__ inline GuLayout gu_layout(int K, int n_books, int T, int H, int r, const StagePlan& pl,
                                              int warps, int E, int k, int S) {
  GuLayout L;
  size_t o = 0;
  L.cb_u = n_books == 2 ? (size_t)K * 16 : 0;
  o = (size_t)n_books * K * 16;
  L.x = o;      o += (size_t)T * (H / 8 + 1) * 16;
  L.ring = o;   o += (size_t)warps * pl.depth * 2 * 32 * 16;
  L.fring = o;  o += (size_t)pl.n_teams * (pl.n_lr > 0 ? pl.n_lr : 0) * pl.depth * 2 * 32 * 16;
  L.z = o;      o += (size_t)2 * T * 2 * ((r + 7) / 8) * 16;            // hi and lo blocks of z
  L.part = o;   o += (size_t)2 * pl.n_teams * 2 * pl.team_warps * 32 * 8;
  L.route = o;  o += route_smem_bytes(T, E, k, S);
  L.total = o;
  return L;
}

template <typename IdxT, bool DENSE>
__global__ void __launch_bounds__(DENSE ? kDenseThreads : kFastThreads, 1)
k_gateup_mma(const Params P, const bf16* __restrict__ x, int T, const StagePlan pl, int n_books) {
  extern __shared__ uint4 s_u4[];
  char* s_base = reinterpret_cast<char*>(s_u4);
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, g = lane >> 2, c = lane & 3;
  const int nb = pl.nb, xs = nb + 1, D = pl.depth, rb = (P.r + 7) / 8;
  const GuLayout L = gu_layout(P.K, n_books, T, P.H, P.r, pl, blockDim.x >> 5, P.E, P.k, P.S);
  uint4* s_cb_g = s_u4;
  uint4* s_cb_u = reinterpret_cast<uint4*>(s_base + L.cb_u);
  uint4* s_x = reinterpret_cast<uint4*>(s_base + L.x);
  uint4* s_ring = reinterpret_cast<uint4*>(s_base + L.ring);
  uint4* s_fring = reinterpret_cast<uint4*>(s_base + L.fring);
  uint4* s_zh = reinterpret_cast<uint4*>(s_base + L.z);          // [T][2][rb]
  uint4* s_zl = s_zh + (size_t)T * 2 * rb;
  float2* s_part = reinterpret_cast<float2*>(s_base + L.part);
  const RouteSmem R = carve_route(s_base + L.route, T, P.E, P.k, P.S);

  // ---- prologue that does not depend on the routing: code books and tokens -------------------
  if (!DENSE) {
    for (int i = tid; i < P.K; i += blockDim.x) s_cb_g[i] = __ldg(P.gate.codebook + i);
    if (n_books == 2)
      for (int i = tid; i < P.K; i += blockDim.x) s_cb_u[i] = __ldg(P.up.codebook + i);
  }
  {
    const uint4* x4 = reinterpret_cast<const uint4*>(x);
    for (int i = tid; i < T * nb; i += blockDim.x) {
      const int t = i / nb, b = i - t * nb;
      s_x[t * xs + b] = __ldg(x4 + i);
    }
  }
  pdl_wait();      // logits and z of this call are complete
  if (pl.n_lr > 0)
    for (int i = tid; i < T * 2 * rb; i += blockDim.x) {      // z as bf16 hi / lo blocks
      const float* zp = P.z + (size_t)i * 8;                   // z is [T][2][r], r a multiple of 8
      split_hi_lo(*reinterpret_cast<const float4*>(zp), *reinterpret_cast<const float4*>(zp + 4), s_zh[i], s_zl[i]);
    }
  route_in_block(P, T, R, blockIdx.x == 0);
  pdl_launch();

  const int team = warp / pl.team_warps, wi = warp - team * pl.team_warps;
  const int team_threads = pl.team_warps * 32;
  const int tid_team = tid - team * team_threads;
  const int n_act = *R.n_act;
  const long long U = (long long)n_act * pl.tiles;
  const long long G = (long long)gridDim.x * pl.n_teams, tau = (long long)blockIdx.x * pl.n_teams + team;
  const long long u_begin = tau * U / G;
  const int n_my = team < pl.n_teams ? (int)((tau + 1) * U / G - u_begin) : 0;
  const bool spw_one = pl.n_slices <= pl.team_warps;         // one slice per warp: fragments stay put
  const bool ringed = !DENSE && spw_one;
  // low-rank group handled by this warp (groups are dealt from the last warp of the team down)
  const int lr_group = pl.team_warps - 1 - wi;
  const bool has_lr = lr_group < pl.n_lr;                    // n_lr is 0 for a dense projection
  const int b_first = wi * 32 + 8 * c, rho_first = lr_group * 32 + 8 * c;
  const bool idx_live = b_first < nb, fac_live = has_lr && rho_first < P.r;

  const IdxT* idx_g = static_cast<const IdxT*>(P.gate.idx);
  const IdxT* idx_u = static_cast<const IdxT*>(P.up.idx);
  uint4* ring = s_ring + (size_t)warp * D * 2 * 32;                                   // [slot][proj][lane]
  uint4* fring = s_fring + (size_t)(team * pl.n_lr + (has_lr ? lr_group : 0)) * D * 2 * 32;

  auto tile_row = [&](int i) -> size_t {                     // this lane's weight row of the team's i-th tile
    const long long u = u_begin + i;
    const int a = (int)(u / pl.tiles), jt = (int)(u - (long long)a * pl.tiles);
    return (size_t)R.act_e[a] * P.I + jt * 8 + g;
  };
  auto issue = [&](int i) {
    const size_t row = tile_row(i);
    const int slot = i % D;
    if (ringed && idx_live) {
      cp_async_idx8<IdxT>(ring + (slot * 2 + 0) * 32 + lane, idx_g + row * nb + b_first);
      cp_async_idx8<IdxT>(ring + (slot * 2 + 1) * 32 + lane, idx_u + row * nb + b_first);
    }
    if (fac_live) {
      cp_async16(fring + (slot * 2 + 0) * 32 + lane, P.gate.factor + row * P.r + rho_first);
      cp_async16(fring + (slot * 2 + 1) * 32 + lane, P.up.factor + row * P.r + rho_first);
    }
  };

  uint4 fx[8];                       // activation fragments of the current slice
  int frag_a = -1, frag_pass = -1, frag_slice = -1;
  int buf = 0;

  for (int i = 0; i < D - 1; ++i) { if (i < n_my) issue(i); cp_async_commit(); }
  for (int i = 0; i < n_my; ++i) {
    if (i + D - 1 < n_my) issue(i + D - 1);
    cp_async_commit();
    cp_async_wait_pending(D - 1);
    const long long u = u_begin + i;
    const int a = (int)(u / pl.tiles), jt = (int)(u - (long long)a * pl.tiles);
    const int e = R.act_e[a], off = R.act_off[a], cnt = R.act_cnt[a];
    const size_t row = (size_t)e * P.I + jt * 8 + g;       // this lane's weight row
    const int slot = i % D;
    uint4 raw_g = {0, 0, 0, 0}, raw_u = {0, 0, 0, 0};
    uint4 fac_g = {0, 0, 0, 0}, fac_u = {0, 0, 0, 0};
    if (ringed && idx_live) {
      raw_g = ring_idx8<IdxT>(ring + (slot * 2 + 0) * 32 + lane);
      raw_u = ring_idx8<IdxT>(ring + (slot * 2 + 1) * 32 + lane);
    }
    if (fac_live) {
      fac_g = fring[(slot * 2 + 0) * 32 + lane];
      fac_u = fring[(slot * 2 + 1) * 32 + lane];
    }
    for (int pass = 0; pass * 8 < cnt; ++pass) {
      const int n_tok = min(8, cnt - pass * 8);
      const int tok = g < n_tok ? R.pair_token[off + pass * 8 + g] : -1;
      float acc_g[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
      float acc_u[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
      for (int sl = wi; sl < pl.n_slices; sl += pl.team_warps) {
        const int b0 = sl * 32 + (DENSE ? c : 8 * c);
        if (frag_a != a || frag_pass != pass || frag_slice != sl) {
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            const int b = b0 + (DENSE ? 4 * j : j);
            fx[j] = (tok >= 0 && b < nb) ? s_x[tok * xs + b] : make_uint4(0, 0, 0, 0);
          }
          frag_a = a; frag_pass = pass; frag_slice = sl;
        }
        if (DENSE) {
          const uint4* wg = reinterpret_cast<const uint4*>(P.gate.dense + row * P.H);
          const uint4* wu = reinterpret_cast<const uint4*>(P.up.dense + row * P.H);
          uint4 vg[8], vu[8];
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            const int b = b0 + 4 * j;
            vg[j] = b < nb ? __ldg(wg + b) : make_uint4(0, 0, 0, 0);
            vu[j] = b < nb ? __ldg(wu + b) : make_uint4(0, 0, 0, 0);
          }
#pragma unroll
          for (int j = 0; j < 8; ++j) { mma_block(acc_g[j & 1], fx[j], vg[j]); mma_block(acc_u[j & 1], fx[j], vu[j]); }
        } else {
          if (!ringed) {
            if (b0 < nb) {
              raw_g = load_idx_raw<IdxT>(idx_g + row * nb + b0);
              raw_u = load_idx_raw<IdxT>(idx_u + row * nb + b0);
            } else {
              raw_g = raw_u = make_uint4(0, 0, 0, 0);
            }
          }
          // mma.sync needs the whole warp: lanes whose group lies beyond the row run it with
          // index 0 and zero activation fragments
          uint32_t ig[8], iu[8];
          unpack_idx8<IdxT>(raw_g, ig);
          unpack_idx8<IdxT>(raw_u, iu);
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            mma_block(acc_g[j & 1], fx[j], s_cb_g[ig[j]]);
            mma_block(acc_u[j & 1], fx[j], s_cb_u[iu[j]]);
          }
        }
      }
      // joint accumulation of the low-rank term: more k for the same tile
      for (int lg = lr_group; lg < pl.n_lr; lg += pl.team_warps) {
        const int rho0 = lg * 32 + 8 * c;
        uint4 fg = fac_g, fu = fac_u;
        if (lg != lr_group) {
          fg = fu = make_uint4(0, 0, 0, 0);
          if (rho0 < P.r) {
            fg = __ldg(reinterpret_cast<const uint4*>(P.gate.factor + row * P.r + rho0));
            fu = __ldg(reinterpret_cast<const uint4*>(P.up.factor + row * P.r + rho0));
          }
        }
        uint4 zgh = {0, 0, 0, 0}, zgl = {0, 0, 0, 0}, zuh = {0, 0, 0, 0}, zul = {0, 0, 0, 0};
        if (tok >= 0 && rho0 < P.r) {
          const int ig2 = (tok * 2 + P.gate.zslot) * rb + (rho0 >> 3), iu2 = (tok * 2 + P.up.zslot) * rb + (rho0 >> 3);
          zgh = s_zh[ig2]; zgl = s_zl[ig2]; zuh = s_zh[iu2]; zul = s_zl[iu2];
        }
        mma_block(acc_g[0], zgh, fg); mma_block(acc_g[1], zgl, fg);
        mma_block(acc_u[0], zuh, fu); mma_block(acc_u[1], zul, fu);
      }
      // ---- add the team's partial tiles and apply SwiGLU -----------------------------------
      float2* part = s_part + ((size_t)(buf * pl.n_teams + team) * 2) * pl.team_warps * 32;
      part[(0 * pl.team_warps + wi) * 32 + lane] = make_float2(acc_g[0][0] + acc_g[1][0], acc_g[0][1] + acc_g[1][1]);
      part[(1 * pl.team_warps + wi) * 32 + lane] = make_float2(acc_u[0][0] + acc_u[1][0], acc_u[0][1] + acc_u[1][1]);
      if (pl.team_warps > 1) team_sync(1 + team, team_threads); else __syncwarp();
      for (int q = tid_team; q < 64; q += team_threads) {
        const int m = q >> 3, n = q & 7;                      // token m of this pass, row n of the tile
        if (m < n_tok) {
          const int src = 4 * m + (n >> 1);
          float gs = 0.f, us = 0.f;
          for (int w = 0; w < pl.team_warps; ++w) {
            const float2 pg = part[(0 * pl.team_warps + w) * 32 + src];
            const float2 pu = part[(1 * pl.team_warps + w) * 32 + src];
            gs += (n & 1) ? pg.y : pg.x;
            us += (n & 1) ? pu.y : pu.x;
          }
          P.p[(size_t)(off + pass * 8 + m) * P.I + jt * 8 + n] = gs / (1.f + expf(-gs)) * us;
        }
      }
      buf ^= 1;
    }
  }
  cp_async_wait_pending(0);
}

// ---------------------------------------------------------------------------------------------
// k_down_mma: y[token][slot][h] for every (expert, 8-row tile of H); activations are the fp32
// intermediates p split into bf16 hi + lo fragments.
// ---------------------------------------------------------------------------------------------
struct DnLayout {
  size_t ring, fring, part, yrow, total;
  int slot_u4;      // uint4 per lane per ring slot: 1 (indices) or 8 (a dense 256-value slice of a row)
};

__host__ __device__ inline DnLayout dn_layout(int K, bool vq, const StagePlan& pl, int warps) {
  DnLayout L;
  size_t o = vq ? (size_t)K * 16 : 0;
  L.slot_u4 = vq ? 1 : 8;
  L.ring = o;   o += (size_t)warps * pl.depth * L.slot_u4 * 32 * 16;
  L.fring = o;  o += (size_t)pl.n_teams * (pl.n_lr > 0 ? pl.n_lr : 0) * pl.depth * 32 * 16;
  L.part = o;   o += (size_t)2 * pl.n_teams * pl.team_warps * 32 * 8;
  L.yrow = o;   o += (size_t)2 * pl.n_teams * 8 * 8;
  L.total = o;
  return L;
}

template <typename IdxT, bool DENSE>
__global__ void __launch_bounds__(kDownThreads, 1)
k_down_mma(const Params P, int T, const StagePlan pl) {
  extern __shared__ uint4 s_u4[];
  char* s_base = reinterpret_cast<char*>(s_u4);
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, g = lane >> 2, c = lane & 3;
  const int nb = pl.nb, D = pl.depth;
  const DnLayout L = dn_layout(P.K, !DENSE, pl, blockDim.x >> 5);
  uint4* s_cb = s_u4;
  uint4* s_ring = reinterpret_cast<uint4*>(s_base + L.ring);
  uint4* s_fring = reinterpret_cast<uint4*>(s_base + L.fring);
  float2* s_part = reinterpret_cast<float2*>(s_base + L.part);
  long long* s_yrow = reinterpret_cast<long long*>(s_base + L.yrow);   // [buf][team][8] output row offsets
  if (!DENSE)
    for (int i = tid; i < P.K; i += blockDim.x) s_cb[i] = __ldg(P.down.codebook + i);
  pdl_wait();      // p (and z_d) and the routing lists are complete
  pdl_launch();
  __syncthreads();

  const int team = warp / pl.team_warps, wi = warp - team * pl.team_warps;
  const int team_threads = pl.team_warps * 32;
  const int tid_team = tid - team * team_threads;
  const int n_act = *P.act_n;
  const int n_slots = P.k + P.S;
  const long long U = (long long)n_act * pl.tiles;
  const long long G = (long long)gridDim.x * pl.n_teams, tau = (long long)blockIdx.x * pl.n_teams + team;
  const long long u_begin = tau * U / G;
  const int n_my = team < pl.n_teams ? (int)((tau + 1) * U / G - u_begin) : 0;
  const bool spw_one = pl.n_slices <= pl.team_warps;
  const bool ringed = spw_one;
  const int lr_group = pl.team_warps - 1 - wi;
  const bool has_lr = lr_group < pl.n_lr;
  const int b_first = wi * 32 + (DENSE ? c : 8 * c), rho_first = lr_group * 32 + 8 * c;
  const bool idx_live = DENSE ? (wi * 32 < nb) : (b_first < nb), fac_live = has_lr && rho_first < P.r;

  const IdxT* idx_d = static_cast<const IdxT*>(P.down.idx);
  uint4* ring = s_ring + (size_t)warp * D * L.slot_u4 * 32;                        // [slot][chunk][lane]
  uint4* fring = s_fring + (size_t)(team * pl.n_lr + (has_lr ? lr_group : 0)) * D * 32;

  auto issue = [&](int i) {
    const long long u = u_begin + i;
    const int a = (int)(u / pl.tiles), jt = (int)(u - (long long)a * pl.tiles);
    const size_t row = (size_t)P.act_e[a] * P.H + jt * 8 + g;
    const int slot = i % D;
    if (ringed && idx_live) {
      if (DENSE) {
        const uint4* wd = reinterpret_cast<const uint4*>(P.down.dense + row * P.I);
#pragma unroll
        for (int j = 0; j < 8; ++j)
          if (b_first + 4 * j < nb) cp_async16(ring + (slot * 8 + j) * 32 + lane, wd + b_first + 4 * j);
      } else {
        cp_async_idx8<IdxT>(ring + slot * 32 + lane, idx_d + row * nb + b_first);
      }
    }
    if (fac_live) cp_async16(fring + slot * 32 + lane, P.down.factor + row * P.r + rho_first);
  };

  uint4 fh[8], fl[8];
  uint4 zh = {0, 0, 0, 0}, zl = {0, 0, 0, 0};
  int frag_a = -1, frag_pass = -1, frag_slice = -1, z_a = -1, z_pass = -1, z_lg = -1;
  int buf = 0;

  for (int i = 0; i < D - 1; ++i) { if (i < n_my) issue(i); cp_async_commit(); }
  for (int i = 0; i < n_my; ++i) {
    if (i + D - 1 < n_my) issue(i + D - 1);
    cp_async_commit();
    cp_async_wait_pending(D - 1);
    const long long u = u_begin + i;
    const int a = (int)(u / pl.tiles), jt = (int)(u - (long long)a * pl.tiles);
    const int e = P.act_e[a], off = P.act_off[a], cnt = P.act_cnt[a];
    const size_t row = (size_t)e * P.H + jt * 8 + g;
    const int slot = i % D;
    uint4 raw = {0, 0, 0, 0}, fac = {0, 0, 0, 0};
    if (!DENSE && ringed && idx_live) raw = ring_idx8<IdxT>(ring + slot * 32 + lane);
    if (fac_live) fac = fring[slot * 32 + lane];
    for (int pass = 0; pass * 8 < cnt; ++pass) {
      const int n_tok = min(8, cnt - pass * 8);
      const int pos = g < n_tok ? off + pass * 8 + g : -1;
      float acc[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
      for (int sl = wi; sl < pl.n_slices; sl += pl.team_warps) {
        const int b0 = sl * 32 + (DENSE ? c : 8 * c);
        if (frag_a != a || frag_pass != pass || frag_slice != sl) {
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            const int b = b0 + (DENSE ? 4 * j : j);
            if (pos >= 0 && b < nb) {
              const float4* pp = reinterpret_cast<const float4*>(P.p + (size_t)pos * P.I + b * 8);
              split_hi_lo(pp[0], pp[1], fh[j], fl[j]);
            } else {
              fh[j] = fl[j] = make_uint4(0, 0, 0, 0);
            }
          }
          frag_a = a; frag_pass = pass; frag_slice = sl;
        }
        if (DENSE) {
          const uint4* wd = reinterpret_cast<const uint4*>(P.down.dense + row * P.I);
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            const int b = b0 + 4 * j;
            uint4 v = make_uint4(0, 0, 0, 0);
            if (b < nb) v = ringed ? ring[(slot * 8 + j) * 32 + lane] : __ldg(wd + b);
            mma_block(acc[0], fh[j], v);
            mma_block(acc[1], fl[j], v);
          }
        } else {
          if (!ringed) raw = b0 < nb ? load_idx_raw<IdxT>(idx_d + row * nb + b0) : make_uint4(0, 0, 0, 0);
          uint32_t id[8];                      // out-of-range groups: index 0, zero fragments
          unpack_idx8<IdxT>(raw, id);
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            const uint4 w = s_cb[id[j]];
            mma_block(acc[0], fh[j], w);
            mma_block(acc[1], fl[j], w);
          }
        }
      }
      for (int lg = lr_group; lg < pl.n_lr; lg += pl.team_warps) {
        const int rho0 = lg * 32 + 8 * c;
        uint4 f = fac;
        if (lg != lr_group)
          f = rho0 < P.r ? __ldg(reinterpret_cast<const uint4*>(P.down.factor + row * P.r + rho0)) : make_uint4(0, 0, 0, 0);
        if (z_a != a || z_pass != pass || z_lg != lg) {
          if (pos >= 0 && rho0 < P.r) {
            const float* zp = P.zd + (size_t)pos * P.r + rho0;
            split_hi_lo(*reinterpret_cast<const float4*>(zp), *reinterpret_cast<const float4*>(zp + 4), zh, zl);
          } else {
            zh = zl = make_uint4(0, 0, 0, 0);
          }
          z_a = a; z_pass = pass; z_lg = lg;
        }
        mma_block(acc[0], zh, f);
        mma_block(acc[1], zl, f);
      }
      float2* part = s_part + (size_t)(buf * pl.n_teams + team) * pl.team_warps * 32;
      long long* yrow = s_yrow + (size_t)(buf * pl.n_teams + team) * 8;
      part[wi * 32 + lane] = make_float2(acc[0][0] + acc[1][0], acc[0][1] + acc[1][1]);
      if (tid_team < n_tok) {                    // output rows of this pass's tokens
        const int ps = off + pass * 8 + tid_team;
        yrow[tid_team] = ((long long)P.pair_token[ps] * n_slots + P.pair_slot[ps]) * P.H;
      }
      if (pl.team_warps > 1) team_sync(1 + team, team_threads); else __syncwarp();
      for (int q = tid_team; q < 64; q += team_threads) {
        const int m = q >> 3, n = q & 7;
        if (m < n_tok) {
          const int src = 4 * m + (n >> 1);
          float sum = 0.f;
          for (int w = 0; w < pl.team_warps; ++w) {
            const float2 v = part[w * 32 + src];
            sum += (n & 1) ? v.y : v.x;
          }
          P.y[yrow[m] + jt * 8 + n] = sum;
        }
      }
      buf ^= 1;
    }
  }
  cp_async_wait_pending(0);
}

// z_d[pos][rho] = <basis_down[rho], p[pos]> (link of the chain between gate/up and down).
__global__ void __launch_bounds__(256) k_zdown_pdl(const Params P, int n_pos) {
  pdl_wait();
  pdl_launch();
  const int lane = threadIdx.x & 31;
  const int w = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  if (w >= n_pos * P.r) return;
  const int pos = w / P.r, rho = w - pos * P.r;
  const uint4* brow = reinterpret_cast<const uint4*>(P.down.basis + (size_t)rho * P.I);
  const float4* prow = reinterpret_cast<const float4*>(P.p + (size_t)pos * P.I);
  float acc = 0.f;
  for (int cidx = lane; cidx < P.I / 8; cidx += 32) {
    float wf[8];
    unpack8(__ldg(brow + cidx), wf);
    const float4 p0 = prow[2 * cidx], p1 = prow[2 * cidx + 1];
    const float pf[8] = {p0.x, p0.y, p0.z, p0.w, p1.x, p1.y, p1.z, p1.w};
    acc = dot8(wf, pf, acc);
  }
  acc = warp_sum(acc);
  if (lane == 0) P.zd[(size_t)pos * P.r + rho] = acc;
}

// out[t][h] = sum over slots (in slot order) of affinity * y[t][slot][h]; shared experts weigh 1.
__global__ void __launch_bounds__(256) k_combine(const Params P, bf16* __restrict__ out, int T) {
  pdl_wait();
  pdl_launch();
  const int n_slots = P.k + P.S, H2 = P.H / 2;
  for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < T * H2; i += gridDim.x * blockDim.x) {
    const int t = i / H2, h2 = i - t * H2;
    float a0 = 0.f, a1 = 0.f;
    for (int s = 0; s < n_slots; ++s) {
      const float w = s < P.k ? P.topk_w[t * P.k + s] : 1.f;
      const float2 v = *reinterpret_cast<const float2*>(P.y + ((size_t)t * n_slots + s) * P.H + 2 * h2);
      a0 = fmaf(w, v.x, a0);
      a1 = fmaf(w, v.y, a1);
    }
    *reinterpret_cast<__nv_bfloat162*>(out + (size_t)t * P.H + 2 * h2) = __floats2bfloat162_rn(a0, a1);
  }
}

}  // namespace
