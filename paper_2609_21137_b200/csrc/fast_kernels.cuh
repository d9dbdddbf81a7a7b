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
constexpr int kDenseThreads = 384;   // dense weight tiles in flight need more registers per thread

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
// k_router_z_pdl: same arithmetic and summation order as k_router_z, as the head of the chain.
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) k_router_z_pdl(const Params P, const bf16* __restrict__ x, int T) {
  pdl_wait();      // the previous call's kernels may still read logits / z
  pdl_launch();
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
// k_gateup_mma
// ---------------------------------------------------------------------------------------------
__host__ __device__ inline size_t gu_part_bytes(const StagePlan& pl) {
  // [buffer 2][team][projection 2][warp][lane 32] float2
  return (size_t)2 * pl.n_teams * 2 * pl.team_warps * 32 * 8;
}

__host__ __device__ inline size_t gu_smem_bytes(int K, int n_books, int T, int H, const StagePlan& pl,
                                                int E, int k, int S) {
  return (size_t)n_books * K * 16 + (size_t)T * (H / 8 + 1) * 16 + gu_part_bytes(pl) +
         route_smem_bytes(T, E, k, S);
}

template <typename IdxT, bool DENSE>
__global__ void __launch_bounds__(DENSE ? kDenseThreads : kFastThreads, 1)
k_gateup_mma(const Params P, const bf16* __restrict__ x, int T, const StagePlan pl, int n_books) {
  extern __shared__ uint4 s_u4[];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, g = lane >> 2, c = lane & 3;
  const int nb = pl.nb, xs = nb + 1;
  uint4* s_cb_g = s_u4;
  uint4* s_cb_u = n_books == 2 ? s_u4 + P.K : s_u4;
  uint4* s_x = s_u4 + (size_t)n_books * P.K;
  float2* s_part = reinterpret_cast<float2*>(s_x + (size_t)T * xs);
  char* s_route = reinterpret_cast<char*>(s_part) + gu_part_bytes(pl);
  const RouteSmem R = carve_route(s_route, T, P.E, P.k, P.S);

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
  route_in_block(P, T, R, blockIdx.x == 0);
  pdl_launch();

  const int team = warp / pl.team_warps, wi = warp - team * pl.team_warps;
  const int team_threads = pl.team_warps * 32;
  const int tid_team = tid - team * team_threads;
  const int n_act = *R.n_act;
  const long long U = (long long)n_act * pl.tiles;
  const long long G = (long long)gridDim.x * pl.n_teams, tau = (long long)blockIdx.x * pl.n_teams + team;
  const long long u_begin = tau * U / G, u_end = (tau + 1) * U / G;
  const int spw_one = pl.n_slices <= pl.team_warps;          // one slice per warp: fragments stay put
  // low-rank group handled by this warp (groups are dealt from the last warp of the team down)
  const int lr_group = pl.team_warps - 1 - wi;
  const bool has_lr = lr_group < pl.n_lr;   // n_lr is 0 for a dense projection

  uint4 fx[8];                       // activation fragments of the current slice
  uint4 zgh = {0, 0, 0, 0}, zgl = {0, 0, 0, 0}, zuh = {0, 0, 0, 0}, zul = {0, 0, 0, 0};
  int frag_a = -1, frag_pass = -1, frag_slice = -1, z_a = -1, z_pass = -1, z_lg = -1;
  int buf = 0;

  const IdxT* idx_g = static_cast<const IdxT*>(P.gate.idx);
  const IdxT* idx_u = static_cast<const IdxT*>(P.up.idx);

  for (long long u = u_begin; u < u_end; ++u) {
    const int a = (int)(u / pl.tiles), jt = (int)(u - (long long)a * pl.tiles);
    const int e = R.act_e[a], off = R.act_off[a], cnt = R.act_cnt[a];
    const size_t row = (size_t)e * P.I + jt * 8 + g;       // this lane's weight row
    // index registers of the first slice are fetched once per tile and reused by every pass
    uint4 raw_g = {0, 0, 0, 0}, raw_u = {0, 0, 0, 0};
    uint4 fac_g = {0, 0, 0, 0}, fac_u = {0, 0, 0, 0};
    const int b_first = wi * 32 + 8 * c;
    if (!DENSE && spw_one && b_first < nb) {
      raw_g = load_idx_raw<IdxT>(idx_g + row * nb + b_first);
      raw_u = load_idx_raw<IdxT>(idx_u + row * nb + b_first);
    }
    if (has_lr && lr_group * 32 + 8 * c < P.r) {
      fac_g = __ldg(reinterpret_cast<const uint4*>(P.gate.factor + row * P.r + lr_group * 32 + 8 * c));
      fac_u = __ldg(reinterpret_cast<const uint4*>(P.up.factor + row * P.r + lr_group * 32 + 8 * c));
    }
    for (int pass = 0; pass * 8 < cnt; ++pass) {
      const int n_tok = min(8, cnt - pass * 8);
      const int tok = g < n_tok ? R.pair_token[off + pass * 8 + g] : -1;
      float acc_g[4] = {0.f, 0.f, 0.f, 0.f}, acc_u[4] = {0.f, 0.f, 0.f, 0.f};
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
          for (int j = 0; j < 8; ++j) { mma_block(acc_g, fx[j], vg[j]); mma_block(acc_u, fx[j], vu[j]); }
        } else {
          if (!spw_one) {
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
            mma_block(acc_g, fx[j], s_cb_g[ig[j]]);
            mma_block(acc_u, fx[j], s_cb_u[iu[j]]);
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
        if (z_a != a || z_pass != pass || z_lg != lg) {
          if (tok >= 0 && rho0 < P.r) {
            const float* zg = P.z + ((size_t)tok * 2 + P.gate.zslot) * P.r + rho0;
            const float* zu = P.z + ((size_t)tok * 2 + P.up.zslot) * P.r + rho0;
            split_hi_lo(*reinterpret_cast<const float4*>(zg), *reinterpret_cast<const float4*>(zg + 4), zgh, zgl);
            split_hi_lo(*reinterpret_cast<const float4*>(zu), *reinterpret_cast<const float4*>(zu + 4), zuh, zul);
          } else {
            zgh = zgl = zuh = zul = make_uint4(0, 0, 0, 0);
          }
          z_a = a; z_pass = pass; z_lg = lg;
        }
        mma_block(acc_g, zgh, fg); mma_block(acc_g, zgl, fg);
        mma_block(acc_u, zuh, fu); mma_block(acc_u, zul, fu);
      }
      // ---- add the team's partial tiles and apply SwiGLU -----------------------------------
      float2* part = s_part + ((size_t)(buf * pl.n_teams + team) * 2) * pl.team_warps * 32;
      part[(0 * pl.team_warps + wi) * 32 + lane] = make_float2(acc_g[0], acc_g[1]);
      part[(1 * pl.team_warps + wi) * 32 + lane] = make_float2(acc_u[0], acc_u[1]);
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
}

// ---------------------------------------------------------------------------------------------
// k_down_mma: y[token][slot][h] for every (expert, 8-row tile of H); activations are the fp32
// intermediates p split into bf16 hi + lo fragments.
// ---------------------------------------------------------------------------------------------
__host__ __device__ inline size_t dn_part_bytes(const StagePlan& pl) {
  return (size_t)2 * pl.n_teams * pl.team_warps * 32 * 8;
}

__host__ __device__ inline size_t dn_smem_bytes(int K, bool vq, const StagePlan& pl) {
  return (vq ? (size_t)K * 16 : 0) + dn_part_bytes(pl);
}

template <typename IdxT, bool DENSE>
__global__ void __launch_bounds__(DENSE ? kDenseThreads : kFastThreads, 1)
k_down_mma(const Params P, int T, const StagePlan pl) {
  extern __shared__ uint4 s_u4[];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, g = lane >> 2, c = lane & 3;
  const int nb = pl.nb;
  uint4* s_cb = s_u4;
  float2* s_part = reinterpret_cast<float2*>(s_u4 + (DENSE ? 0 : P.K));
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
  const long long u_begin = tau * U / G, u_end = (tau + 1) * U / G;
  const int spw_one = pl.n_slices <= pl.team_warps;
  const int lr_group = pl.team_warps - 1 - wi;
  const bool has_lr = lr_group < pl.n_lr;

  uint4 fh[8], fl[8];
  uint4 zh = {0, 0, 0, 0}, zl = {0, 0, 0, 0};
  int frag_a = -1, frag_pass = -1, frag_slice = -1, z_a = -1, z_pass = -1, z_lg = -1;
  int buf = 0;
  const IdxT* idx_d = static_cast<const IdxT*>(P.down.idx);

  for (long long u = u_begin; u < u_end; ++u) {
    const int a = (int)(u / pl.tiles), jt = (int)(u - (long long)a * pl.tiles);
    const int e = P.act_e[a], off = P.act_off[a], cnt = P.act_cnt[a];
    const size_t row = (size_t)e * P.H + jt * 8 + g;
    uint4 raw = {0, 0, 0, 0}, fac = {0, 0, 0, 0};
    const int b_first = wi * 32 + 8 * c;
    if (!DENSE && spw_one && b_first < nb) raw = load_idx_raw<IdxT>(idx_d + row * nb + b_first);
    if (has_lr && lr_group * 32 + 8 * c < P.r)
      fac = __ldg(reinterpret_cast<const uint4*>(P.down.factor + row * P.r + lr_group * 32 + 8 * c));
    for (int pass = 0; pass * 8 < cnt; ++pass) {
      const int n_tok = min(8, cnt - pass * 8);
      const int pos = g < n_tok ? off + pass * 8 + g : -1;
      float acc[4] = {0.f, 0.f, 0.f, 0.f};
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
          uint4 v[8];
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            const int b = b0 + 4 * j;
            v[j] = b < nb ? __ldg(wd + b) : make_uint4(0, 0, 0, 0);
          }
#pragma unroll
          for (int j = 0; j < 8; ++j) { mma_block(acc, fh[j], v[j]); mma_block(acc, fl[j], v[j]); }
        } else {
          if (!spw_one) raw = b0 < nb ? load_idx_raw<IdxT>(idx_d + row * nb + b0) : make_uint4(0, 0, 0, 0);
          uint32_t id[8];                      // out-of-range groups: index 0, zero fragments
          unpack_idx8<IdxT>(raw, id);
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            const uint4 w = s_cb[id[j]];
            mma_block(acc, fh[j], w);
            mma_block(acc, fl[j], w);
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
        mma_block(acc, zh, f);
        mma_block(acc, zl, f);
      }
      float2* part = s_part + (size_t)(buf * pl.n_teams + team) * pl.team_warps * 32;
      part[wi * 32 + lane] = make_float2(acc[0], acc[1]);
      if (pl.team_warps > 1) team_sync(1 + team, team_threads); else __syncwarp();
      for (int q = tid_team; q < 64; q += team_threads) {
        const int m = q >> 3, n = q & 7;
        if (m < n_tok) {
          const int src = 4 * m + (n >> 1);
          float s = 0.f;
          for (int w = 0; w < pl.team_warps; ++w) {
            const float2 v = part[w * 32 + src];
            s += (n & 1) ? v.y : v.x;
          }
          const int ps = off + pass * 8 + m;
          P.y[((size_t)P.pair_token[ps] * n_slots + P.pair_slot[ps]) * P.H + jt * 8 + n] = s;
        }
      }
      buf ^= 1;
    }
  }
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
